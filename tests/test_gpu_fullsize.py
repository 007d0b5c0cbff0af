"""Parity at the full sizes of the benchmark configurations, in the launch configuration bench.py times.

The source buffers are filled on the device with a counter hash; the tables are compared whole with the oracle's.
KV: whole layers of EVERY destination pool are compared element by element - live blocks, idle blocks and foreign blocks
alike - with the oracle's transformation of the same layers, streamed through host memory a few layers at a time (the
oracle's layer loop on as many threads): ALL layers of the headline configuration (on a host so slow that this would
take more than four minutes: as many groups of layers as fit, never fewer than three), three layers (the first, the
last, one drawn at random) of the others; on the remaining layers sampled (layer, sequence, block) units are re-laid-out by
the oracle one by one.  Weights: all layers of the headline configuration, three of the others, compared whole."""
import os
import time
from concurrent.futures import ThreadPoolExecutor

import numpy as np
import pytest

import workloads as wl
from harness import pairs_in_destination_order

pytestmark = pytest.mark.gpu

FULL = ["llama3_8b_1to4", "llama3_8b_2to8", "llama2_7b_1to2", "llama2_13b_4to1", "llama3_70b_slice_8to2"]


HEADLINE = "llama3_8b_1to4"  # compared completely: every layer of every destination buffer
GROUP_BYTES = 12 << 30       # source KV bytes streamed through host memory per oracle call (less on a small host)
WHOLE_LAYER_BUDGET_S = 240.0  # the headline's every-layer comparison takes about 135 s with 16 host cores


@pytest.fixture(autouse=True)
def _device_memory_given_back():
    """These tests take most of the device memory in a few buffers of tens of GiB.  A small buffer carved out of a
    cached segment of that size would pin it, so nothing cached is carried from one test into the next."""
    import gc

    import torch

    gc.collect()
    torch.cuda.empty_cache()
    yield
    gc.collect()
    torch.cuda.empty_cache()


def _host_available() -> int:
    """Bytes of host memory that can still be taken (MemAvailable), or a large number if it cannot be read."""
    try:
        for line in open("/proc/meminfo"):
            if line.startswith("MemAvailable"):
                return int(line.split()[1]) * 1024
    except OSError:
        pass
    return 1 << 40


def _group_bytes() -> int:
    # an oracle call holds the sources, the expected destinations and its own logical copy: about 3.5 x the sources
    return max(1 << 30, min(GROUP_BYTES, _host_available() // 8))


def _picked_layers(g, L):
    """The layers compared whole: the first, the last and one drawn at random; with fewer than 12 host cores (the
    oracle's layer loop then takes twice as long) the first and the last."""
    drawn = int(g.integers(L))  # drawn either way, so that the later draws of a test do not depend on the host
    return sorted({0, L - 1, drawn} if (os.cpu_count() or 1) >= 12 else {0, L - 1})


def _whole_layers(g, L, bytes_per_layer):
    """The picked layers - or fewer when they (held twice) do not fit the host comfortably."""
    layers = _picked_layers(g, L)
    while len(layers) > 1 and 4 * len(layers) * bytes_per_layer > _host_available() // 2:
        layers.pop()
    return layers

CASES = [(n, "head") for n in FULL] + [("llama3_8b_1to4", "token"), ("llama3_70b_slice_8to2", "token2head"),
                                       ("llama2_7b_1to2", "head2token")]


class _BlockView:
    """One worker's pool addressed as [layer, block] -> the bytes of that block, as a pool holding only that block
    would store them (header-centric: one slab per block; token-first: the block's K slab then its V slab)."""

    def __init__(self, pool, n_layers, NB, token_first):
        self.tf = token_first
        self.v = pool.view(n_layers, 2, NB, -1) if token_first else pool.view(n_layers, NB, -1)

    def __getitem__(self, idx):
        l, blk = idx
        return self.v[l, :, blk].reshape(-1) if self.tf else self.v[l, blk]


@pytest.mark.parametrize("name,kv_order", CASES)
def test_full_size_config(name, kv_order, oracle):
    import torch

    import bench

    assert torch.cuda.is_available()
    cfg = wl.CONFIGS[name]
    m, a, b, T = cfg["model"], cfg["a"], cfg["b"], wl.BLOCK_TOKENS
    device = torch.device("cuda:0")
    so, do = bench.KV_ORDERS[kv_order]
    s, st = bench.build_session(name, device, kv_order=kv_order)
    try:
        s.status.zero_()
        s.step()
        torch.cuda.synchronize()

        # ---- tables: whole comparison
        exp_bt, exp_pairs, exp_n, exp_left, exp_status = oracle.assign_blocks(
            st["seq_lens"], T, st["src_bt"], st["NB_src"], st["NB_dst"], free_list=st.get("dst_free_list"),
            free_mask=st.get("dst_free_mask"), pairs_cap=st["n_live"])
        assert exp_status == 0 and int(s.status.item()) == 0
        assert int(s.num_pairs.item()) == exp_n == st["n_live"] and int(s.free_count.item()) == exp_left
        dst_bt = s.dst_bt.cpu().numpy()
        assert np.array_equal(dst_bt, exp_bt)
        assert np.array_equal(s.pairs.cpu().numpy()[:exp_n],
                              pairs_in_destination_order(exp_pairs, exp_bt, st["seq_lens"], T))

        # ---- KV: sampled blocks, each re-laid-out by the oracle on its own
        Lkv = s.kv_layers
        src_v = [_BlockView(p, Lkv, st["NB_src"], so == 1) for p in s.src_pools]
        dst_v = [_BlockView(p, Lkv, st["NB_dst"], do == 1) for p in s.dst_pools]
        g = np.random.default_rng(7)
        one = dict(m, L=1)
        seqs = np.flatnonzero(st["blocks_per_seq"] > 0)
        for _ in range(96):
            l = int(g.integers(Lkv))
            q = int(g.choice(seqs))
            i = int(g.integers(st["blocks_per_seq"][q]))
            sid, did = int(st["src_bt"][q, i]), int(dst_bt[q, i])
            src1 = [v[l, sid].cpu().numpy().view(np.uint16).copy() for v in src_v]  # NB = 1 pools
            exp1 = [np.zeros(d[l, did].numel() // 2, np.uint16) for d in dst_v]
            oracle.kv_transform(one, T, [T], a, 1, [[0]], src1, b, 1, [[0]], exp1, src_order=so, dst_order=do)
            for r in range(b):
                got = dst_v[r][l, did].cpu().numpy().view(np.uint16)
                assert np.array_equal(got, exp1[r]), (name, l, q, i, r)

        # ---- KV: whole layers, every word of every destination pool (live, idle and foreign blocks); consecutive
        # layers go through the oracle together, its layer loop on one thread per layer
        everything = name == HEADLINE and kv_order == "head"
        layers = list(range(Lkv)) if everything else _picked_layers(g, Lkv)
        src_layer_bytes = sum(p.numel() for p in s.src_pools) // Lkv
        per_call = max(1, min(os.cpu_count() or 1, 16, _group_bytes() // src_layer_bytes))
        groups = [[layers[0]]]
        for l in layers[1:]:
            if l == groups[-1][-1] + 1 and len(groups[-1]) < per_call:
                groups[-1].append(l)
            else:
                groups.append([l])
        # the first, the last and the middle group go first; on a host too slow to get through every group of the
        # headline configuration within the budget the remaining layers keep their sampled blocks only
        first3 = [0, len(groups) - 1, len(groups) // 2]
        groups = [groups[i] for i in dict.fromkeys(first3)] + [grp for i, grp in enumerate(groups) if i not in first3]
        t_begin = time.monotonic()
        exp_n_layers, exp_grp = 0, None
        try:
            for gi, grp in enumerate(groups):
                if gi >= 3 and time.monotonic() - t_begin > WHOLE_LAYER_BUDGET_S:
                    print(f"{name}: whole-layer comparison stopped after {gi} of {len(groups)} groups "
                          f"({WHOLE_LAYER_BUDGET_S:.0f} s budget)")
                    break
                l0, nl = grp[0], len(grp)
                oracle.set_threads(nl)
                src_grp = [p.view(Lkv, -1)[l0:l0 + nl].cpu().numpy().view(np.uint16).reshape(-1) for p in s.src_pools]
                if exp_n_layers != nl:
                    exp_grp = [np.empty(p.numel() // Lkv // 2 * nl, np.uint16) for p in s.dst_pools]
                    exp_n_layers = nl
                for e in exp_grp:
                    e.fill(0xA5A5)
                oracle.kv_transform(dict(m, L=nl), T, st["seq_lens"], a, st["NB_src"], st["src_bt"], src_grp, b,
                                    st["NB_dst"], exp_bt, exp_grp, src_order=so, dst_order=do)
                del src_grp
                for r in range(b):
                    got = s.dst_pools[r].view(Lkv, -1)[l0:l0 + nl].cpu().numpy().view(np.uint16).reshape(-1)
                    if not np.array_equal(got, exp_grp[r]):
                        bad = np.flatnonzero(got != exp_grp[r])
                        raise AssertionError(f"{name} layers {l0}..{l0 + nl - 1} dst pool {r}: {bad.size} words differ, "
                                             f"first at {bad[0]}")
                    del got
        finally:
            oracle.set_threads(1)
            del exp_grp

        # ---- weights: whole layers (the C calls release the interpreter lock: a few layers at a time)
        w_layers = list(range(m["L"])) if everything else _picked_layers(g, m["L"])

        def check_weights(l):
            src_sh = [{n: t.cpu().numpy().view(np.uint16).reshape(oracle.shard_shapes(m, a)[n])
                       for n, t in s.src_w[r][l].items()} for r in range(a)]
            exp = oracle.weights_transform(src_sh, m, a, b)
            for r in range(b):
                for n, e in exp[r].items():
                    got = s.dst_w[r][l][n].cpu().numpy().view(np.uint16)
                    assert np.array_equal(got, e.reshape(-1)), (name, "weights", l, r, n)

        with ThreadPoolExecutor(max_workers=min(os.cpu_count() or 1, 8)) as pool:
            list(pool.map(check_weights, w_layers))
    finally:
        del s
        torch.cuda.empty_cache()


def test_full_size_inplace_merge(oracle):
    """The benchmark's in-place merge workload (4 x TP1 -> TP4) at full size: merged tables and live marks compared
    whole; three whole layers (first, last, one at random) of every pool compared word by word with the oracle's merge
    of the same layer; on the other layers sampled old blocks (with whatever mix of live / free they have across the
    instances) compared with the oracle's merge of just those blocks."""
    import torch

    import bench

    name = "llama3_8b_merge_4x1to4"
    cfg = wl.MERGE_CONFIGS[name]
    m, N, a, T = cfg["model"], cfg["N"], cfg["a"], wl.BLOCK_TOKENS
    device = torch.device("cuda:0")
    s, st = bench.build_merge_session(name, device)
    try:
        NB, L = st["NB"], s.kv_layers
        exp_bt, exp_live, exp_status = oracle.kv_merge_inplace(dict(m, L=0), T, N, a, NB, st["seq_lens"], st["src_bt"],
                                                               [np.zeros(0, np.uint16) for _ in range(N * a)])
        assert exp_status == 0
        g = np.random.default_rng(11)
        old_v = [p.view(L, NB, -1) for p in s.pools]            # [layer][old block][bytes]
        samples = [(int(g.integers(L)), int(g.integers(NB))) for _ in range(64)]
        before = {(l, p): [v[l, p].cpu().numpy().view(np.uint16).copy() for v in old_v] for l, p in samples}
        whole_layers = _whole_layers(g, L, sum(p.numel() for p in s.pools) // L)
        layer_before = {l: [v[l].cpu().numpy().view(np.uint16).reshape(-1).copy() for v in old_v] for l in whole_layers}

        s.status.zero_()
        s.step()
        torch.cuda.synchronize()
        assert int(s.status.item()) == 0
        assert np.array_equal(s.dst_bt.cpu().numpy(), exp_bt)
        assert np.array_equal(s.live.cpu().numpy()[:N * NB].reshape(N, NB), exp_live)

        one = dict(m, L=1)
        for (l, p), olds in before.items():
            lens1 = np.array([[T if exp_live[i, p] else 0] for i in range(N)], np.int32)
            mini = [o.copy() for o in olds]                      # N*a pools of one old block each
            _, _, st1 = oracle.kv_merge_inplace(one, T, N, a, 1, lens1, np.zeros((N, 1, 1), np.int32), mini)
            assert st1 == 0
            for w in range(N * a):
                got = old_v[w][l, p].cpu().numpy().view(np.uint16)
                assert np.array_equal(got, mini[w]), (l, p, w)

        for l in whole_layers:
            exp = layer_before.pop(l)
            _, _, st1 = oracle.kv_merge_inplace(one, T, N, a, NB, st["seq_lens"], st["src_bt"], exp)
            assert st1 == 0
            for w in range(N * a):
                got = old_v[w][l].cpu().numpy().view(np.uint16).reshape(-1)
                if not np.array_equal(got, exp[w]):
                    bad = np.flatnonzero(got != exp[w])
                    raise AssertionError(f"layer {l} pool {w}: {bad.size} words differ, first at {bad[0]}")
    finally:
        del s
        torch.cuda.empty_cache()


@pytest.mark.parametrize("name", ["llama3_8b_1to4", "llama3_8b_2to8", "llama3_70b_slice_8to2"])
def test_full_size_inplace_reshape(name, oracle):
    """In-place block reshaping of one instance with the benchmark configuration's sequences, in the launch
    configuration bench.py --inplace times: tables, pair list and free mask compared whole; three whole layers of every
    pool (old workers' memory and new workers' pools) compared word by word with the oracle."""
    import torch

    import bench

    cfg = wl.CONFIGS[name]
    m, T = cfg["model"], wl.BLOCK_TOKENS
    s, st = bench.build_reshape_session(name, torch.device("cuda:0"))
    try:
        N, a, NB, L = s.N, s.a, s.NB, s.kv_layers
        src_bt = s.src_bt.cpu().numpy()
        g = np.random.default_rng(13)
        whole_layers = _whole_layers(g, L, sum(p.numel() for p in s.pools) // L)
        views = [p.view(L, -1) for p in s.pools]
        before = {l: [v[l].cpu().numpy().view(np.uint16).copy() for v in views] for l in whole_layers}
        s.status.zero_()
        s.step()
        torch.cuda.synchronize()
        one = dict(m, L=1)
        first = True
        for l in whole_layers:
            exp = before.pop(l)
            e_bt, e_pairs, e_n, e_mask, e_left, e_status = oracle.kv_reshape_inplace(
                s.direction, one, T, N, a, NB, st["seq_lens"], src_bt, exp, pairs_cap=st["n_live"])
            if first:
                assert e_status == 0 and int(s.status.item()) == 0
                assert np.array_equal(s.dst_bt.cpu().numpy(), e_bt)
                assert int(s.num_pairs.item()) == e_n and np.array_equal(s.pairs.cpu().numpy()[:e_n], e_pairs)
                assert np.array_equal(s.free_mask.cpu().numpy(), e_mask) and int(s.free_count.item()) == e_left
                first = False
            for w in range(N * a):
                got = views[w][l].cpu().numpy().view(np.uint16)
                if not np.array_equal(got, exp[w]):
                    bad = np.flatnonzero(got != exp[w])
                    raise AssertionError(f"{name} layer {l} pool {w}: {bad.size} words differ, first at {bad[0]}")
    finally:
        del s
        torch.cuda.empty_cache()


def test_full_size_padded_weights(oracle):
    """Llama-3-8B-shaped weights held as 4 padded partitions per tensor (2 MiB pages) on both sides, TP 1 -> 4: two
    layers compared whole with the oracle, pad bytes included (they keep the destination's fill)."""
    import torch

    import bench

    name, P = "llama3_8b_1to4", 4
    cfg = wl.CONFIGS[name]
    m, a, b = cfg["model"], cfg["a"], cfg["b"]
    s, st = bench.build_session(name, torch.device("cuda:0"), kv=False, weight_pad=P)
    try:
        s.status.zero_()
        s.reshard_weights()
        torch.cuda.synchronize()
        assert int(s.status.item()) == 0
        page_elems = (2 << 20) // 2
        for l in (0, m["L"] - 1):
            src_sh = [{n: t.cpu().numpy().view(np.uint16) for n, t in s.src_w[r][l].items()} for r in range(a)]
            exp = oracle.weights_transform_any(src_sh, m, a, b, src_pad=(P, page_elems), dst_pad=(P, page_elems),
                                               fill=0xA5A5)
            for r in range(b):
                for n, e in exp[r].items():
                    got = s.dst_w[r][l][n].cpu().numpy().view(np.uint16)
                    assert np.array_equal(got, e), (l, r, n)
    finally:
        del s
        torch.cuda.empty_cache()


@pytest.mark.parametrize("name,keep", [("llama3_8b_1to4", [2]), ("llama3_8b_2to8", [3, 0])])
def test_full_size_weight_compaction_in_place(name, keep, oracle):
    """Partial swap at the Llama-3-8B shape (4096 rows: 7 or 13 ordered waves for the column tensors, thousands of
    concurrent work items per wave): the front of every source buffer becomes the kept worker's dense shard."""
    import torch

    import bench
    import paper_2509_19729_b200 as A

    cfg = wl.CONFIGS[name]
    m, a, b = dict(cfg["model"]), cfg["a"], cfg["b"]
    N = b // a
    s, st = bench.build_session(name, torch.device("cuda:0"), layers=3, kv=False)
    try:
        m["L"] = 3
        before = {l: [{n: t.cpu().numpy().view(np.uint16).reshape(oracle.shard_shapes(m, a)[n]).copy()
                       for n, t in s.src_w[r][l].items()} for r in range(a)] for l in (0, 2)}
        s.status.zero_()
        A.amoeba_compact_weights_inplace(s.plan, s._src_w_packed, keep, 0, 3, s.status)
        torch.cuda.synchronize()
        assert int(s.status.item()) == 0
        for l in (0, 2):
            exp = oracle.weights_transform(before[l], m, a, b)
            for r in range(a):
                for n, e in exp[r * N + keep[r]].items():
                    got = s.src_w[r][l][n].cpu().numpy().view(np.uint16)[:e.size]
                    assert np.array_equal(got, e.reshape(-1)), (l, r, n)
    finally:
        del s
        torch.cuda.empty_cache()

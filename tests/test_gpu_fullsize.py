"""Parity at the full sizes of the benchmark configurations, in the launch configuration bench.py times.

The source buffers are filled on the device with a counter hash; the tables are compared whole with the oracle's;
the KV result is compared on sampled (layer, sequence, block) units - for each, the source worker slices are fetched,
the oracle re-lays-out that one block on the CPU, and the destination worker slices must equal it; the weights of
sampled layers are compared whole.  Size-independent properties: word sums are conserved, untouched destination
blocks keep their fill."""
import numpy as np
import pytest

import workloads as wl

pytestmark = pytest.mark.gpu

FULL = ["llama3_8b_1to4", "llama3_8b_2to8", "llama2_7b_1to2", "llama2_13b_4to1", "llama3_70b_slice_8to2"]


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

    def layer_blocks(self, l, NB, ids):
        """int64 words of the given blocks of layer l, [len(ids), words]."""
        import torch

        if self.tf:
            return torch.cat([self.v[l, c].view(torch.int64).view(NB, -1).index_select(0, ids) for c in range(2)], 1)
        return self.v[l].view(torch.int64).view(NB, -1).index_select(0, ids)


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
        assert np.array_equal(s.pairs.cpu().numpy()[:exp_n], exp_pairs)

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

        # ---- untouched destination blocks keep the fill (sampled)
        used = np.zeros(st["NB_dst"], bool)
        used[exp_pairs[:, 1]] = True
        idle = np.flatnonzero(~used)
        if idle.size:
            for did in g.choice(idle, size=min(16, idle.size), replace=False):
                for v in dst_v:
                    assert bool((v[int(g.integers(Lkv)), int(did)] == 0xA5).all())

        # ---- word sums are conserved over the live blocks of every layer (any size, any permutation)
        live_src = torch.as_tensor(exp_pairs[:, 0].astype(np.int64), device=device)
        live_dst = torch.as_tensor(exp_pairs[:, 1].astype(np.int64), device=device)
        for l in sorted(set(int(x) for x in g.integers(Lkv, size=3))):
            ssum = sum(int(v.layer_blocks(l, st["NB_src"], live_src).sum().item()) for v in src_v)
            dsum = sum(int(v.layer_blocks(l, st["NB_dst"], live_dst).sum().item()) for v in dst_v)
            assert (ssum - dsum) % (1 << 64) == 0

        # ---- weights: whole comparison of sampled layers
        for l in sorted(set([0, m["L"] - 1, int(g.integers(m["L"]))])):
            src_sh = [{n: t.cpu().numpy().view(np.uint16).reshape(oracle.shard_shapes(m, a)[n])
                       for n, t in s.src_w[r][l].items()} for r in range(a)]
            exp = oracle.weights_transform(src_sh, m, a, b)
            for r in range(b):
                for n, e in exp[r].items():
                    got = s.dst_w[r][l][n].cpu().numpy().view(np.uint16)
                    assert np.array_equal(got, e.reshape(-1)), (name, "weights", l, r, n)
    finally:
        del s
        torch.cuda.empty_cache()


def test_full_size_inplace_merge(oracle):
    """The benchmark's in-place merge workload (4 x TP1 -> TP4) at full size: merged tables and live marks compared
    whole; sampled old blocks (with whatever mix of live / free they have across the instances) compared with the
    oracle's merge of just those blocks; word sums of the live blocks conserved per layer."""
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
        live_old = [torch.as_tensor(np.flatnonzero(exp_live[i]).astype(np.int64), device=device) for i in range(N)]
        sum_layers = sorted(set(int(x) for x in g.integers(L, size=2)))
        sums_before = {l: sum(int(old_v[i * a + r][l].view(torch.int64).view(NB, -1).index_select(0, live_old[i]).sum())
                              for i in range(N) for r in range(a)) for l in sum_layers}

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

        new_v = [p.view(L, NB * N, -1) for p in s.pools]        # [layer][new block][bytes]
        for l in sum_layers:
            after = 0
            for i in range(N):
                ids = live_old[i] * N + i
                after += sum(int(v[l].view(torch.int64).view(NB * N, -1).index_select(0, ids).sum()) for v in new_v)
            assert (after - sums_before[l]) % (1 << 64) == 0
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

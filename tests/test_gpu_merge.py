"""Parity of the in-place merge of N instances (Sec. 3.1, Improvement 1) with the CPU oracle: every byte of every
pool, the merged block table, the live marks and the status word."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

MHA8 = dict(L=2, hidden=64, Hq=8, Hkv=8, D=16, I=64)
GQA = dict(L=3, hidden=512, Hq=16, Hkv=8, D=128, I=1792)


def _instances(oracle, m, T, N, a, NB, lens_per_instance, seed=0):
    g = np.random.default_rng(seed)
    S = max(len(l) for l in lens_per_instance)
    lens = np.zeros((N, S), np.int32)
    for i, l in enumerate(lens_per_instance):
        lens[i, :len(l)] = l
    nblk = (np.maximum(lens, 0) + T - 1) // T
    maxb = max(int(nblk.max()), 1)
    bt = np.full((N, S, maxb), -1, np.int32)
    pools = []
    for i in range(N):
        ids = g.permutation(NB)
        k = 0
        for s in range(S):
            bt[i, s, :nblk[i, s]] = ids[k:k + nblk[i, s]]
            k += int(nblk[i, s])
        G = int(nblk[i].sum()) * T
        KV = g.integers(0, 65536, size=(m["L"], G, m["Hkv"], 2, m["D"]), dtype=np.uint16)
        pools += oracle.kv_shard(KV, m, T, a, NB, np.maximum(lens[i], 0), bt[i], fill=0x1000 + i)
    return lens, bt, pools


def _run(m, T, N, a, NB, lens, bt, pools, options=(), layer_ranges=None, stream=None, steps=1):
    import torch

    import paper_2509_19729_b200 as A

    dev = torch.device("cuda:0")
    plan = A.amoeba_plan_create(A.make_layout(m, a, NB, block_tokens=T), A.make_layout(m, N * a, NB * N, block_tokens=T))
    for o, v in options:
        A.amoeba_plan_set_option(plan, o, v)
    d_pools = [torch.from_numpy(p.view(np.uint8).copy()).to(dev) for p in pools]
    d_bt = torch.from_numpy(bt).to(dev)
    d_lens = torch.from_numpy(lens).to(dev)
    d_new = torch.full(bt.shape, -9, dtype=torch.int32, device=dev)
    d_live = torch.full((A.amoeba_merge_live_bytes(plan),), 7, dtype=torch.uint8, device=dev)
    d_status = torch.zeros(1, dtype=torch.int32, device=dev)
    for _ in range(steps):
        A.amoeba_merge_block_tables(plan, d_bt, d_lens, bt.shape[1], bt.shape[2], d_new, d_live, d_status, stream)
        for lo, hi in (layer_ranges or [(0, m["L"])]):
            A.amoeba_merge_kv_inplace(plan, d_pools, d_live, lo, hi, d_status, stream)
    torch.cuda.synchronize()
    return ([p.cpu().numpy().view(np.uint16) for p in d_pools], d_new.cpu().numpy(),
            d_live.cpu().numpy()[:N * NB].reshape(N, NB), int(d_status.item()))


def _check(oracle, m, T, N, a, NB, lens, bt, pools, **kw):
    exp_pools = [p.copy() for p in pools]
    exp_bt, exp_live, exp_status = oracle.kv_merge_inplace(m, T, N, a, NB, lens, bt, exp_pools)
    got_pools, got_bt, got_live, got_status = _run(m, T, N, a, NB, lens, bt, pools, **kw)
    assert got_status == exp_status
    assert np.array_equal(got_bt, exp_bt)
    assert np.array_equal(got_live, exp_live)
    for w, (g, e) in enumerate(zip(got_pools, exp_pools)):
        if not np.array_equal(g, e):
            bad = np.flatnonzero(g != e)
            raise AssertionError(f"pool {w}: {bad.size} words differ, first at {bad[0]}")


LENS = [[5, 9, 1, 40], [64], [3, 3, 3], [0, 7], [33], [12, 12], [1], [80, 2]]


@pytest.mark.parametrize("path", [2, 3])
@pytest.mark.parametrize("N,a", [(2, 1), (4, 1), (8, 1), (2, 2), (4, 2), (2, 4)])
def test_merge_matches_oracle(oracle, path, N, a):
    import paper_2509_19729_b200 as A

    m, T, NB = MHA8, 4, 23
    lens, bt, pools = _instances(oracle, m, T, N, a, NB, LENS[:N], seed=N * 8 + a)
    _check(oracle, m, T, N, a, NB, lens, bt, pools, options=[(A.OPT_COPY_PATH, path)])


@pytest.mark.parametrize("chunk", [32, 256, 2048, 8192, 65536])
def test_merge_gqa_shape_and_chunk_sizes(oracle, chunk):
    """Segments of 16 KiB (2 headers of head_dim 128) cut into chunks from 16 bytes up to the whole segment."""
    import paper_2509_19729_b200 as A

    m, T, N, a, NB = GQA, 16, 4, 1, 37
    lens, bt, pools = _instances(oracle, m, T, N, a, NB, [[300, 17], [512], [1, 16, 33, 90], [250]], seed=chunk)
    _check(oracle, m, T, N, a, NB, lens, bt, pools, options=[(A.OPT_CHUNK_BYTES, chunk)])


def test_merge_all_blocks_live_and_none_live(oracle):
    m, T, N, a, NB = MHA8, 4, 4, 1, 10
    lens, bt, pools = _instances(oracle, m, T, N, a, NB, [[NB * T]] * N, seed=1)
    _check(oracle, m, T, N, a, NB, lens, bt, pools)
    lens0 = np.zeros_like(lens)
    _check(oracle, m, T, N, a, NB, lens0, bt, pools)


def test_merge_layer_ranges_and_side_stream(oracle):
    import torch

    m, T, N, a, NB = GQA, 16, 2, 2, 19
    lens, bt, pools = _instances(oracle, m, T, N, a, NB, [[100, 60], [150]], seed=6)
    _check(oracle, m, T, N, a, NB, lens, bt, pools, layer_ranges=[(0, 1), (1, 3)])
    st = torch.cuda.Stream()
    _check(oracle, m, T, N, a, NB, lens, bt, pools, stream=st)


def test_merge_twice_restores_exchanged_segments(oracle):
    """Where both blocks of a pair are live the kernel exchanges them, so a second pass over the same tables puts
    them back: with every block live in every instance all pools return to their first bytes."""
    m, T, N, a, NB = MHA8, 4, 2, 1, 6
    lens, bt, pools = _instances(oracle, m, T, N, a, NB, [[NB * T]] * N, seed=4)
    got_pools, _, _, st = _run(m, T, N, a, NB, lens, bt, pools, steps=2)
    assert st == 0
    for g, p in zip(got_pools, pools):
        assert np.array_equal(g, p)


def test_merge_device_detected_errors(oracle):
    m, T, N, a, NB = MHA8, 4, 2, 1, 9
    lens, bt, pools = _instances(oracle, m, T, N, a, NB, [[8, 4, 20], [5, 9]], seed=2)
    bad = lens.copy()
    bad[1, 0] = -3                       # whole-call error: nothing moves
    _check(oracle, m, T, N, a, NB, bad, bt, pools)
    bad = lens.copy()
    bad[0, 1] = (bt.shape[2] + 1) * T
    _check(oracle, m, T, N, a, NB, bad, bt, pools)
    bt2 = bt.copy()
    bt2[0, 0, 0] = NB                    # out of range
    bt2[0, 2, 1] = -1                    # hole inside a sequence
    bt2[1, 1, 0] = bt2[1, 1, 1]          # named twice by one instance
    _check(oracle, m, T, N, a, NB, lens, bt2, pools)


def test_merge_host_detected_errors():
    import torch

    import paper_2509_19729_b200 as A

    m, T = MHA8, 4
    dev = torch.device("cuda:0")
    z = torch.zeros(64, dtype=torch.int32, device=dev)
    live = torch.zeros(64, dtype=torch.uint8, device=dev)
    pool = [torch.zeros(1 << 16, dtype=torch.uint8, device=dev) for _ in range(4)]

    def status_of(fn):
        with pytest.raises(A.AmoebaError) as e:
            fn()
        return e.value.status

    # not a merge: destination pool is not N times the source pool, token-first order, TP not a multiple
    for src, dst in ((A.make_layout(m, 1, 8, T), A.make_layout(m, 4, 8, T)),
                     (A.make_layout(m, 1, 8, T, kv_order=1), A.make_layout(m, 4, 32, T, kv_order=1)),
                     (A.make_layout(m, 2, 8, T), A.make_layout(m, 2, 8, T))):
        plan = A.amoeba_plan_create(src, dst)
        assert status_of(lambda: A.amoeba_merge_live_bytes(plan)) == A.ERR_UNSUPPORTED
        assert status_of(lambda: A.amoeba_merge_block_tables(plan, z, z, 2, 4, z, live, z)) == A.ERR_UNSUPPORTED
        if dst.tp == 4:
            assert status_of(lambda: A.amoeba_merge_kv_inplace(plan, pool, live, 0, 1, z)) == A.ERR_UNSUPPORTED
    plan = A.amoeba_plan_create(A.make_layout(m, 1, 8, T), A.make_layout(m, 4, 32, T))
    assert A.amoeba_merge_live_bytes(plan) == 32
    assert A.amoeba_merge_bytes(plan, 10) == 2 * 10 * m["L"] * 6 * (2 * T * m["D"] * 2)
    assert status_of(lambda: A.amoeba_merge_kv_inplace(plan, pool, live, 0, 3, z)) == A.ERR_INVALID_ARG   # layers
    assert status_of(lambda: A.amoeba_merge_kv_inplace(plan, [pool[0], pool[1], pool[2], pool[0]], live, 0, 1, z)) \
        == A.ERR_INVALID_ARG                                                                            # shared pool
    assert status_of(lambda: A.amoeba_merge_kv_inplace(plan, [pool[0], pool[1], pool[2], pool[3].data_ptr() + 8],
                                                       live, 0, 1, z)) == A.ERR_ALIGNMENT
    assert status_of(lambda: A.amoeba_merge_block_tables(plan, z, z, 2, 4, z, live.data_ptr() + 4, z)) == A.ERR_ALIGNMENT
    assert status_of(lambda: A.amoeba_merge_block_tables(plan, z, z, 2, 0, z, live, z)) == A.ERR_INVALID_ARG


def test_merge_replayed_from_a_cuda_graph(oracle):
    """The merge's two calls (a memset, the table kernel, the exchange kernel) recorded into a CUDA graph: one replay
    gives the oracle's result, a second replay exchanges the live segments back where every instance holds the block."""
    import torch

    import paper_2509_19729_b200 as A

    m, T, N, a, NB = GQA, 16, 2, 1, 11
    lens, bt, pools = _instances(oracle, m, T, N, a, NB, [[100, 60], [150, 3]], seed=8)
    exp_pools = [p.copy() for p in pools]
    exp_bt, exp_live, exp_status = oracle.kv_merge_inplace(m, T, N, a, NB, lens, bt, exp_pools)
    dev = torch.device("cuda:0")
    plan = A.amoeba_plan_create(A.make_layout(m, a, NB, block_tokens=T), A.make_layout(m, N * a, NB * N, block_tokens=T))
    d_bt, d_lens = torch.from_numpy(bt).to(dev), torch.from_numpy(lens).to(dev)
    d_new = torch.full(bt.shape, -9, dtype=torch.int32, device=dev)
    d_live = torch.zeros(A.amoeba_merge_live_bytes(plan), dtype=torch.uint8, device=dev)
    d_status = torch.zeros(1, dtype=torch.int32, device=dev)
    scratch = [torch.zeros(p.size * 2, dtype=torch.uint8, device=dev) for p in pools]
    A.amoeba_merge_block_tables(plan, d_bt, d_lens, bt.shape[1], bt.shape[2], d_new, d_live, d_status)  # one-time set-up
    A.amoeba_merge_kv_inplace(plan, scratch, d_live, 0, m["L"], d_status)
    torch.cuda.synchronize()
    d_pools = [torch.from_numpy(p.view(np.uint8).copy()).to(dev) for p in pools]
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        A.amoeba_merge_block_tables(plan, d_bt, d_lens, bt.shape[1], bt.shape[2], d_new, d_live, d_status)
        A.amoeba_merge_kv_inplace(plan, d_pools, d_live, 0, m["L"], d_status)
    graph.replay()
    torch.cuda.synchronize()
    assert int(d_status.item()) == exp_status == 0
    assert np.array_equal(d_new.cpu().numpy(), exp_bt)
    for g, e in zip(d_pools, exp_pools):
        assert np.array_equal(g.cpu().numpy().view(np.uint16), e)


# ---- the way back: one instance of TP = N*a -> N instances of TP = a, in place
def _run_split(m, T, N, a, NB, lens, bt, pools):
    import torch

    import paper_2509_19729_b200 as A

    dev = torch.device("cuda:0")
    plan = A.amoeba_plan_create(A.make_layout(m, a, NB, block_tokens=T), A.make_layout(m, N * a, NB * N, block_tokens=T))
    d_pools = [torch.from_numpy(p.view(np.uint8).copy()).to(dev) for p in pools]
    d_bt, d_lens = torch.from_numpy(bt).to(dev), torch.from_numpy(lens).to(dev)
    d_old = torch.full(bt.shape, -9, dtype=torch.int32, device=dev)
    d_live = torch.full((A.amoeba_merge_live_bytes(plan),), 7, dtype=torch.uint8, device=dev)
    d_status = torch.zeros(1, dtype=torch.int32, device=dev)
    A.amoeba_split_block_tables(plan, d_bt, d_lens, bt.shape[1], bt.shape[2], d_old, d_live, d_status)
    A.amoeba_split_kv_inplace(plan, d_pools, d_live, 0, m["L"], d_status)
    torch.cuda.synchronize()
    return ([p.cpu().numpy().view(np.uint16) for p in d_pools], d_old.cpu().numpy(),
            d_live.cpu().numpy()[:N * NB].reshape(N, NB), int(d_status.item()))


def _scribble_free_blocks(m, T, N, a, NB, merged_bt, pools, seed=99):
    """Overwrite every merged-size block no table names (the merge leaves stale copies there, a running instance would
    have reused them): a split that moved a segment the wrong way would now fetch garbage."""
    g = np.random.default_rng(seed)
    used = np.zeros(NB * N, bool)
    used[merged_bt[merged_bt >= 0]] = True
    per = (m["Hkv"] // (N * a)) * 2 * T * m["D"]
    for p in pools:
        v = p.reshape(m["L"], NB * N, per)
        v[:, ~used] = g.integers(0, 65536, size=(m["L"], int((~used).sum()), per), dtype=np.uint16)


@pytest.mark.parametrize("N,a", [(2, 1), (4, 1), (2, 2), (4, 2)])
def test_split_matches_oracle(oracle, N, a):
    """Start from the oracle's merged state (so block ids have the residue of their instance), split on the GPU."""
    m, T, NB = MHA8, 4, 23
    lens, bt, pools = _instances(oracle, m, T, N, a, NB, LENS[:N], seed=N * 8 + a)
    merged_bt, _, st = oracle.kv_merge_inplace(m, T, N, a, NB, lens, bt, pools)   # pools are now the merged instance
    assert st == 0
    _scribble_free_blocks(m, T, N, a, NB, merged_bt, pools)
    exp_pools = [p.copy() for p in pools]
    exp_bt, exp_live, exp_status = oracle.kv_split_inplace(m, T, N, a, NB, lens, merged_bt, exp_pools)
    got_pools, got_bt, got_live, got_status = _run_split(m, T, N, a, NB, lens, merged_bt, pools)
    assert got_status == exp_status == 0
    assert np.array_equal(got_bt, exp_bt) and np.array_equal(got_bt, bt)
    assert np.array_equal(got_live, exp_live)
    for w, (g, e) in enumerate(zip(got_pools, exp_pools)):
        assert np.array_equal(g, e), w


def _random_instances(oracle, seed):
    g = np.random.default_rng(9100 + seed)
    Hkv = int(g.choice([2, 4, 8, 16]))
    N = int(g.choice([x for x in (2, 4, 8) if Hkv % x == 0]))
    a = int(g.choice([x for x in (1, 2, 4) if Hkv % (x * N) == 0]))
    m = dict(L=int(g.integers(1, 4)), hidden=64, Hq=Hkv, Hkv=Hkv, D=int(g.choice([16, 32, 64])), I=64 * N * a)
    T = int(g.choice([4, 8, 16]))
    lens_pi = [[int(x) for x in g.integers(0, 12 * T, size=int(g.integers(1, 6)))] for _ in range(N)]
    NB = max(sum((l + T - 1) // T for l in li) for li in lens_pi) + int(g.integers(1, 9))
    lens, bt, pools = _instances(oracle, m, T, N, a, NB, lens_pi, seed=seed)
    return g, m, T, N, a, NB, lens, bt, pools


@pytest.mark.parametrize("seed", range(24))
def test_random_merges_and_splits(oracle, seed):
    """Seeded random shapes, instance counts, worker counts, block sizes, lengths and ring shapes: the merge against the
    oracle, then - from the oracle's merged state with every unnamed block overwritten - the split back."""
    import paper_2509_19729_b200 as A

    g, m, T, N, a, NB, lens, bt, pools = _random_instances(oracle, seed)
    opts = [(A.OPT_COPY_PATH, int(g.choice([2, 3]))), (A.OPT_CHUNK_BYTES, int(g.choice([32, 256, 2048, 8192, 65536]))),
            (A.OPT_WARPS, int(g.integers(1, 8))), (A.OPT_STAGES, int(g.integers(2, 8)))]
    _check(oracle, m, T, N, a, NB, lens, bt, [p.copy() for p in pools], options=opts)
    merged_bt, _, st = oracle.kv_merge_inplace(m, T, N, a, NB, lens, bt, pools)
    assert st == 0
    _scribble_free_blocks(m, T, N, a, NB, merged_bt, pools, seed=seed)
    exp_pools = [p.copy() for p in pools]
    exp_bt, exp_live, exp_status = oracle.kv_split_inplace(m, T, N, a, NB, lens, merged_bt, exp_pools)
    got_pools, got_bt, got_live, got_status = _run_split(m, T, N, a, NB, lens, merged_bt, pools)
    assert got_status == exp_status == 0
    assert np.array_equal(got_bt, exp_bt) and np.array_equal(got_live, exp_live)
    for w, (x, e) in enumerate(zip(got_pools, exp_pools)):
        assert np.array_equal(x, e), (w, m, T, N, a, NB)


def test_split_device_detected_errors(oracle):
    m, T, N, a, NB = MHA8, 4, 2, 1, 9
    lens, bt, pools = _instances(oracle, m, T, N, a, NB, [[8, 4, 20], [5, 9]], seed=2)
    merged_bt, _, _ = oracle.kv_merge_inplace(m, T, N, a, NB, lens, bt, pools)
    _scribble_free_blocks(m, T, N, a, NB, merged_bt, pools)
    bad = merged_bt.copy()
    bad[0, 0, 0] += 1            # residue of the other instance
    bad[1, 1, 0] = NB * N        # out of range
    bad[0, 2, 1] = -1            # hole inside a sequence
    exp_pools = [p.copy() for p in pools]
    exp_bt, exp_live, exp_status = oracle.kv_split_inplace(m, T, N, a, NB, lens, bad, exp_pools)
    got_pools, got_bt, got_live, got_status = _run_split(m, T, N, a, NB, lens, bad, pools)
    assert got_status == exp_status == 5
    assert np.array_equal(got_bt, exp_bt) and np.array_equal(got_live, exp_live)
    for g, e in zip(got_pools, exp_pools):
        assert np.array_equal(g, e)
    neg = lens.copy()
    neg[1, 0] = -2
    exp_pools = [p.copy() for p in pools]
    exp_bt, exp_live, exp_status = oracle.kv_split_inplace(m, T, N, a, NB, neg, merged_bt, exp_pools)
    got_pools, got_bt, got_live, got_status = _run_split(m, T, N, a, NB, neg, merged_bt, pools)
    assert got_status == exp_status == 1 and np.array_equal(got_bt, exp_bt) and not got_live.any()
    for g, e in zip(got_pools, exp_pools):
        assert np.array_equal(g, e)


@pytest.mark.parametrize("order", ["head", "token"])
def test_out_of_place_merge_session_matches_oracle(oracle, order):
    """The benchmark's out-of-place merge plumbing on the tiny merge workload: every destination pool equals the
    oracle's a -> N*a transformation of each instance with the free list advanced by the earlier instances."""
    import torch

    import bench
    import workloads as wl

    name = "tiny_merge_2x1to2"
    cfg = wl.MERGE_CONFIGS[name]
    m, N, a, T = cfg["model"], cfg["N"], cfg["a"], wl.BLOCK_TOKENS
    so, do = bench.KV_ORDERS[order]
    s, st = bench.build_merge_copy_session(name, torch.device("cuda:0"), kv_order=order)
    s.status.zero_()
    s.step()
    torch.cuda.synchronize()
    assert int(s.status.item()) == 0
    NB_dst = s.dst_layout.num_blocks
    free = s.free_list.cpu().numpy()
    exp = [np.full(m["L"] * oracle.pool_elems_per_layer(m, T, N * a, NB_dst), 0xA5A5, np.uint16) for _ in range(N * a)]
    for i in range(N):
        src = [p.cpu().numpy().view(np.uint16) for p in s.src_pools[i]]
        exp_bt, _, n, _, status = oracle.assign_blocks(st["seq_lens"][i], T, st["src_bt"][i], st["NB"], NB_dst,
                                                       free_list=free[s.offsets[i]:])
        assert status == 0 and n == s.counts[i]
        assert np.array_equal(s.dst_bt[i].cpu().numpy(), exp_bt)
        oracle.kv_transform(m, T, st["seq_lens"][i], a, st["NB"], st["src_bt"][i], src, N * a, NB_dst, exp_bt, exp,
                            src_order=so, dst_order=do)
    for w in range(N * a):
        assert np.array_equal(s.dst_pools[w].cpu().numpy().view(np.uint16), exp[w]), w

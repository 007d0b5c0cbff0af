"""Parity of the in-place block reshaping of one instance (Sec. 3.1, Improvement 1) with the CPU oracle: every byte
of every pool (the old workers' memory and the new workers' pools, guard regions around each), the new block table,
the pair list, the free mask and count, the status word - split (TP a -> N*a) and the merge back, all copy paths."""
import numpy as np
import pytest

from harness import pairs_in_destination_order

pytestmark = pytest.mark.gpu

MHA8 = dict(L=2, hidden=64, Hq=8, Hkv=8, D=16, I=64)
GQA = dict(L=3, hidden=512, Hq=16, Hkv=8, D=128, I=1792)
FRESH = 0x3C3C
GUARD = 4096  # bytes of sentinel before and after every pool


def _coarse_instance(oracle, m, T, a, NB, lens, seed=0, ids=None):
    g = np.random.default_rng(seed)
    lens = np.asarray(lens, np.int32)
    nblk = (np.maximum(lens, 0) + T - 1) // T
    maxb = max(int(nblk.max()), 1)
    bt = np.full((len(lens), maxb), -1, np.int32)
    ids = g.permutation(NB) if ids is None else ids
    k = 0
    for s, n in enumerate(nblk):
        bt[s, :n] = ids[k:k + n]
        k += int(n)
    G = int(nblk.sum()) * T
    KV = g.integers(0, 65536, size=(m["L"], G, m["Hkv"], 2, m["D"]), dtype=np.uint16)
    pools = oracle.kv_shard(KV, m, T, a, NB, np.maximum(lens, 0), bt, fill=0x1000)
    return lens, bt, pools


def _with_fresh(old_pools, N):
    out = []
    for p in old_pools:
        out.append(p)
        out += [np.full(p.size, FRESH, np.uint16) for _ in range(N - 1)]
    return out


def _fine_instance(oracle, m, T, N, a, NB, lens, seed=0):
    """One instance at TP = N*a whose live blocks all have ids = 0 (mod N); the other blocks hold a fill."""
    g = np.random.default_rng(seed)
    lens = np.asarray(lens, np.int32)
    nblk = (lens + T - 1) // T
    bt = np.full((len(lens), max(int(nblk.max()), 1)), -1, np.int32)
    ids = g.permutation(NB) * N
    k = 0
    for s, n in enumerate(nblk):
        bt[s, :n] = ids[k:k + n]
        k += int(n)
    KV = g.integers(0, 65536, size=(m["L"], int(nblk.sum()) * T, m["Hkv"], 2, m["D"]), dtype=np.uint16)
    return lens, bt, oracle.kv_shard(KV, m, T, N * a, NB * N, lens, bt, fill=0x2222)


def _run(direction, m, T, N, a, NB, lens, bt, pools, options=(), layer_ranges=None, stream=None, pairs_cap=None):
    import torch

    import paper_2509_19729_b200 as A
    from paper_2509_19729_b200.session import ReshapeSession

    cap = bt.size if pairs_cap is None else pairs_cap
    s = ReshapeSession(m, N, a, NB, len(lens), bt.shape[1], cap, direction=direction, block_tokens=T)
    for o, v in options:
        s.set_option(o, v)
    s.set_tables(lens, bt)
    # every pool sits between two guard regions
    guarded = []
    for i, p in enumerate(pools):
        buf = torch.full((GUARD + p.nbytes + GUARD,), 0xC7, dtype=torch.uint8, device=s.device)
        buf[GUARD:GUARD + p.nbytes].copy_(torch.from_numpy(p.view(np.uint8).copy()))
        guarded.append(buf)
        s.pools[i] = buf[GUARD:GUARD + p.nbytes]
    s.reshape_block_tables(stream)
    for lo, hi in (layer_ranges or [(0, m["L"])]):
        s.reshape_kv(stream, lo, hi)
    torch.cuda.synchronize()
    for buf in guarded:
        assert bool((buf[:GUARD] == 0xC7).all()) and bool((buf[-GUARD:] == 0xC7).all())
    n = int(s.num_pairs.item())
    return dict(pools=[p.cpu().numpy().view(np.uint16) for p in s.pools], bt=s.dst_bt.cpu().numpy(),
                pairs=s.pairs.cpu().numpy(), n=n, mask=s.free_mask.cpu().numpy(), left=int(s.free_count.item()),
                status=int(s.status.item()))


def _check(oracle, direction, m, T, N, a, NB, lens, bt, pools, pairs_cap=None, **kw):
    exp_pools = [p.copy() for p in pools]
    e_bt, e_pairs, e_n, e_mask, e_left, e_status = oracle.kv_reshape_inplace(direction, m, T, N, a, NB, lens, bt,
                                                                             exp_pools, pairs_cap=pairs_cap)
    got = _run(direction, m, T, N, a, NB, lens, bt, pools, pairs_cap=pairs_cap, **kw)
    assert got["status"] == e_status
    assert np.array_equal(got["bt"], e_bt)
    assert got["n"] == e_n and np.array_equal(got["pairs"][:e_n], e_pairs)
    assert np.all(got["pairs"][e_n:] == -3)
    assert np.array_equal(got["mask"], e_mask) and got["left"] == e_left
    for w, (g, e) in enumerate(zip(got["pools"], exp_pools)):
        if not np.array_equal(g, e):
            bad = np.flatnonzero(g != e)
            raise AssertionError(f"pool {w}: {bad.size} words differ, first at {bad[0]}")


LENS = [5, 9, 0, 1, 40, 64, 3]


@pytest.mark.parametrize("path", [1, 2, 3])
@pytest.mark.parametrize("N,a", [(2, 1), (4, 1), (8, 1), (2, 2), (4, 2), (2, 4)])
def test_split_matches_oracle(oracle, path, N, a):
    import paper_2509_19729_b200 as A

    m, T, NB = MHA8, 4, 41
    lens, bt, old = _coarse_instance(oracle, m, T, a, NB, LENS, seed=N * 8 + a)
    _check(oracle, "split", m, T, N, a, NB, lens, bt, _with_fresh(old, N), options=[(A.OPT_COPY_PATH, path)])


@pytest.mark.parametrize("path", [1, 2, 3])
@pytest.mark.parametrize("N,a", [(2, 1), (4, 1), (2, 2), (4, 2)])
def test_merge_back_matches_oracle(oracle, path, N, a):
    import paper_2509_19729_b200 as A

    m, T, NB = MHA8, 4, 41
    lens, bt, pools = _fine_instance(oracle, m, T, N, a, NB, [x for x in LENS if x], seed=N * 16 + a)
    _check(oracle, "merge", m, T, N, a, NB, lens, bt, pools, options=[(A.OPT_COPY_PATH, path)])


@pytest.mark.parametrize("chunk", [32, 2048, 8192, 65536])
@pytest.mark.parametrize("direction,N,a", [("split", 4, 1), ("split", 4, 2), ("merge", 2, 2), ("merge", 8, 1)])
def test_gqa_shape_chunk_sizes_layer_ranges(oracle, direction, N, a, chunk):
    """The Llama-3-8B header geometry (8 K/V heads x 128) at a few layers: segments of 8-32 KiB cut into chunks from
    32 bytes to a whole segment, two layer ranges, a side stream."""
    import torch

    import paper_2509_19729_b200 as A

    m, T, NB = GQA, 16, 29
    lens_in = [300, 17, 1, 16, 33]
    if direction == "split":
        lens, bt, old = _coarse_instance(oracle, m, T, a, NB, lens_in, seed=chunk + N)
        pools = _with_fresh(old, N)
    else:
        lens, bt, pools = _fine_instance(oracle, m, T, N, a, NB, lens_in, seed=chunk + N)
    _check(oracle, direction, m, T, N, a, NB, lens, bt, pools, options=[(A.OPT_CHUNK_BYTES, chunk)],
           layer_ranges=[(0, 1), (1, 3)], stream=torch.cuda.Stream())


def test_split_then_merge_restores_the_instance(oracle):
    """Through the library only: split, scribble over the vacated segments, merge back - every live block is whole
    again where it was."""
    import torch

    import paper_2509_19729_b200 as A
    from paper_2509_19729_b200.session import ReshapeSession

    m, T, N, a, NB = GQA, 16, 4, 2, 23
    lens, bt, old = _coarse_instance(oracle, m, T, a, NB, [100, 60, 7], seed=9)
    sp = ReshapeSession(m, N, a, NB, len(lens), bt.shape[1], bt.size, "split", block_tokens=T)
    sp.set_tables(lens, bt)
    for i, p in enumerate(_with_fresh(old, N)):
        sp.pools[i].copy_(torch.from_numpy(p.view(np.uint8).copy()))
    sp.step()
    torch.cuda.synchronize()
    assert int(sp.status.item()) == 0
    live = torch.as_tensor(bt[bt >= 0].astype(np.int64), device=sp.device)
    for r in range(a):
        v = sp.pools[r * N].view(m["L"], NB, N, -1)
        v[:, live, 1:] = 0xEE
    mg = ReshapeSession(m, N, a, NB, len(lens), bt.shape[1], bt.size, "merge", block_tokens=T)
    mg.pools = sp.pools
    mg.seq_lens.copy_(sp.seq_lens)
    mg.src_bt.copy_(sp.dst_bt)
    mg.step()
    torch.cuda.synchronize()
    assert int(mg.status.item()) == 0 and np.array_equal(mg.dst_bt.cpu().numpy(), bt)
    per_block = (m["Hkv"] // a) * 2 * T * m["D"]
    for r in range(a):
        now = mg.pools[r * N].cpu().numpy().view(np.uint16).reshape(m["L"], NB, per_block)
        was = old[r].reshape(m["L"], NB, per_block)
        assert np.array_equal(now[:, bt[bt >= 0]], was[:, bt[bt >= 0]])


def test_reshape_errors(oracle):
    import paper_2509_19729_b200 as A

    m, T, N, a, NB = MHA8, 4, 2, 1, 12
    lens, bt, old = _coarse_instance(oracle, m, T, a, NB, [8, 4, 5, 16], seed=2)
    pools = _with_fresh(old, N)
    # whole-call errors: nothing moves
    for bad_lens, cap in (([8, -3, 5, 16], None), ([(bt.shape[1] + 1) * T, 4, 5, 16], None), ([8, 4, 5, 16], 5)):
        _check(oracle, "split", m, T, N, a, NB, np.array(bad_lens, np.int32), bt, pools, pairs_cap=cap)
    # per-block errors: out of range, a hole, an id named twice
    bt2 = bt.copy()
    bt2[0, 0] = NB
    bt2[1, 0] = -1
    bt2[2, 0] = bt2[3, 1]
    _check(oracle, "split", m, T, N, a, NB, lens, bt2, pools)
    # merge: ids that are not multiples of N
    lens_f, bt_f, pools_f = _fine_instance(oracle, m, T, N, a, NB, [8, 12], seed=5)
    bt_f2 = bt_f.copy()
    bt_f2[0, 1] += 1
    _check(oracle, "merge", m, T, N, a, NB, lens_f, bt_f2, pools_f)
    # host-side refusals
    plan = A.amoeba_plan_create(A.make_layout(m, 1, NB, block_tokens=T), A.make_layout(m, 2, NB * 2 + 1, block_tokens=T))
    with pytest.raises(A.AmoebaError) as e:
        A.amoeba_reshape_bytes(plan, 1)
    assert e.value.status == A.ERR_UNSUPPORTED
    plan = A.amoeba_plan_create(A.make_layout(m, 1, NB, block_tokens=T), A.make_layout(m, 2, NB * 2, block_tokens=T))
    with pytest.raises(A.AmoebaError) as e:  # the same pool twice
        A.amoeba_reshape_kv_inplace(plan, [4096, 4096], 4096, 4096, 4, 0, 1, 4096, stream=0)
    assert e.value.status == A.ERR_INVALID_ARG
    assert A.amoeba_reshape_bytes(plan, 3) == 2 * 3 * m["L"] * (m["Hkv"] // 2) * 2 * T * m["D"] * 2


def test_empty_and_single_block(oracle):
    m, T, N, a, NB = MHA8, 4, 4, 1, 5
    lens, bt, old = _coarse_instance(oracle, m, T, a, NB, [0, 0], seed=3)
    _check(oracle, "split", m, T, N, a, NB, lens, bt, _with_fresh(old, N))
    lens, bt, old = _coarse_instance(oracle, m, T, a, NB, [1], seed=3)
    _check(oracle, "split", m, T, N, a, NB, lens, bt, _with_fresh(old, N))


def test_large_tables_take_the_two_launch_path(oracle):
    """A table of 600 rows x 260 columns (> 128 Ki entries) next to a 1000-block row: scan and assign as two launches."""
    m, T, N, a = dict(L=1, hidden=32, Hq=4, Hkv=4, D=8, I=32), 4, 2, 1
    g = np.random.default_rng(8)
    lens_in = np.concatenate([[1040], g.integers(0, 40, size=599)]).astype(np.int32)
    NB = int(((lens_in + T - 1) // T).sum()) + 50
    lens, bt, old = _coarse_instance(oracle, m, T, a, NB, lens_in, seed=8)
    assert bt.size > 128 * 1024
    _check(oracle, "split", m, T, N, a, NB, lens, bt, _with_fresh(old, N))


@pytest.mark.parametrize("seed", range(10))
def test_random_reshapes_with_layer_strides(oracle, seed):
    """Random factor, TP degree, lengths, direction, copy path, item size and a layer stride larger than a dense
    layer: every byte of every (strided) pool, the words between the layers included."""
    import torch

    import paper_2509_19729_b200 as A

    g = np.random.default_rng(1000 + seed)
    m = dict(L=3, hidden=64, Hq=16, Hkv=16, D=16, I=256)
    T = int(g.choice([4, 8, 16]))
    N = int(g.choice([2, 4, 8]))
    a = int(g.choice([x for x in (1, 2, 4, 8) if x * N <= 16]))
    direction = str(g.choice(["split", "merge"]))
    lens = g.integers(0 if direction == "split" else 1, 12 * T, size=int(g.integers(1, 9))).astype(np.int32)
    NB = int(((lens + T - 1) // T).sum()) + int(g.integers(1, 9))
    dense = oracle.pool_elems_per_layer(m, T, a, NB)
    stride = dense + 8 * int(g.integers(0, 40))  # elements; a multiple of 16 bytes
    if direction == "split":
        lens, bt, old = _coarse_instance(oracle, m, T, a, NB, lens, seed=seed)
        dense_pools = _with_fresh(old, N)
    else:
        lens, bt, dense_pools = _fine_instance(oracle, m, T, N, a, NB, lens, seed=seed)
    pools = []
    for w, p in enumerate(dense_pools):
        q = np.full(m["L"] * stride, 0x7000 + w, np.uint16)
        q.reshape(m["L"], stride)[:, :dense] = p.reshape(m["L"], dense)
        pools.append(q)
    exp = [p.copy() for p in pools]
    e_bt, e_pairs, e_n, e_mask, e_left, e_status = oracle.kv_reshape_inplace(direction, m, T, N, a, NB, lens, bt, exp,
                                                                             layer_stride=stride)
    coarse = A.make_layout(m, a, NB, T, kv_layer_stride_bytes=stride * 2)
    fine = A.make_layout(m, N * a, NB * N, T, kv_layer_stride_bytes=stride * 2)
    plan = A.amoeba_plan_create(*((coarse, fine) if direction == "split" else (fine, coarse)))
    A.amoeba_plan_set_option(plan, A.OPT_COPY_PATH, int(g.choice([1, 2, 3])))
    A.amoeba_plan_set_option(plan, A.OPT_CHUNK_BYTES, int(g.choice([64, 512, 8192])))
    by_destination = seed % 2 == 1  # half the seeds ask for the pair list in destination order
    if by_destination:
        A.amoeba_plan_set_option(plan, A.OPT_PAIR_ORDER, A.PAIR_ORDER_DESTINATION)
    dev = torch.device("cuda:0")
    i32 = dict(dtype=torch.int32, device=dev)
    d_pools = [torch.from_numpy(p.view(np.uint8).copy()).to(dev) for p in pools]
    d_bt, d_lens = torch.from_numpy(bt).to(dev), torch.from_numpy(lens).to(dev)
    d_new = torch.full(bt.shape, -2, **i32)
    d_pairs = torch.full((bt.size, 2), -3, **i32)
    d_n, d_left, d_status = torch.zeros(1, **i32), torch.zeros(1, **i32), torch.zeros(1, **i32)
    d_mask = torch.full((NB * N if direction == "split" else NB,), 7, dtype=torch.uint8, device=dev)
    ws_bytes = A.amoeba_rewrite_workspace_bytes(plan, len(lens), 0)
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device=dev)
    A.amoeba_reshape_block_tables(plan, d_bt, d_lens, len(lens), bt.shape[1], d_new, d_pairs, bt.size, d_n, d_mask,
                                  d_left, d_status, ws, ws_bytes)
    A.amoeba_reshape_kv_inplace(plan, d_pools, d_pairs, d_n, bt.size, 0, m["L"], d_status)
    torch.cuda.synchronize()
    assert int(d_status.item()) == e_status == 0
    assert np.array_equal(d_new.cpu().numpy(), e_bt) and int(d_n.item()) == e_n and int(d_left.item()) == e_left
    assert np.array_equal(d_pairs.cpu().numpy()[:e_n],
                          pairs_in_destination_order(e_pairs, e_bt, lens, T) if by_destination else e_pairs)
    assert np.array_equal(d_mask.cpu().numpy(), e_mask)
    for w, (t, e) in enumerate(zip(d_pools, exp)):
        assert np.array_equal(t.cpu().numpy().view(np.uint16), e), (w, direction, N, a, T)

"""Pins for the oracle's in-place block reshaping of ONE instance (Sec. 3.1, Improvement 1): TP = a -> TP = N*a on the
instance's own memory plus fresh pools for the new workers, and the way back.  No GPU, no CUDA library.

What fixes the functions from outside themselves: the paper's worked example (H = 8, TP4: the headers split
H1-2 / H3-4 / H5-6 / H7-8 over W1..W4); a closed form written with numpy reshapes; the reconstruction invariant
through the independent shard / reconstruct functions; equality with the out-of-place transformation on every word
that moves; and what must NOT change (the old workers' memory, every block no table names)."""
import numpy as np
import pytest

MHA8 = dict(L=2, hidden=32, Hq=8, Hkv=8, D=4, I=32)
GQA = dict(L=2, hidden=32, Hq=16, Hkv=4, D=4, I=32)
FRESH = 0x3C3C


def _instance(oracle, m, T, a, NB, lens, seed=0, layer_stride=None):
    g = np.random.default_rng(seed)
    lens = np.asarray(lens, np.int32)
    nblk = (lens + T - 1) // T
    maxb = max(int(nblk.max()), 1)
    bt = np.full((len(lens), maxb), -1, np.int32)
    ids = g.permutation(NB)
    k = 0
    for s, n in enumerate(nblk):
        bt[s, :n] = ids[k:k + n]
        k += int(n)
    G = int(nblk.sum()) * T
    KV = g.integers(0, 65536, size=(m["L"], G, m["Hkv"], 2, m["D"]), dtype=np.uint16)
    pools = oracle.kv_shard(KV, m, T, a, NB, lens, bt, fill=0x1000, layer_stride=layer_stride)
    return lens, bt, KV, pools


def _with_fresh(old_pools, N):
    """pools[w] of the TP = N*a side: old worker r at r*N, fresh pools (same size) elsewhere."""
    out = []
    for p in old_pools:
        out.append(p)
        out += [np.full(p.size, FRESH, np.uint16) for _ in range(N - 1)]
    return out


@pytest.mark.parametrize("m,N,a", [(MHA8, 4, 1), (MHA8, 2, 2), (MHA8, 4, 2), (GQA, 2, 1), (GQA, 2, 2), (GQA, 4, 1)])
def test_split_reconstructs_and_moves_only_what_leaves(oracle, m, N, a):
    T, NB = 4, 12
    lens, bt, KV, old = _instance(oracle, m, T, a, NB, [5, 9, 0, 1, 13], seed=N * 8 + a)
    before = [p.copy() for p in old]
    pools = _with_fresh(old, N)
    new_bt, pairs, n, free_mask, left, st = oracle.kv_reshape_inplace("split", m, T, N, a, NB, lens, bt, pools)
    assert st == 0
    live = bt[bt >= 0]
    # table: p -> p*N, padding stays -1; pairs in (sequence, block) order; free ids = everything but the p*N
    assert np.array_equal(new_bt[bt >= 0], live * N) and np.all(new_bt[bt < 0] == -1)
    assert n == live.size and np.array_equal(pairs, np.stack([live, live * N], 1))
    assert np.array_equal(np.flatnonzero(free_mask == 0), np.sort(live * N)) and left == NB * N - live.size
    for p in live:
        assert all(free_mask[p * N + k] == 1 for k in range(1, N))  # the segments the migrated headers left
    # the instance's logical KV reads back from the N*a pools through the independent reconstruct
    assert np.array_equal(oracle.kv_reconstruct(pools, m, T, N * a, NB * N, lens, new_bt), KV)
    # the memory of the old workers is untouched, bit for bit and address for address (retained headers do not
    # move, vacated segments keep stale words)
    for r in range(a):
        assert np.array_equal(pools[r * N], before[r])
    # the same blocks as the out-of-place a -> N*a transformation writes into fresh pools
    fresh = [np.full(p.size, 0xEEEE, np.uint16) for p in pools]
    oracle.kv_transform(m, T, lens, a, NB, bt, before, N * a, NB * N, new_bt, fresh)
    seg = (m["Hkv"] // (N * a)) * 2 * T * m["D"]
    used = np.zeros(NB * N, bool)
    used[live * N] = True
    for w in range(N * a):
        now = pools[w].reshape(m["L"], NB * N, seg)
        assert np.array_equal(now[:, used], fresh[w].reshape(m["L"], NB * N, seg)[:, used])
        if w % N:  # a fresh pool: nothing but the live new blocks was written
            assert np.all(now[:, ~used] == FRESH)


@pytest.mark.parametrize("N,a", [(4, 1), (2, 2)])
def test_split_closed_form(oracle, N, a):
    """new pool r*N+k, viewed [L][NB*N][segment], holds at block p*N what old pool r, viewed [L][NB][N][segment],
    holds at (p, k)."""
    m, T, NB = MHA8, 4, 6
    lens, bt, KV, old = _instance(oracle, m, T, a, NB, [NB * T], seed=3)
    before = [p.copy() for p in old]
    pools = _with_fresh(old, N)
    *_, st = oracle.kv_reshape_inplace("split", m, T, N, a, NB, lens, bt, pools)
    assert st == 0
    seg = (m["Hkv"] // (N * a)) * 2 * T * m["D"]
    for r in range(a):
        was = before[r].reshape(m["L"], NB, N, seg)
        for k in range(N):
            now = pools[r * N + k].reshape(m["L"], NB, N, seg)  # block p*N = (p, slot 0)
            assert np.array_equal(now[:, :, 0], was[:, :, k])


def test_paper_example_h8_tp4_from_one_worker(oracle):
    """TP1 -> TP4 with H = 8 (the partition of Sec. 3.1's example): the old worker becomes W1 and keeps H1,H2 where
    they are; H3,H4 / H5,H6 / H7,H8 of every live block end on W2 / W3 / W4 at block p*4."""
    m, T, NB, N = MHA8, 4, 5, 4
    lens, bt, KV, old = _instance(oracle, m, T, 1, NB, [8, 7], seed=5)
    before = old[0].copy()
    pools = _with_fresh(old, N)
    new_bt, *_ , st = oracle.kv_reshape_inplace("split", m, T, N, 1, NB, lens, bt, pools)
    assert st == 0
    unit = 2 * T * m["D"]
    was = before.reshape(m["L"], NB, 8, unit)  # [layer][block][header][words]
    for p in bt[bt >= 0]:
        assert np.array_equal(pools[0].reshape(m["L"], NB, 8, unit)[:, p, 0:2], was[:, p, 0:2])
        for w in (1, 2, 3):
            got = pools[w].reshape(m["L"], NB * 4, 2, unit)[:, p * 4]
            assert np.array_equal(got, was[:, p, 2 * w:2 * w + 2])
            first, last = oracle.header_range(8, 4, w + 1)
            assert (first, last) == (2 * w + 1, 2 * w + 2)


@pytest.mark.parametrize("m,N,a", [(MHA8, 4, 1), (MHA8, 2, 2), (GQA, 2, 2)])
def test_merge_back_undoes_split(oracle, m, N, a):
    T, NB = 4, 8
    lens, bt, KV, old = _instance(oracle, m, T, a, NB, [5, 9, 1, 0, 6], seed=17)
    before = [p.copy() for p in old]
    pools = _with_fresh(old, N)
    new_bt, *_ = oracle.kv_reshape_inplace("split", m, T, N, a, NB, lens, bt, pools)
    for r in range(a):  # scribble over the vacated segments: the merge must bring the headers back from the others
        v = pools[r * N].reshape(m["L"], NB, N, -1)
        v[:, bt[bt >= 0], 1:] = 0xDEAD
    fresh_before = [p.copy() for p in pools]
    back_bt, pairs, n, free_mask, left, st = oracle.kv_reshape_inplace("merge", m, T, N, a, NB, lens, new_bt, pools)
    assert st == 0 and np.array_equal(back_bt, bt)
    live = bt[bt >= 0]
    assert np.array_equal(pairs, np.stack([live * N, live], 1))
    assert np.array_equal(np.flatnonzero(free_mask == 0), np.sort(live)) and left == NB - live.size
    per_block = (m["Hkv"] // a) * 2 * T * m["D"]
    for r in range(a):
        now = pools[r * N].reshape(m["L"], NB, per_block)
        was = before[r].reshape(m["L"], NB, per_block)
        assert np.array_equal(now[:, live], was[:, live])  # every live block is whole again, where it was
        dead = np.setdiff1d(np.arange(NB), live)
        assert np.array_equal(now[:, dead], was[:, dead])
        for k in range(1, N):  # the other workers' memory is only read
            assert np.array_equal(pools[r * N + k], fresh_before[r * N + k])
    assert np.array_equal(oracle.kv_reconstruct([pools[r * N] for r in range(a)], m, T, a, NB, lens, back_bt), KV)


def test_merge_equals_out_of_place_transformation(oracle):
    m, T, N, a, NB = GQA, 4, 2, 1, 7
    g = np.random.default_rng(4)
    lens = np.array([9, 4, 0, 7], np.int32)
    nblk = (lens + T - 1) // T
    bt = np.full((4, int(nblk.max())), -1, np.int32)
    ids = g.permutation(NB) * N  # ids = 0 (mod N)
    k = 0
    for s, nb in enumerate(nblk):
        bt[s, :nb] = ids[k:k + nb]
        k += int(nb)
    KV = g.integers(0, 65536, size=(m["L"], int(nblk.sum()) * T, m["Hkv"], 2, m["D"]), dtype=np.uint16)
    pools = oracle.kv_shard(KV, m, T, N * a, NB * N, lens, bt, fill=0x4444)
    before = [p.copy() for p in pools]
    new_bt, *_, st = oracle.kv_reshape_inplace("merge", m, T, N, a, NB, lens, bt, pools)
    assert st == 0
    fresh = [np.full(before[0].size, 0xEEEE, np.uint16)]
    oracle.kv_transform(m, T, lens, N * a, NB * N, bt, before, a, NB, new_bt, fresh)
    per_block = m["Hkv"] * 2 * T * m["D"]
    live = new_bt[new_bt >= 0]
    assert np.array_equal(pools[0].reshape(m["L"], NB, per_block)[:, live], fresh[0].reshape(m["L"], NB, per_block)[:, live])


def test_reshape_error_cases(oracle):
    m, T, N, a, NB = MHA8, 4, 2, 1, 6
    lens, bt, KV, old = _instance(oracle, m, T, a, NB, [8, 4, 5], seed=2)
    pools = _with_fresh(old, N)
    before = [p.copy() for p in pools]
    # whole-call errors: nothing moves
    for bad_lens, cap in (([8, -3, 5], None), ([(bt.shape[1] + 1) * T, 4, 5], None), ([8, 4, 5], 4)):
        new_bt, pairs, n, fm, left, st = oracle.kv_reshape_inplace("split", m, T, N, a, NB, bad_lens, bt, pools,
                                                                   pairs_cap=cap)
        assert st == oracle.INVALID_ARG and np.all(new_bt == -1) and n == 0 and np.all(fm == 1) and left == NB * N
        assert all(np.array_equal(p, q) for p, q in zip(pools, before))
    # per-block errors: out of range, a hole, an id named twice -> those entries -1, the others move
    bt2 = bt.copy()
    dup = int(bt2[0, 1])
    bt2[0, 0] = NB
    bt2[1, 0] = -1
    bt2[2, 0] = dup
    new_bt, pairs, n, fm, left, st = oracle.kv_reshape_inplace("split", m, T, N, a, NB, lens, bt2, pools)
    assert st == oracle.BAD_BLOCK_ID and n == 5
    assert new_bt[0, 0] == -1 and new_bt[1, 0] == -1 and new_bt[2, 0] == -1 and new_bt[0, 1] == dup * N
    assert [tuple(p) for p in pairs[[0, 2, 3]]] == [(-1, -1)] * 3 and tuple(pairs[1]) == (dup, dup * N)
    assert left == NB * N - 2
    # merge: an id that is not a multiple of N cannot be reshaped back
    lens_m = np.array([8], np.int32)
    bt_m = np.array([[4, 5]], np.int32)
    pools_m = [np.zeros(m["L"] * NB * N * 4 * 2 * T * m["D"], np.uint16) for _ in range(N)]
    new_bt, pairs, n, fm, left, st = oracle.kv_reshape_inplace("merge", m, T, N, a, NB, lens_m, bt_m, pools_m)
    assert st == oracle.BAD_BLOCK_ID and list(new_bt[0]) == [2, -1] and left == NB - 1
    # sticky status
    *_, st = oracle.kv_reshape_inplace("split", m, T, N, a, NB, lens, bt, [p.copy() for p in before], status=9)
    assert st == 9


def test_reshape_with_a_layer_stride(oracle):
    m, T, N, a, NB = dict(GQA, L=3), 4, 2, 2, 7
    dense = oracle.pool_elems_per_layer(m, T, a, NB)
    stride = dense + 40
    lens, bt, KV, old_d = _instance(oracle, m, T, a, NB, [5, 9, 1], seed=23)
    _, _, _, old_s = _instance(oracle, m, T, a, NB, [5, 9, 1], seed=23, layer_stride=stride)
    pd, ps = _with_fresh(old_d, N), _with_fresh(old_s, N)
    rd = oracle.kv_reshape_inplace("split", m, T, N, a, NB, lens, bt, pd)
    rs = oracle.kv_reshape_inplace("split", m, T, N, a, NB, lens, bt, ps, layer_stride=stride)
    assert rs[5] == 0 and np.array_equal(rd[0], rs[0]) and np.array_equal(rd[3], rs[3])
    for x, y in zip(pd, ps):
        v = y.reshape(m["L"], stride)
        assert np.array_equal(v[:, :dense], x.reshape(m["L"], dense))
    for w in range(N * a):
        if w % N:
            assert np.all(ps[w].reshape(m["L"], stride)[:, dense:] == FRESH)
    assert np.array_equal(oracle.kv_reconstruct(ps, m, T, N * a, NB * N, lens, rs[0], layer_stride=stride), KV)

"""Pins for the oracle's in-place merge of N instances (Sec. 3.1, Improvement 1: in-place migration with the
header-centric layout and block reshaping).  No GPU, no CUDA library.

What fixes the function from outside itself: the paper's worked example (H = 8, TP4: W2 retains H3,H4 and sends
H1-2 / H5-6 / H7-8 to W1 / W3 / W4); a closed form (with every block live the merge is a transposition of the
(instance, segment) axes, written with numpy); the reconstruction invariant through the independent shard /
reconstruct functions; equality with the out-of-place transformation; and what must NOT change."""
import numpy as np
import pytest

MHA8 = dict(L=2, hidden=32, Hq=8, Hkv=8, D=4, I=32)


def _instances(oracle, m, T, N, a, NB, lens_per_instance, seed=0):
    """N independent instances at TP=a: logical KV, block tables over each instance's own pool, pools."""
    g = np.random.default_rng(seed)
    S = max(len(l) for l in lens_per_instance)
    lens = np.zeros((N, S), np.int32)
    for i, l in enumerate(lens_per_instance):
        lens[i, :len(l)] = l
    nblk = (lens + T - 1) // T
    maxb = max(int(nblk.max()), 1)
    bt = np.full((N, S, maxb), -1, np.int32)
    KVs, pools = [], []
    for i in range(N):
        ids = g.permutation(NB)
        k = 0
        for s in range(S):
            bt[i, s, :nblk[i, s]] = ids[k:k + nblk[i, s]]
            k += int(nblk[i, s])
        G = int(nblk[i].sum()) * T
        KV = g.integers(0, 65536, size=(m["L"], G, m["Hkv"], 2, m["D"]), dtype=np.uint16)
        KVs.append(KV)
        pools += oracle.kv_shard(KV, m, T, a, NB, lens[i], bt[i], fill=0x1000 + i)  # worker r of instance i
    return lens, bt, KVs, pools


def _merged_order(pools, N, a):
    """pools[i*a + r] is worker r*N+i of the merged instance: the list in merged-worker order."""
    return [pools[(w % N) * a + (w // N)] for w in range(N * a)]


@pytest.mark.parametrize("N,a", [(4, 1), (2, 1), (2, 2), (4, 2)])
def test_merged_state_reconstructs_every_instance(oracle, N, a):
    m, T, NB = MHA8, 4, 9
    lens, bt, KVs, pools = _instances(oracle, m, T, N, a, NB, [[5, 9, 1], [16], [3, 3, 3, 3][:3], [0, 7]][:N], seed=N * 8 + a)
    new_bt, live, st = oracle.kv_merge_inplace(m, T, N, a, NB, lens, bt, pools)
    assert st == 0
    merged = _merged_order(pools, N, a)
    for i in range(N):
        assert np.array_equal(new_bt[i][bt[i] >= 0], bt[i][bt[i] >= 0] * N + i)
        assert np.all(new_bt[i][bt[i] < 0] == -1)
        back = oracle.kv_reconstruct(merged, m, T, N * a, NB * N, lens[i], new_bt[i])
        assert np.array_equal(back, KVs[i])
        assert np.array_equal(np.flatnonzero(live[i]), np.sort(bt[i][bt[i] >= 0]))
    # the new tables of different instances never name the same block
    used = np.concatenate([new_bt[i][new_bt[i] >= 0] for i in range(N)])
    assert len(set(used.tolist())) == used.size


@pytest.mark.parametrize("N,a", [(4, 1), (2, 2)])
def test_all_live_merge_is_a_transposition(oracle, N, a):
    """Every block of every instance live: old pool (i, r) viewed [L][NB][N segments][...] and new pool (k, r) viewed
    the same way satisfy new[k][.., p, i] = old[i][.., p, k] - a swap of the (instance, segment) axes."""
    m, T, NB = MHA8, 4, 6
    lens, bt, KVs, pools = _instances(oracle, m, T, N, a, NB, [[NB * T]] * N, seed=3)
    old = np.stack([np.stack([pools[i * a + r].copy() for r in range(a)]) for i in range(N)])  # [i][r][words]
    _, _, st = oracle.kv_merge_inplace(m, T, N, a, NB, lens, bt, pools)
    assert st == 0
    new = np.stack([np.stack([pools[i * a + r] for r in range(a)]) for i in range(N)])
    seg = (m["Hkv"] // (N * a)) * 2 * T * m["D"]
    old = old.reshape(N, a, m["L"], NB, N, seg)   # [instance][rank][layer][block][segment][words]
    new = new.reshape(N, a, m["L"], NB, N, seg)
    assert np.array_equal(new, old.transpose(4, 1, 2, 3, 0, 5))


def test_paper_example_w2_retains_h3_h4(oracle):
    """4 x TP1 -> TP4 with H = 8 (Sec. 3.1): W2 keeps H3,H4 of its own requests where they are, and receives H3,H4
    of the other workers' requests; H1,H2 / H5,H6 / H7,H8 of its requests end on W1 / W3 / W4."""
    m, T, NB, N = MHA8, 4, 5, 4
    lens, bt, KVs, pools = _instances(oracle, m, T, N, 1, NB, [[8], [7, 4], [12], [2]], seed=5)
    before = [p.copy() for p in pools]
    new_bt, live, st = oracle.kv_merge_inplace(m, T, N, 1, NB, lens, bt, pools)
    unit = 2 * T * m["D"]                       # one (block, header)
    L = m["L"]
    W2 = 1                                      # 0-indexed instance / worker
    old2 = before[W2].reshape(L, NB, 8, unit)   # [layer][block][header][words]
    for p in bt[W2][bt[W2] >= 0]:
        # retained in place: H3,H4 (0-indexed headers 2,3) at the same words of W2's memory
        assert np.array_equal(pools[W2].reshape(L, NB, 8, unit)[:, p, 2:4], old2[:, p, 2:4])
        # sent: header group g of the block now sits on worker g, block p*4 + 1, as its 2 local headers
        for gw in (0, 2, 3):
            got = pools[gw].reshape(L, NB * 4, 2, unit)[:, p * 4 + W2]
            assert np.array_equal(got, old2[:, p, 2 * gw:2 * gw + 2])
    # received: H3,H4 of every other worker's live blocks
    for other in (0, 2, 3):
        oldo = before[other].reshape(L, NB, 8, unit)
        for p in bt[other][bt[other] >= 0]:
            assert np.array_equal(pools[W2].reshape(L, NB * 4, 2, unit)[:, p * 4 + other], oldo[:, p, 2:4])


def test_merge_equals_out_of_place_transformation_and_leaves_the_rest_alone(oracle):
    m, T, NB, N, a = MHA8, 4, 8, 2, 2
    lens, bt, KVs, pools = _instances(oracle, m, T, N, a, NB, [[6, 5], [9]], seed=11)
    before = [p.copy() for p in pools]
    new_bt, live, st = oracle.kv_merge_inplace(m, T, N, a, NB, lens, bt, pools)
    assert st == 0
    merged = _merged_order(pools, N, a)
    # the same blocks written by the out-of-place a -> N*a transformation of each instance into fresh pools
    fresh = [np.full(p.size, 0xEEEE, np.uint16) for p in merged]
    for i in range(N):
        oracle.kv_transform(m, T, lens[i], a, NB, bt[i], before[i * a:(i + 1) * a], N * a, NB * N, new_bt[i], fresh)
    written = [f != 0xEEEE for f in fresh]  # random words: a written word equals the marker with probability 2^-16
    for w in range(N * a):
        assert np.array_equal(merged[w][written[w]], fresh[w][written[w]])
    # words of the merged pools that belong to no live new block keep what they held
    per_new_block = (m["Hkv"] // (N * a)) * 2 * T * m["D"]
    for i in range(N):
        for r in range(a):
            now = pools[i * a + r].reshape(m["L"], NB * N, per_new_block)
            was = before[i * a + r].reshape(m["L"], NB * N, per_new_block)
            used = np.zeros(NB * N, bool)
            for j in range(N):
                used[new_bt[j][new_bt[j] >= 0]] = True
            assert np.array_equal(now[:, ~used], was[:, ~used])


def test_merge_error_cases(oracle):
    m, T, NB, N, a = MHA8, 4, 6, 2, 1
    lens, bt, KVs, pools = _instances(oracle, m, T, N, a, NB, [[8, 4], [5]], seed=2)
    before = [p.copy() for p in pools]
    # negative length: whole-call error, nothing moves
    bad = lens.copy()
    bad[1, 0] = -3
    new_bt, live, st = oracle.kv_merge_inplace(m, T, N, a, NB, bad, bt, pools)
    assert st == oracle.INVALID_ARG and np.all(new_bt == -1) and not live.any()
    assert all(np.array_equal(p, q) for p, q in zip(pools, before))
    # a sequence that needs more blocks than the table has columns
    bad = lens.copy()
    bad[0, 0] = (bt.shape[2] + 1) * T
    _, _, st = oracle.kv_merge_inplace(m, T, N, a, NB, bad, bt, pools)
    assert st == oracle.INVALID_ARG and all(np.array_equal(p, q) for p, q in zip(pools, before))
    # an id out of range and a hole inside a sequence: those blocks stay, the others move
    bt2 = bt.copy()
    good = int(bt2[0, 0, 1])
    bt2[0, 0, 0] = NB
    bt2[0, 1, 0] = -1
    new_bt, live, st = oracle.kv_merge_inplace(m, T, N, a, NB, lens, bt2, pools)
    assert st == oracle.BAD_BLOCK_ID
    assert new_bt[0, 0, 0] == -1 and new_bt[0, 1, 0] == -1 and new_bt[0, 0, 1] == good * N
    assert live[0].sum() == 1 and live[0, good] == 1
    # sticky status
    _, _, st = oracle.kv_merge_inplace(m, T, N, a, NB, lens, bt, [p.copy() for p in before], status=7)
    assert st == 7


def test_merge_decode_attention_unchanged(oracle):
    """One decode step of attention for instance 1's requests gives the same bits from its TP1 pools before the
    merge and from the merged TP2 pools after it (read through the block tables of each state)."""
    m, T, NB, N = dict(L=1, hidden=16, Hq=4, Hkv=4, D=8, I=16), 4, 6, 2
    g = np.random.default_rng(9)
    S = 2
    lens = np.array([[7, 3], [10, 0]], np.int32)
    nblk = (lens + T - 1) // T
    maxb = int(nblk.max())
    bt = np.full((N, S, maxb), -1, np.int32)
    KVs, pools = [], []
    import workloads as wl

    for i in range(N):
        ids = g.permutation(NB)
        k = 0
        for s in range(S):
            bt[i, s, :nblk[i, s]] = ids[k:k + nblk[i, s]]
            k += int(nblk[i, s])
        G = int(nblk[i].sum()) * T
        KV = wl.to_bits(g.standard_normal((1, G, 4, 2, 8)).astype(np.float32), "fp16")
        KVs.append(KV)
        pools += oracle.kv_shard(KV, m, T, 1, NB, lens[i], bt[i], fill=0)

    def attend(KV, lens_i, q):
        out, g0 = [], 0
        for s, n in enumerate(lens_i):
            kv = wl.from_bits(KV[0, g0:g0 + n], "fp16").astype(np.float32)  # [n][H][2][D]
            g0 += ((n + T - 1) // T) * T
            for h in range(4):
                sc = (kv[:, h, 0] @ q[s, h]) / np.float32(np.sqrt(8.0))
                w = np.exp(sc - sc.max()) if n else sc
                out.append((w / w.sum()) @ kv[:, h, 1] if n else np.zeros(8, np.float32))
        return np.array(out, np.float32)

    q = g.standard_normal((S, 4, 8)).astype(np.float32)
    ref = attend(KVs[1], lens[1], q)
    new_bt, _, st = oracle.kv_merge_inplace(m, T, N, 1, NB, lens, bt, pools)
    assert st == 0
    back = oracle.kv_reconstruct(pools, m, T, N, NB * N, lens[1], new_bt[1])
    assert np.array_equal(attend(back, lens[1], q).view(np.uint32), ref.view(np.uint32))


# ---------------- the way back: one instance of TP = N*a -> N instances of TP = a, in place ----------------
def _merged_instance(oracle, m, T, N, a, NB, lens_per_group, seed=0):
    """One instance at TP = N*a whose requests are already grouped by the instance they will go to: group i's blocks
    have ids = i (mod N).  Returns lens [N][S], bt [N][S][maxb], the logical KV of each group, and the pools in the
    order pools[i*a + r] = merged worker r*N+i."""
    g = np.random.default_rng(seed)
    S = max(len(l) for l in lens_per_group)
    lens = np.zeros((N, S), np.int32)
    for i, l in enumerate(lens_per_group):
        lens[i, :len(l)] = l
    nblk = (lens + T - 1) // T
    maxb = max(int(nblk.max()), 1)
    bt = np.full((N, S, maxb), -1, np.int32)
    merged = [np.full(m["L"] * oracle.pool_elems_per_layer(m, T, N * a, NB * N), 0x2000 + w, np.uint16)
              for w in range(N * a)]
    KVs = []
    for i in range(N):
        ids = g.permutation(NB) * N + i
        k = 0
        for s in range(S):
            bt[i, s, :nblk[i, s]] = ids[k:k + nblk[i, s]]
            k += int(nblk[i, s])
        G = int(nblk[i].sum()) * T
        KV = g.integers(0, 65536, size=(m["L"], G, m["Hkv"], 2, m["D"]), dtype=np.uint16)
        KVs.append(KV)
        part = oracle.kv_shard(KV, m, T, N * a, NB * N, lens[i], bt[i], fill=0)
        where = oracle.kv_shard(np.full_like(KV, 1), m, T, N * a, NB * N, lens[i], bt[i], fill=0)  # 1 = written word
        for w in range(N * a):
            merged[w][where[w] != 0] = part[w][where[w] != 0]
    pools = [None] * (N * a)
    for w in range(N * a):
        pools[(w % N) * a + (w // N)] = merged[w]
    return lens, bt, KVs, pools


@pytest.mark.parametrize("N,a", [(4, 1), (2, 1), (2, 2)])
def test_split_gives_every_instance_all_headers_of_its_requests(oracle, N, a):
    m, T, NB = MHA8, 4, 7
    lens, bt, KVs, pools = _merged_instance(oracle, m, T, N, a, NB, [[5, 9], [16], [3, 3, 3], [7]][:N], seed=N + a)
    old_bt, live, st = oracle.kv_split_inplace(m, T, N, a, NB, lens, bt, pools)
    assert st == 0
    for i in range(N):
        assert np.array_equal(old_bt[i][bt[i] >= 0], bt[i][bt[i] >= 0] // N)
        back = oracle.kv_reconstruct(pools[i * a:(i + 1) * a], m, T, a, NB, lens[i], old_bt[i])
        assert np.array_equal(back, KVs[i])
        assert np.array_equal(np.flatnonzero(live[i]), np.sort(old_bt[i][old_bt[i] >= 0]))


@pytest.mark.parametrize("N,a", [(4, 1), (2, 2)])
def test_split_undoes_merge_and_merge_undoes_split(oracle, N, a):
    m, T, NB = MHA8, 4, 9
    lens, bt, KVs, pools = _instances(oracle, m, T, N, a, NB, [[5, 9, 1], [16], [3, 3, 3], [0, 7]][:N], seed=21)
    first = [p.copy() for p in pools]
    new_bt, live_m, st = oracle.kv_merge_inplace(m, T, N, a, NB, lens, bt, pools)
    assert st == 0
    old_bt, live_s, st = oracle.kv_split_inplace(m, T, N, a, NB, lens, new_bt, pools)
    assert st == 0 and np.array_equal(old_bt, bt) and np.array_equal(live_s, live_m)
    per_block = (m["Hkv"] // a) * 2 * T * m["D"]
    for i in range(N):
        for r in range(a):
            now = pools[i * a + r].reshape(m["L"], NB, per_block)
            was = first[i * a + r].reshape(m["L"], NB, per_block)
            assert np.array_equal(now[:, live_m[i] != 0], was[:, live_m[i] != 0])  # every live block is back, whole


def test_split_rejects_blocks_of_the_wrong_residue(oracle):
    m, T, N, a, NB = MHA8, 4, 2, 1, 5
    lens, bt, KVs, pools = _merged_instance(oracle, m, T, N, a, NB, [[8], [4, 4]], seed=3)
    before = [p.copy() for p in pools]
    bad = bt.copy()
    good = int(bad[0, 0, 1])
    bad[0, 0, 0] = int(bad[0, 0, 0]) + 1           # an id = 1 (mod 2) in the rows of instance 0
    bad[1, 1, 0] = NB * N                          # out of range
    old_bt, live, st = oracle.kv_split_inplace(m, T, N, a, NB, lens, bad, pools)
    assert st == oracle.BAD_BLOCK_ID
    assert old_bt[0, 0, 0] == -1 and old_bt[1, 1, 0] == -1 and old_bt[0, 0, 1] == good // N
    assert live[0].sum() == 1 and live[1].sum() == 1
    neg = lens.copy()
    neg[0, 0] = -1
    pools2 = [p.copy() for p in before]
    old_bt, live, st = oracle.kv_split_inplace(m, T, N, a, NB, neg, bt, pools2)
    assert st == oracle.INVALID_ARG and np.all(old_bt == -1) and not live.any()
    assert all(np.array_equal(p, q) for p, q in zip(pools2, before))


# ---------------- layer stride of the in-place merge and split ----------------
@pytest.mark.parametrize("N,a", [(4, 1), (2, 2)])
def test_inplace_merge_and_split_with_a_layer_stride(oracle, N, a):
    """Pools whose layers are `stride` elements apart: layer l of the result sits at l*stride and equals layer l of
    the dense result; the words between layers keep their values; and the split brings every live block back."""
    m, T, NB = dict(MHA8, L=3), 4, 7
    lens, bt, KVs, dense_pools = _instances(oracle, m, T, N, a, NB, [[5, 9, 1], [16], [3, 3, 3], [0, 7]][:N], seed=31)
    dense = oracle.pool_elems_per_layer(m, T, a, NB)
    stride = dense + 56
    strided = []
    for w, p in enumerate(dense_pools):
        q = np.full(m["L"] * stride, 0x7000 + w, np.uint16)
        q.reshape(m["L"], stride)[:, :dense] = p.reshape(m["L"], dense)
        strided.append(q)
    first = [q.copy() for q in strided]
    bt_d, live_d, st = oracle.kv_merge_inplace(m, T, N, a, NB, lens, bt, dense_pools)
    assert st == 0
    bt_s, live_s, st = oracle.kv_merge_inplace(m, T, N, a, NB, lens, bt, strided, layer_stride=stride)
    assert st == 0 and np.array_equal(bt_s, bt_d) and np.array_equal(live_s, live_d)
    for w in range(N * a):
        v = strided[w].reshape(m["L"], stride)
        assert np.array_equal(v[:, :dense], dense_pools[w].reshape(m["L"], dense))
        assert np.all(v[:, dense:] == 0x7000 + w)
    # every instance's logical KV can be read back from the strided merged pools through the independent reconstruct
    merged = _merged_order(strided, N, a)
    for i in range(N):
        back = oracle.kv_reconstruct(merged, m, T, N * a, NB * N, lens[i], bt_s[i], layer_stride=stride)
        assert np.array_equal(back, KVs[i])
    old_bt, _, st = oracle.kv_split_inplace(m, T, N, a, NB, lens, bt_s, strided, layer_stride=stride)
    assert st == 0 and np.array_equal(old_bt, bt)
    per_block = (m["Hkv"] // a) * 2 * T * m["D"]
    for i in range(N):
        for r in range(a):
            now = strided[i * a + r].reshape(m["L"], stride)
            was = first[i * a + r].reshape(m["L"], stride)
            live = live_d[i] != 0
            assert np.array_equal(now[:, :dense].reshape(m["L"], NB, per_block)[:, live],
                                  was[:, :dense].reshape(m["L"], NB, per_block)[:, live])
            assert np.array_equal(now[:, dense:], was[:, dense:])

"""Pins for the CPU oracle: the paper's worked example, the stated storage order, library-routine special cases,
round trips, Eq. 1, and the decode-attention invariant.  No GPU, no CUDA library."""
import itertools
import os

import numpy as np
import pytest

import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")

SMALL = dict(L=2, hidden=16, Hq=8, Hkv=4, D=4, I=24)


def _state(seq_lens, T, NB, seed=1):
    g = np.random.default_rng(seed)
    nblk = (np.asarray(seq_lens) + T - 1) // T
    maxb = max(int(nblk.max()), 1)
    ids = g.permutation(NB)
    bt = np.full((len(seq_lens), maxb), -1, dtype=np.int32)
    k = 0
    for s, n in enumerate(nblk):
        bt[s, :n] = ids[k:k + n]
        k += n
    return bt, nblk


# ---------------- head partition (Sec. 3.1) ----------------
def test_worked_example_h8_tp4(oracle):
    rows = [l.split() for l in open(os.path.join(GOLDEN, "head_partition_example.txt")) if not l.startswith("#")]
    assert len(rows) == 4
    for H, TP, w, first, last in (map(int, r) for r in rows):
        assert oracle.header_range(H, TP, w) == (first, last)
        for h in range(first, last + 1):
            assert oracle.worker_of_header(H, TP, h) == w
    # W2 retains H3,H4 and sends H1,H2 -> W1; H5,H6 -> W3; H7,H8 -> W4
    assert [oracle.worker_of_header(8, 4, h) for h in range(1, 9)] == [1, 1, 2, 2, 3, 3, 4, 4]


@pytest.mark.parametrize("H,TP", [(8, 1), (8, 2), (8, 8), (40, 5), (40, 8), (32, 4)])
def test_partition_is_even_and_exact(oracle, H, TP):
    owners = [oracle.worker_of_header(H, TP, h) for h in range(1, H + 1)]
    assert sorted(set(owners)) == list(range(1, TP + 1))
    assert all(owners.count(w) == H // TP for w in range(1, TP + 1))
    assert owners == sorted(owners)  # contiguous ranges in worker order


# ---------------- storage order [Block, Header, K/V, Token] (Sec. 3.1, Improvement 1) ----------------
@pytest.mark.parametrize("TP", [1, 2, 4])
def test_memory_order_is_block_header_kv_token(oracle, TP):
    m, T, NB = SMALL, 4, 7
    seq_lens = [5, 0, 9, 4]
    bt, nblk = _state(seq_lens, T, NB)
    G = int(nblk.sum()) * T
    n = m["L"] * G * m["Hkv"] * 2 * m["D"]
    assert n < 65535
    KV = np.arange(n, dtype=np.uint16).reshape(m["L"], G, m["Hkv"], 2, m["D"])  # stamp = logical linear index
    FILL = 0xFFFF
    pools = oracle.kv_shard(KV, m, T, TP, NB, seq_lens, bt, fill=FILL)
    Hs = m["Hkv"] // TP
    blk_elems = Hs * 2 * T * m["D"]
    # logical block -> (sequence-local) table
    tok_block = {}  # global token -> physical block
    g0 = 0
    for s, nb in enumerate(nblk):
        for t in range(nb * T):
            tok_block[g0 + t] = (bt[s, t // T], t % T)
        g0 += nb * T
    seen = 0
    for r, pool in enumerate(pools):
        assert pool.size == m["L"] * NB * blk_elems
        written = np.flatnonzero(pool != FILL)
        seen += written.size
        stamps = pool[written].astype(np.int64)
        l, g, h, c, d = np.unravel_index(stamps, KV.shape)
        blk = np.array([tok_block[x][0] for x in g])
        tok = np.array([tok_block[x][1] for x in g])
        # memory order == lexicographic order of (layer, block, header, K/V, token, dim)
        keys = np.stack([l, blk, h, c, tok, d], axis=1)
        order = np.lexsort(keys.T[::-1])
        assert np.array_equal(order, np.arange(len(order)))
        # the worker holds exactly its own headers (0-indexed form of the 1-indexed range)
        first, last = oracle.header_range(m["Hkv"], TP, r + 1)
        assert set(np.unique(h)) == set(range(first - 1, last))
        # every live block is one dense segment starting at (layer*NB + block) * block size
        for ll, bb in set(zip(l.tolist(), blk.tolist())):
            lo = (ll * NB + bb) * blk_elems
            seg = pool[lo:lo + blk_elems]
            assert np.all(seg != FILL)
            # and inside it each header's K then V, T tokens each, is one compact run
            hh, cc = np.unravel_index(seg.astype(np.int64), KV.shape)[2:4]
            assert np.array_equal(hh, np.repeat(np.arange(first - 1, last), 2 * T * m["D"]))
            assert np.array_equal(cc, np.tile(np.repeat([0, 1], T * m["D"]), Hs))
    assert seen == n  # every logical element stored exactly once across the workers


# ---------------- special case: TP shards are numpy splits along the head axis ----------------
@pytest.mark.parametrize("TP", [1, 2, 4])
def test_kv_shard_equals_numpy_split(oracle, TP):
    m, T, NB = SMALL, 4, 9
    seq_lens = [7, 3, 0, 16, 1]
    bt, nblk = _state(seq_lens, T, NB, seed=3)
    G = int(nblk.sum()) * T
    KV = np.random.default_rng(0).integers(0, 65536, size=(m["L"], G, m["Hkv"], 2, m["D"]), dtype=np.uint16)
    pools = oracle.kv_shard(KV, m, T, TP, NB, seq_lens, bt, fill=0)
    parts = np.split(KV, TP, axis=2)
    Hs = m["Hkv"] // TP
    for r in range(TP):
        pool = pools[r].reshape(m["L"], NB, Hs, 2, T, m["D"])
        g0 = 0
        for s, nb in enumerate(nblk):
            for i in range(nb):
                blk_logical = parts[r][:, g0 + i * T:g0 + (i + 1) * T]  # [L, T, Hs, 2, D]
                assert np.array_equal(pool[:, bt[s, i]], blk_logical.transpose(0, 2, 3, 1, 4))
            g0 += nb * T


# ---------------- invariant (i): reconstruct(shard(X)) == X ----------------
@pytest.mark.parametrize("Hkv,TP", [(4, 1), (4, 2), (4, 4), (40, 5), (40, 8), (40, 20)])
def test_reconstruct_inverts_shard(oracle, Hkv, TP):
    m = dict(SMALL, Hkv=Hkv, Hq=Hkv)
    T, NB = 4, 11
    seq_lens = [9, 4, 0, 13]
    bt, nblk = _state(seq_lens, T, NB, seed=5)
    G = int(nblk.sum()) * T
    KV = np.random.default_rng(1).integers(0, 65536, size=(m["L"], G, Hkv, 2, m["D"]), dtype=np.uint16)
    pools = oracle.kv_shard(KV, m, T, TP, NB, seq_lens, bt)
    assert np.array_equal(oracle.kv_reconstruct(pools, m, T, TP, NB, seq_lens, bt), KV)


# ---------------- invariant (ii): a -> b -> a is the identity ----------------
@pytest.mark.parametrize("a,b", [(2, 1), (1, 4), (4, 2), (2, 4), (4, 4)])
def test_round_trip_identity(oracle, a, b):
    m, T = SMALL, 4
    seq_lens = [9, 4, 0, 13, 2]
    NB_a, NB_b = 10, 13
    bt_a, nblk = _state(seq_lens, T, NB_a, seed=7)
    G = int(nblk.sum()) * T
    KV = np.random.default_rng(2).integers(0, 65536, size=(m["L"], G, m["Hkv"], 2, m["D"]), dtype=np.uint16)
    pools_a = oracle.kv_shard(KV, m, T, a, NB_a, seq_lens, bt_a)
    free_b = np.random.default_rng(3).permutation(NB_b).astype(np.int32)
    bt_b, pairs, N, left, st = oracle.assign_blocks(seq_lens, T, bt_a, NB_a, NB_b, free_list=free_b)
    assert st == 0 and N == nblk.sum() and left == NB_b - N
    pools_b = [np.full(m["L"] * oracle.pool_elems_per_layer(m, T, b, NB_b), 0xA5A5, np.uint16) for _ in range(b)]
    oracle.kv_transform(m, T, seq_lens, a, NB_a, bt_a, pools_a, b, NB_b, bt_b, pools_b)
    # logical content survives
    assert np.array_equal(oracle.kv_reconstruct(pools_b, m, T, b, NB_b, seq_lens, bt_b), KV)
    # it equals a direct shard of the logical state for TP=b
    direct = oracle.kv_shard(KV, m, T, b, NB_b, seq_lens, bt_b)
    for x, y in zip(pools_b, direct):
        assert np.array_equal(x, y)
    # return trip with the original ids, in original order, as the free list: physical bytes identical
    back_free = bt_a[bt_a >= 0]
    bt_a2, _, N2, _, st2 = oracle.assign_blocks(seq_lens, T, bt_b, NB_b, NB_a, free_list=back_free)
    assert st2 == 0 and np.array_equal(bt_a2, bt_a)
    pools_a2 = [np.full_like(p, 0xA5A5) for p in pools_a]
    oracle.kv_transform(m, T, seq_lens, b, NB_b, bt_b, pools_b, a, NB_a, bt_a2, pools_a2)
    for x, y in zip(pools_a2, pools_a):
        assert np.array_equal(x, y)


def test_same_tp_identity_free_list_copies_used_blocks(oracle):
    m, T, NB = SMALL, 4, 9
    seq_lens = [5, 8, 3]
    bt, nblk = _state(seq_lens, T, NB, seed=11)
    G = int(nblk.sum()) * T
    KV = np.random.default_rng(4).integers(0, 65536, size=(m["L"], G, m["Hkv"], 2, m["D"]), dtype=np.uint16)
    src = oracle.kv_shard(KV, m, T, 2, NB, seq_lens, bt)
    dst_bt, pairs, N, _, st = oracle.assign_blocks(seq_lens, T, bt, NB, NB, free_list=bt[bt >= 0])
    assert st == 0 and np.array_equal(dst_bt, bt) and np.array_equal(pairs[:, 0], pairs[:, 1])
    dst = [np.full_like(p, 0xA5A5) for p in src]
    oracle.kv_copy_pairs(m, T, 2, NB, src, 2, NB, dst, pairs, N)
    for x, y in zip(src, dst):
        assert np.array_equal(x, y)


def test_copy_pairs_matches_transform(oracle):
    m, T = SMALL, 4
    seq_lens = [9, 0, 13, 2]
    NB_a, NB_b = 8, 12
    bt_a, nblk = _state(seq_lens, T, NB_a, seed=13)
    G = int(nblk.sum()) * T
    KV = np.random.default_rng(5).integers(0, 65536, size=(m["L"], G, m["Hkv"], 2, m["D"]), dtype=np.uint16)
    for a, b in [(1, 4), (4, 2), (2, 1)]:
        src = oracle.kv_shard(KV, m, T, a, NB_a, seq_lens, bt_a)
        mask = np.ones(NB_b, np.uint8)
        mask[[1, 5]] = 0
        bt_b, pairs, N, left, st = oracle.assign_blocks(seq_lens, T, bt_a, NB_a, NB_b, free_mask=mask)
        assert st == 0 and left == 10 - N
        d1 = [np.full(m["L"] * oracle.pool_elems_per_layer(m, T, b, NB_b), 0xA5A5, np.uint16) for _ in range(b)]
        d2 = [x.copy() for x in d1]
        oracle.kv_transform(m, T, seq_lens, a, NB_a, bt_a, src, b, NB_b, bt_b, d1)
        assert oracle.kv_copy_pairs(m, T, a, NB_a, src, b, NB_b, d2, pairs, N) == 0
        for x, y in zip(d1, d2):
            assert np.array_equal(x, y)
        # occupied (foreign) blocks 1 and 5 were never touched
        for p in d1:
            v = p.reshape(m["L"], NB_b, -1)
            assert np.all(v[:, [1, 5]] == 0xA5A5)


# ---------------- invariant (iii): decode-step attention from resharded KV == from unsharded KV ----------------
def test_decode_attention_invariant_tiny(oracle):
    cfg = wl.CONFIGS["tiny_2to1"]
    m, T = cfg["model"], wl.BLOCK_TOKENS
    st = wl.draw_kv_state(cfg, name="tiny_2to1")
    seq_lens, src_bt = st["seq_lens"], st["src_bt"]
    G = int(st["blocks_per_seq"].sum()) * T
    KV = wl.draw_kv_logical(cfg, G, range(m["L"]))
    a, b = cfg["a"], cfg["b"]
    src = oracle.kv_shard(KV, m, T, a, st["NB_src"], seq_lens, src_bt)
    dst_bt, pairs, N, _, status = oracle.assign_blocks(seq_lens, T, src_bt, st["NB_src"], st["NB_dst"],
                                                       free_list=st["dst_free_list"])
    assert status == 0
    dst = [np.full(m["L"] * oracle.pool_elems_per_layer(m, T, b, st["NB_dst"]), 0xA5A5, np.uint16) for _ in range(b)]
    oracle.kv_transform(m, T, seq_lens, a, st["NB_src"], src_bt, src, b, st["NB_dst"], dst_bt, dst)

    q = wl.rng(7, "q").standard_normal(size=(m["L"], len(seq_lens), m["Hq"], m["D"])).astype(np.float32)
    group = m["Hq"] // m["Hkv"]

    def attend(K, V, qv):  # fixed-order fp32 decode attention on contiguous [len, D] arrays
        s = (K.astype(np.float32) @ qv) / np.float32(np.sqrt(m["D"]))
        p = np.exp(s - s.max())
        return (p / p.sum()) @ V.astype(np.float32)

    def from_logical(l, s, j):
        g0 = int(st["blocks_per_seq"][:s].sum()) * T
        h = j // group
        x = KV[l, g0:g0 + seq_lens[s], h]  # [len, 2, D]
        return np.ascontiguousarray(x[:, 0]), np.ascontiguousarray(x[:, 1])

    def from_pools(pools, TP, NB, bt, l, s, j):
        h = j // group
        Hs = m["Hkv"] // TP
        pool = pools[h // Hs].reshape(m["L"], NB, Hs, 2, T, m["D"])  # strides the attention kernel would be given
        blocks = bt[s, :st["blocks_per_seq"][s]]
        x = pool[l, blocks, h % Hs]  # [nblk, 2, T, D]
        K = x[:, 0].reshape(-1, m["D"])[:seq_lens[s]]
        V = x[:, 1].reshape(-1, m["D"])[:seq_lens[s]]
        return np.ascontiguousarray(K), np.ascontiguousarray(V)

    f16 = lambda w: w.view(np.float16)
    for l, s, j in itertools.product(range(m["L"]), range(len(seq_lens)), range(m["Hq"])):
        K0, V0 = from_logical(l, s, j)
        ref = attend(f16(K0), f16(V0), q[l, s, j])
        for pools, TP, NB, bt in ((src, a, st["NB_src"], src_bt), (dst, b, st["NB_dst"], dst_bt)):
            K1, V1 = from_pools(pools, TP, NB, bt, l, s, j)
            out = attend(f16(K1), f16(V1), q[l, s, j])
            assert np.array_equal(out.view(np.uint32), ref.view(np.uint32))


# ---------------- weights ----------------
def _rand_weights(m, seed=0):
    g = np.random.default_rng(seed)
    import oracle as o
    return {n: g.integers(0, 65536, size=s, dtype=np.uint16) for n, s in o.logical_shapes(m).items()}


@pytest.mark.parametrize("fq,fg", [(True, True), (False, False), (True, False)])
@pytest.mark.parametrize("TP", [1, 2, 4])
def test_weight_shards_are_numpy_splits(oracle, TP, fq, fg):
    m = SMALL
    W = _rand_weights(m)
    sh = oracle.weights_shard(W, m, TP, fq, fg)
    for r in range(TP):
        q, k, v = (np.split(W[n], TP, axis=0)[r] for n in "qkv")
        gate, up = (np.split(W[n], TP, axis=0)[r] for n in ("gate", "up"))
        if fq:
            assert np.array_equal(sh[r]["q"], np.concatenate([q, k, v], axis=0))
        else:
            assert all(np.array_equal(sh[r][n], x) for n, x in zip("qkv", (q, k, v)))
        if fg:
            assert np.array_equal(sh[r]["gate"], np.concatenate([gate, up], axis=0))
        else:
            assert np.array_equal(sh[r]["gate"], gate) and np.array_equal(sh[r]["up"], up)
        assert np.array_equal(sh[r]["o"], np.split(W["o"], TP, axis=1)[r])
        assert np.array_equal(sh[r]["down"], np.split(W["down"], TP, axis=1)[r])
    if TP == 1 and not fq and not fg:
        assert all(np.array_equal(sh[0][n], W[n]) for n in W)  # TP1 unfused shard is the logical tensor
    back = oracle.weights_reconstruct(sh, m, TP, fq, fg)
    assert all(np.array_equal(back[n], W[n]) for n in W)


@pytest.mark.parametrize("a,b", [(1, 2), (2, 1), (4, 1), (1, 4), (2, 4), (4, 2)])
def test_weight_transform_round_trip(oracle, a, b):
    m = SMALL
    W = _rand_weights(m, seed=3)
    sa = oracle.weights_shard(W, m, a)
    sb = oracle.weights_transform(sa, m, a, b)
    direct = oracle.weights_shard(W, m, b)
    for x, y in zip(sb, direct):
        assert all(np.array_equal(x[n], y[n]) for n in x)
    sa2 = oracle.weights_transform(sb, m, b, a)
    for x, y in zip(sa2, sa):
        assert all(np.array_equal(x[n], y[n]) for n in x)


@pytest.mark.parametrize("TP", [1, 2, 4])
def test_eq1_ffn_sum_over_shards(oracle, TP):
    """Eq. 1: FFN = f(I x U) x D; with U split by columns and D by rows the shard results add up to it."""
    cfg = dict(model=SMALL, dtype="bf16")
    m = SMALL
    Wb = wl.draw_weights_logical(cfg, 0, std=0.5)
    sh = oracle.weights_shard(Wb, m, TP, fused_qkv=True, fused_gate_up=False)
    F = lambda w: wl.from_bits(w, "bf16")
    x = np.random.default_rng(9).standard_normal((3, m["hidden"]))
    f = lambda z: z / (1.0 + np.exp(-z))
    # storage is [out,in]: the paper's U is up^T, its D is down^T
    full = f(x @ F(Wb["up"]).T) @ F(Wb["down"]).T
    parts = sum(f(x @ F(s["up"]).T) @ F(s["down"]).T for s in sh)
    assert np.allclose(parts, full, rtol=1e-12, atol=1e-12)
    # gated form used by the Llama-shaped configs
    full_g = (f(x @ F(Wb["gate"]).T) * (x @ F(Wb["up"]).T)) @ F(Wb["down"]).T
    parts_g = sum((f(x @ F(s["gate"]).T) * (x @ F(s["up"]).T)) @ F(s["down"]).T for s in sh)
    assert np.allclose(parts_g, full_g, rtol=1e-12, atol=1e-12)
    # attention projections split by heads: q rows per head, o columns per head
    D, Hq, Hkv = m["D"], m["Hq"], m["Hkv"]
    ctx = np.random.default_rng(10).standard_normal((3, Hq * D))  # per-head attention outputs, concatenated
    full_o = ctx @ F(Wb["o"]).T
    parts_o = sum(np.split(ctx, TP, axis=1)[r] @ F(sh[r]["o"]).T for r in range(TP))
    assert np.allclose(parts_o, full_o, rtol=1e-12, atol=1e-12)
    qr, kr = Hq * D // TP, Hkv * D // TP
    full_q = x @ F(Wb["q"]).T
    cat_q = np.concatenate([x @ F(s["q"][:qr]).T for s in sh], axis=1)
    assert np.array_equal(cat_q, full_q)
    cat_v = np.concatenate([x @ F(s["q"][qr + kr:]).T for s in sh], axis=1)
    assert np.array_equal(cat_v, x @ F(Wb["v"]).T)


# ---------------- destination block bookkeeping ----------------
def test_assign_blocks_closed_forms(oracle):
    T = 16
    for seed in range(5):
        g = np.random.default_rng(seed)
        S = int(g.integers(1, 9))
        seq_lens = g.integers(0, 100, size=S)
        NB_src = 64
        bt, nblk = _state(seq_lens, T, NB_src, seed=seed)
        N = int(nblk.sum())
        NB_dst = N + 5
        free = g.permutation(NB_dst).astype(np.int32)
        dst_bt, pairs, n, left, st = oracle.assign_blocks(seq_lens, T, bt, NB_src, NB_dst, free_list=free)
        assert st == 0 and n == N and left == NB_dst - N
        assert np.array_equal(dst_bt[bt >= 0], free[:N])  # row-major valid entries == prefix of the free list
        assert np.all(dst_bt[bt < 0] == -1)
        assert np.array_equal(pairs[:, 0], bt[bt >= 0]) and np.array_equal(pairs[:, 1], free[:N])
        mask = (g.random(NB_dst + 40) < 0.6).astype(np.uint8)
        mask[:N] = 1
        dst_bt, pairs, n, left, st = oracle.assign_blocks(seq_lens, T, bt, NB_src, len(mask), free_mask=mask)
        assert st == 0 and left == int(mask.sum()) - N
        assert np.array_equal(pairs[:, 1], np.flatnonzero(mask)[:N])  # ascending ids of the set bytes


def test_assign_blocks_errors(oracle):
    T, NB = 16, 32
    seq_lens = [40, 16, 0]
    bt, nblk = _state(seq_lens, T, NB)
    N = int(nblk.sum())
    free = np.arange(N - 1, dtype=np.int32)
    dst_bt, pairs, n, left, st = oracle.assign_blocks(seq_lens, T, bt, NB, NB, free_list=free)
    assert st == oracle.NO_FREE_BLOCKS and n == 0 and left == N - 1 and np.all(dst_bt == -1)
    free = np.arange(N, dtype=np.int32)
    *_, st = oracle.assign_blocks([40, -1, 0], T, bt, NB, NB, free_list=free)
    assert st == oracle.INVALID_ARG
    *_, st = oracle.assign_blocks([40, 16, 0], T, bt, NB, NB, free_list=free, pairs_cap=N - 1)
    assert st == oracle.INVALID_ARG
    *_, st = oracle.assign_blocks([40, 16, 0], T, bt, NB, NB, free_list=free, status=9)
    assert st == 9  # sticky
    bad = free.copy()
    bad[1] = NB
    dst_bt, pairs, n, left, st = oracle.assign_blocks(seq_lens, T, bt, NB, NB, free_list=bad)
    assert st == oracle.BAD_BLOCK_ID and n == N and dst_bt[0, 1] == -1 and tuple(pairs[1]) == (-1, -1)
    bt2 = bt.copy()
    bt2[1, 0] = -1
    dst_bt, pairs, n, left, st = oracle.assign_blocks(seq_lens, T, bt2, NB, NB, free_list=free)
    assert st == oracle.BAD_BLOCK_ID and dst_bt[1, 0] == free[3] and tuple(pairs[3]) == (-1, -1)


# ---------------- the input generators are reproducible and shaped as stated ----------------
def test_workload_generators():
    for name, cfg in wl.CONFIGS.items():
        lens = wl.draw_seq_lens(cfg, name=name)
        assert len(lens) == cfg["S"] and np.array_equal(lens, wl.draw_seq_lens(cfg, name=name))
        assert lens.min() >= 1
    cfg = wl.CONFIGS["llama3_70b_slice_8to2"]
    lens = wl.draw_seq_lens(cfg, name="x")
    assert lens[0] == 131072 and lens[1:].max() <= 2048 and lens[1:].min() >= 256
    st = wl.draw_kv_state(wl.CONFIGS["llama2_13b_4to1"], name="c3")
    live = st["src_bt"][st["src_bt"] >= 0]
    assert len(np.unique(live)) == st["n_live"] == len(live)
    assert 0.28 < 1 - st["n_live"] / st["NB_src"] < 0.32
    assert int(st["dst_free_mask"].sum()) >= st["n_live"]
    x = np.array([1.0, -2.5, 3.1415926, 1e-3], dtype=np.float32)
    assert np.allclose(wl.from_bits(wl.to_bits(x, "bf16"), "bf16"), x, rtol=2 ** -8)
    assert np.allclose(wl.from_bits(wl.to_bits(x, "fp16"), "fp16"), x, rtol=2 ** -10)


# ---------------- token-first storage order (Sec. 3.1: the mainstream-engine layout the paper starts from) ----------------
@pytest.mark.parametrize("TP", [1, 2, 4])
def test_token_first_memory_order_and_two_regions(oracle, TP):
    m, T, NB = SMALL, 4, 7
    seq_lens = [5, 0, 9, 4]
    bt, nblk = _state(seq_lens, T, NB)
    G = int(nblk.sum()) * T
    n = m["L"] * G * m["Hkv"] * 2 * m["D"]
    KV = np.arange(n, dtype=np.uint16).reshape(m["L"], G, m["Hkv"], 2, m["D"])
    FILL = 0xFFFF
    pools = oracle.kv_shard(KV, m, T, TP, NB, seq_lens, bt, fill=FILL, order=oracle.TOKEN_FIRST)
    Hs = m["Hkv"] // TP
    region = NB * T * Hs * m["D"]  # one of K / V for one layer
    tok_block = {}
    g0 = 0
    for s, nb in enumerate(nblk):
        for t in range(nb * T):
            tok_block[g0 + t] = (bt[s, t // T], t % T)
        g0 += nb * T
    seen = 0
    for r, pool in enumerate(pools):
        assert pool.size == m["L"] * 2 * region
        written = np.flatnonzero(pool != FILL)
        seen += written.size
        l, g, h, c, d = np.unravel_index(pool[written].astype(np.int64), KV.shape)
        blk = np.array([tok_block[x][0] for x in g])
        tok = np.array([tok_block[x][1] for x in g])
        # memory order == lexicographic order of (layer, K/V, block, token, header, dim)
        keys = np.stack([l, c, blk, tok, h, d], axis=1)
        assert np.array_equal(np.lexsort(keys.T[::-1]), np.arange(len(keys)))
        # K and V live in two separate contiguous regions of each layer
        assert np.array_equal(c, (written // region) % 2)
        assert np.array_equal(l, written // (2 * region))
        # a token's headers are stored together: Hs*D consecutive words share (block, token)
        runs = (written // (Hs * m["D"]))
        for run in np.unique(runs)[:50]:
            sel = runs == run
            assert len(set(zip(blk[sel].tolist(), tok[sel].tolist(), c[sel].tolist()))) == 1 and sel.sum() == Hs * m["D"]
    assert seen == n


@pytest.mark.parametrize("TP", [1, 2, 4])
def test_token_first_equals_numpy_split(oracle, TP):
    m, T, NB = SMALL, 4, 9
    seq_lens = [7, 3, 0, 16, 1]
    bt, nblk = _state(seq_lens, T, NB, seed=3)
    G = int(nblk.sum()) * T
    KV = np.random.default_rng(0).integers(0, 65536, size=(m["L"], G, m["Hkv"], 2, m["D"]), dtype=np.uint16)
    pools = oracle.kv_shard(KV, m, T, TP, NB, seq_lens, bt, fill=0, order=oracle.TOKEN_FIRST)
    parts = np.split(KV, TP, axis=2)
    Hs = m["Hkv"] // TP
    for r in range(TP):
        pool = pools[r].reshape(m["L"], 2, NB, T, Hs, m["D"])
        g0 = 0
        for s, nb in enumerate(nblk):
            for i in range(nb):
                blk_logical = parts[r][:, g0 + i * T:g0 + (i + 1) * T]  # [L, T, Hs, 2, D]
                assert np.array_equal(pool[:, :, bt[s, i]], blk_logical.transpose(0, 3, 1, 2, 4))
            g0 += nb * T
    assert np.array_equal(oracle.kv_reconstruct(pools, m, T, TP, NB, seq_lens, bt, order=oracle.TOKEN_FIRST), KV)


@pytest.mark.parametrize("a,b,so,do", [(1, 4, 1, 1), (4, 2, 1, 1), (2, 2, 1, 0), (2, 4, 0, 1), (4, 1, 1, 0), (1, 2, 0, 1)])
def test_storage_order_conversions_round_trip(oracle, a, b, so, do):
    m, T = SMALL, 4
    seq_lens = [9, 4, 0, 13, 2]
    NB_a, NB_b = 10, 13
    bt_a, nblk = _state(seq_lens, T, NB_a, seed=7)
    G = int(nblk.sum()) * T
    KV = np.random.default_rng(2).integers(0, 65536, size=(m["L"], G, m["Hkv"], 2, m["D"]), dtype=np.uint16)
    pools_a = oracle.kv_shard(KV, m, T, a, NB_a, seq_lens, bt_a, order=so)
    free_b = np.random.default_rng(3).permutation(NB_b).astype(np.int32)
    bt_b, pairs, N, left, st = oracle.assign_blocks(seq_lens, T, bt_a, NB_a, NB_b, free_list=free_b)
    pools_b = [np.full(m["L"] * oracle.pool_elems_per_layer(m, T, b, NB_b), 0xA5A5, np.uint16) for _ in range(b)]
    oracle.kv_transform(m, T, seq_lens, a, NB_a, bt_a, pools_a, b, NB_b, bt_b, pools_b, src_order=so, dst_order=do)
    direct = oracle.kv_shard(KV, m, T, b, NB_b, seq_lens, bt_b, order=do)
    for x, y in zip(pools_b, direct):
        assert np.array_equal(x, y)
    via_pairs = [np.full_like(p, 0xA5A5) for p in pools_b]
    assert oracle.kv_copy_pairs(m, T, a, NB_a, pools_a, b, NB_b, via_pairs, pairs, N, src_order=so, dst_order=do) == 0
    for x, y in zip(pools_b, via_pairs):
        assert np.array_equal(x, y)
    # back again with the original ids: physical bytes identical
    bt_a2, _, _, _, st2 = oracle.assign_blocks(seq_lens, T, bt_b, NB_b, NB_a, free_list=bt_a[bt_a >= 0])
    back = [np.full_like(p, 0xA5A5) for p in pools_a]
    oracle.kv_transform(m, T, seq_lens, b, NB_b, bt_b, pools_b, a, NB_a, bt_a2, back, src_order=do, dst_order=so)
    for x, y in zip(back, pools_a):
        assert np.array_equal(x, y)


def test_decode_attention_from_token_first_strides(oracle):
    """The same decode-step attention, read through the token-first strides, gives the same bits."""
    cfg = wl.CONFIGS["tiny_2to1"]
    m, T = cfg["model"], wl.BLOCK_TOKENS
    st = wl.draw_kv_state(cfg, name="tiny_2to1")
    seq_lens, bt = st["seq_lens"], st["src_bt"]
    G = int(st["blocks_per_seq"].sum()) * T
    KV = wl.draw_kv_logical(cfg, G, range(m["L"]))
    TP, NB = 2, st["NB_src"]
    Hs = m["Hkv"] // TP
    tf = oracle.kv_shard(KV, m, T, TP, NB, seq_lens, bt, order=oracle.TOKEN_FIRST)
    hc = oracle.kv_shard(KV, m, T, TP, NB, seq_lens, bt, order=oracle.HEADER_CENTRIC)
    q = wl.rng(7, "q").standard_normal(size=(m["D"],)).astype(np.float32)

    def attend(K, V):
        s = (K.view(np.float16).astype(np.float32) @ q) / np.float32(np.sqrt(m["D"]))
        p = np.exp(s - s.max())
        return (p / p.sum()) @ V.view(np.float16).astype(np.float32)

    for l, s, h in itertools.product(range(m["L"]), range(len(seq_lens)), range(m["Hkv"])):
        blocks = bt[s, :st["blocks_per_seq"][s]]
        a_tf = tf[h // Hs].reshape(m["L"], 2, NB, T, Hs, m["D"])[l][:, blocks][:, :, :, h % Hs]  # [2, nblk, T, D]
        a_hc = hc[h // Hs].reshape(m["L"], NB, Hs, 2, T, m["D"])[l, blocks, h % Hs]        # [nblk, 2, T, D]
        n = seq_lens[s]
        K1, V1 = (np.ascontiguousarray(a_tf[c].reshape(-1, m["D"])[:n]) for c in (0, 1))
        K2, V2 = (np.ascontiguousarray(a_hc[:, c].reshape(-1, m["D"])[:n]) for c in (0, 1))
        assert np.array_equal(attend(K1, V1).view(np.uint32), attend(K2, V2).view(np.uint32))


# ---------------- layer stride: layers further apart than one dense layer (every layer has its own block array) -------
def _strided_views(pool, L, stride, dense):
    v = pool.reshape(L, stride)
    return v[:, :dense], v[:, dense:]


@pytest.mark.parametrize("order", [0, 1])
@pytest.mark.parametrize("TP", [1, 2, 4])
def test_layer_stride_places_layer_l_at_l_times_stride(oracle, TP, order):
    """A pool whose layers are `stride` elements apart holds, at l*stride, exactly what the dense pool holds at
    l*dense, and the words between two layers are never written (nor read back)."""
    m, T, NB = dict(SMALL, L=3), 4, 7
    seq_lens = [5, 0, 9, 4]
    bt, nblk = _state(seq_lens, T, NB)
    G = int(nblk.sum()) * T
    KV = np.random.default_rng(21).integers(0, 65536, size=(m["L"], G, m["Hkv"], 2, m["D"]), dtype=np.uint16)
    dense = oracle.pool_elems_per_layer(m, T, TP, NB)
    gap = 24
    stride = dense + gap
    FILL = 0xBEEF
    ref = oracle.kv_shard(KV, m, T, TP, NB, seq_lens, bt, fill=FILL, order=order)
    got = oracle.kv_shard(KV, m, T, TP, NB, seq_lens, bt, fill=FILL, order=order, layer_stride=stride)
    for r in range(TP):
        assert got[r].size == m["L"] * stride
        body, between = _strided_views(got[r], m["L"], stride, dense)
        assert np.array_equal(body, ref[r].reshape(m["L"], dense))
        assert np.all(between == FILL)
    # the inverse reads the same places: poison the gaps, the logical state must not change
    for r in range(TP):
        _strided_views(got[r], m["L"], stride, dense)[1][:] = 0x0BAD
    assert np.array_equal(oracle.kv_reconstruct(got, m, T, TP, NB, seq_lens, bt, order=order, layer_stride=stride), KV)
    # a stride counted in the wrong unit (bytes instead of elements) would land layer 1 elsewhere: the stamp of the
    # first word of layer 1 sits at element `stride`, not at 2*stride or stride/2
    l1 = oracle.kv_shard(KV[:2], dict(m, L=2), T, TP, NB, seq_lens, bt, fill=FILL, order=order, layer_stride=stride)
    for r in range(TP):
        assert np.array_equal(l1[r][stride:stride + dense], ref[r][dense:2 * dense])


@pytest.mark.parametrize("a,b,so,do", [(1, 4, 0, 0), (4, 2, 0, 0), (2, 4, 1, 0), (2, 1, 0, 1)])
def test_transform_with_layer_strides_equals_dense_transform(oracle, a, b, so, do):
    m, T = dict(SMALL, L=3), 4
    seq_lens = [9, 4, 0, 13, 2]
    NB_a, NB_b = 10, 13
    bt_a, nblk = _state(seq_lens, T, NB_a, seed=7)
    G = int(nblk.sum()) * T
    KV = np.random.default_rng(22).integers(0, 65536, size=(m["L"], G, m["Hkv"], 2, m["D"]), dtype=np.uint16)
    da, db = oracle.pool_elems_per_layer(m, T, a, NB_a), oracle.pool_elems_per_layer(m, T, b, NB_b)
    sa, sb = da + 40, db + 8
    free_b = np.random.default_rng(3).permutation(NB_b).astype(np.int32)
    bt_b, *_ = oracle.assign_blocks(seq_lens, T, bt_a, NB_a, NB_b, free_list=free_b)
    src_d = oracle.kv_shard(KV, m, T, a, NB_a, seq_lens, bt_a, order=so)
    src_s = oracle.kv_shard(KV, m, T, a, NB_a, seq_lens, bt_a, order=so, layer_stride=sa, fill=0x1111)
    dst_d = [np.full(m["L"] * db, 0xA5A5, np.uint16) for _ in range(b)]
    dst_s = [np.full(m["L"] * sb, 0xA5A5, np.uint16) for _ in range(b)]
    oracle.kv_transform(m, T, seq_lens, a, NB_a, bt_a, src_d, b, NB_b, bt_b, dst_d, src_order=so, dst_order=do)
    oracle.kv_transform(m, T, seq_lens, a, NB_a, bt_a, src_s, b, NB_b, bt_b, dst_s, src_order=so, dst_order=do,
                        src_layer_stride=sa, dst_layer_stride=sb)
    for r in range(b):
        body, between = _strided_views(dst_s[r], m["L"], sb, db)
        assert np.array_equal(body, dst_d[r].reshape(m["L"], db))
        assert np.all(between == 0xA5A5)
    # and it is the direct shard of the logical state at that stride
    direct = oracle.kv_shard(KV, m, T, b, NB_b, seq_lens, bt_b, order=do, layer_stride=sb, fill=0xA5A5)
    for x, y in zip(dst_s, direct):
        assert np.array_equal(x, y)


def test_assign_blocks_refuses_an_id_handed_out_twice(oracle):
    """Brute force on a tiny input: a free list that names id 7 twice.  The first block that is given 7 keeps it, the
    later one gets no destination (entry -1, pair (-1,-1)), so no two blocks ever share a destination block."""
    T, NB = 16, 32
    seq_lens = [40, 16, 20]                       # 3 + 1 + 2 blocks
    bt, nblk = _state(seq_lens, T, NB)
    free = np.array([3, 7, 9, 7, 11, 12, 13], np.int32)
    dst_bt, pairs, n, left, st = oracle.assign_blocks(seq_lens, T, bt, NB, NB, free_list=free)
    assert st == oracle.BAD_BLOCK_ID and n == 6 and left == 1
    flat = [int(dst_bt[s, i]) for s in range(3) for i in range(nblk[s])]
    assert flat == [3, 7, 9, -1, 11, 12]
    assert tuple(pairs[3]) == (-1, -1) and tuple(pairs[1]) == (int(bt[0, 1]), 7)
    given = [x for x in flat if x >= 0]
    assert len(set(given)) == len(given)


def test_pairs_by_destination_worked_by_hand(oracle):
    """The other order of the work list, on an input small enough to sort by hand: five blocks, one of which is refused
    its destination (id 7 is named twice) and one of which has a bad source id but a good destination."""
    T, NB = 4, 12
    seq_lens = [12, 7]                                   # 3 + 2 blocks
    bt = np.array([[5, 1, 9], [2, 30, -1]], np.int32)    # block 4 names source id 30 of a pool with 12 blocks
    free = np.array([7, 3, 7, 0, 4, 6], np.int32)
    dst_bt, pairs, n, left, st = oracle.assign_blocks(seq_lens, T, bt, NB, NB, free_list=free)
    assert st == oracle.BAD_BLOCK_ID and n == 5
    assert dst_bt.tolist() == [[7, 3, -1], [0, 4, -1]]
    assert pairs.tolist() == [[5, 7], [1, 3], [-1, -1], [2, 0], [-1, -1]]          # (sequence, block) order
    by_dst = oracle.pairs_by_destination(pairs, dst_bt, seq_lens, T)
    #          dst 0    dst 3   dst 4: bad source   dst 7   the refused block
    assert by_dst.tolist() == [[2, 0], [1, 3], [-1, -1], [5, 7], [-1, -1]]
    # a call that failed as a whole lists nothing in either order
    dst_bt, pairs, n, _, st = oracle.assign_blocks(seq_lens, T, bt, NB, NB, free_list=free[:2])
    assert st == oracle.NO_FREE_BLOCKS and n == 0 and len(oracle.pairs_by_destination(pairs, dst_bt, seq_lens, T)) == 0

"""Pins for the oracle's padded weight partitions (Sec. 3.2, Improvement 1).  No GPU, no CUDA library.

Fixed from outside the oracle: the paper's Table 2 (pages per tensor), numpy's split / concatenate for what a
partition holds and where it starts, the reduction to the dense shards when there is nothing to pad, round trips,
and Eq. 2 (the padded FFN equals the unpadded one)."""
import os

import numpy as np
import pytest

import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
M = dict(L=1, hidden=16, Hq=8, Hkv=4, D=4, I=48)


def _logical(oracle, m, seed=0):
    g = np.random.default_rng(seed)
    return {n: g.integers(0, 65536, size=s, dtype=np.uint16) for n, s in oracle.logical_shapes(m).items()}


def test_table2_pages_per_tensor(oracle):
    rows = [l.split() for l in open(os.path.join(GOLDEN, "table2_pages.txt")) if l.strip() and not l.startswith("#")]
    assert len(rows) == 6
    for name, hidden, inter, experts, fused, p1, p4 in rows:
        cols = int(inter) * int(experts) * int(fused)
        for tp, printed in ((1, p1), (4, p4)):
            pages = oracle.pages_per_tensor(int(hidden), cols, 2, tp)
            digits = len(printed.split(".")[1]) if "." in printed else 0
            # the paper prints up to three decimals (126.5625 appears as 126.563)
            assert abs(pages - float(printed)) <= 0.5 * 10.0 ** -digits + 1e-9, (name, tp, pages, printed)
    # "decimals mean unaligned placements": the pitch rounds a 33.75-page partition up to 34 pages
    page_elems = (2 << 20) // 2
    assert oracle.padded_pitch(5120 * 27648 // 4, page_elems) == 34 * page_elems
    assert oracle.padded_pitch(8192 * 28672 // 4, page_elems) == 56 * page_elems  # already aligned: no padding


@pytest.mark.parametrize("fq,fg", [(False, False), (True, True)])
@pytest.mark.parametrize("TP,P", [(1, 4), (2, 4), (4, 4), (1, 1), (2, 2)])
def test_partitions_are_numpy_splits_at_page_pitch(oracle, TP, P, fq, fg):
    m, page = M, 40  # elements; none of the partition sizes is a multiple of it
    W = _logical(oracle, m, TP * 8 + P)
    FILL = 0xBEEF
    sh = oracle.weights_shard_padded(W, m, TP, P, page, fq, fg, fill=FILL)
    n = P // TP
    rows = lambda name: np.split(W[name], P, axis=0)
    cols = lambda name: [np.ascontiguousarray(x) for x in np.split(W[name], P, axis=1)]
    for r in range(TP):
        for j in range(n):
            p = r * n + j
            expect = {"o": cols("o")[p], "down": cols("down")[p]}
            if fq:
                expect["q"] = np.concatenate([rows("q")[p], rows("k")[p], rows("v")[p]])
            else:
                expect.update(q=rows("q")[p], k=rows("k")[p], v=rows("v")[p])
            if fg:
                expect["gate"] = np.concatenate([rows("gate")[p], rows("up")[p]])
            else:
                expect.update(gate=rows("gate")[p], up=rows("up")[p])
            assert set(expect) == set(sh[r])
            for name, e in expect.items():
                pitch = -(-e.size // page) * page
                assert sh[r][name].size == n * pitch
                got = sh[r][name][j * pitch:(j + 1) * pitch]
                assert np.array_equal(got[:e.size], e.reshape(-1)), (r, j, name)
                assert np.all(got[e.size:] == FILL)  # pad words are not written
    back = oracle.weights_reconstruct_padded(sh, m, TP, P, page, fq, fg)
    for name in W:
        assert np.array_equal(back[name], W[name])


@pytest.mark.parametrize("TP", [1, 2, 4])
def test_nothing_to_pad_reduces_to_dense_shards(oracle, TP):
    """P = TP with a page of one element: one partition per worker at pitch = its size: the dense shard."""
    W = _logical(oracle, M, 3)
    dense = oracle.weights_shard(W, M, TP)
    padded = oracle.weights_shard_padded(W, M, TP, TP, 1)
    for r in range(TP):
        for name in dense[r]:
            assert np.array_equal(padded[r][name], dense[r][name].reshape(-1))


@pytest.mark.parametrize("a,b,src_pad,dst_pad", [(1, 4, (4, 40), (4, 40)), (4, 1, (4, 40), (4, 40)), (1, 4, (4, 40), None),
                                                  (4, 2, None, (4, 24)), (2, 4, (8, 16), (4, 40)), (2, 1, (2, 40), (4, 8))])
def test_transform_between_forms_equals_direct_shard(oracle, a, b, src_pad, dst_pad):
    W = _logical(oracle, M | dict(Hq=8, Hkv=8, I=64), 5)
    m = M | dict(Hq=8, Hkv=8, I=64)
    src = oracle.weights_shard_padded(W, m, a, *src_pad) if src_pad else oracle.weights_shard(W, m, a)
    got = oracle.weights_transform_any(src, m, a, b, src_pad=src_pad, dst_pad=dst_pad, fill=0)
    direct = oracle.weights_shard_padded(W, m, b, *dst_pad, fill=0) if dst_pad else oracle.weights_shard(W, m, b)
    for r in range(b):
        for name in direct[r]:
            assert np.array_equal(got[r][name].reshape(-1), direct[r][name].reshape(-1))


def test_eq2_padded_ffn_equals_ffn(oracle):
    """Eq. 2: with U' = [U_1,0,U_2,0,...] and D' = [D_1^T,0,D_2^T,0,...]^T, f(I x U') x D' = f(I x U) x D.  U' is
    read straight from the oracle's padded TP1 buffers (zero-filled pads, a page of whole rows); D' puts the
    oracle's dense partitions D_p side by side with the same number of zero columns."""
    m, P = dict(L=1, hidden=16, Hq=8, Hkv=4, D=4, I=40), 4
    hid, I = m["hidden"], m["I"]
    g = np.random.default_rng(8)
    Wf = {n: g.standard_normal(s).astype(np.float32) * 0.3 for n, s in oracle.logical_shapes(m).items()}
    W = {n: wl.to_bits(x, "bf16") for n, x in Wf.items()}
    val = lambda bits: wl.from_bits(bits, "bf16")
    page = 6 * hid                                        # 6 rows of `hidden`: partitions of 10 rows pad to 12
    sh = oracle.weights_shard_padded(W, m, 1, P, page, fused_qkv=False, fused_gate_up=False, fill=0)[0]
    rows_p = oracle.padded_pitch(I // P * hid, page) // hid
    assert rows_p == 12
    gate_pad = val(sh["gate"]).reshape(P * rows_p, hid)   # U' (gate), [out', in]
    up_pad = val(sh["up"]).reshape(P * rows_p, hid)
    pitch_down = oracle.padded_pitch(hid * I // P, page)
    D_parts = [val(sh["down"][p * pitch_down:p * pitch_down + hid * I // P]).reshape(hid, I // P) for p in range(P)]
    down_pad = np.concatenate([np.concatenate([d, np.zeros((hid, rows_p - I // P))], axis=1) for d in D_parts], axis=1)
    x = g.standard_normal((5, hid))
    silu = lambda z: z / (1.0 + np.exp(-z))
    ffn = (silu(x @ val(W["gate"]).T) * (x @ val(W["up"]).T)) @ val(W["down"]).T
    ffn_pad = (silu(x @ gate_pad.T) * (x @ up_pad.T)) @ down_pad.T
    assert gate_pad.shape[0] == I + P * 2 and np.count_nonzero(gate_pad[10:12]) == 0
    assert np.allclose(ffn_pad, ffn, rtol=1e-12, atol=1e-12)
    # the padding changes the result as soon as a pad word is not zero
    gate_bad = gate_pad.copy()
    gate_bad[10] = 1.0
    up_bad = up_pad.copy()
    up_bad[10] = 1.0
    down_bad = down_pad.copy()
    down_bad[:, 10] = 1.0
    assert not np.allclose((silu(x @ gate_bad.T) * (x @ up_bad.T)) @ down_bad.T, ffn, rtol=1e-6)

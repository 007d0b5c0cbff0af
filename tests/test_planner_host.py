"""Host-side checks that need no GPU: the shared library loads and exports every declared symbol; the planner's
descriptors, applied with plain numpy byte copies, reproduce the oracle's result; layout validation."""
import ctypes as C
import os
import re

import numpy as np
import pytest

import paper_2509_19729_b200 as A

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SMALL40 = dict(L=1, hidden=40, Hq=40, Hkv=40, D=8, I=320)
GQA = dict(L=1, hidden=64, Hq=16, Hkv=8, D=16, I=192)


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "amoeba.h")).read()
    names = re.findall(r"AMOEBA_API\s+[\w\s\*]+?\b(amoeba_\w+)\s*\(", header)
    assert len(names) >= 15 and len(set(names)) == len(names)
    lib = C.CDLL(str(A.library_path()))
    for n in names:
        assert hasattr(lib, n), n
    assert A.amoeba_status_string(0) == "ok" and "block" in A.amoeba_status_string(A.ERR_BAD_BLOCK_ID)


def _apply_descs(plan, src_bufs, dst_bufs):
    """src_bufs / dst_bufs: [rank][tensor index] -> uint8 arrays.  Returns per-destination write counts."""
    counts = [[np.zeros(len(b), np.int32) if b is not None else None for b in r] for r in dst_bufs]
    for i in range(A.amoeba_plan_num_weight_descs(plan)):
        d = A.amoeba_plan_weight_desc(plan, i)
        s, t = src_bufs[d.src_rank][d.src_tensor], dst_bufs[d.dst_rank][d.dst_tensor]
        for r in range(d.n_rows):
            so, to = d.src_off + r * d.src_pitch, d.dst_off + r * d.dst_pitch
            t[to:to + d.row_bytes] = s[so:so + d.row_bytes]
            counts[d.dst_rank][d.dst_tensor][to:to + d.row_bytes] += 1
    return counts


@pytest.mark.parametrize("fq,fg", [(True, True), (False, False)])
@pytest.mark.parametrize("model,a,b", [(GQA, 1, 2), (GQA, 2, 1), (GQA, 1, 4), (GQA, 2, 8), (GQA, 8, 2), (GQA, 4, 4),
                                       (SMALL40, 4, 5), (SMALL40, 5, 8), (SMALL40, 8, 5), (SMALL40, 10, 20),
                                       (SMALL40, 20, 1)])
def test_weight_descriptors_reproduce_oracle(oracle, model, a, b, fq, fg):
    g = np.random.default_rng(a * 100 + b)
    W = {n: g.integers(0, 65536, size=s, dtype=np.uint16) for n, s in oracle.logical_shapes(model).items()}
    src = oracle.weights_shard(W, model, a, fq, fg)
    exp = oracle.weights_transform(src, model, a, b, fq, fg)
    plan = A.amoeba_plan_create(A.make_layout(model, a, 4, fused_qkv=fq, fused_gate_up=fg),
                                A.make_layout(model, b, 4, fused_qkv=fq, fused_gate_up=fg))
    as_bytes = lambda sh: [[sh_r[n].reshape(-1).view(np.uint8) if n in sh_r else None for n in A.TENSOR_NAMES]
                           for sh_r in sh]
    dst = [[np.full(e.size, 0xA5, np.uint8) if e is not None else None for e in r] for r in as_bytes(exp)]
    counts = _apply_descs(plan, as_bytes(src), dst)
    for r in range(b):
        for t, n in enumerate(A.TENSOR_NAMES):
            if n in exp[r]:
                assert np.array_equal(dst[r][t], exp[r][n].reshape(-1).view(np.uint8)), (r, n)
                assert np.all(counts[r][t] == 1)  # every destination byte written exactly once
                lay = A.make_layout(model, b, 4, fused_qkv=fq, fused_gate_up=fg)
                assert A.amoeba_layout_weight_bytes(lay, t) == exp[r][n].size * 2
    kv, w = A.amoeba_plan_bytes(plan, 3)
    assert w == 2 * sum(x.size * 2 for x in W.values())
    assert kv == 2 * 3 * model["L"] * model["Hkv"] * 2 * 16 * model["D"] * 2


@pytest.mark.parametrize("Hkv,a,b", [(8, 1, 4), (8, 2, 8), (8, 8, 2), (40, 4, 5), (40, 5, 8), (40, 10, 20), (32, 1, 2)])
def test_kv_runs_never_straddle_a_worker(oracle, Hkv, a, b):
    m = dict(L=2, hidden=Hkv * 8, Hq=Hkv, Hkv=Hkv, D=8, I=Hkv * 8)
    plan = A.amoeba_plan_create(A.make_layout(m, a, 10), A.make_layout(m, b, 12))
    info = A.amoeba_plan_kv_info(plan)
    g = info.heads_per_run
    assert g * info.runs_per_block == Hkv
    unit = 2 * 16 * m["D"] * 2
    assert info.run_bytes == g * unit and info.run_bytes % info.chunk_bytes == 0 and info.chunk_bytes % 16 == 0
    assert info.src_block_bytes == Hkv // a * unit and info.dst_block_bytes == Hkv // b * unit
    assert info.src_layer_stride == 10 * info.src_block_bytes and info.dst_layer_stride == 12 * info.dst_block_bytes
    for run in range(info.runs_per_block):
        heads = range(run * g + 1, (run + 1) * g + 1)  # 1-indexed headers of this run
        assert len({oracle.worker_of_header(Hkv, a, h) for h in heads}) == 1
        assert len({oracle.worker_of_header(Hkv, b, h) for h in heads}) == 1
    # and no larger uniform run would do
    if g < Hkv:
        bigger = [k for k in range(g + 1, Hkv + 1) if Hkv % k == 0 and (Hkv // a) % k == 0 and (Hkv // b) % k == 0]
        assert not bigger


def test_layout_validation():
    m = GQA
    ok = A.make_layout(m, 2, 8)
    for bad, code in [
        (A.make_layout(m, 3, 8), A.ERR_UNSUPPORTED),                     # 3 does not divide the head counts
        (A.make_layout(m, 16, 8), A.ERR_UNSUPPORTED),                    # more workers than K/V heads
        (A.make_layout(m, 2, 0), A.ERR_INVALID_ARG),                     # empty pool
        (A.make_layout(dict(m, D=12), 2, 8), A.ERR_INVALID_ARG),         # different model on the two sides
        (A.make_layout(m, 2, 8, block_tokens=8), A.ERR_INVALID_ARG),     # different block size
        (A.make_layout(m, 2, 8, elem_bytes=3), A.ERR_UNSUPPORTED),                 # 1, 2 and 4 are the sizes taken
        (A.make_layout(m, 2, 8, kv_layer_stride_bytes=1024), A.ERR_INVALID_ARG),  # stride smaller than a layer
    ]:
        with pytest.raises(A.AmoebaError) as e:
            A.amoeba_plan_create(ok, bad)
        assert e.value.status == code, (e.value.status, code)
    tiny_rows = dict(L=1, hidden=4, Hq=2, Hkv=2, D=2, I=4)  # 8-byte rows: not copyable in 16-byte units
    with pytest.raises(A.AmoebaError) as e:
        A.amoeba_plan_create(A.make_layout(tiny_rows, 1, 8), A.make_layout(tiny_rows, 2, 8))
    assert e.value.status == A.ERR_ALIGNMENT
    plan = A.amoeba_plan_create(ok, A.make_layout(m, 4, 8))
    with pytest.raises(A.AmoebaError):
        A.amoeba_plan_set_option(plan, A.OPT_CHUNK_BYTES, 24)  # not a multiple of 16
    A.amoeba_plan_set_option(plan, A.OPT_CHUNK_BYTES, 1024)
    assert A.amoeba_plan_kv_info(plan).chunk_bytes == 1024
    assert A.amoeba_rewrite_workspace_bytes(plan, 10, 100) >= 64 + 44 + 4 * 8  # header, offsets, one word per block id
    for order in (0, A.PAIR_ORDER_TABLE, A.PAIR_ORDER_DESTINATION):
        A.amoeba_plan_set_option(plan, A.OPT_PAIR_ORDER, order)
    with pytest.raises(A.AmoebaError) as e:
        A.amoeba_plan_set_option(plan, A.OPT_PAIR_ORDER, 3)  # no such order
    assert e.value.status == A.ERR_INVALID_ARG


def test_no_device_means_cuda_error_not_a_fallback():
    import torch

    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    m = GQA
    plan = A.amoeba_plan_create(A.make_layout(m, 2, 8), A.make_layout(m, 1, 8))
    with pytest.raises(A.AmoebaError) as e:  # non-null fake addresses, aligned: passes validation, then no device
        A.amoeba_reshard_kv(plan, [4096, 8192], [12288], 4096, 4096, 4, 0, 1, 4096, stream=0)
    assert e.value.status == A.ERR_CUDA


@pytest.mark.parametrize("so,do", [(0, 0), (1, 1), (1, 0), (0, 1)])
@pytest.mark.parametrize("a,b", [(1, 4), (8, 2), (4, 5), (2, 2)])
def test_kv_geometry_covers_each_block_once_for_both_orders(so, do, a, b):
    """The planner's work-item size never exceeds the cap and the plan accepts both storage orders on both sides."""
    import paper_2509_19729_b200 as A

    model = dict(L=2, hidden=320, Hq=40, Hkv=40, D=16, I=640)
    src = A.make_layout(model, a, 64, block_tokens=8, kv_order=so)
    dst = A.make_layout(model, b, 64, block_tokens=8, kv_order=do)
    plan = A.amoeba_plan_create(src, dst)
    info = A.amoeba_plan_kv_info(plan)
    assert 16 <= info.chunk_bytes <= 8192 and info.chunk_bytes % 16 == 0
    for cap in (16, 64, 4096):
        A.amoeba_plan_set_option(plan, A.OPT_CHUNK_BYTES, cap)
        assert A.amoeba_plan_kv_info(plan).chunk_bytes <= max(cap, 16)
    kv_rw, _ = A.amoeba_plan_bytes(plan, 10)
    assert kv_rw == 2 * 10 * 2 * 40 * 2 * 8 * 16 * 2  # both ways x blocks x layers x Hkv x (K,V) x T x D x e


def test_unknown_kv_order_is_unsupported():
    import paper_2509_19729_b200 as A

    model = dict(L=1, hidden=64, Hq=4, Hkv=4, D=16, I=128)
    with pytest.raises(A.AmoebaError) as e:
        A.amoeba_plan_create(A.make_layout(model, 1, 8, kv_order=2), A.make_layout(model, 2, 8))
    assert e.value.status == A.ERR_UNSUPPORTED
    # token-first needs head_dim * elem_bytes to be a multiple of 16
    odd = dict(model, D=4)
    with pytest.raises(A.AmoebaError) as e:
        A.amoeba_plan_create(A.make_layout(odd, 1, 8, kv_order=1), A.make_layout(odd, 2, 8, kv_order=1))
    assert e.value.status == A.ERR_ALIGNMENT


# ---- padded weight partitions (Sec. 3.2, Improvement 1)
PADM = dict(L=1, hidden=32, Hq=16, Hkv=8, D=8, I=192)  # every partition size is a multiple of 16 bytes down to P = 8
PAD_CASES = [  # a, b, source (P, page bytes) or None, destination (P, page bytes) or None
    (1, 4, (4, 2048), (4, 2048)), (4, 1, (4, 2048), (4, 2048)), (2, 4, (8, 1024), (8, 1024)), (1, 4, (4, 2048), None),
    (4, 2, None, (4, 2048)), (2, 4, (8, 4096), (4, 2048)), (2, 1, (2, 2048), (8, 512)), (1, 1, None, (8, 4096)),
    (8, 8, (8, 2048), None), (4, 4, (4, 2048), (4, 512)),
]


@pytest.mark.parametrize("fq,fg", [(True, True), (False, False)])
@pytest.mark.parametrize("a,b,sp,dp", PAD_CASES)
def test_padded_weight_descriptors_reproduce_oracle(oracle, a, b, sp, dp, fq, fg):
    m = PADM
    g = np.random.default_rng(a * 100 + b)
    W = {n: g.integers(0, 65536, size=s, dtype=np.uint16) for n, s in oracle.logical_shapes(m).items()}
    opad = lambda pad: (pad[0], pad[1] // 2) if pad else None   # the oracle counts pages in elements
    src = oracle.weights_shard_padded(W, m, a, *opad(sp), fq, fg) if sp else oracle.weights_shard(W, m, a, fq, fg)
    exp = oracle.weights_transform_any(src, m, a, b, fq, fg, src_pad=opad(sp), dst_pad=opad(dp), fill=0xA5A5)
    lay = lambda tp, pad: A.make_layout(m, tp, 4, fused_qkv=fq, fused_gate_up=fg, weight_pad_parts=pad[0] if pad else 0,
                                        weight_page_bytes=pad[1] if pad else 0)
    plan = A.amoeba_plan_create(lay(a, sp), lay(b, dp))
    as_bytes = lambda sh: [[sh_r[n].reshape(-1).view(np.uint8) if n in sh_r else None for n in A.TENSOR_NAMES]
                           for sh_r in sh]
    dst = [[np.full(e.size, 0xA5, np.uint8) if e is not None else None for e in r] for r in as_bytes(exp)]
    counts = _apply_descs(plan, as_bytes(src), dst)
    total = 0
    for r in range(b):
        for t, n in enumerate(A.TENSOR_NAMES):
            if n in exp[r]:
                assert A.amoeba_layout_weight_bytes(lay(b, dp), t) == exp[r][n].size * 2, (r, n)
                assert np.array_equal(dst[r][t], exp[r][n].reshape(-1).view(np.uint8)), (r, n)
                assert counts[r][t].max() == 1      # no byte written twice; pad bytes never written
                total += int(counts[r][t].sum())
            else:
                assert A.amoeba_layout_weight_bytes(lay(b, dp), t) == 0
    assert total == sum(x.size * 2 for x in W.values())  # every weight byte written exactly once
    _, w = A.amoeba_plan_bytes(plan, 0)
    assert w == 2 * total


def test_padded_partitions_fold_into_few_descriptors():
    """Padded -> padded moves whole partitions: per (source worker, destination worker, tensor) one 2-D descriptor whose
    rows are the partitions, not one descriptor per partition."""
    m = dict(L=1, hidden=64, Hq=32, Hkv=32, D=8, I=512)
    lay = lambda tp: A.make_layout(m, tp, 4, weight_pad_parts=32, weight_page_bytes=4096)
    plan = A.amoeba_plan_create(lay(1), lay(4))
    n = A.amoeba_plan_num_weight_descs(plan)
    assert n == 7 * 4
    d = A.amoeba_plan_weight_desc(plan, 0)
    assert d.n_rows == 8 and d.src_pitch == d.dst_pitch  # 8 partitions per destination worker, same pitch both sides


def test_pad_info_reproduces_table2():
    rows = [l.split() for l in open(os.path.join(ROOT, "tests", "golden", "table2_pages.txt"))
            if l.strip() and not l.startswith("#")]
    for name, hidden, inter, experts, fused, p1, p4 in rows:
        # an expert-parallel FFN tensor holds `experts` matrices: the page arithmetic sees hidden x (inter * experts)
        I = int(inter) * int(experts) * int(fused)
        m = dict(L=1, hidden=int(hidden), Hq=64, Hkv=64, D=int(hidden) // 64, I=I)
        for tp, printed in ((1, p1), (4, p4)):
            info = A.amoeba_layout_pad_info(A.make_layout(m, tp, 4, fused_gate_up=False, weight_pad_parts=tp), 6)
            digits = len(printed.split(".")[1]) if "." in printed else 0
            assert abs(info.pages - float(printed)) <= 0.5 * 10.0 ** -digits + 1e-9, (name, tp, info.pages)
            assert info.page_bytes == 2 << 20 and info.partitions_per_worker == 1
            assert info.pitch_bytes == -(-info.partition_bytes // info.page_bytes) * info.page_bytes
    # Qwen2.5-32B at TP4: 33.75 pages per partition -> padded to 34; Llama-3.1-70B: 56, already aligned
    qwen = A.make_layout(dict(L=1, hidden=5120, Hq=40, Hkv=8, D=128, I=27648), 1, 4, weight_pad_parts=4)
    assert A.amoeba_layout_pad_info(qwen, 6).pitch_bytes == 34 * (2 << 20)
    assert A.amoeba_layout_weight_bytes(qwen, 6) == 4 * 34 * (2 << 20)
    llama = A.make_layout(dict(L=1, hidden=8192, Hq=64, Hkv=8, D=128, I=28672), 4, 4, weight_pad_parts=4)
    assert A.amoeba_layout_pad_info(llama, 6).pitch_bytes == 56 * (2 << 20) == A.amoeba_layout_weight_bytes(llama, 6)


def test_padded_layout_validation():
    m = PADM
    for kw, status in ((dict(weight_pad_parts=3), A.ERR_UNSUPPORTED),          # tp = 2 does not divide P = 3
                       (dict(weight_pad_parts=16), A.ERR_UNSUPPORTED),         # P = 16 does not divide Hkv = 8
                       (dict(weight_pad_parts=-1), A.ERR_INVALID_ARG),
                       (dict(weight_pad_parts=4, weight_page_bytes=100), A.ERR_ALIGNMENT)):
        with pytest.raises(A.AmoebaError) as e:
            A.amoeba_plan_create(A.make_layout(m, 2, 4, **kw), A.make_layout(m, 2, 4))
        assert e.value.status == status, kw


@pytest.mark.parametrize("fq,fg", [(True, True), (False, False)])
@pytest.mark.parametrize("a,b,P", [(1, 4, 4), (2, 8, 8), (1, 2, 8), (4, 4, 8)])
def test_padded_scale_up_is_an_alias_of_the_source_buffers(oracle, a, b, P, fq, fg):
    """Sec. 3.2 Improvement 1: with padded partitions every destination shard already sits in a source buffer."""
    m, page = PADM, 1024
    g = np.random.default_rng(P)
    W = {n: g.integers(0, 65536, size=s, dtype=np.uint16) for n, s in oracle.logical_shapes(m).items()}
    src = oracle.weights_shard_padded(W, m, a, P, page // 2, fq, fg, fill=0)
    dst = oracle.weights_shard_padded(W, m, b, P, page // 2, fq, fg, fill=0)
    lay = lambda tp: A.make_layout(m, tp, 4, fused_qkv=fq, fused_gate_up=fg, weight_pad_parts=P, weight_page_bytes=page)
    plan = A.amoeba_plan_create(lay(a), lay(b))
    for j in range(b):
        for t, n in enumerate(A.TENSOR_NAMES):
            r, off, nbytes = A.amoeba_plan_weight_alias(plan, j, t)
            if n not in dst[j]:
                assert nbytes == 0
                continue
            assert nbytes == dst[j][n].size * 2 and off % page == 0
            assert np.array_equal(src[r][n].view(np.uint8)[off:off + nbytes], dst[j][n].view(np.uint8))
    for other in (A.make_layout(m, b, 4, fused_qkv=fq, fused_gate_up=fg),                                   # dense
                  A.make_layout(m, b, 4, fused_qkv=fq, fused_gate_up=fg, weight_pad_parts=P, weight_page_bytes=512)):
        with pytest.raises(A.AmoebaError) as e:
            A.amoeba_plan_weight_alias(A.amoeba_plan_create(lay(a), other), 0, 0)
        assert e.value.status == A.ERR_UNSUPPORTED
    if a > 1:  # scale-down gathers partitions of several workers: a copy
        with pytest.raises(A.AmoebaError) as e:
            A.amoeba_plan_weight_alias(A.amoeba_plan_create(lay(b), lay(1)), 0, 0)
        assert e.value.status == A.ERR_UNSUPPORTED or b == 1


def test_random_layout_pairs_reproduce_oracle(oracle):
    """Seeded random shapes, TP degrees, fused / unfused buffers and dense / padded forms on either side: the planner's
    descriptors, applied as plain byte copies, give the oracle's destination buffers and write no byte twice."""
    g = np.random.default_rng(20250919)
    done = 0
    while done < 40:
        Hkv = int(g.choice([4, 8, 12, 16, 24]))
        m = dict(L=1, hidden=int(g.choice([16, 24, 40])), Hq=Hkv * int(g.choice([1, 2])), Hkv=Hkv,
                 D=int(g.choice([8, 16])), I=Hkv * int(g.choice([8, 24])))
        divs = [d for d in (1, 2, 3, 4, 6, 8, 12) if Hkv % d == 0]
        a, b = int(g.choice(divs)), int(g.choice(divs))
        fq, fg = bool(g.integers(2)), bool(g.integers(2))

        def pick_pad(tp):
            if g.integers(3) == 0:
                return None
            P = int(g.choice([d for d in divs if d % tp == 0]))
            return (P, int(g.choice([64, 256, 1024])))

        sp, dp = pick_pad(a), pick_pad(b)
        W = {n: g.integers(0, 65536, size=s, dtype=np.uint16) for n, s in oracle.logical_shapes(m).items()}
        opad = lambda pad: (pad[0], pad[1] // 2) if pad else None
        src = oracle.weights_shard_padded(W, m, a, *opad(sp), fq, fg) if sp else oracle.weights_shard(W, m, a, fq, fg)
        exp = oracle.weights_transform_any(src, m, a, b, fq, fg, src_pad=opad(sp), dst_pad=opad(dp), fill=0xA5A5)
        lay = lambda tp, pad: A.make_layout(m, tp, 4, fused_qkv=fq, fused_gate_up=fg,
                                            weight_pad_parts=pad[0] if pad else 0, weight_page_bytes=pad[1] if pad else 0)
        try:
            plan = A.amoeba_plan_create(lay(a, sp), lay(b, dp))
        except A.AmoebaError as e:  # more descriptors than one launch carries: refused, not mis-planned
            assert e.status == A.ERR_UNSUPPORTED, (m, a, b, sp, dp)
            continue
        as_bytes = lambda sh: [[r[n].reshape(-1).view(np.uint8) if n in r else None for n in A.TENSOR_NAMES] for r in sh]
        dst = [[np.full(e.size, 0xA5, np.uint8) if e is not None else None for e in r] for r in as_bytes(exp)]
        counts = _apply_descs(plan, as_bytes(src), dst)
        for r in range(b):
            for t, n in enumerate(A.TENSOR_NAMES):
                if n in exp[r]:
                    assert np.array_equal(dst[r][t], exp[r][n].reshape(-1).view(np.uint8)), (m, a, b, sp, dp, fq, fg, r, n)
                    assert counts[r][t].max() == 1
        done += 1


def test_compact_bytes_counts_only_what_moves():
    """Partial swap, TP 1 -> 4, fused buffers: with keep = 0 the q and gate sections and row 0 of o_proj / down_proj
    already sit where they belong and are not counted; with keep > 0 everything kept moves."""
    m = dict(L=3, hidden=64, Hq=16, Hkv=8, D=16, I=192)
    plan = A.amoeba_plan_create(A.make_layout(m, 1, 4), A.make_layout(m, 4, 16))
    e, hid, N = 2, m["hidden"], 4
    rb = hid * e
    q, kv, ffn = m["Hq"] * m["D"] // N * rb, m["Hkv"] * m["D"] // N * rb, m["I"] // N * rb
    wo, wd = m["Hq"] * m["D"] // N * e, m["I"] // N * e
    everything = q + 2 * kv + 2 * ffn + hid * (wo + wd)
    assert A.amoeba_compact_bytes(plan, [2]) == 2 * m["L"] * everything
    assert A.amoeba_compact_bytes(plan, [0]) == 2 * m["L"] * (everything - q - ffn - wo - wd)
    _, w = A.amoeba_plan_bytes(plan, 0)
    assert A.amoeba_compact_bytes(plan, [3]) * N == w  # one N-th of the weights, read and written
    with pytest.raises(A.AmoebaError) as err:
        A.amoeba_compact_bytes(plan, [4])
    assert err.value.status == A.ERR_INVALID_ARG


def test_reshape_plans_are_recognised_on_the_host():
    """In-place reshaping needs TP degrees and block counts that are multiples of each other by the same factor,
    header-centric pools and one layer stride; the bytes it moves are (N-1)/N of the blocks."""
    m = GQA
    unit = 2 * 16 * m["D"] * 2
    for a, N, NB in ((1, 4, 10), (2, 2, 7), (2, 4, 3)):
        split = A.amoeba_plan_create(A.make_layout(m, a, NB), A.make_layout(m, a * N, NB * N))
        back = A.amoeba_plan_create(A.make_layout(m, a * N, NB * N), A.make_layout(m, a, NB))
        expect = 2 * 5 * m["L"] * (m["Hkv"] // N) * (N - 1) * unit
        assert A.amoeba_reshape_bytes(split, 5) == expect == A.amoeba_reshape_bytes(back, 5)
        kv, _ = A.amoeba_plan_bytes(split, 5)
        assert expect * N == kv * (N - 1)
    for src, dst in ((A.make_layout(m, 1, 10), A.make_layout(m, 4, 41)),                 # block counts do not match
                     (A.make_layout(m, 2, 10), A.make_layout(m, 2, 10)),                 # same TP degree
                     (A.make_layout(m, 1, 10, kv_order=A.KV_TOKEN_MAJOR), A.make_layout(m, 4, 40)),
                     (A.make_layout(m, 1, 10), A.make_layout(m, 4, 40, kv_layer_stride_bytes=1 << 20))):
        plan = A.amoeba_plan_create(src, dst)
        with pytest.raises(A.AmoebaError) as e:
            A.amoeba_reshape_bytes(plan, 1)
        assert e.value.status == A.ERR_UNSUPPORTED

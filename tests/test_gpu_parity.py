"""Parity of the CUDA path (through the C ABI) with the CPU oracle: bit-exact on every output byte."""
import numpy as np
import pytest

import workloads as wl
from harness import check_case, make_case, pairs_in_destination_order, run_case

pytestmark = pytest.mark.gpu

LDST, BULK, PAIR = 1, 2, 3
PATHS = [LDST, BULK, PAIR]
SMALL40 = dict(L=2, hidden=320, Hq=40, Hkv=40, D=16, I=640)  # 40-head shape: divisors 1,2,4,5,8,10,20,40
GQA = dict(L=3, hidden=512, Hq=16, Hkv=8, D=128, I=1792)


@pytest.fixture(scope="module", autouse=True)
def _need_gpu():
    import torch

    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    import paper_2509_19729_b200 as A

    assert A.library_path().exists()


@pytest.mark.parametrize("path", PATHS)
def test_tiny_config_end_to_end(path):
    cfg = wl.CONFIGS["tiny_2to1"]
    lens = wl.draw_seq_lens(cfg, name="tiny_2to1")
    c = make_case(cfg["model"], cfg["a"], cfg["b"], lens, src_free=0.25, dst_slack=0.25, dtype="fp16", seed=1)
    check_case(c, run_case(c, path))


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("a,b", [(1, 2), (2, 1), (1, 4), (4, 1), (2, 8), (8, 2), (4, 4), (1, 1), (8, 1), (1, 8)])
def test_gqa_shapes_all_directions(path, a, b):
    lens = [1, 16, 17, 300, 0, 77, 1024, 5]
    c = make_case(GQA, a, b, lens, seed=a * 16 + b)
    check_case(c, run_case(c, path))


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("a,b", [(4, 5), (5, 8), (8, 5), (10, 4), (10, 20), (20, 1), (5, 5)])
def test_non_nested_partitions(path, a, b):
    lens = [33, 7, 0, 64, 129]
    c = make_case(SMALL40, a, b, lens, T=8, seed=a * 64 + b)
    check_case(c, run_case(c, path))


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("fq,fg", [(False, False), (True, False), (False, True)])
def test_unfused_weight_buffers(path, fq, fg):
    c = make_case(GQA, 2, 4, [40], fused_qkv=fq, fused_gate_up=fg, kv=True, seed=5)
    check_case(c, run_case(c, path))


@pytest.mark.parametrize("path", PATHS)
def test_free_mask_compaction_and_foreign_blocks(path):
    lens = list(np.random.default_rng(3).integers(1, 600, size=200))
    c = make_case(dict(GQA, L=1), 4, 1, lens, dst_form="mask", dst_occupied=0.3, src_free=0.3, weights=False, seed=9)
    s = run_case(c, path)
    check_case(c, s)  # foreign (occupied) blocks keep the fill: whole-pool comparison


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("chunk", [1024, 4096, 8192, 32768])
def test_chunk_sizes_and_ragged_tails(path, chunk):
    import paper_2509_19729_b200 as A

    lens = [16 * 37 + 3, 1, 16 * 64]
    c = make_case(dict(L=2, hidden=1024 + 64, Hq=8, Hkv=8, D=128, I=2816 + 256), 2, 4, lens, seed=chunk)
    check_case(c, run_case(c, path, options=[(A.OPT_CHUNK_BYTES, chunk)]))


@pytest.mark.parametrize("path", [BULK, PAIR])
@pytest.mark.parametrize("stages,lag,warps", [(2, 1, 1), (3, 2, 2), (4, 2, 3), (6, 3, 0), (8, 1, 2), (12, 11, 1),
                                              (16, 8, 1), (5, 4, 16)])
def test_bulk_ring_shapes(path, stages, lag, warps):
    import paper_2509_19729_b200 as A

    c = make_case(GQA, 1, 4, [500, 20, 1000], seed=stages)
    opts = [(A.OPT_STAGES, stages), (A.OPT_LAG, lag), (A.OPT_WARPS, warps)]
    check_case(c, run_case(c, path, options=opts))
    check_case(c, run_case(c, path, options=opts + [(A.OPT_CHUNK_BYTES, 4096), (A.OPT_CTAS_PER_SM, 2),
                                                    (A.OPT_L2_HINT, 4)]))


def test_per_kernel_options():
    import paper_2509_19729_b200 as A

    c = make_case(GQA, 2, 4, [300, 20], seed=77)
    opts = [(A.OPT_COPY_PATH + A.OPT_KV_ONLY, PAIR), (A.OPT_COPY_PATH + A.OPT_WEIGHTS_ONLY, LDST),
            (A.OPT_CHUNK_BYTES + A.OPT_WEIGHTS_ONLY, 2048), (A.OPT_L2_HINT + A.OPT_KV_ONLY, 2)]
    s = run_case(c, None, options=opts)
    assert A.amoeba_plan_kv_info(s.plan).chunk_bytes == 8192  # the weights-only chunk option left KV alone
    check_case(c, s)


def test_long_single_row_and_many_sequences():
    # one very long row (many 128-entry segments) next to many short ones; > 1024 sequences (several scan tiles)
    lens = [16 * 3000] + list(np.random.default_rng(4).integers(0, 40, size=2500))
    c = make_case(dict(L=1, hidden=128, Hq=2, Hkv=2, D=64, I=256), 1, 2, lens, weights=False, seed=11)
    check_case(c, run_case(c, BULK))


def test_empty_inputs():
    c = make_case(GQA, 2, 1, [0, 0, 0], weights=False, seed=2)
    check_case(c, run_case(c, BULK))


def test_repeated_steps_are_idempotent():
    c = make_case(GQA, 2, 4, [100, 200, 300], seed=21)
    check_case(c, run_case(c, BULK, steps=3))


# ---------------- device-detected errors (values, never traps) ----------------
def test_not_enough_free_blocks():
    lens = [160, 160]
    free = (np.arange(19, dtype=np.int32), None)  # need 20
    c = make_case(GQA, 2, 1, lens, free_override=free, weights=False, seed=3)
    assert c.exp_status == 4
    check_case(c, run_case(c, BULK))


def test_invalid_lengths_and_pairs_cap():
    c = make_case(GQA, 2, 1, [160, -5, 16], weights=False, seed=3)
    assert c.exp_status == 1
    check_case(c, run_case(c, LDST))
    c = make_case(GQA, 2, 1, [160, 160], weights=False, seed=3, pairs_cap=19)
    assert c.exp_status == 1
    check_case(c, run_case(c, LDST))


@pytest.mark.parametrize("path", PATHS)
def test_bad_block_ids_are_skipped(path):
    lens = [160, 48]
    base = make_case(GQA, 2, 1, lens, weights=False, seed=4)
    bt = base.src_bt.copy()
    bt[0, 3] = base.NB_src + 7  # out of range source id
    bt[1, 1] = -1               # hole inside a sequence
    free = base.free_list.copy()
    free[5] = base.NB_dst       # out of range destination id
    c = make_case(GQA, 2, 1, lens, weights=False, seed=4, src_bt_override=bt, free_override=(free, None))
    assert c.exp_status == 5
    check_case(c, run_case(c, path))


def test_host_detected_errors():
    import torch

    import paper_2509_19729_b200 as A

    m = GQA
    with pytest.raises(A.AmoebaError) as e:
        A.amoeba_plan_create(A.make_layout(m, 3, 8), A.make_layout(m, 1, 8))
    assert e.value.status == A.ERR_UNSUPPORTED
    c = make_case(m, 2, 1, [40], weights=False, seed=1)
    s = run_case(c, BULK)
    with pytest.raises(A.AmoebaError) as e:  # misaligned pool pointer
        A.amoeba_reshard_kv(s.plan, [s.src_pools[0].data_ptr() + 4, s.src_pools[1]], s.dst_pools, s.pairs,
                            s.num_pairs, s.pairs_cap, 0, 1, s.status)
    assert e.value.status == A.ERR_ALIGNMENT
    with pytest.raises(A.AmoebaError) as e:  # layer range outside the model
        A.amoeba_reshard_kv(s.plan, s.src_pools, s.dst_pools, s.pairs, s.num_pairs, s.pairs_cap, 0, m["L"] + 1,
                            s.status)
    assert e.value.status == A.ERR_INVALID_ARG
    with pytest.raises(A.AmoebaError) as e:  # workspace too small
        A.amoeba_rewrite_block_tables(s.plan, s.src_bt, s.seq_lens, s.num_seqs, s.maxb, s.free_list, None,
                                      s.n_free_or_nb, s.dst_bt, s.pairs, s.pairs_cap, s.num_pairs, s.free_count,
                                      s.status, s.workspace, 8)
    assert e.value.status == A.ERR_INVALID_ARG
    torch.cuda.synchronize()
    check_case(c, s)  # the failed calls launched nothing


def test_layer_ranges_compose():
    """Transforming layer ranges one after the other (a few layers per inference step) equals one full call."""
    import torch

    c = make_case(GQA, 1, 2, [100, 37], seed=8)
    s = run_case(c, BULK, steps=0)
    s.status.zero_()
    s.rewrite_block_tables()
    for l in range(c.model["L"]):
        s.reshard_kv(layer_begin=l, layer_end=l + 1)
        s.reshard_weights(layer_begin=l, layer_end=l + 1)
    torch.cuda.synchronize()
    check_case(c, s)


def test_side_stream():
    import torch

    c = make_case(GQA, 4, 2, [100, 37, 900], seed=12)
    s = run_case(c, BULK, steps=0)
    st = torch.cuda.Stream()
    st.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(st):
        s.step(st)
    st.synchronize()
    check_case(c, s)


def test_host_threads_with_their_own_plans_and_streams():
    """The library is thread-compatible: host threads that use different plans may call it at the same time (the
    binding releases the interpreter lock inside every call).  Four threads, each with its own plan, buffers and
    stream - two of them with token-first pools, whose tensor maps are cached per plan - run their transformation
    twenty times while the others do; every result is compared with the oracle."""
    import threading

    import torch

    cases = [make_case(GQA, 1, 4, [300, 77, 45], seed=31), make_case(GQA, 4, 2, [100, 37, 200], seed=32),
             make_case(GQA, 2, 4, [64, 500], seed=33, weights=False, src_order=TF, dst_order=HC),
             make_case(GQA, 2, 1, [250, 9, 9], seed=34, weights=False, src_order=TF, dst_order=TF)]
    paths = [PAIR, LDST, PAIR, BULK]
    sessions = [run_case(c, p, steps=0) for c, p in zip(cases, paths)]
    streams = [torch.cuda.Stream() for _ in cases]
    errors = []
    go = threading.Barrier(len(cases))

    def work(s, st):
        try:
            torch.cuda.set_device(0)
            go.wait()
            for _ in range(20):
                s.step(st)
            st.synchronize()
        except Exception as e:  # surfaced below: an exception in a thread would otherwise be lost
            errors.append(e)

    threads = [threading.Thread(target=work, args=(s, st)) for s, st in zip(sessions, streams)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not errors, errors
    torch.cuda.synchronize()
    for c, s in zip(cases, sessions):
        check_case(c, s)


# ---- token-first storage order (Sec. 3.1: the layout of mainstream engines) on either or both sides
HC, TF = 0, 1
ORDERS = [(TF, TF), (TF, HC), (HC, TF)]
# (copy path, token-first addressing in the bulk-copy kernels: 1 = one bulk copy per token row, 2 = tensor-map boxes)
VARIANTS = [(LDST, 0), (BULK, 1), (BULK, 2), (PAIR, 1), (PAIR, 2)]


def _opts(tm, extra=()):
    import paper_2509_19729_b200 as A

    return ([(A.OPT_TENSOR_MAPS, tm)] if tm else []) + list(extra)


@pytest.mark.parametrize("path,tm", VARIANTS)
@pytest.mark.parametrize("so,do", ORDERS)
@pytest.mark.parametrize("a,b", [(1, 4), (4, 1), (2, 8), (8, 2), (2, 2), (1, 1)])
def test_token_first_orders_gqa(path, tm, so, do, a, b):
    lens = [1, 16, 17, 300, 0, 77, 513, 5]
    c = make_case(GQA, a, b, lens, weights=False, seed=a * 16 + b + 100 * so + 1000 * do, src_order=so, dst_order=do)
    check_case(c, run_case(c, path, options=_opts(tm)))


@pytest.mark.parametrize("path,tm", VARIANTS)
@pytest.mark.parametrize("so,do", ORDERS)
@pytest.mark.parametrize("a,b", [(4, 5), (8, 5), (10, 4), (20, 1), (5, 5)])
def test_token_first_non_nested_partitions(path, tm, so, do, a, b):
    c = make_case(SMALL40, a, b, [33, 7, 0, 64, 129], T=8, weights=False, seed=a * 64 + b, src_order=so, dst_order=do)
    check_case(c, run_case(c, path, options=_opts(tm)))


@pytest.mark.parametrize("path,tm", VARIANTS)
@pytest.mark.parametrize("so,do", ORDERS)
@pytest.mark.parametrize("chunk", [256, 1024, 4096, 32768])
def test_token_first_chunk_sizes(path, tm, so, do, chunk):
    """Work items from a quarter of a token row up to several rows (row copies) and from one token of one header up to
    a whole run of headers (boxes): column chunks, row groups, ragged groups, token groups, header groups."""
    import paper_2509_19729_b200 as A

    wide = dict(L=2, hidden=256, Hq=16, Hkv=16, D=64, I=512)  # 1->2: token rows of 8 headers = 1 KiB
    c = make_case(wide, 1, 2, [100, 3, 48], T=12, weights=False, seed=chunk, src_order=so, dst_order=do)
    check_case(c, run_case(c, path, options=_opts(tm, [(A.OPT_CHUNK_BYTES, chunk)])))


@pytest.mark.parametrize("so,do", ORDERS)
def test_token_first_bad_block_ids_are_skipped(so, do):
    """A pair with an id outside its pool moves nothing and reports BAD_BLOCK_ID, with boxes as with rows."""
    lens = [40, 40, 40]
    c0 = make_case(dict(GQA, L=1), 2, 4, lens, weights=False, seed=3)
    bt = c0.src_bt.copy()
    bt[1, 1] = c0.NB_src + 5
    c = make_case(dict(GQA, L=1), 2, 4, lens, weights=False, seed=3, src_bt_override=bt, src_order=so, dst_order=do)
    check_case(c, run_case(c))


def test_token_first_full_transformation_with_weights_and_mask():
    lens = list(np.random.default_rng(4).integers(1, 400, size=60))
    c = make_case(GQA, 2, 4, lens, dst_form="mask", dst_occupied=0.3, src_free=0.3, seed=21, src_order=TF, dst_order=TF)
    check_case(c, run_case(c))


# ---- padded weight partitions (Sec. 3.2, Improvement 1): every byte of every padded buffer, pads included
PADM = dict(L=2, hidden=256, Hq=16, Hkv=8, D=32, I=768)
PAD_CASES = [(1, 4, (4, 4096), (4, 4096)), (4, 1, (4, 4096), (4, 4096)), (2, 4, (8, 2048), (8, 2048)),
             (1, 4, (4, 4096), None), (4, 2, None, (4, 4096)), (2, 4, (8, 8192), (4, 4096)), (2, 1, (2, 4096), (8, 1024)),
             (1, 1, None, (8, 8192)), (8, 8, (8, 4096), None)]


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("a,b,sp,dp", PAD_CASES)
def test_padded_weight_partitions(path, a, b, sp, dp):
    c = make_case(PADM, a, b, [20], kv=False, seed=a * 8 + b, src_pad=sp, dst_pad=dp)
    check_case(c, run_case(c, path))


@pytest.mark.parametrize("fq,fg", [(False, False), (True, False)])
def test_padded_unfused_buffers_and_kv_together(fq, fg):
    c = make_case(PADM, 2, 4, [40, 3], fused_qkv=fq, fused_gate_up=fg, seed=12, src_pad=(4, 4096), dst_pad=(4, 4096))
    check_case(c, run_case(c))


# ---- stream capture: the data calls only enqueue work, so a transformation can be recorded once and replayed
@pytest.mark.parametrize("so,do", [(HC, HC), (TF, TF), (TF, HC)])
def test_step_replayed_from_a_cuda_graph(so, do):
    import torch

    c = make_case(GQA, 2, 4, [300, 17, 64, 5], seed=31, src_order=so, dst_order=do)
    s = run_case(c)          # one plain run first: one-time set-up (function attributes, entry points) happens here
    check_case(c, s)

    def wipe():
        for t in s.dst_pools + s._wbufs[c.a:]:
            t.fill_(0xA5)
        s.dst_bt.fill_(-2)
        s.pairs.fill_(-3)
        s.num_pairs.zero_()
        s.free_count.zero_()

    wipe()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        s.status.zero_()
        s.step()
    for _ in range(2):       # replay twice, wiping the outputs in between
        graph.replay()
        torch.cuda.synchronize()
        check_case(c, s)
        wipe()


# ---- out-of-place merge of N instances into one (distinct request sets, one shared destination free list)
def test_out_of_place_merge_of_instances_by_composition():
    """N instances of TP = a become one instance of TP = N*a in fresh pools: one table rewrite and one KV call per
    instance, each taking the part of the shared free list the earlier instances left (the caller knows the block counts
    from the sequence lengths).  Expected: the oracle's a -> N*a transformation of each instance into the same pools."""
    import torch

    import oracle as O
    import paper_2509_19729_b200 as A

    m, T, N, a = GQA, 16, 3, 2
    b = 4  # destination TP (the three instances need not fill a multiple of their own TP)
    dev = torch.device("cuda:0")
    g = np.random.default_rng(17)
    lens_all = [[100, 17, 300], [64], [5, 5, 5, 200]]
    NB_src, need = 40, sum(sum((l + T - 1) // T for l in ls) for ls in lens_all)
    NB_dst = need + 9
    free = g.permutation(NB_dst).astype(np.int32)
    exp_pools = [np.full(m["L"] * O.pool_elems_per_layer(m, T, b, NB_dst), 0xA5A5, np.uint16) for _ in range(b)]
    d_dst = [torch.full((p.size * 2,), 0xA5, dtype=torch.uint8, device=dev) for p in exp_pools]
    d_free = torch.from_numpy(free).to(dev)
    d_status = torch.zeros(1, dtype=torch.int32, device=dev)
    plan = A.amoeba_plan_create(A.make_layout(m, a, NB_src, T), A.make_layout(m, b, NB_dst, T))
    consumed, keep = 0, []
    for i, ls in enumerate(lens_all):
        lens = np.array(ls, np.int32)
        nblk = (lens + T - 1) // T
        maxb = int(nblk.max())
        bt = np.full((len(ls), maxb), -1, np.int32)
        ids = g.permutation(NB_src)
        k = 0
        for s, n in enumerate(nblk):
            bt[s, :n] = ids[k:k + n]
            k += int(n)
        KV = g.integers(0, 65536, size=(m["L"], int(nblk.sum()) * T, m["Hkv"], 2, m["D"]), dtype=np.uint16)
        src = O.kv_shard(KV, m, T, a, NB_src, lens, bt)
        # expected: this instance's blocks take the next ids of the shared list
        exp_bt, exp_pairs, n_pairs, left, st = O.assign_blocks(lens, T, bt, NB_src, NB_dst, free_list=free[consumed:])
        assert st == 0
        O.kv_transform(m, T, lens, a, NB_src, bt, src, b, NB_dst, exp_bt, exp_pools)
        # device: the same with the free list advanced by what the earlier instances took
        d_src = [torch.from_numpy(p.view(np.uint8)).to(dev) for p in src]
        d_bt, d_lens = torch.from_numpy(bt).to(dev), torch.from_numpy(lens).to(dev)
        d_new = torch.empty_like(d_bt)
        d_pairs = torch.empty((n_pairs, 2), dtype=torch.int32, device=dev)
        d_n, d_left = torch.zeros(1, dtype=torch.int32, device=dev), torch.zeros(1, dtype=torch.int32, device=dev)
        ws_bytes = A.amoeba_rewrite_workspace_bytes(plan, len(ls), NB_dst - consumed)
        ws = torch.empty(ws_bytes, dtype=torch.uint8, device=dev)
        A.amoeba_rewrite_block_tables(plan, d_bt, d_lens, len(ls), maxb, d_free[consumed:], None, NB_dst - consumed,
                                      d_new, d_pairs, n_pairs, d_n, d_left, d_status, ws, ws_bytes)
        A.amoeba_reshard_kv(plan, d_src, d_dst, d_pairs, d_n, n_pairs, 0, m["L"], d_status)
        torch.cuda.synchronize()
        assert np.array_equal(d_new.cpu().numpy(), exp_bt) and int(d_left.item()) == left
        keep.append((d_src, d_bt, d_lens, d_new, d_pairs, ws))
        consumed += n_pairs
    assert int(d_status.item()) == 0
    for r in range(b):
        assert np.array_equal(d_dst[r].cpu().numpy().view(np.uint16), exp_pools[r]), r


def test_writes_stay_inside_the_buffers():
    """Every destination buffer sits between guard regions inside one allocation; after a whole transformation (KV in
    both storage orders, weights) the guards still hold their pattern."""
    import torch

    import oracle as O
    import paper_2509_19729_b200 as A

    m, T, a, b, NB_s, NB_d = GQA, 16, 2, 4, 12, 15
    dev = torch.device("cuda:0")
    GUARD = 4096
    for order in (0, 1):
        src_l = A.make_layout(m, a, NB_s, T, kv_order=order)
        dst_l = A.make_layout(m, b, NB_d, T, kv_order=order)
        plan = A.amoeba_plan_create(src_l, dst_l)
        pool_bytes = A.amoeba_layout_kv_pool_bytes(dst_l)
        w_sizes = [A.amoeba_layout_weight_bytes(dst_l, t) for t in range(7)]
        per_rank = [pool_bytes] + [s for s in w_sizes if s] * m["L"]
        total = sum(GUARD + (s + 255) // 256 * 256 for s in per_rank) * b + GUARD
        arena = torch.full((total,), 0xC3, dtype=torch.uint8, device=dev)
        off, dst_pools, dst_w, spans = GUARD, [], [], []
        for r in range(b):
            dst_pools.append(arena[off:off + pool_bytes])
            spans.append((off, pool_bytes))
            off += (pool_bytes + 255) // 256 * 256 + GUARD
            layers = []
            for l in range(m["L"]):
                d = {}
                for t, s in enumerate(w_sizes):
                    if s:
                        d[A.TENSOR_NAMES[t]] = arena[off:off + s]
                        spans.append((off, s))
                        off += (s + 255) // 256 * 256 + GUARD
                layers.append(d)
            dst_w.append(layers)
        g = torch.Generator(device=dev).manual_seed(5)
        src_pools = [torch.randint(0, 256, (A.amoeba_layout_kv_pool_bytes(src_l),), dtype=torch.uint8, device=dev,
                                   generator=g) for _ in range(a)]
        src_w = [[{A.TENSOR_NAMES[t]: torch.randint(0, 256, (A.amoeba_layout_weight_bytes(src_l, t),), dtype=torch.uint8,
                                                    device=dev, generator=g)
                   for t in range(7) if A.amoeba_layout_weight_bytes(src_l, t)} for _ in range(m["L"])] for _ in range(a)]
        pairs = torch.tensor([[i, NB_d - 1 - i] for i in range(NB_s)], dtype=torch.int32, device=dev)
        n = torch.tensor([NB_s], dtype=torch.int32, device=dev)
        status = torch.zeros(1, dtype=torch.int32, device=dev)
        for path in PATHS:
            A.amoeba_plan_set_option(plan, A.OPT_COPY_PATH, path)
            A.amoeba_reshard_kv(plan, src_pools, dst_pools, pairs, n, NB_s, 0, m["L"], status)
            A.amoeba_reshard_weights(plan, src_w, dst_w, 0, m["L"], status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        inside = torch.zeros(total, dtype=torch.bool, device=dev)
        for o, s in spans:
            inside[o:o + s] = True
        assert bool((arena[~inside] == 0xC3).all())
        assert not bool((arena[inside] == 0xC3).all())  # and the buffers themselves were written


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("cap", [1, 7, 100000])
def test_grid_cap_leaves_results_unchanged(path, cap):
    import paper_2509_19729_b200 as A

    c = make_case(GQA, 2, 4, [300, 17, 64, 5], seed=41)
    check_case(c, run_case(c, path, options=[(A.OPT_MAX_CTAS, cap)]))


def test_random_shapes_orders_and_options():
    """Seeded random small cases: block sizes from 1 token, head dims from 8, any divisor pair of TP degrees, either
    storage order on either side, every copy path, odd chunk sizes."""
    import paper_2509_19729_b200 as A

    g = np.random.default_rng(2509)
    for trial in range(48):
        Hkv = int(g.choice([1, 2, 4, 6, 8, 12]))
        D = int(g.choice([8, 16, 40, 64, 128]))
        T = int(g.choice([1, 3, 8, 16, 32]))
        divs = [d for d in (1, 2, 3, 4, 6, 8, 12) if Hkv % d == 0]
        a, b = int(g.choice(divs)), int(g.choice(divs))
        m = dict(L=int(g.integers(1, 4)), hidden=64, Hq=Hkv * int(g.choice([1, 2])), Hkv=Hkv, D=D, I=Hkv * 16)
        so, do = int(g.integers(2)), int(g.integers(2))
        path, tm = VARIANTS[int(g.integers(len(VARIANTS)))]
        chunk = int(g.choice([16, 48, 256, 4096, 8192, 65536]))
        lens = [int(x) for x in g.integers(0, 6 * T, size=int(g.integers(1, 7)))]
        c = make_case(m, a, b, lens, T=T, weights=bool(g.integers(2)), seed=trial, src_order=so, dst_order=do)
        try:
            check_case(c, run_case(c, path, options=_opts(tm, [(A.OPT_CHUNK_BYTES, chunk)])))
        except Exception as e:
            raise AssertionError(f"trial {trial}: m={m} T={T} {a}->{b} orders {so}{do} path {path} tm {tm} chunk {chunk} "
                                 f"lens {lens}: {e}") from e


@pytest.mark.parametrize("seed", range(64))
def test_random_cases_with_ring_shapes_and_injected_errors(seed):
    """One seeded random case per seed: model shape, TP pair, block size, lengths up to hundreds of blocks, free list or
    mask, storage orders, weights, copy path, item size, ring shape, grid cap - and in a third of the cases one damaged
    input (an id twice or out of range in the free list, a bad source id, a pair list or a free list that is too short,
    a negative length).  Everything is compared with the oracle, the untouched bytes included."""
    import paper_2509_19729_b200 as A

    g = np.random.default_rng(77000 + seed)
    Hkv = int(g.choice([1, 2, 4, 6, 8, 12, 20, 40]))
    tps = [d for d in range(1, 33) if Hkv % d == 0]
    a, b = int(g.choice(tps)), int(g.choice(tps))
    m = dict(L=int(g.integers(1, 4)), hidden=64 * int(g.integers(1, 9)), Hq=Hkv * int(g.choice([1, 2, 4])), Hkv=Hkv,
             D=int(g.choice([16, 32, 64, 128])), I=int(np.lcm(a, b)) * 8 * int(g.integers(1, 12)))
    T = int(g.choice([8, 16, 32]))
    S = int(g.integers(1, 10))
    lens = [int(x) for x in g.integers(0, int(g.choice([3, 40, 300])) * T, size=S)]
    form = "mask" if g.random() < 0.35 else "list"
    kw = dict(T=T, dst_form=form, seed=seed, fused_qkv=bool(g.integers(2)), fused_gate_up=bool(g.integers(2)),
              weights=bool(g.integers(2)) and m["hidden"] * max(m["I"], m["Hq"] * m["D"]) < 3e6,
              src_order=int(g.random() < 0.3), dst_order=int(g.random() < 0.3), src_free=float(g.choice([0.0, 0.2, 0.5])))
    path = int(g.choice([LDST, BULK, PAIR, PAIR]))
    opts = [(A.OPT_CHUNK_BYTES, int(g.choice([256, 1024, 2048, 4096, 8192, 16384, 32768])))]
    for opt, lo, hi, p in ((A.OPT_STAGES, 2, 9, 0.5), (A.OPT_WARPS, 1, 9, 0.5), (A.OPT_LAG, 1, 4, 0.5),
                           (A.OPT_TENSOR_MAPS, 1, 2, 0.3), (A.OPT_L2_HINT, 1, 5, 0.3)):
        if g.random() < p:
            opts.append((opt, int(g.integers(lo, hi))))
    if g.random() < 0.3:
        opts.append((A.OPT_MAX_CTAS, int(g.choice([1, 3, 17, 100]))))
    c = make_case(m, a, b, lens, **kw)
    kind = int(g.integers(0, 6)) if g.random() < 0.35 and c.n_live > 2 else -1
    free, bt, cap = None, None, None
    if kind == 0 and form == "list":
        fl = c.free_list.copy()
        i, j = g.choice(c.n_live, 2, replace=False)
        fl[i] = fl[j]
        free = (fl, None)
    elif kind == 1 and form == "list":
        fl = c.free_list.copy()
        fl[int(g.integers(0, c.n_live))] = int(g.choice([-1, -7, c.NB_dst, c.NB_dst + 5, 2**31 - 1]))
        free = (fl, None)
    elif kind == 2:
        bt = c.src_bt.copy()
        rows, cols = np.nonzero(bt >= 0)
        k = int(g.integers(0, len(rows)))
        bt[rows[k], cols[k]] = int(g.choice([-1, -5, c.NB_src, c.NB_src + 3, 2**31 - 1]))
    elif kind == 3:
        cap = int(g.integers(0, c.n_live))
    elif kind == 4 and form == "list":
        free = (c.free_list[:int(g.integers(1, c.n_live))].copy(), None)
    elif kind == 5:
        lens[int(g.integers(0, S))] = -int(g.integers(1, 50))
    if kind >= 0:
        c = make_case(m, a, b, lens, free_override=free, src_bt_override=bt, pairs_cap=cap, **kw)
    try:
        check_case(c, run_case(c, path, options=opts))
    except Exception as e:
        raise AssertionError(f"m={m} T={T} {a}->{b} lens {lens} {kw} path {path} opts {opts} damaged {kind}: {e}") from e


@pytest.mark.parametrize("a,b", [(32, 1), (1, 32), (32, 32), (16, 32)])
def test_largest_tp_degrees(a, b):
    """The largest worker counts the library accepts: 32 pools on a side, one header per worker."""
    wide = dict(L=2, hidden=128, Hq=32, Hkv=32, D=16, I=512)
    c = make_case(wide, a, b, [70, 9, 33], T=8, seed=a + b)
    check_case(c, run_case(c))
    c = make_case(wide, a, b, [70, 9], T=8, weights=False, seed=a + b, src_order=TF, dst_order=HC)
    check_case(c, run_case(c))


@pytest.mark.parametrize("path", PATHS)
def test_weights_for_a_subset_of_destination_workers(path):
    """Each worker of a merge only needs its own new shard: destination workers passed as all-NULL are left out, the
    others get exactly what a full call gives them; a half-given worker is an error."""
    import torch

    import oracle as O
    import paper_2509_19729_b200 as A

    m, a, b = dict(GQA, L=2), 1, 4
    dev = torch.device("cuda:0")
    g = np.random.default_rng(77)
    plan = A.amoeba_plan_create(A.make_layout(m, a, 4), A.make_layout(m, b, 4))
    A.amoeba_plan_set_option(plan, A.OPT_COPY_PATH, path)
    src, exp = [], []
    for l in range(m["L"]):
        W = {n: g.integers(0, 65536, size=s, dtype=np.uint16) for n, s in O.logical_shapes(m).items()}
        sa = O.weights_shard(W, m, a)
        src.append(sa)
        exp.append(O.weights_transform(sa, m, a, b))
    d_src = [[{n: torch.from_numpy(x.reshape(-1).view(np.uint8)).to(dev) for n, x in src[l][0].items()}
              for l in range(m["L"])]]
    keep = (1, 3)  # the destination workers this call produces
    d_dst = [[({n: torch.full((x.size * 2,), 0xA5, dtype=torch.uint8, device=dev) for n, x in exp[l][r].items()}
               if r in keep else {}) for l in range(m["L"])] for r in range(b)]
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    A.amoeba_reshard_weights(plan, d_src, d_dst, 0, m["L"], status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    for r in keep:
        for l in range(m["L"]):
            for n, e in exp[l][r].items():
                assert np.array_equal(d_dst[r][l][n].cpu().numpy().view(np.uint16), e.reshape(-1)), (r, l, n)
    half = [[dict(d) for d in row] for row in d_dst]
    del half[1][0]["o"]
    with pytest.raises(A.AmoebaError) as e:
        A.amoeba_reshard_weights(plan, d_src, half, 0, m["L"], status)
    assert e.value.status == A.ERR_INVALID_ARG


@pytest.mark.parametrize("path,tm", VARIANTS)
@pytest.mark.parametrize("so,do", [(HC, HC)] + ORDERS)
def test_layers_further_apart_than_their_size(path, tm, so, do):
    """kv_layer_stride_bytes larger than a layer on both sides: the gaps between layers keep their bytes."""
    import torch

    import oracle as O
    import paper_2509_19729_b200 as A

    m, T, a, b, NB_s, NB_d = dict(GQA, L=3), 16, 2, 4, 9, 11
    lens = np.array([40, 7, 64], np.int32)
    nblk = (lens + T - 1) // T
    g = np.random.default_rng(so * 2 + do)
    bt = np.full((3, int(nblk.max())), -1, np.int32)
    ids, k = g.permutation(NB_s), 0
    for s, n in enumerate(nblk):
        bt[s, :n] = ids[k:k + n]
        k += int(n)
    s_stride = O.pool_elems_per_layer(m, T, a, NB_s) + 2048   # elements
    d_stride = O.pool_elems_per_layer(m, T, b, NB_d) + 512
    KV = g.integers(0, 65536, size=(m["L"], int(nblk.sum()) * T, m["Hkv"], 2, m["D"]), dtype=np.uint16)
    src = O.kv_shard(KV, m, T, a, NB_s, lens, bt, fill=0x5A5A, layer_stride=s_stride, order=so)
    free = g.permutation(NB_d).astype(np.int32)
    exp_bt, exp_pairs, n, _, st = O.assign_blocks(lens, T, bt, NB_s, NB_d, free_list=free)
    exp = [np.full(m["L"] * d_stride, 0xA5A5, np.uint16) for _ in range(b)]
    O.kv_transform(m, T, lens, a, NB_s, bt, src, b, NB_d, exp_bt, exp, src_order=so, dst_order=do,
                   src_layer_stride=s_stride, dst_layer_stride=d_stride)
    dev = torch.device("cuda:0")
    plan = A.amoeba_plan_create(A.make_layout(m, a, NB_s, T, kv_order=so, kv_layer_stride_bytes=2 * s_stride),
                                A.make_layout(m, b, NB_d, T, kv_order=do, kv_layer_stride_bytes=2 * d_stride))
    for o, v in [(A.OPT_COPY_PATH, path)] + _opts(tm):
        A.amoeba_plan_set_option(plan, o, v)
    assert A.amoeba_layout_kv_pool_bytes(plan.dst) == 2 * d_stride * m["L"]
    d_src = [torch.from_numpy(p.view(np.uint8)).to(dev) for p in src]
    d_dst = [torch.full((p.size * 2,), 0xA5, dtype=torch.uint8, device=dev) for p in exp]
    d_pairs = torch.from_numpy(exp_pairs).to(dev)
    d_n = torch.tensor([n], dtype=torch.int32, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    A.amoeba_reshard_kv(plan, d_src, d_dst, d_pairs, d_n, n, 0, m["L"], status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    for r in range(b):
        assert np.array_equal(d_dst[r].cpu().numpy().view(np.uint16), exp[r]), r


@pytest.mark.parametrize("hint", [1, 2, 3, 4])
@pytest.mark.parametrize("so,do", [(HC, HC), (TF, TF), (TF, HC), (HC, TF)])
def test_l2_hints_on_bulk_and_tiled_copies(hint, so, do):
    import paper_2509_19729_b200 as A

    c = make_case(GQA, 2, 4, [100, 3, 48], seed=hint, src_order=so, dst_order=do)
    check_case(c, run_case(c, PAIR, options=[(A.OPT_L2_HINT, hint)]))


# ---- partial swap (Sec. 3.2, base solution): the kept N-th of every shard moves to the front of its buffer, in place
@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("fq,fg", [(True, True), (False, False)])
@pytest.mark.parametrize("a,b,keep", [(1, 2, [1]), (1, 4, [2]), (1, 4, [0]), (2, 4, [1, 0]), (2, 8, [3, 1]), (4, 8, [1, 0, 1, 1]),
                                      (1, 8, [7])])
def test_weights_compacted_in_place(path, fq, fg, a, b, keep):
    """After the call the front of worker r's buffers is the dense TP = b shard of worker r*N + keep[r], byte for byte
    what the oracle's a -> b transformation gives that worker."""
    m = dict(L=2, hidden=96, Hq=16, Hkv=8, D=16, I=320)   # 96 rows: the waves of the column tensors end raggedly
    _compact_case(m, path, fq, fg, a, b, keep)


@pytest.mark.parametrize("fq", [True, False])
@pytest.mark.parametrize("hidden", [96, 1200])
@pytest.mark.parametrize("a,b,keep", [(1, 2, [0]), (1, 2, [1]), (2, 4, [0, 1]), (1, 4, [0]), (1, 4, [3])])
def test_weights_compacted_in_place_mha(fq, hidden, a, b, keep):
    """As many K/V heads as query heads: with N = 2 the new v section would land on rows k is still read from, so v
    moves one launch after k; hidden = 1200 takes the column tensors past the rows one CTA moves alone, with a ragged
    last wave."""
    m = dict(L=2, hidden=hidden, Hq=8, Hkv=8, D=16, I=320)
    _compact_case(m, PAIR, fq, True, a, b, keep)


@pytest.mark.parametrize("seed", range(40))
def test_random_compactions(seed):
    """Seeded random shapes for the partial swap: factor, worker count, kept parts, head counts, row counts from 16 to
    2500 (a quarter of the seeds pass the rows one CTA moves alone), fused or separate buffers, copy path, item size."""
    g = np.random.default_rng(4400 + seed)
    N, a = int(g.choice([2, 4, 8])), int(g.choice([1, 2, 4]))
    b = a * N
    Hkv = b * int(g.choice([1, 2]))
    big = seed % 4 == 0
    m = dict(L=int(g.integers(1, 3)), hidden=16 * int(g.integers(1, 160 if big else 24)), Hq=Hkv * int(g.choice([1, 2, 4])),
             Hkv=Hkv, D=int(g.choice([16, 32, 64])), I=b * 8 * int(g.integers(1, 64 if big else 12)))
    keep = [int(g.integers(0, N)) for _ in range(a)]
    _compact_case(m, int(g.choice([LDST, BULK, PAIR, PAIR])), bool(g.integers(2)), bool(g.integers(2)), a, b, keep,
                  chunk=int(g.choice([256, 1024, 4096, 8192, 16384])))


def _compact_case(m, path, fq, fg, a, b, keep, chunk=1024):
    import torch

    import oracle as O
    import paper_2509_19729_b200 as A

    N = b // a
    dev = torch.device("cuda:0")
    g = np.random.default_rng(a * 31 + b + sum(keep))
    plan = A.amoeba_plan_create(A.make_layout(m, a, 4, fused_qkv=fq, fused_gate_up=fg),
                                A.make_layout(m, b, 4, fused_qkv=fq, fused_gate_up=fg))
    A.amoeba_plan_set_option(plan, A.OPT_COPY_PATH, path)
    A.amoeba_plan_set_option(plan, A.OPT_CHUNK_BYTES, chunk)
    bufs, exp = [[None] * m["L"] for _ in range(a)], []
    for l in range(m["L"]):
        W = {n: g.integers(0, 65536, size=s, dtype=np.uint16) for n, s in O.logical_shapes(m).items()}
        sa = O.weights_shard(W, m, a, fq, fg)
        exp.append(O.weights_transform(sa, m, a, b, fq, fg))
        for r in range(a):
            bufs[r][l] = {n: torch.from_numpy(x.reshape(-1).view(np.uint8).copy()).to(dev) for n, x in sa[r].items()}
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    A.amoeba_compact_weights_inplace(plan, bufs, keep, 0, m["L"], status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    for r in range(a):
        w = r * N + keep[r]
        for l in range(m["L"]):
            for n, e in exp[l][w].items():
                got = bufs[r][l][n].cpu().numpy().view(np.uint16)[:e.size]
                assert np.array_equal(got, e.reshape(-1)), (r, l, n, m, a, b, keep, path, fq, fg, chunk)


def test_weights_compaction_host_errors():
    import torch

    import paper_2509_19729_b200 as A

    m = dict(L=1, hidden=64, Hq=8, Hkv=8, D=16, I=128)
    dev = torch.device("cuda:0")
    z = torch.zeros(1, dtype=torch.int32, device=dev)
    buf = lambda lay: [[{A.TENSOR_NAMES[t]: torch.zeros(A.amoeba_layout_weight_bytes(lay, t), dtype=torch.uint8, device=dev)
                         for t in range(7) if A.amoeba_layout_weight_bytes(lay, t)}] for _ in range(lay.tp)]

    def status_of(fn):
        with pytest.raises(A.AmoebaError) as e:
            fn()
        return e.value.status

    src = A.make_layout(m, 2, 4)
    plan = A.amoeba_plan_create(src, A.make_layout(m, 4, 4))
    assert status_of(lambda: A.amoeba_compact_weights_inplace(plan, buf(src), [0, 2], 0, 1, z)) == A.ERR_INVALID_ARG
    assert status_of(lambda: A.amoeba_compact_weights_inplace(plan, buf(src), [0, 1], 0, 2, z)) == A.ERR_INVALID_ARG
    half = buf(src)
    del half[1][0]["down"]
    assert status_of(lambda: A.amoeba_compact_weights_inplace(plan, half, [0, 1], 0, 1, z)) == A.ERR_INVALID_ARG
    for dst in (A.make_layout(m, 2, 4, weight_pad_parts=4), A.make_layout(m, 4, 4, fused_qkv=False)):
        p2 = A.amoeba_plan_create(src, dst)
        assert status_of(lambda: A.amoeba_compact_weights_inplace(p2, buf(src), [0, 0], 0, 1, z)) == A.ERR_UNSUPPORTED
    p3 = A.amoeba_plan_create(A.make_layout(m, 4, 4), A.make_layout(m, 2, 4))  # scale-down is not a compaction
    assert status_of(lambda: A.amoeba_compact_weights_inplace(p3, buf(A.make_layout(m, 4, 4)), [0] * 4, 0, 1, z)) \
        == A.ERR_UNSUPPORTED


@pytest.mark.parametrize("form", ["list", "mask"])
def test_pair_list_order_option(form):
    """The pair list comes ascending by destination id (the default; the tail holds the (-1,-1) pairs of blocks that
    were given no id) or, with the option set, in (sequence, block) order.  Tables, counts, status and the copied
    pools are the same either way."""
    import paper_2509_19729_b200 as A

    lens = [160, 48, 0, 300, 7]
    base = make_case(GQA, 2, 4, lens, weights=False, seed=8, dst_form=form)
    if form == "list":
        free = base.free_list.copy()
        free[5] = free[1]          # one block is refused: its pair goes to the tail in destination order
        c = make_case(GQA, 2, 4, lens, weights=False, seed=8, free_override=(free, None))
        assert c.exp_status == 5
    else:
        c = base
    for order in (A.PAIR_ORDER_DESTINATION, A.PAIR_ORDER_TABLE):
        s = run_case(c, PAIR, options=[(A.OPT_PAIR_ORDER, order)])
        got = s.pairs.cpu().numpy()[:c.exp_n]
        if order == A.PAIR_ORDER_TABLE:
            assert np.array_equal(got, c.exp_pairs)
        else:
            live = got[got[:, 1] >= 0, 1]
            assert np.all(np.diff(live) > 0) and np.all(got[len(live):] == -1)
            assert sorted(map(tuple, got)) == sorted(map(tuple, c.exp_pairs))
        assert int(s.num_pairs.item()) == c.exp_n and int(s.status.item()) == c.exp_status
        assert np.array_equal(s.dst_bt.cpu().numpy(), c.exp_dst_bt)
        for t, e in zip(s.dst_pools, c.exp_dst_pools):
            assert np.array_equal(t.cpu().numpy().view(np.uint16), e)


@pytest.mark.parametrize("path", PATHS)
def test_free_list_that_names_an_id_twice(path):
    """Two blocks must never share a destination: the first block (in sequence, block order) given an id keeps it,
    a later one gets none (entry -1, pair (-1,-1), BAD_BLOCK_ID) and is not copied."""
    lens = [160, 48, 300]
    base = make_case(GQA, 2, 1, lens, weights=False, seed=6)
    free = base.free_list.copy()
    free[7] = free[2]
    free[20] = free[2]
    free[11] = free[30]  # the later entry (30) loses
    c = make_case(GQA, 2, 1, lens, weights=False, seed=6, free_override=(free, None))
    assert c.exp_status == 5 and (c.exp_pairs[[7, 20, 30]] == -1).all() and c.exp_pairs[11, 1] == free[30]
    check_case(c, run_case(c, path))


def test_out_of_place_calls_refuse_a_buffer_on_both_sides():
    import paper_2509_19729_b200 as A

    c = make_case(GQA, 2, 2, [40], seed=1)
    s = run_case(c, PAIR)
    with pytest.raises(A.AmoebaError) as e:
        A.amoeba_reshard_kv(s.plan, s.src_pools, [s.dst_pools[0], s.src_pools[1]], s.pairs, s.num_pairs, s.pairs_cap,
                            0, 1, s.status)
    assert e.value.status == A.ERR_INVALID_ARG
    dst = [[dict(d) for d in r] for r in s.dst_w]
    dst[1][0]["o"] = s.src_w[1][0]["o"]
    with pytest.raises(A.AmoebaError) as e:
        A.amoeba_reshard_weights(s.plan, s.src_w, dst, 0, 1, s.status)
    assert e.value.status == A.ERR_INVALID_ARG
    check_case(c, s)  # the refused calls launched nothing


@pytest.mark.parametrize("path", [BULK, PAIR])
def test_wait_budget_running_out_is_reported_and_the_next_call_is_exact(path):
    """Every wait of a copy kernel on its own bulk copies is bounded.  With the smallest budget (give up without
    polling) the first wait of every ring runs out although its load is healthy: the kernel must record TIMEOUT, let
    the copies it has in flight land, and return - nothing outside the destination buffers is touched, the context
    stays usable, and the same call with the default budget then gives the exact result."""
    import torch

    import paper_2509_19729_b200 as A

    c = make_case(GQA, 2, 4, [300, 77, 1024, 5, 640], seed=12)
    s = run_case(c, path, options=[(A.OPT_WAIT_TRIES, 1)])
    assert int(s.status.item()) == A.ERR_TIMEOUT
    for t, e in zip(s.src_pools, c.src_pools):  # sources are never written
        assert np.array_equal(t.cpu().numpy().view(np.uint16), e)
    for t, e in zip(s.dst_pools, c.exp_dst_pools):  # every destination word is either untouched or already right
        got = t.cpu().numpy().view(np.uint16)
        assert np.all((got == e) | (got == 0xA5A5))
    s.set_option(A.OPT_WAIT_TRIES, 0)
    s.status.zero_()
    s.step()
    torch.cuda.synchronize()
    check_case(c, s)


@pytest.mark.parametrize("seed", range(24))
def test_random_tables_with_damaged_inputs(seed):
    """The table kernels alone on random inputs, small enough for one launch or large enough for three: lengths with
    zeros, free lists with repeated and out-of-range ids, source tables with holes and out-of-range ids, masks, too
    few free blocks, a pair capacity that is too small - every output word against the oracle."""
    import torch

    import oracle as O
    import paper_2509_19729_b200 as A

    g = np.random.default_rng(5000 + seed)
    T = 16
    big = seed % 3 == 2
    S = int(g.integers(1, 400 if big else 40))
    lens = g.integers(0, (60 if big else 12) * T, size=S).astype(np.int32)
    lens[g.random(S) < 0.15] = 0
    nblk = (lens + T - 1) // T
    maxb = max(int(nblk.max()), 1) + int(g.integers(0, 3))
    total = int(nblk.sum())
    NB_src = total + int(g.integers(1, 50))
    NB_dst = max(1, total + int(g.integers(-3, 60)))
    bt = np.full((S, maxb), -1, np.int32)
    ids, k = g.permutation(NB_src), 0
    for s, n in enumerate(nblk):
        bt[s, :n] = ids[k:k + n]
        k += int(n)
    live = np.argwhere(bt >= 0)
    for s, i in live[g.random(len(live)) < 0.03]:      # holes and out-of-range source ids
        bt[s, i] = int(g.choice([-1, NB_src, NB_src + 7]))
    use_mask = seed % 2 == 1
    free_list = free_mask = None
    if use_mask:
        free_mask = (g.random(NB_dst) < 0.8).astype(np.uint8)
    else:
        n_free = max(0, total + int(g.integers(-2, 20)))
        free_list = g.integers(0, NB_dst, size=n_free).astype(np.int32) if seed % 4 == 0 \
            else g.permutation(max(NB_dst, n_free))[:n_free].astype(np.int32)   # repeats / ids beyond the pool
        if n_free:
            free_list[g.random(n_free) < 0.02] = NB_dst + 3
    pairs_cap = total if seed % 5 else max(0, total - 1)
    if seed % 7 == 3 and S > 1:
        lens[1] = -5
    m = dict(L=1, hidden=128, Hq=8, Hkv=8, D=64, I=256)
    plan = A.amoeba_plan_create(A.make_layout(m, 2, NB_src, T), A.make_layout(m, 4, NB_dst, T))
    if seed % 2 == 0 and seed % 3 != 0:
        A.amoeba_plan_set_option(plan, A.OPT_PAIR_ORDER, A.PAIR_ORDER_TABLE)
    e_bt, e_pairs, e_n, e_left, e_st = O.assign_blocks(lens, T, bt, NB_src, NB_dst, free_list=free_list,
                                                       free_mask=free_mask, pairs_cap=pairs_cap)
    dev = torch.device("cuda:0")
    i32 = dict(dtype=torch.int32, device=dev)
    d_bt, d_lens = torch.from_numpy(bt).to(dev), torch.from_numpy(lens).to(dev)
    d_new = torch.full(bt.shape, -2, **i32)
    d_pairs = torch.full((max(pairs_cap, 1), 2), -3, **i32)
    d_n, d_left, d_status = torch.zeros(1, **i32), torch.zeros(1, **i32), torch.zeros(1, **i32)
    d_free = torch.from_numpy(free_list).to(dev) if free_list is not None and len(free_list) else \
        (torch.zeros(1, **i32) if free_list is not None else None)
    d_mask = torch.from_numpy(free_mask).to(dev) if use_mask else None
    n_arg = NB_dst if use_mask else len(free_list)
    ws_bytes = A.amoeba_rewrite_workspace_bytes(plan, S, n_arg)
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device=dev)
    A.amoeba_rewrite_block_tables(plan, d_bt, d_lens, S, maxb, d_free, d_mask, n_arg, d_new, d_pairs, pairs_cap, d_n,
                                  d_left, d_status, ws, ws_bytes)
    torch.cuda.synchronize()
    assert int(d_status.item()) == e_st
    assert int(d_n.item()) == e_n and int(d_left.item()) == e_left
    assert np.array_equal(d_new.cpu().numpy(), e_bt)
    table_order = seed % 2 == 0 and seed % 3 != 0   # both pair orders get their share of the seeds
    assert np.array_equal(d_pairs.cpu().numpy()[:e_n],
                          e_pairs if table_order else pairs_in_destination_order(e_pairs, e_bt, lens, T))


@pytest.mark.parametrize("so,do", [(HC, HC), (TF, HC), (HC, TF)])
@pytest.mark.parametrize("e,a,b", [(1, 2, 4), (1, 4, 1), (4, 1, 2), (4, 8, 2)])
def test_element_sizes_one_and_four_bytes(e, a, b, so, do):
    """Elements are opaque, so a state of e-byte elements is byte for byte a 16-bit state with the innermost extent
    scaled by e/2: head_dim for the KV cache, the input width for the row-split weights, the column count for the
    column-split ones.  The 16-bit oracle gives the expected bytes; the library runs with elem_bytes = e."""
    import torch

    import oracle as O
    from paper_2509_19729_b200.session import Session

    m = dict(L=2, hidden=256, Hq=16, Hkv=8, D=64, I=512)           # the model as the library sees it
    scale = lambda x: x * e // 2
    lens = [1, 16, 17, 200, 0, 77]
    # ---- KV: the same bytes as 16-bit words with head_dim * e / 2
    ckv = make_case(dict(m, D=scale(m["D"])), a, b, lens, weights=False, seed=e * 10 + a, src_order=so, dst_order=do)
    s = Session(m, a, b, ckv.NB_src, ckv.NB_dst, len(lens), ckv.maxb, ckv.pairs_cap, weights=False, elem_bytes=e,
                src_kv_order=so, dst_kv_order=do)
    s.set_tables(ckv.seq_lens, ckv.src_bt, ckv.free_list, ckv.free_mask)
    for t, p in zip(s.src_pools, ckv.src_pools):
        assert t.numel() == p.nbytes
        t.copy_(torch.from_numpy(p.view(np.uint8)))
    s.step()
    torch.cuda.synchronize()
    check_case(ckv, s)
    # ---- weights: row-split tensors as 16-bit rows of hidden * e / 2, column-split ones with head_dim and I scaled
    rows_m = dict(m, hidden=scale(m["hidden"]))
    cols_m = dict(m, D=scale(m["D"]), I=scale(m["I"]))
    g = np.random.default_rng(e)
    w = Session(m, a, b, 4, 4, 1, 1, 1, kv=False, elem_bytes=e)
    expected = []
    for l in range(m["L"]):
        Wr = {n: g.integers(0, 65536, size=sh, dtype=np.uint16) for n, sh in O.logical_shapes(rows_m).items()}
        Wc = {n: g.integers(0, 65536, size=sh, dtype=np.uint16) for n, sh in O.logical_shapes(cols_m).items()}
        src_r, src_c = O.weights_shard(Wr, rows_m, a), O.weights_shard(Wc, cols_m, a)
        exp_r, exp_c = O.weights_transform(src_r, rows_m, a, b), O.weights_transform(src_c, cols_m, a, b)
        pick = lambda rs, cs: {"q": rs["q"], "gate": rs["gate"], "o": cs["o"], "down": cs["down"]}
        for r in range(a):
            for n, arr in pick(src_r[r], src_c[r]).items():
                assert w.src_w[r][l][n].numel() == arr.nbytes, (n, w.src_w[r][l][n].numel(), arr.nbytes)
                w.src_w[r][l][n].copy_(torch.from_numpy(arr.reshape(-1).view(np.uint8)))
        expected.append([pick(exp_r[r], exp_c[r]) for r in range(b)])
    w.reshard_weights()
    torch.cuda.synchronize()
    assert int(w.status.item()) == 0
    for l in range(m["L"]):
        for r in range(b):
            for n, arr in expected[l][r].items():
                got = w.dst_w[r][l][n].cpu().numpy().view(np.uint16)
                assert np.array_equal(got, arr.reshape(-1)), (l, r, n)

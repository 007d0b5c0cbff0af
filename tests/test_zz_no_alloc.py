"""The built-in-scratch variant of the block-table rewrite, for callers that cannot allocate device memory (a
serving process whose pool already owns the GPU, a no-allocation region, a plug-in without an allocator).

It must give exactly what the ordinary entry point gives and what the CPU oracle gives (integer outputs: bit-exact,
the tolerance every table test here uses), on two calls in a row that share the library's scratch array; it must
take no device memory; and it must refuse problems larger than the array.  Collected last so that a run stopping at
the first failure has already run everything else."""
import numpy as np
import pytest

import workloads as wl
from harness import pairs_in_destination_order

pytestmark = pytest.mark.gpu


def _outputs(s):
    import torch

    torch.cuda.synchronize()
    return [t.cpu().numpy().copy() for t in (s.dst_bt, s.pairs, s.num_pairs, s.free_count, s.status)]


def _session(model, a, b, lens, dst_form, seed):
    from paper_2509_19729_b200.session import Session

    cfg = dict(model=model, S=len(lens), src_free=0.2, dst_form=dst_form, dst_slack=0.1, dst_occupied=0.3)
    st = wl.draw_kv_state(cfg, seed=seed, name="noalloc", seq_lens=lens)
    s = Session(model, a, b, st["NB_src"], st["NB_dst"], len(lens), st["maxb"], st["n_live"], kv=False, weights=False)
    s.set_tables(st["seq_lens"], st["src_bt"], st.get("dst_free_list"), st.get("dst_free_mask"))
    s.state = st
    return s


def _oracle_outputs(oracle, s, T=16):
    st = s.state
    dst_bt, pairs, n, left, status = oracle.assign_blocks(st["seq_lens"], T, st["src_bt"], st["NB_src"], st["NB_dst"],
                                                          free_list=st.get("dst_free_list"),
                                                          free_mask=st.get("dst_free_mask"), pairs_cap=s.pairs_cap)
    return dst_bt, pairs, n, left, status


def _reset(s):
    s.dst_bt.fill_(-2)
    s.pairs.fill_(-3)
    s.num_pairs.zero_()
    s.free_count.zero_()
    s.status.zero_()


def test_builtin_scratch_matches_workspace_entry_point_twice_in_a_row(oracle):
    import torch

    import paper_2509_19729_b200 as A

    assert torch.cuda.is_available()
    model = dict(L=1, hidden=128, Hq=8, Hkv=8, D=64, I=256)
    g = np.random.default_rng(5)
    # two different problems back to back: the second call sees whatever the first left in the shared scratch
    cases = [(_session(model, 2, 4, g.integers(0, 700, size=300).astype(np.int32), "list", 1), "list"),
             (_session(model, 4, 1, g.integers(1, 90, size=1500).astype(np.int32), "mask", 2), "mask")]
    expected = []
    for s, _ in cases:
        _reset(s)
        s.rewrite_block_tables()  # the existing entry point, caller-supplied workspace
        expected.append(_outputs(s))
        assert int(expected[-1][4][0]) == 0 and int(expected[-1][2][0]) > 0
    # the first call on the device resolves the scratch array's address; from then on no call may take device memory
    s0 = cases[0][0]
    _reset(s0)
    A.amoeba_rewrite_block_tables_builtin_scratch(s0.plan, s0.src_bt, s0.seq_lens, s0.num_seqs, s0.maxb, s0.free_list,
                                                  s0.free_mask, s0.n_free_or_nb, s0.dst_bt, s0.pairs, s0.pairs_cap,
                                                  s0.num_pairs, s0.free_count, s0.status)
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    torch_before = torch.cuda.memory_allocated()
    got = []
    for s, _ in cases:  # issued back to back on one stream, no synchronisation in between
        _reset(s)
        A.amoeba_rewrite_block_tables_builtin_scratch(s.plan, s.src_bt, s.seq_lens, s.num_seqs, s.maxb, s.free_list,
                                                      s.free_mask, s.n_free_or_nb, s.dst_bt, s.pairs, s.pairs_cap,
                                                      s.num_pairs, s.free_count, s.status)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before and torch.cuda.memory_allocated() == torch_before
    for s, _ in cases:
        got.append(_outputs(s))
    for e, o in zip(expected, got):
        for x, y in zip(e, o):
            assert np.array_equal(x, y)
    for (s, _), o in zip(cases, got):  # and against the CPU oracle directly
        e_bt, e_pairs, e_n, e_left, e_status = _oracle_outputs(oracle, s)
        assert e_status == 0 and int(o[4][0]) == 0
        assert np.array_equal(o[0], e_bt) and int(o[2][0]) == e_n and int(o[3][0]) == e_left
        assert np.array_equal(o[1][:e_n], pairs_in_destination_order(e_pairs, e_bt, s.state["seq_lens"], 16))
        assert np.all(o[1][e_n:] == -3)
    # and once more in the opposite order
    for (s, _), e in reversed(list(zip(cases, expected))):
        _reset(s)
        A.amoeba_rewrite_block_tables_builtin_scratch(s.plan, s.src_bt, s.seq_lens, s.num_seqs, s.maxb, s.free_list,
                                                      s.free_mask, s.n_free_or_nb, s.dst_bt, s.pairs, s.pairs_cap,
                                                      s.num_pairs, s.free_count, s.status)
        for x, y in zip(e, _outputs(s)):
            assert np.array_equal(x, y)


def test_builtin_scratch_refuses_oversized_problems():
    import paper_2509_19729_b200 as A

    model = dict(L=1, hidden=128, Hq=8, Hkv=8, D=64, I=256)
    s = _session(model, 1, 2, np.array([16, 32], np.int32), "list", 3)
    _reset(s)
    # a destination pool of this many blocks needs one scratch word per block id: more than the array holds
    too_many = A.BUILTIN_SCRATCH_BYTES // 4
    big = A.amoeba_plan_create(A.make_layout(model, 1, s.src_layout.num_blocks), A.make_layout(model, 2, too_many))
    assert A.amoeba_rewrite_workspace_bytes(big, s.num_seqs, s.n_free_or_nb) > A.BUILTIN_SCRATCH_BYTES
    with pytest.raises(A.AmoebaError) as e:
        A.amoeba_rewrite_block_tables_builtin_scratch(big, s.src_bt, s.seq_lens, s.num_seqs, s.maxb, s.free_list,
                                                      None, s.n_free_or_nb, s.dst_bt, s.pairs, s.pairs_cap,
                                                      s.num_pairs, s.free_count, s.status)
    assert e.value.status == A.ERR_TOO_LARGE
    out = _outputs(s)
    assert np.all(out[0] == -2) and np.all(out[1] == -3) and int(out[4][0]) == 0  # nothing was launched
    # a long free LIST alone is no reason to refuse: the scratch does not hold the list
    assert A.amoeba_rewrite_workspace_bytes(s.plan, s.num_seqs, 10 * too_many) <= A.BUILTIN_SCRATCH_BYTES

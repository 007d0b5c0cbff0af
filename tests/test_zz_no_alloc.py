"""The built-in-scratch variant of the block-table rewrite, for callers that cannot allocate device memory (a
serving process whose pool already owns the GPU, a no-allocation region, a plug-in without an allocator).

It must give exactly what the ordinary entry point gives (integer outputs: bit-exact, the tolerance every table
test here uses), on two calls in a row that share the library's scratch array, and must refuse problems larger
than the array.  Collected last so that a run stopping at the first failure has already run everything else."""
import numpy as np
import pytest

import workloads as wl

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
    return s


def _reset(s):
    s.dst_bt.fill_(-2)
    s.pairs.fill_(-3)
    s.num_pairs.zero_()
    s.free_count.zero_()
    s.status.zero_()


def test_builtin_scratch_matches_workspace_entry_point_twice_in_a_row():
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
    got = []
    for s, _ in cases:  # issued back to back on one stream, no synchronisation in between
        _reset(s)
        A.amoeba_rewrite_block_tables_builtin_scratch(s.plan, s.src_bt, s.seq_lens, s.num_seqs, s.maxb, s.free_list,
                                                      s.free_mask, s.n_free_or_nb, s.dst_bt, s.pairs, s.pairs_cap,
                                                      s.num_pairs, s.free_count, s.status)
    for s, _ in cases:
        got.append(_outputs(s))
    for e, o in zip(expected, got):
        for x, y in zip(e, o):
            assert np.array_equal(x, y)
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
    too_many = A.BUILTIN_SCRATCH_BYTES // 4  # this many free-list entries alone overflow the array
    assert A.amoeba_rewrite_workspace_bytes(s.plan, s.num_seqs, too_many) > A.BUILTIN_SCRATCH_BYTES
    with pytest.raises(A.AmoebaError) as e:
        A.amoeba_rewrite_block_tables_builtin_scratch(s.plan, s.src_bt, s.seq_lens, s.num_seqs, s.maxb, s.free_list,
                                                      None, too_many, s.dst_bt, s.pairs, s.pairs_cap, s.num_pairs,
                                                      s.free_count, s.status)
    assert e.value.status == A.ERR_TOO_LARGE
    out = _outputs(s)
    assert np.all(out[0] == -2) and np.all(out[1] == -3) and int(out[4][0]) == 0  # nothing was launched

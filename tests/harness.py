"""Shared test plumbing: build a seeded case, get the expected result from the CPU oracle, run the CUDA path
through the C-ABI binding, and compare everything byte for byte."""
from __future__ import annotations

import numpy as np

import oracle
import workloads as wl

FILL16 = 0xA5A5  # destination words before the call (0xA5 bytes)


class Case:
    pass


def pairs_in_destination_order(pairs, dst_bt, seq_lens, T):
    """The oracle's pair list in the order the library writes it by default (ascending by destination id)."""
    return oracle.pairs_by_destination(pairs, dst_bt, seq_lens, T)


def make_case(model, a, b, seq_lens, T=16, src_free=0.2, dst_form="list", dst_slack=0.25, dst_occupied=0.3, seed=0,
              fused_qkv=True, fused_gate_up=True, weights=True, kv=True, dtype="bf16", free_override=None,
              src_bt_override=None, pairs_cap=None, src_order=0, dst_order=0, src_pad=None, dst_pad=None):
    """Seeded inputs + the oracle's expected outputs for one TP a->b transformation."""
    c = Case()
    c.model, c.a, c.b, c.T, c.fq, c.fg = model, a, b, T, fused_qkv, fused_gate_up
    c.src_order, c.dst_order = src_order, dst_order  # 0 header-centric, 1 token-first (same codes on both sides)
    c.src_pad, c.dst_pad = src_pad, dst_pad          # (partitions P, page bytes) of padded weight buffers, or None
    cfg = dict(model=model, dtype=dtype, S=len(seq_lens), src_free=src_free, dst_form=dst_form, dst_slack=dst_slack,
               dst_occupied=dst_occupied)
    st = wl.draw_kv_state(cfg, seed=seed, name="case", seq_lens=np.maximum(np.asarray(seq_lens), 0), T=T)
    c.seq_lens = np.asarray(seq_lens, dtype=np.int32)
    c.src_bt = st["src_bt"] if src_bt_override is None else src_bt_override
    c.NB_src, c.NB_dst, c.maxb, c.n_live = st["NB_src"], st["NB_dst"], st["maxb"], st["n_live"]
    c.free_list = st.get("dst_free_list")
    c.free_mask = st.get("dst_free_mask")
    if free_override is not None:
        c.free_list, c.free_mask = free_override
        c.NB_dst = len(c.free_mask) if c.free_mask is not None else c.NB_dst
    c.pairs_cap = c.src_bt.size if pairs_cap is None else pairs_cap
    L = model["L"]
    g = wl.rng(seed, "case_values")
    # source state: logical tensors drawn, sharded for TP=a by the oracle
    c.kv = kv
    if kv:
        G = int(st["blocks_per_seq"].sum()) * T
        c.KV = g.integers(0, 65536, size=(L, G, model["Hkv"], 2, model["D"]), dtype=np.uint16)
        valid_lens = np.maximum(c.seq_lens, 0)
        c.src_pools = oracle.kv_shard(c.KV, model, T, a, c.NB_src, valid_lens, st["src_bt"], fill=0x5A5A,
                                      order=src_order)
    # expected tables
    c.exp_dst_bt, c.exp_pairs, c.exp_n, c.exp_left, c.exp_status = oracle.assign_blocks(
        c.seq_lens, T, c.src_bt, c.NB_src, c.NB_dst, free_list=c.free_list, free_mask=c.free_mask,
        pairs_cap=c.pairs_cap)
    if kv:
        c.exp_dst_pools = [np.full(L * oracle.pool_elems_per_layer(model, T, b, c.NB_dst), FILL16, np.uint16)
                           for _ in range(b)]
        if c.exp_status == 0:
            oracle.kv_transform(model, T, c.seq_lens, a, c.NB_src, c.src_bt, c.src_pools, b, c.NB_dst, c.exp_dst_bt,
                                c.exp_dst_pools, src_order=src_order, dst_order=dst_order)
        else:
            st2 = oracle.kv_copy_pairs(model, T, a, c.NB_src, c.src_pools, b, c.NB_dst, c.exp_dst_pools, c.exp_pairs,
                                       c.exp_n, status=c.exp_status, src_order=src_order, dst_order=dst_order)
            assert st2 == c.exp_status
    c.weights = weights
    if weights:
        c.src_w, c.exp_dst_w = [], []
        for l in range(L):
            W = {n: g.integers(0, 65536, size=s, dtype=np.uint16) for n, s in oracle.logical_shapes(model).items()}
            if src_pad or dst_pad:
                opad = lambda pad: (pad[0], pad[1] // 2) if pad else None  # the oracle counts pages in elements
                sa = (oracle.weights_shard_padded(W, model, a, *opad(src_pad), fused_qkv, fused_gate_up, fill=0x5A5A)
                      if src_pad else oracle.weights_shard(W, model, a, fused_qkv, fused_gate_up))
                c.src_w.append(sa)
                c.exp_dst_w.append(oracle.weights_transform_any(sa, model, a, b, fused_qkv, fused_gate_up,
                                                                src_pad=opad(src_pad), dst_pad=opad(dst_pad),
                                                                fill=FILL16))
                continue
            sa = oracle.weights_shard(W, model, a, fused_qkv, fused_gate_up)
            c.src_w.append(sa)
            c.exp_dst_w.append(oracle.weights_transform(sa, model, a, b, fused_qkv, fused_gate_up))
    return c


def run_case(c, copy_path=None, options=(), device="cuda:0", steps=1):
    """Run the case on the GPU; returns the Session (synchronised)."""
    import torch

    import paper_2509_19729_b200 as A
    from paper_2509_19729_b200.session import Session

    s = Session(c.model, c.a, c.b, c.NB_src, c.NB_dst, len(c.seq_lens), c.maxb, c.pairs_cap, kv=c.kv,
                weights=c.weights, fused_qkv=c.fq, fused_gate_up=c.fg, block_tokens=c.T, device=device,
                src_kv_order=c.src_order, dst_kv_order=c.dst_order, src_weight_pad=c.src_pad,
                dst_weight_pad=c.dst_pad)
    if copy_path is not None:
        s.set_option(A.OPT_COPY_PATH, copy_path)
    for opt, val in options:
        s.set_option(opt, val)
    s.set_tables(c.seq_lens, c.src_bt, c.free_list, c.free_mask)
    if c.kv:
        for t, p in zip(s.src_pools, c.src_pools):
            t.copy_(torch.from_numpy(p.view(np.uint8)))
    if c.weights:
        for r in range(c.a):
            for l in range(c.model["L"]):
                for n, arr in c.src_w[l][r].items():
                    s.src_w[r][l][n].copy_(torch.from_numpy(arr.reshape(-1).view(np.uint8)))
    for _ in range(steps):
        s.status.zero_()
        s.step()
    torch.cuda.synchronize()
    return s


def check_case(c, s):
    """Bit-exact comparison of every output buffer with the oracle's."""
    st = int(s.status.item())
    assert st == c.exp_status, f"status {st} != {c.exp_status}"
    assert int(s.num_pairs.item()) == c.exp_n
    assert int(s.free_count.item()) == c.exp_left
    assert np.array_equal(s.dst_bt.cpu().numpy(), c.exp_dst_bt)
    assert np.array_equal(s.pairs.cpu().numpy()[:c.exp_n],
                          pairs_in_destination_order(c.exp_pairs, c.exp_dst_bt, c.seq_lens, c.T))
    assert np.all(s.pairs.cpu().numpy()[c.exp_n:] == -3)  # pair slots past N untouched
    if c.kv:
        for r, (t, e) in enumerate(zip(s.dst_pools, c.exp_dst_pools)):
            got = t.cpu().numpy().view(np.uint16)
            if not np.array_equal(got, e):
                bad = np.flatnonzero(got != e)
                raise AssertionError(f"dst pool {r}: {bad.size} words differ, first at {bad[0]}")
        for t, e in zip(s.src_pools, c.src_pools):  # sources are read-only
            assert np.array_equal(t.cpu().numpy().view(np.uint16), e)
    if c.weights:
        for r in range(c.b):
            for l in range(c.model["L"]):
                for n, e in c.exp_dst_w[l][r].items():
                    got = s.dst_w[r][l][n].cpu().numpy().view(np.uint16)
                    if not np.array_equal(got, e.reshape(-1)):
                        bad = np.flatnonzero(got != e.reshape(-1))
                        raise AssertionError(f"dst weight rank {r} layer {l} {n}: {bad.size} words differ, first {bad[0]}")
        # carved gaps between weight buffers keep the fill
        for r, buf in enumerate(s._wbufs[c.a:]):
            total = buf.numel()
            used = sum(v.numel() for lay in s.dst_w[r] for v in lay.values())
            assert int((buf == 0xA5).sum().item()) >= total - used

"""Device-side state of one TP a->b transformation and the calls that run it.

Plumbing only: allocates the source and destination buffers with torch (sizes come from the C library), uploads
tables, and issues the three C-ABI calls of one transformation in order.  No re-layout arithmetic lives here.
"""
from __future__ import annotations

from typing import Optional

import torch

from . import binding as A


def _carve(buf: torch.Tensor, sizes, align: int = 256):
    """Views of `sizes` bytes each into one uint8 buffer, each starting on an `align` boundary."""
    out, off = [], 0
    for n in sizes:
        out.append(buf[off:off + n])
        off += (n + align - 1) // align * align
    return out


def _carved_bytes(sizes, align: int = 256) -> int:
    return sum((n + align - 1) // align * align for n in sizes)


class Session:
    """All buffers of one transformation on one GPU.

    model: shape dict (L, hidden, Hq, Hkv, D, I); a, b: source / destination TP; NB_src / NB_dst: pool capacities;
    kv_layers: number of layers the KV pools hold (the first kv_layers layers; None = all); weights: allocate the
    weight shards too; src_weight_pad / dst_weight_pad: (partitions P, page bytes) for padded weight buffers.  Buffers are uint8 tensors; KV pools are one tensor per worker.
    """

    def __init__(self, model: dict, a: int, b: int, NB_src: int, NB_dst: int, num_seqs: int, max_blocks_per_seq: int,
                 pairs_cap: int, kv_layers: Optional[int] = None, kv: bool = True, weights: bool = True,
                 fused_qkv: bool = True, fused_gate_up: bool = True, block_tokens: int = 16, device="cuda:0",
                 dst_fill: Optional[int] = 0xA5, src_kv_order: int = A.KV_HEAD_MAJOR,
                 dst_kv_order: int = A.KV_HEAD_MAJOR, src_weight_pad=None, dst_weight_pad=None, elem_bytes: int = 2):
        self.model, self.a, self.b = model, a, b
        self.device = torch.device(device)
        pad = lambda p: dict(weight_pad_parts=p[0], weight_page_bytes=p[1]) if p else {}  # (P, page bytes) or None
        self.src_layout = A.make_layout(model, a, NB_src, block_tokens, fused_qkv, fused_gate_up, elem_bytes,
                                        kv_order=src_kv_order, **pad(src_weight_pad))
        self.dst_layout = A.make_layout(model, b, NB_dst, block_tokens, fused_qkv, fused_gate_up, elem_bytes,
                                        kv_order=dst_kv_order, **pad(dst_weight_pad))
        self.plan = A.amoeba_plan_create(self.src_layout, self.dst_layout)
        self.info = A.amoeba_plan_kv_info(self.plan)
        self.L = model["L"]
        self.kv_layers = self.L if kv_layers is None else kv_layers
        self.num_seqs, self.maxb, self.pairs_cap = num_seqs, max_blocks_per_seq, pairs_cap
        dev = self.device
        i32 = dict(dtype=torch.int32, device=dev)
        # tables
        self.src_bt = torch.full((num_seqs, max_blocks_per_seq), -1, **i32)
        self.dst_bt = torch.full((num_seqs, max_blocks_per_seq), -2, **i32)
        self.seq_lens = torch.zeros(num_seqs, **i32)
        self.pairs = torch.full((max(pairs_cap, 1), 2), -3, **i32)
        self.num_pairs = torch.zeros(1, **i32)
        self.free_count = torch.zeros(1, **i32)
        self.status = torch.zeros(1, **i32)
        self.free_list = None
        self.free_mask = None
        self.workspace = None
        # KV pools: only the first kv_layers layers are held
        self.src_pools, self.dst_pools = [], []
        if kv:
            for lay, tp, pools in ((self.src_layout, a, self.src_pools), (self.dst_layout, b, self.dst_pools)):
                per_layer = A.amoeba_layout_kv_pool_bytes(lay) // self.L
                for _ in range(tp):
                    pools.append(torch.empty(per_layer * self.kv_layers, dtype=torch.uint8, device=dev))
            if dst_fill is not None:
                for p in self.dst_pools:
                    p.fill_(dst_fill)
        # weights: one buffer per worker, carved into [layer][tensor] views
        self.src_w, self.dst_w, self._wbufs = [], [], []
        if weights:
            for lay, tp, out in ((self.src_layout, a, self.src_w), (self.dst_layout, b, self.dst_w)):
                sizes = [A.amoeba_layout_weight_bytes(lay, t) for t in range(len(A.TENSOR_NAMES))]
                used = [(n, s) for n, s in zip(A.TENSOR_NAMES, sizes) if s]
                for _ in range(tp):
                    buf = torch.empty(_carved_bytes([s for _, s in used]) * self.L, dtype=torch.uint8, device=dev)
                    views = _carve(buf, [s for _, s in used] * self.L)
                    self._wbufs.append(buf)
                    out.append([{n: views[l * len(used) + i] for i, (n, _) in enumerate(used)} for l in range(self.L)])
            if dst_fill is not None:
                for buf in self._wbufs[a:]:
                    buf.fill_(dst_fill)
            self._src_w_packed = A.pack_weights(self.src_w)
            self._dst_w_packed = A.pack_weights(self.dst_w)

    # ---- inputs
    def set_tables(self, seq_lens, src_bt, free_list=None, free_mask=None) -> None:
        """Upload sequence lengths, the source block table and the destination free blocks (numpy or torch, host)."""
        self.seq_lens.copy_(torch.as_tensor(seq_lens, dtype=torch.int32))
        self.src_bt.copy_(torch.as_tensor(src_bt, dtype=torch.int32))
        assert (free_list is None) != (free_mask is None)
        if free_list is not None:
            self.free_list = torch.as_tensor(free_list, dtype=torch.int32).to(self.device)
            self.free_mask, n = None, self.free_list.numel()
        else:
            self.free_mask = torch.as_tensor(free_mask, dtype=torch.uint8).to(self.device)
            self.free_list, n = None, self.free_mask.numel()
        self.n_free_or_nb = n
        self.workspace_bytes = A.amoeba_rewrite_workspace_bytes(self.plan, self.num_seqs, n)
        self.workspace = torch.empty(self.workspace_bytes, dtype=torch.uint8, device=self.device)

    # ---- the three calls of one transformation
    def rewrite_block_tables(self, stream=None) -> None:
        A.amoeba_rewrite_block_tables(self.plan, self.src_bt, self.seq_lens, self.num_seqs, self.maxb, self.free_list,
                                      self.free_mask, self.n_free_or_nb, self.dst_bt, self.pairs, self.pairs_cap,
                                      self.num_pairs, self.free_count, self.status, self.workspace,
                                      self.workspace_bytes, stream)

    def reshard_kv(self, stream=None, layer_begin: int = 0, layer_end: Optional[int] = None) -> None:
        A.amoeba_reshard_kv(self.plan, self.src_pools, self.dst_pools, self.pairs, self.num_pairs, self.pairs_cap,
                            layer_begin, self.kv_layers if layer_end is None else layer_end, self.status, stream)

    def reshard_weights(self, stream=None, layer_begin: int = 0, layer_end: Optional[int] = None) -> None:
        A.amoeba_reshard_weights(self.plan, self._src_w_packed, self._dst_w_packed, layer_begin,
                                 self.L if layer_end is None else layer_end, self.status, stream)

    def step(self, stream=None) -> None:
        """One whole transformation: table rewrite, KV migration, weight re-partition (asynchronous)."""
        self.rewrite_block_tables(stream)
        if self.src_pools:
            self.reshard_kv(stream)
        if self.src_w:
            self.reshard_weights(stream)

    def set_option(self, option: int, value: int) -> None:
        A.amoeba_plan_set_option(self.plan, option, value)
        self.info = A.amoeba_plan_kv_info(self.plan)

    def bytes_rw(self, n_blocks: int):
        """(KV bytes, weight bytes) read+written by one step with n_blocks live blocks over the held KV layers."""
        kv, w = A.amoeba_plan_bytes(self.plan, n_blocks)
        return kv * self.kv_layers // self.L if self.src_pools else 0, w if self.src_w else 0



class ReshapeSession:
    """Buffers of the in-place block reshaping of ONE instance between TP=a (NB blocks) and TP=N*a (NB*N blocks).

    pools[w] is worker w of the TP=N*a side; worker r of the TP=a side is pools[r*N].  direction "split": the tables
    are over NB ids and the instance goes a -> N*a; "merge": over NB*N ids and it goes N*a -> a."""

    def __init__(self, model: dict, N: int, a: int, NB: int, num_seqs: int, max_blocks_per_seq: int, pairs_cap: int,
                 direction: str = "split", kv_layers: Optional[int] = None, block_tokens: int = 16, device="cuda:0"):
        assert direction in ("split", "merge")
        self.model, self.N, self.a, self.NB, self.direction = model, N, a, NB, direction
        self.device = dev = torch.device(device)
        coarse = A.make_layout(model, a, NB, block_tokens)
        fine = A.make_layout(model, N * a, NB * N, block_tokens)
        self.src_layout, self.dst_layout = (coarse, fine) if direction == "split" else (fine, coarse)
        self.plan = A.amoeba_plan_create(self.src_layout, self.dst_layout)
        self.L = model["L"]
        self.kv_layers = self.L if kv_layers is None else kv_layers
        self.num_seqs, self.maxb, self.pairs_cap = num_seqs, max_blocks_per_seq, pairs_cap
        i32 = dict(dtype=torch.int32, device=dev)
        self.src_bt = torch.full((num_seqs, max_blocks_per_seq), -1, **i32)
        self.dst_bt = torch.full((num_seqs, max_blocks_per_seq), -2, **i32)
        self.seq_lens = torch.zeros(num_seqs, **i32)
        self.pairs = torch.full((max(pairs_cap, 1), 2), -3, **i32)
        self.num_pairs = torch.zeros(1, **i32)
        self.free_count = torch.zeros(1, **i32)
        self.status = torch.zeros(1, **i32)
        self.free_mask = torch.full((self.dst_layout.num_blocks,), 7, dtype=torch.uint8, device=dev)
        self.workspace_bytes = A.amoeba_rewrite_workspace_bytes(self.plan, num_seqs, 0)
        self.workspace = torch.empty(self.workspace_bytes, dtype=torch.uint8, device=dev)
        per_layer = A.amoeba_layout_kv_pool_bytes(coarse) // self.L
        self.pools = [torch.empty(per_layer * self.kv_layers, dtype=torch.uint8, device=dev) for _ in range(N * a)]

    def set_tables(self, seq_lens, src_bt) -> None:
        self.seq_lens.copy_(torch.as_tensor(seq_lens, dtype=torch.int32))
        self.src_bt.copy_(torch.as_tensor(src_bt, dtype=torch.int32))

    def reshape_block_tables(self, stream=None) -> None:
        A.amoeba_reshape_block_tables(self.plan, self.src_bt, self.seq_lens, self.num_seqs, self.maxb, self.dst_bt,
                                      self.pairs, self.pairs_cap, self.num_pairs, self.free_mask, self.free_count,
                                      self.status, self.workspace, self.workspace_bytes, stream)

    def reshape_kv(self, stream=None, layer_begin: int = 0, layer_end: Optional[int] = None) -> None:
        A.amoeba_reshape_kv_inplace(self.plan, self.pools, self.pairs, self.num_pairs, self.pairs_cap, layer_begin,
                                    self.kv_layers if layer_end is None else layer_end, self.status, stream)

    def step(self, stream=None) -> None:
        self.reshape_block_tables(stream)
        self.reshape_kv(stream)

    def set_option(self, option: int, value: int) -> None:
        A.amoeba_plan_set_option(self.plan, option, value)

    def bytes_rw(self, n_live: int) -> int:
        return A.amoeba_reshape_bytes(self.plan, n_live) * self.kv_layers // self.L


class MergeSession:
    """Buffers of one in-place merge of N instances of TP=a into one instance of TP=N*a on one GPU.

    pools[i*a + r] is the pool of worker r of instance i before the merge and of worker r*N+i of the merged instance
    after it.  kv_layers: layers the pools hold (None = all)."""

    def __init__(self, model: dict, N: int, a: int, NB: int, num_seqs: int, max_blocks_per_seq: int,
                 kv_layers: Optional[int] = None, block_tokens: int = 16, device="cuda:0", weights: bool = False):
        self.model, self.N, self.a, self.NB = model, N, a, NB
        self.device = torch.device(device)
        self.src_layout = A.make_layout(model, a, NB, block_tokens)
        self.dst_layout = A.make_layout(model, N * a, NB * N, block_tokens)
        self.plan = A.amoeba_plan_create(self.src_layout, self.dst_layout)
        self.L = model["L"]
        self.kv_layers = self.L if kv_layers is None else kv_layers
        self.num_seqs, self.maxb = num_seqs, max_blocks_per_seq
        i32 = dict(dtype=torch.int32, device=self.device)
        self.src_bt = torch.full((N, num_seqs, max_blocks_per_seq), -1, **i32)
        self.dst_bt = torch.full((N, num_seqs, max_blocks_per_seq), -2, **i32)
        self.seq_lens = torch.zeros((N, num_seqs), **i32)
        self.status = torch.zeros(1, **i32)
        self.live = torch.zeros(A.amoeba_merge_live_bytes(self.plan), dtype=torch.uint8, device=self.device)
        per_layer = A.amoeba_layout_kv_pool_bytes(self.src_layout) // self.L
        self.pools = [torch.empty(per_layer * self.kv_layers, dtype=torch.uint8, device=self.device)
                      for _ in range(N * a)]
        # weights: every instance holds the whole model as dense TP=a shards; instance i's worker r keeps sub-shard i
        self.inst_w, self._inst_w_packed, self._wbufs = [], [], []
        if weights:
            sizes = [A.amoeba_layout_weight_bytes(self.src_layout, t) for t in range(len(A.TENSOR_NAMES))]
            used = [(n, sz) for n, sz in zip(A.TENSOR_NAMES, sizes) if sz]
            for _ in range(N):
                shards = []
                for _ in range(a):
                    buf = torch.empty(_carved_bytes([sz for _, sz in used]) * self.L, dtype=torch.uint8,
                                      device=self.device)
                    views = _carve(buf, [sz for _, sz in used] * self.L)
                    self._wbufs.append(buf)
                    shards.append([{n: views[l * len(used) + j] for j, (n, _) in enumerate(used)}
                                   for l in range(self.L)])
                self.inst_w.append(shards)
                self._inst_w_packed.append(A.pack_weights(shards))

    def set_tables(self, seq_lens, src_bt) -> None:
        self.seq_lens.copy_(torch.as_tensor(seq_lens, dtype=torch.int32))
        self.src_bt.copy_(torch.as_tensor(src_bt, dtype=torch.int32))

    def compact_weights(self, stream=None) -> None:
        """Every worker of every instance moves the part of its weight shards it keeps to the front, in place."""
        for i, packed in enumerate(self._inst_w_packed):
            A.amoeba_compact_weights_inplace(self.plan, packed, [i] * self.a, 0, self.L, self.status, stream)

    def weight_bytes_rw(self) -> int:
        """Bytes read + written by compact_weights, as the library counts them (what already is in place - e.g. the
        first section of every buffer of instance 0 - is not moved and not counted)."""
        if not self.inst_w:
            return 0
        return sum(A.amoeba_compact_bytes(self.plan, [i] * self.a) for i in range(self.N))

    def merge_block_tables(self, stream=None) -> None:
        A.amoeba_merge_block_tables(self.plan, self.src_bt, self.seq_lens, self.num_seqs, self.maxb, self.dst_bt,
                                    self.live, self.status, stream)

    def merge_kv(self, stream=None, layer_begin: int = 0, layer_end: Optional[int] = None) -> None:
        A.amoeba_merge_kv_inplace(self.plan, self.pools, self.live, layer_begin,
                                  self.kv_layers if layer_end is None else layer_end, self.status, stream)

    def step(self, stream=None) -> None:
        """Weights first, then the KV cache: the order the paper gives for raising the TP degree (Sec. 3.3)."""
        if self.inst_w:
            self.compact_weights(stream)
        self.merge_block_tables(stream)
        self.merge_kv(stream)

    def set_option(self, option: int, value: int) -> None:
        A.amoeba_plan_set_option(self.plan, option, value)

    def bytes_rw(self, n_live: int) -> int:
        """Bytes read + written by one merge with n_live live old blocks (summed over instances), held layers."""
        return A.amoeba_merge_bytes(self.plan, n_live) * self.kv_layers // self.L



class MergeCopySession:
    """N instances of TP=a become one instance of TP=N*a in FRESH pools (out of place): one table rewrite and one KV
    call per instance, each given the part of the shared destination free list the earlier instances left.  This is
    what a merge costs without in-place block reshaping (and the only way with token-first pools); it needs a second
    set of pools.  seq_lens [N][S] and src_bt [N][S][maxb] are host arrays; counts[i] = number of blocks instance i's
    table names (the caller's bookkeeping: it is what advances the shared free list from one instance to the next)."""

    def __init__(self, model: dict, N: int, a: int, NB_src: int, NB_dst: int, seq_lens, src_bt, free_list, counts,
                 kv_layers: Optional[int] = None, block_tokens: int = 16, device="cuda:0",
                 src_kv_order: int = A.KV_HEAD_MAJOR, dst_kv_order: int = A.KV_HEAD_MAJOR):
        self.model, self.N, self.a = model, N, a
        self.device = dev = torch.device(device)
        self.src_layout = A.make_layout(model, a, NB_src, block_tokens, kv_order=src_kv_order)
        self.dst_layout = A.make_layout(model, N * a, NB_dst, block_tokens, kv_order=dst_kv_order)
        self.plan = A.amoeba_plan_create(self.src_layout, self.dst_layout)
        self.L = model["L"]
        self.kv_layers = self.L if kv_layers is None else kv_layers
        lens = torch.as_tensor(seq_lens, dtype=torch.int32)
        bt = torch.as_tensor(src_bt, dtype=torch.int32)
        self.num_seqs, self.maxb = int(bt.shape[1]), int(bt.shape[2])
        i32 = dict(dtype=torch.int32, device=dev)
        counts = [int(c) for c in counts]
        assert len(counts) == N
        self.counts, self.offsets = counts, [sum(counts[:i]) for i in range(N)]
        self.free_list = torch.as_tensor(free_list, dtype=torch.int32).to(dev)
        assert self.free_list.numel() >= sum(counts)
        self.seq_lens, self.src_bt = lens.to(dev), bt.to(dev)
        self.dst_bt = torch.full(tuple(bt.shape), -2, **i32)
        self.pairs = [torch.full((max(c, 1), 2), -3, **i32) for c in counts]
        self.num_pairs = torch.zeros(N, **i32)
        self.free_count = torch.zeros(N, **i32)
        self.status = torch.zeros(1, **i32)
        self.ws_bytes = A.amoeba_rewrite_workspace_bytes(self.plan, self.num_seqs, self.free_list.numel())
        self.workspace = torch.empty(self.ws_bytes, dtype=torch.uint8, device=dev)
        src_per_layer = A.amoeba_layout_kv_pool_bytes(self.src_layout) // self.L
        dst_per_layer = A.amoeba_layout_kv_pool_bytes(self.dst_layout) // self.L
        self.src_pools = [[torch.empty(src_per_layer * self.kv_layers, dtype=torch.uint8, device=dev) for _ in range(a)]
                          for _ in range(N)]
        self.dst_pools = [torch.empty(dst_per_layer * self.kv_layers, dtype=torch.uint8, device=dev)
                          for _ in range(N * a)]

    def step(self, stream=None) -> None:
        n_free = self.free_list.numel()
        for i in range(self.N):
            off = self.offsets[i]
            A.amoeba_rewrite_block_tables(self.plan, self.src_bt[i], self.seq_lens[i], self.num_seqs, self.maxb,
                                          self.free_list[off:], None, n_free - off, self.dst_bt[i], self.pairs[i],
                                          self.counts[i], self.num_pairs[i:i + 1], self.free_count[i:i + 1],
                                          self.status, self.workspace, self.ws_bytes, stream)
            A.amoeba_reshard_kv(self.plan, self.src_pools[i], self.dst_pools, self.pairs[i], self.num_pairs[i:i + 1],
                                self.counts[i], 0, self.kv_layers, self.status, stream)

    def set_option(self, option: int, value: int) -> None:
        A.amoeba_plan_set_option(self.plan, option, value)

    def bytes_rw(self) -> int:
        kv, _ = A.amoeba_plan_bytes(self.plan, sum(self.counts))
        return kv * self.kv_layers // self.L

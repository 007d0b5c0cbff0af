"""ctypes binding of ``libamoeba.so``: argument marshalling only, every step runs in the CUDA kernels.

Device buffers are ``torch`` CUDA tensors (or raw integer device addresses); the stream defaults to torch's
current stream.  Every function raises :class:`AmoebaError` when the C call returns a non-zero status.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

from . import build as _build

__all__ = [
    "AmoebaError", "Model", "Layout", "LayerWeights", "KvInfo", "WeightDesc", "Plan", "STATUS_NAMES", "TENSOR_NAMES",
    "OPT_COPY_PATH", "OPT_CTAS_PER_SM", "OPT_CHUNK_BYTES", "OPT_STAGES", "OPT_LAG", "OPT_WARPS", "OPT_L2_HINT", "OPT_TENSOR_MAPS", "OPT_MAX_CTAS",
    "OPT_WEIGHTS_ONLY", "OPT_KV_ONLY", "COPY_PATH_LDST", "COPY_PATH_BULK", "COPY_PATH_PAIR",
    "amoeba_plan_create", "amoeba_plan_destroy", "amoeba_layout_kv_pool_bytes", "amoeba_layout_weight_bytes", "amoeba_plan_bytes", "amoeba_plan_kv_info",
    "amoeba_plan_num_weight_descs", "amoeba_plan_weight_desc", "amoeba_plan_set_option",
    "amoeba_rewrite_workspace_bytes", "amoeba_rewrite_block_tables", "amoeba_reshard_kv", "amoeba_reshard_weights",
    "amoeba_launch_count", "amoeba_status_string", "library_path", "make_layout",
]

(OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_ALIGNMENT, ERR_NO_FREE_BLOCKS, ERR_BAD_BLOCK_ID, ERR_CUDA, ERR_TIMEOUT,
 ERR_TOO_LARGE, ERR_NO_MEMORY, ERR_INTERNAL) = range(11)
STATUS_NAMES = ["OK", "INVALID_ARG", "UNSUPPORTED", "ALIGNMENT", "NO_FREE_BLOCKS", "BAD_BLOCK_ID", "CUDA", "TIMEOUT",
                "TOO_LARGE", "NO_MEMORY", "INTERNAL"]
BUILTIN_SCRATCH_BYTES = 1 << 20
__all__ += ["OK", "ERR_INVALID_ARG", "ERR_UNSUPPORTED", "ERR_ALIGNMENT", "ERR_NO_FREE_BLOCKS", "ERR_BAD_BLOCK_ID",
            "ERR_CUDA", "ERR_TIMEOUT", "ERR_TOO_LARGE", "ERR_NO_MEMORY", "ERR_INTERNAL", "BUILTIN_SCRATCH_BYTES", "OPT_WAIT_TRIES", "OPT_L2_PROMOTION", "OPT_PAIR_ORDER", "PAIR_ORDER_TABLE", "PAIR_ORDER_DESTINATION",
            "amoeba_rewrite_block_tables_builtin_scratch", "amoeba_reshape_block_tables", "amoeba_reshape_kv_inplace",
            "amoeba_reshape_bytes"]
(OPT_COPY_PATH, OPT_CTAS_PER_SM, OPT_CHUNK_BYTES, OPT_STAGES, OPT_LAG, OPT_WARPS, OPT_L2_HINT, OPT_TENSOR_MAPS,
 OPT_MAX_CTAS, OPT_WAIT_TRIES, OPT_L2_PROMOTION, OPT_PAIR_ORDER) = range(12)
PAIR_ORDER_TABLE, PAIR_ORDER_DESTINATION = 1, 2
OPT_WEIGHTS_ONLY, OPT_KV_ONLY = 16, 32  # add to an option id to set one kernel only
COPY_PATH_LDST, COPY_PATH_BULK, COPY_PATH_PAIR = 1, 2, 3
KV_HEAD_MAJOR, KV_TOKEN_MAJOR = 0, 1  # [block][header][K/V][token][dim] / [K/V][block][token][header][dim]
__all__ += ["KV_HEAD_MAJOR", "KV_TOKEN_MAJOR"]
TENSOR_NAMES = ("q", "k", "v", "o", "gate", "up", "down")


class AmoebaError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {amoeba_status_string(status)} (status {status})")


class Model(C.Structure):
    _fields_ = [(n, C.c_int32) for n in
                ("num_layers", "hidden", "num_q_heads", "num_kv_heads", "head_dim", "intermediate", "elem_bytes")]


class Layout(C.Structure):
    _fields_ = [("model", Model), ("tp", C.c_int32), ("block_tokens", C.c_int32), ("num_blocks", C.c_int32),
                ("kv_order", C.c_int32), ("fused_qkv", C.c_int32), ("fused_gate_up", C.c_int32),
                ("kv_layer_stride_bytes", C.c_int64), ("weight_pad_parts", C.c_int32), ("reserved", C.c_int32),
                ("weight_page_bytes", C.c_int64)]


class PadInfo(C.Structure):
    _fields_ = [("partitions_per_worker", C.c_int32), ("reserved", C.c_int32), ("partition_bytes", C.c_int64),
                ("pitch_bytes", C.c_int64), ("page_bytes", C.c_int64), ("pages", C.c_double)]


class LayerWeights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in TENSOR_NAMES]


class KvInfo(C.Structure):
    _fields_ = [("heads_per_run", C.c_int32), ("runs_per_block", C.c_int32), ("run_bytes", C.c_int64),
                ("chunk_bytes", C.c_int64), ("src_block_bytes", C.c_int64), ("dst_block_bytes", C.c_int64),
                ("src_layer_stride", C.c_int64), ("dst_layer_stride", C.c_int64)]


class WeightDesc(C.Structure):
    _fields_ = [("src_rank", C.c_int32), ("src_tensor", C.c_int32), ("dst_rank", C.c_int32), ("dst_tensor", C.c_int32),
                ("src_off", C.c_int64), ("dst_off", C.c_int64), ("row_bytes", C.c_int64), ("src_pitch", C.c_int64),
                ("dst_pitch", C.c_int64), ("n_rows", C.c_int32), ("reserved", C.c_int32)]


_lib = None


# AMOEBA_BINDING_BUILD=checked makes this binding load the checked build of the library (every work item tested against
# the extent of its buffers, see build.py) instead of the normal one: a switch of the Python binding for test runs,
# the C library itself reads no environment variable.
_CHECKED = os.environ.get("AMOEBA_BINDING_BUILD", "") == "checked"


def library_path():
    return _build.LIB_CHECKED if _CHECKED else _build.LIB


def _load():
    global _lib
    if _lib is not None:
        return _lib
    if _build.needs_build(_CHECKED):
        try:
            _build.build(checked=_CHECKED)
        except Exception as e:  # no silent fallback: the product is the CUDA library
            raise ImportError(f"{library_path().name} is missing or stale and could not be built: {e}") from e
    lib = C.CDLL(str(library_path()))
    P, I32, I64, VP = C.POINTER, C.c_int32, C.c_int64, C.c_void_p
    sig = {
        "amoeba_plan_create": (I32, [P(Layout), P(Layout), P(VP)]),
        "amoeba_plan_destroy": (None, [VP]),
        "amoeba_layout_kv_pool_bytes": (I32, [P(Layout), P(I64)]),
        "amoeba_layout_weight_bytes": (I32, [P(Layout), I32, P(I64)]),
        "amoeba_layout_pad_info": (I32, [P(Layout), I32, P(PadInfo)]),
        "amoeba_plan_bytes": (I32, [VP, I64, P(I64), P(I64)]),
        "amoeba_plan_kv_info": (I32, [VP, P(KvInfo)]),
        "amoeba_plan_num_weight_descs": (I32, [VP]),
        "amoeba_plan_weight_desc": (I32, [VP, I32, P(WeightDesc)]),
        "amoeba_plan_set_option": (I32, [VP, I32, I64]),
        "amoeba_rewrite_workspace_bytes": (I32, [VP, I32, I32, P(I64)]),
        "amoeba_rewrite_block_tables": (I32, [VP, VP, VP, I32, I32, VP, VP, I32, VP, VP, I32, VP, VP, VP, VP, I64, VP]),
        "amoeba_rewrite_block_tables_builtin_scratch": (I32, [VP, VP, VP, I32, I32, VP, VP, I32, VP, VP, I32, VP, VP, VP, VP]),
        "amoeba_reshard_kv": (I32, [VP, P(VP), P(VP), VP, VP, I32, I32, I32, VP, VP]),
        "amoeba_reshape_block_tables": (I32, [VP, VP, VP, I32, I32, VP, VP, I32, VP, VP, VP, VP, VP, I64, VP]),
        "amoeba_reshape_kv_inplace": (I32, [VP, P(VP), VP, VP, I32, I32, I32, VP, VP]),
        "amoeba_reshape_bytes": (I32, [VP, I64, P(I64)]),
        "amoeba_reshard_weights": (I32, [VP, P(LayerWeights), P(LayerWeights), I32, I32, VP, VP]),
        "amoeba_merge_live_bytes": (I32, [VP, P(I64)]),
        "amoeba_merge_bytes": (I32, [VP, I64, P(I64)]),
        "amoeba_merge_block_tables": (I32, [VP, VP, VP, I32, I32, VP, VP, VP, VP]),
        "amoeba_split_block_tables": (I32, [VP, VP, VP, I32, I32, VP, VP, VP, VP]),
        "amoeba_merge_kv_inplace": (I32, [VP, P(VP), VP, I32, I32, VP, VP]),
        "amoeba_split_kv_inplace": (I32, [VP, P(VP), VP, I32, I32, VP, VP]),
        "amoeba_compact_weights_inplace": (I32, [VP, P(LayerWeights), P(I32), I32, I32, VP, VP]),
        "amoeba_compact_bytes": (I32, [VP, P(I32), P(I64)]),
        "amoeba_plan_weight_alias": (I32, [VP, I32, I32, P(I32), P(I64), P(I64)]),
        "amoeba_launch_count": (I64, []),
        "amoeba_status_string": (C.c_char_p, [I32]),
    }
    for name, (res, args) in sig.items():
        f = getattr(lib, name)
        f.restype, f.argtypes = res, args
    _lib = lib
    return lib


def _ptr(x) -> Optional[int]:
    """Device address of a torch tensor, an int address, or None."""
    if x is None:
        return None
    if isinstance(x, int):
        return x
    return x.data_ptr()


def _stream(stream) -> Optional[int]:
    if stream is None:
        import torch

        return torch.cuda.current_stream().cuda_stream
    return stream if isinstance(stream, int) else stream.cuda_stream


def _check(status: int, where: str) -> None:
    if status != OK:
        raise AmoebaError(status, where)


class Plan:
    """Owner of an ``amoeba_plan*``."""

    def __init__(self, handle: int, src: Layout, dst: Layout):
        self.handle, self.src, self.dst = handle, src, dst

    def __del__(self):
        if getattr(self, "handle", None):
            _load().amoeba_plan_destroy(self.handle)
            self.handle = None


def make_layout(model: dict, tp: int, num_blocks: int, block_tokens: int = 16, fused_qkv: bool = True,
                fused_gate_up: bool = True, elem_bytes: int = 2, kv_layer_stride_bytes: int = 0,
                kv_order: int = 0, weight_pad_parts: int = 0, weight_page_bytes: int = 0) -> Layout:
    """Layout from a shape dict with keys L, hidden, Hq, Hkv, D, I; kv_order KV_HEAD_MAJOR or KV_TOKEN_MAJOR;
    weight_pad_parts > 0: padded weight partitions (page 0 = 2 MiB)."""
    m = Model(model["L"], model["hidden"], model["Hq"], model["Hkv"], model["D"], model["I"], elem_bytes)
    return Layout(m, tp, block_tokens, num_blocks, int(kv_order), int(fused_qkv), int(fused_gate_up),
                  kv_layer_stride_bytes, int(weight_pad_parts), 0, int(weight_page_bytes))


def amoeba_status_string(status: int) -> str:
    return _load().amoeba_status_string(int(status)).decode()


def amoeba_plan_create(src: Layout, dst: Layout) -> Plan:
    h = C.c_void_p()
    _check(_load().amoeba_plan_create(C.byref(src), C.byref(dst), C.byref(h)), "amoeba_plan_create")
    return Plan(h.value, src, dst)


def amoeba_layout_kv_pool_bytes(layout: Layout) -> int:
    out = C.c_int64()
    _check(_load().amoeba_layout_kv_pool_bytes(C.byref(layout), C.byref(out)), "amoeba_layout_kv_pool_bytes")
    return out.value


def amoeba_layout_weight_bytes(layout: Layout, tensor: int) -> int:
    out = C.c_int64()
    _check(_load().amoeba_layout_weight_bytes(C.byref(layout), tensor, C.byref(out)), "amoeba_layout_weight_bytes")
    return out.value


def amoeba_layout_pad_info(layout: Layout, tensor: int) -> PadInfo:
    out = PadInfo()
    _check(_load().amoeba_layout_pad_info(C.byref(layout), tensor, C.byref(out)), "amoeba_layout_pad_info")
    return out


__all__ += ["PadInfo", "amoeba_layout_pad_info"]


def amoeba_plan_destroy(plan: Plan) -> None:
    plan.__del__()


def amoeba_plan_bytes(plan: Plan, n_blocks: int):
    kv, w = C.c_int64(), C.c_int64()
    _check(_load().amoeba_plan_bytes(plan.handle, n_blocks, C.byref(kv), C.byref(w)), "amoeba_plan_bytes")
    return kv.value, w.value


def amoeba_plan_kv_info(plan: Plan) -> KvInfo:
    out = KvInfo()
    _check(_load().amoeba_plan_kv_info(plan.handle, C.byref(out)), "amoeba_plan_kv_info")
    return out


def amoeba_plan_num_weight_descs(plan: Plan) -> int:
    return _load().amoeba_plan_num_weight_descs(plan.handle)


def amoeba_plan_weight_desc(plan: Plan, index: int) -> WeightDesc:
    out = WeightDesc()
    _check(_load().amoeba_plan_weight_desc(plan.handle, index, C.byref(out)), "amoeba_plan_weight_desc")
    return out


def amoeba_plan_set_option(plan: Plan, option: int, value: int) -> None:
    _check(_load().amoeba_plan_set_option(plan.handle, option, value), "amoeba_plan_set_option")


def amoeba_rewrite_workspace_bytes(plan: Plan, num_seqs: int, n_free_or_nb: int) -> int:
    out = C.c_int64()
    _check(_load().amoeba_rewrite_workspace_bytes(plan.handle, num_seqs, n_free_or_nb, C.byref(out)),
           "amoeba_rewrite_workspace_bytes")
    return out.value


def amoeba_rewrite_block_tables(plan: Plan, src_bt, seq_lens, num_seqs: int, max_blocks_per_seq: int, dst_free_list,
                                dst_free_mask, n_free_or_nb: int, dst_bt, pairs, pairs_cap: int, num_pairs,
                                dst_free_count_out, status, workspace, workspace_bytes: int, stream=None) -> None:
    _check(_load().amoeba_rewrite_block_tables(
        plan.handle, _ptr(src_bt), _ptr(seq_lens), num_seqs, max_blocks_per_seq, _ptr(dst_free_list),
        _ptr(dst_free_mask), n_free_or_nb, _ptr(dst_bt), _ptr(pairs), pairs_cap, _ptr(num_pairs),
        _ptr(dst_free_count_out), _ptr(status), _ptr(workspace), workspace_bytes, _stream(stream)),
        "amoeba_rewrite_block_tables")


def amoeba_rewrite_block_tables_builtin_scratch(plan: Plan, src_bt, seq_lens, num_seqs: int, max_blocks_per_seq: int,
                                                dst_free_list, dst_free_mask, n_free_or_nb: int, dst_bt, pairs,
                                                pairs_cap: int, num_pairs, dst_free_count_out, status,
                                                stream=None) -> None:
    """``amoeba_rewrite_block_tables`` for callers that cannot allocate device memory (a serving process whose pool
    owns the whole GPU, code inside a no-allocation region, a plug-in without an allocator): the scratch is a 1 MiB
    array built into the library, so no workspace is passed.  Problems whose workspace would exceed
    ``BUILTIN_SCRATCH_BYTES`` raise ``AmoebaError`` with ``ERR_TOO_LARGE``.  The first call on a device resolves the
    array's address (do it at start-up, outside stream capture); calls that may overlap on the GPU share the array
    and must be ordered by the caller."""
    _check(_load().amoeba_rewrite_block_tables_builtin_scratch(
        plan.handle, _ptr(src_bt), _ptr(seq_lens), num_seqs, max_blocks_per_seq, _ptr(dst_free_list),
        _ptr(dst_free_mask), n_free_or_nb, _ptr(dst_bt), _ptr(pairs), pairs_cap, _ptr(num_pairs),
        _ptr(dst_free_count_out), _ptr(status), _stream(stream)), "amoeba_rewrite_block_tables_builtin_scratch")


def amoeba_reshard_kv(plan: Plan, src_pools: Sequence, dst_pools: Sequence, pairs, num_pairs, pairs_cap: int,
                      layer_begin: int, layer_end: int, status, stream=None) -> None:
    sp = (C.c_void_p * len(src_pools))(*[_ptr(x) for x in src_pools])
    dp = (C.c_void_p * len(dst_pools))(*[_ptr(x) for x in dst_pools])
    if len(src_pools) != plan.src.tp or len(dst_pools) != plan.dst.tp:
        raise AmoebaError(ERR_INVALID_ARG, "amoeba_reshard_kv (pool count != tp)")
    _check(_load().amoeba_reshard_kv(plan.handle, sp, dp, _ptr(pairs), _ptr(num_pairs), pairs_cap, layer_begin,
                                     layer_end, _ptr(status), _stream(stream)), "amoeba_reshard_kv")


def amoeba_reshape_block_tables(plan: Plan, src_bt, seq_lens, num_seqs: int, max_blocks_per_seq: int, dst_bt, pairs,
                                pairs_cap: int, num_pairs, dst_free_mask_out, dst_free_count_out, status, workspace,
                                workspace_bytes: int, stream=None) -> None:
    _check(_load().amoeba_reshape_block_tables(
        plan.handle, _ptr(src_bt), _ptr(seq_lens), num_seqs, max_blocks_per_seq, _ptr(dst_bt), _ptr(pairs), pairs_cap,
        _ptr(num_pairs), _ptr(dst_free_mask_out), _ptr(dst_free_count_out), _ptr(status), _ptr(workspace),
        workspace_bytes, _stream(stream)), "amoeba_reshape_block_tables")


def amoeba_reshape_kv_inplace(plan: Plan, pools: Sequence, pairs, num_pairs, pairs_cap: int, layer_begin: int,
                              layer_end: int, status, stream=None) -> None:
    """pools: max(a, b) tensors or addresses, pools[w] = worker w of the finer side; worker r of the coarser side is
    pools[r * N]."""
    if len(pools) != max(plan.src.tp, plan.dst.tp):
        raise AmoebaError(ERR_INVALID_ARG, "amoeba_reshape_kv_inplace (need one pool per worker of the finer side)")
    pp = (C.c_void_p * len(pools))(*[_ptr(x) for x in pools])
    _check(_load().amoeba_reshape_kv_inplace(plan.handle, pp, _ptr(pairs), _ptr(num_pairs), pairs_cap, layer_begin,
                                             layer_end, _ptr(status), _stream(stream)), "amoeba_reshape_kv_inplace")


def amoeba_reshape_bytes(plan: Plan, n_live_blocks: int) -> int:
    out = C.c_int64()
    _check(_load().amoeba_reshape_bytes(plan.handle, n_live_blocks, C.byref(out)), "amoeba_reshape_bytes")
    return out.value


def pack_weights(shards: Sequence[Sequence[dict]]):
    """[rank][layer] dicts {tensor name: tensor or address} -> C array of LayerWeights, rank-major."""
    n_rank, n_layer = len(shards), len(shards[0])
    arr = (LayerWeights * (n_rank * n_layer))()
    for r in range(n_rank):
        for l in range(n_layer):
            for name in TENSOR_NAMES:
                setattr(arr[r * n_layer + l], name, _ptr(shards[r][l].get(name)))
    return arr


__all__.append("pack_weights")


def amoeba_reshard_weights(plan: Plan, src, dst, layer_begin: int, layer_end: int, status, stream=None) -> None:
    """``src`` / ``dst``: ``pack_weights`` arrays or [rank][layer] lists of dicts."""
    if not isinstance(src, C.Array):
        src = pack_weights(src)
    if not isinstance(dst, C.Array):
        dst = pack_weights(dst)
    L = plan.src.model.num_layers
    if len(src) != plan.src.tp * L or len(dst) != plan.dst.tp * L:
        raise AmoebaError(ERR_INVALID_ARG, "amoeba_reshard_weights (need [tp][num_layers] entries)")
    _check(_load().amoeba_reshard_weights(plan.handle, src, dst, layer_begin, layer_end, _ptr(status),
                                          _stream(stream)), "amoeba_reshard_weights")


def amoeba_merge_live_bytes(plan: Plan) -> int:
    out = C.c_int64()
    _check(_load().amoeba_merge_live_bytes(plan.handle, C.byref(out)), "amoeba_merge_live_bytes")
    return out.value


def amoeba_merge_bytes(plan: Plan, n_live_blocks: int) -> int:
    out = C.c_int64()
    _check(_load().amoeba_merge_bytes(plan.handle, n_live_blocks, C.byref(out)), "amoeba_merge_bytes")
    return out.value


def amoeba_merge_block_tables(plan: Plan, src_bt, seq_lens, num_seqs: int, max_blocks_per_seq: int, dst_bt, live,
                              status, stream=None) -> None:
    _check(_load().amoeba_merge_block_tables(plan.handle, _ptr(src_bt), _ptr(seq_lens), num_seqs, max_blocks_per_seq,
                                             _ptr(dst_bt), _ptr(live), _ptr(status), _stream(stream)),
           "amoeba_merge_block_tables")


def amoeba_split_block_tables(plan: Plan, merged_bt, seq_lens, num_seqs: int, max_blocks_per_seq: int, inst_bt, live,
                              status, stream=None) -> None:
    _check(_load().amoeba_split_block_tables(plan.handle, _ptr(merged_bt), _ptr(seq_lens), num_seqs,
                                             max_blocks_per_seq, _ptr(inst_bt), _ptr(live), _ptr(status),
                                             _stream(stream)), "amoeba_split_block_tables")


__all__.append("amoeba_split_block_tables")


def amoeba_merge_kv_inplace(plan: Plan, pools: Sequence, live, layer_begin: int, layer_end: int, status,
                            stream=None) -> None:
    """pools: N*a tensors or addresses, pools[i*a + r] = worker r of instance i."""
    if len(pools) != plan.dst.tp:
        raise AmoebaError(ERR_INVALID_ARG, "amoeba_merge_kv_inplace (need N*a pools)")
    pp = (C.c_void_p * len(pools))(*[_ptr(x) for x in pools])
    _check(_load().amoeba_merge_kv_inplace(plan.handle, pp, _ptr(live), layer_begin, layer_end, _ptr(status),
                                           _stream(stream)), "amoeba_merge_kv_inplace")


def amoeba_split_kv_inplace(plan: Plan, pools: Sequence, live, layer_begin: int, layer_end: int, status,
                            stream=None) -> None:
    """pools: N*a tensors or addresses, pools[i*a + r] = merged worker r*N+i, afterwards worker r of instance i."""
    if len(pools) != plan.dst.tp:
        raise AmoebaError(ERR_INVALID_ARG, "amoeba_split_kv_inplace (need N*a pools)")
    pp = (C.c_void_p * len(pools))(*[_ptr(x) for x in pools])
    _check(_load().amoeba_split_kv_inplace(plan.handle, pp, _ptr(live), layer_begin, layer_end, _ptr(status),
                                           _stream(stream)), "amoeba_split_kv_inplace")


__all__ += ["amoeba_split_kv_inplace", "amoeba_merge_live_bytes", "amoeba_merge_bytes", "amoeba_merge_block_tables", "amoeba_merge_kv_inplace"]


def amoeba_compact_weights_inplace(plan: Plan, bufs, keep: Sequence[int], layer_begin: int, layer_end: int, status,
                                   stream=None) -> None:
    """``bufs``: ``pack_weights`` array or [rank][layer] list of dicts of the TP=a workers' buffers; ``keep[r]``: which
    N-th of its shards worker r keeps (it becomes worker r*N + keep[r] of TP = N*a)."""
    if not isinstance(bufs, C.Array):
        bufs = pack_weights(bufs)
    if len(bufs) != plan.src.tp * plan.src.model.num_layers or len(keep) != plan.src.tp:
        raise AmoebaError(ERR_INVALID_ARG, "amoeba_compact_weights_inplace (need [tp][num_layers] buffers, tp keeps)")
    k = (C.c_int32 * len(keep))(*[int(x) for x in keep])
    _check(_load().amoeba_compact_weights_inplace(plan.handle, bufs, k, layer_begin, layer_end, _ptr(status),
                                                  _stream(stream)), "amoeba_compact_weights_inplace")


def amoeba_compact_bytes(plan: Plan, keep: Sequence[int]) -> int:
    """Bytes read + written by ``amoeba_compact_weights_inplace`` over all layers for this ``keep``."""
    k = (C.c_int32 * len(keep))(*[int(x) for x in keep])
    out = C.c_int64()
    _check(_load().amoeba_compact_bytes(plan.handle, k, C.byref(out)), "amoeba_compact_bytes")
    return out.value


__all__ += ["amoeba_compact_weights_inplace", "amoeba_compact_bytes"]


def amoeba_plan_weight_alias(plan: Plan, dst_rank: int, tensor: int):
    """(source worker, byte offset, bytes) of the source buffer range that already is the destination worker's
    buffer; raises AmoebaError(ERR_UNSUPPORTED) when the layouts need a copy."""
    r, off, n = C.c_int32(), C.c_int64(), C.c_int64()
    _check(_load().amoeba_plan_weight_alias(plan.handle, dst_rank, tensor, C.byref(r), C.byref(off), C.byref(n)),
           "amoeba_plan_weight_alias")
    return r.value, off.value, n.value


__all__.append("amoeba_plan_weight_alias")


def amoeba_launch_count() -> int:
    return _load().amoeba_launch_count()


_load()

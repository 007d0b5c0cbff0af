"""CPU oracle for the TP a->b re-layout (test infrastructure, not part of the product).

Thin numpy marshalling around ``amoeba_oracle.c`` (plain C element loops, compiled with gcc).  Only the tests,
the smoke check and the benchmark's CPU-baseline leg import this package; the CUDA library and its Python
binding never do, and nothing here imports them.

Conventions (see the C file for the passages of the paper each function follows):
  * elements are opaque 16-bit words, numpy ``uint16``;
  * logical KV is ``KV[L][G][Hkv][2][D]`` with ``G`` the number of block-padded tokens of all sequences;
  * a KV pool of one worker is ``pool[L][NB][Hkv/TP][2][T][D]`` (header-centric) or
    ``pool[L][2][NB][T][Hkv/TP][D]`` (token-first);
  * one layer's logical weights are a dict ``{q,k,v,o,gate,up,down}`` of ``[out,in]`` arrays.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "amoeba_oracle.c"
_LIB = _HERE / "liboracle.so"

OK, INVALID_ARG, NO_FREE_BLOCKS, BAD_BLOCK_ID = 0, 1, 4, 5
HEADER_CENTRIC, TOKEN_FIRST = 0, 1  # KV storage orders (Sec. 3.1)


def build(force: bool = False) -> Path:
    """Compile the C oracle with gcc (no CUDA involved)."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(f".tmp{os.getpid()}.so")
        subprocess.run(["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-o", str(tmp), str(_SRC)],
                       check=True)
        os.replace(tmp, _LIB)
    return _LIB


class _Model(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("L", "hidden", "Hq", "Hkv", "D", "I")]


class _Weights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("q", "k", "v", "o", "gate", "up", "down")]


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(str(build()))
    return _lib


def _model(m: dict) -> _Model:
    return _Model(m["L"], m["hidden"], m["Hq"], m["Hkv"], m["D"], m["I"])


def _i32(a):
    a = np.ascontiguousarray(a, dtype=np.int32)
    return a, a.ctypes.data_as(C.POINTER(C.c_int32))


def _ptr_array(arrs):
    return (C.c_void_p * len(arrs))(*[a.ctypes.data for a in arrs])


def set_threads(n: int) -> None:
    """Number of OpenMP threads the layer loops may use (1 = serial)."""
    os.environ["OMP_NUM_THREADS"] = str(n)
    try:
        omp = C.CDLL("libgomp.so.1")
        omp.omp_set_num_threads(int(n))
    except OSError:
        pass


def header_range(H: int, TP: int, i: int):
    """1-indexed inclusive range of headers kept by worker W_i (Sec. 3.1)."""
    f, l = C.c_int(), C.c_int()
    lib().oracle_header_range(H, TP, i, C.byref(f), C.byref(l))
    return f.value, l.value


def worker_of_header(H: int, TP: int, header: int) -> int:
    return lib().oracle_worker_of_header(H, TP, header)


def padded_tokens(seq_lens, T: int) -> int:
    sl, slp = _i32(seq_lens)
    f = lib().oracle_padded_tokens
    f.restype = C.c_int64
    return f(len(sl), slp, T)


def pool_elems_per_layer(m: dict, T: int, TP: int, NB: int) -> int:
    return NB * (m["Hkv"] // TP) * 2 * T * m["D"]


def kv_shard(KV, m, T, TP, NB, seq_lens, bt, fill=0xA5A5, layer_stride=None, order=HEADER_CENTRIC):
    """Logical KV -> list of TP pools (uint16, ``order`` storage order), untouched words = ``fill``."""
    sl, slp = _i32(seq_lens)
    bt, btp = _i32(bt)
    per = pool_elems_per_layer(m, T, TP, NB)
    stride = per if layer_stride is None else layer_stride
    pools = [np.full(m["L"] * stride, fill, dtype=np.uint16) for _ in range(TP)]
    KV = np.ascontiguousarray(KV, dtype=np.uint16)
    mm = _model(m)
    lib().oracle_kv_shard(KV.ctypes.data_as(C.c_void_p), C.byref(mm), T, TP, NB, order, C.c_int64(stride), len(sl),
                          slp, btp, bt.shape[1], _ptr_array(pools))
    return pools


def kv_reconstruct(pools, m, T, TP, NB, seq_lens, bt, layer_stride=None, order=HEADER_CENTRIC):
    sl, slp = _i32(seq_lens)
    bt, btp = _i32(bt)
    G = padded_tokens(sl, T)
    KV = np.zeros((m["L"], G, m["Hkv"], 2, m["D"]), dtype=np.uint16)
    stride = pool_elems_per_layer(m, T, TP, NB) if layer_stride is None else layer_stride
    mm = _model(m)
    lib().oracle_kv_reconstruct(KV.ctypes.data_as(C.c_void_p), C.byref(mm), T, TP, NB, order, C.c_int64(stride),
                                len(sl), slp, btp, bt.shape[1], _ptr_array(pools))
    return KV


def kv_transform(m, T, seq_lens, a, NB_src, src_bt, src_pools, b, NB_dst, dst_bt, dst_pools,
                 src_order=HEADER_CENTRIC, dst_order=HEADER_CENTRIC, src_layer_stride=None, dst_layer_stride=None):
    """TP a->b on the KV pools: writes the live blocks of ``dst_pools`` in place (reconstruct, then shard)."""
    sl, slp = _i32(seq_lens)
    sbt, sbtp = _i32(src_bt)
    dbt, dbtp = _i32(dst_bt)
    assert sbt.shape == dbt.shape
    mm = _model(m)
    ss = pool_elems_per_layer(m, T, a, NB_src) if src_layer_stride is None else src_layer_stride  # in elements
    ds = pool_elems_per_layer(m, T, b, NB_dst) if dst_layer_stride is None else dst_layer_stride
    rc = lib().oracle_kv_transform(C.byref(mm), T, len(sl), slp, sbt.shape[1], a, NB_src, src_order,
                                   C.c_int64(ss), sbtp, _ptr_array(src_pools), b,
                                   NB_dst, dst_order, C.c_int64(ds), dbtp,
                                   _ptr_array(dst_pools))
    assert rc == 0


def kv_copy_pairs(m, T, a, NB_src, src_pools, b, NB_dst, dst_pools, pairs, num_pairs, status=0,
                  src_order=HEADER_CENTRIC, dst_order=HEADER_CENTRIC):
    pr, prp = _i32(pairs)
    st = C.c_int32(status)
    mm = _model(m)
    lib().oracle_kv_copy_pairs(C.byref(mm), T, a, NB_src, src_order,
                               C.c_int64(pool_elems_per_layer(m, T, a, NB_src)), _ptr_array(src_pools), b, NB_dst,
                               dst_order, C.c_int64(pool_elems_per_layer(m, T, b, NB_dst)), _ptr_array(dst_pools),
                               prp, int(num_pairs), C.byref(st))
    return st.value


WEIGHT_NAMES = ("q", "k", "v", "o", "gate", "up", "down")


def shard_shapes(m: dict, TP: int, fused_qkv=True, fused_gate_up=True) -> dict:
    """Shapes of one worker's weight buffers for one layer."""
    hid, qr, kr, I = m["hidden"], m["Hq"] * m["D"] // TP, m["Hkv"] * m["D"] // TP, m["I"] // TP
    sh = {"o": (hid, qr), "down": (hid, I)}
    if fused_qkv:
        sh["q"] = (qr + 2 * kr, hid)
    else:
        sh.update(q=(qr, hid), k=(kr, hid), v=(kr, hid))
    if fused_gate_up:
        sh["gate"] = (2 * I, hid)
    else:
        sh.update(gate=(I, hid), up=(I, hid))
    return sh


def _wstruct(d: dict) -> _Weights:
    return _Weights(*[(d[n].ctypes.data if n in d else None) for n in WEIGHT_NAMES])


def empty_shards(m, TP, fused_qkv=True, fused_gate_up=True, fill=0xA5A5):
    return [{n: np.full(s, fill, dtype=np.uint16) for n, s in shard_shapes(m, TP, fused_qkv, fused_gate_up).items()}
            for _ in range(TP)]


def weights_shard(logical: dict, m, TP, fused_qkv=True, fused_gate_up=True):
    """One layer's logical weights -> list of TP shard dicts (fused buffers live under 'q' and 'gate')."""
    shards = empty_shards(m, TP, fused_qkv, fused_gate_up)
    lg = _wstruct(logical)
    mm = _model(m)
    for r in range(TP):
        sh = _wstruct(shards[r])
        lib().oracle_weights_shard(C.byref(mm), TP, r, int(fused_qkv), int(fused_gate_up), C.byref(lg), C.byref(sh))
    return shards


def logical_shapes(m: dict) -> dict:
    hid, qr, kr, I = m["hidden"], m["Hq"] * m["D"], m["Hkv"] * m["D"], m["I"]
    return {"q": (qr, hid), "k": (kr, hid), "v": (kr, hid), "o": (hid, qr), "gate": (I, hid), "up": (I, hid),
            "down": (hid, I)}


def weights_reconstruct(shards, m, TP, fused_qkv=True, fused_gate_up=True):
    logical = {n: np.zeros(s, dtype=np.uint16) for n, s in logical_shapes(m).items()}
    lg = _wstruct(logical)
    mm = _model(m)
    for r in range(TP):
        sh = _wstruct(shards[r])
        lib().oracle_weights_reconstruct(C.byref(mm), TP, r, int(fused_qkv), int(fused_gate_up), C.byref(lg),
                                         C.byref(sh))
    return logical


def weights_transform(src_shards, m, a, b, fused_qkv=True, fused_gate_up=True, dst_shards=None):
    """TP a->b on one layer's weights (reconstruct, then shard); returns the b destination shard dicts."""
    if dst_shards is None:
        dst_shards = empty_shards(m, b, fused_qkv, fused_gate_up)
    src = (_Weights * a)(*[_wstruct(s) for s in src_shards])
    dst = (_Weights * b)(*[_wstruct(s) for s in dst_shards])
    mm = _model(m)
    rc = lib().oracle_weights_transform(C.byref(mm), int(fused_qkv), int(fused_gate_up), a, src, b, dst)
    assert rc == 0
    return dst_shards


def assign_blocks(seq_lens, T, src_bt, NB_src, NB_dst, free_list=None, free_mask=None, pairs_cap=None, status=0):
    """Destination block bookkeeping; returns (dst_bt, pairs[N,2], N, free_left, status)."""
    sl, slp = _i32(seq_lens)
    sbt, sbtp = _i32(src_bt)
    S, maxb = sbt.shape
    assert (free_list is None) != (free_mask is None)
    if free_list is not None:
        fl, flp = _i32(free_list)
        n, fmp = len(fl), None
    else:
        fm = np.ascontiguousarray(free_mask, dtype=np.uint8)
        n, flp, fmp = len(fm), None, fm.ctypes.data_as(C.POINTER(C.c_uint8))
    if pairs_cap is None:
        pairs_cap = S * maxb
    dst_bt = np.empty((S, maxb), dtype=np.int32)
    pairs = np.full((max(pairs_cap, 1), 2), -7, dtype=np.int32)
    npairs, nfree, st = C.c_int32(0), C.c_int32(0), C.c_int32(status)
    lib().oracle_assign_blocks(S, slp, T, sbtp, maxb, NB_src, flp, fmp, n, NB_dst,
                               dst_bt.ctypes.data_as(C.POINTER(C.c_int32)),
                               pairs.ctypes.data_as(C.POINTER(C.c_int32)), pairs_cap, C.byref(npairs),
                               C.byref(nfree), C.byref(st))
    return dst_bt, pairs[:npairs.value].copy(), npairs.value, nfree.value, st.value


def pairs_by_destination(pairs, dst_bt, seq_lens, T):
    """The work list of ``assign_blocks`` / ``kv_reshape_inplace`` (entry k = the k-th block in (sequence, block) order)
    listed the other way the table calls offer: ascending by the destination id each block was given, and the blocks
    that were given none - their entries are (-1,-1) - at the end.  The paper fixes no order of the migration work
    (Sec. 3.1); the set of pairs is the same in both orders.  ``dst_bt`` is the destination table of the same call
    (-1 where a block got no id).  Plain loops."""
    pairs = np.asarray(pairs, dtype=np.int32).reshape(-1, 2)
    if len(pairs) == 0:  # a call that failed as a whole lists nothing
        return pairs
    given, k = [], 0
    for s, length in enumerate(seq_lens):
        for i in range((max(int(length), 0) + T - 1) // T):
            given.append((int(dst_bt[s][i]), k))
            k += 1
    assert k == len(pairs)
    with_id = sorted(e for e in given if e[0] >= 0)  # destination ids are distinct: no ties
    out = [pairs[k] for _, k in with_id] + [(-1, -1)] * (len(given) - len(with_id))
    return np.asarray(out, dtype=np.int32).reshape(-1, 2)



def kv_split_inplace(m, T, N, a, NB, seq_lens, bt, pools, status=0, layer_stride=None):
    """The way back from ``kv_merge_inplace``: one instance of TP=N*a becomes N instances of TP=a in place.

    seq_lens [N][S], bt [N][S][maxb]: the merged instance's table rows of the requests that go to instance i (ids over
    NB*N blocks, each = i mod N); pools[i*a + r] = merged worker r*N+i, rewritten into worker r of instance i.
    Returns (old_bt [N][S][maxb] with q -> q // N, live [N][NB], status)."""
    sl = np.ascontiguousarray(seq_lens, dtype=np.int32)
    b = np.ascontiguousarray(bt, dtype=np.int32)
    assert sl.ndim == 2 and b.ndim == 3 and sl.shape[0] == N and b.shape[:2] == sl.shape and len(pools) == N * a
    S, maxb = b.shape[1], b.shape[2]
    stride = pool_elems_per_layer(m, T, a, NB) if layer_stride is None else layer_stride
    old_bt = np.empty_like(b)
    live = np.empty((N, NB), dtype=np.uint8)
    st = C.c_int32(status)
    mm = _model(m)
    lib().oracle_kv_split_inplace(C.byref(mm), T, N, a, NB, C.c_int64(stride), S,
                                  sl.ctypes.data_as(C.POINTER(C.c_int32)), maxb,
                                  b.ctypes.data_as(C.POINTER(C.c_int32)), _ptr_array(pools),
                                  old_bt.ctypes.data_as(C.POINTER(C.c_int32)),
                                  live.ctypes.data_as(C.POINTER(C.c_uint8)), C.byref(st))
    return old_bt, live, st.value


def kv_merge_inplace(m, T, N, a, NB, seq_lens, bt, pools, status=0, layer_stride=None):
    """In-place merge of N instances of TP=a into one of TP=N*a (Sec. 3.1, Improvement 1).

    seq_lens [N][S], bt [N][S][maxb]; pools: list of N*a uint16 arrays, pools[i*a + r] = worker r of instance i
    (header-centric, NB blocks per layer), rewritten in place into worker r*N+i of the merged instance (NB*N blocks of
    Hkv/(N*a) headers).  Returns (new_bt [N][S][maxb], live [N][NB], status)."""
    sl = np.ascontiguousarray(seq_lens, dtype=np.int32)
    b = np.ascontiguousarray(bt, dtype=np.int32)
    assert sl.ndim == 2 and b.ndim == 3 and sl.shape[0] == N and b.shape[:2] == sl.shape and len(pools) == N * a
    S, maxb = b.shape[1], b.shape[2]
    stride = pool_elems_per_layer(m, T, a, NB) if layer_stride is None else layer_stride
    new_bt = np.empty_like(b)
    live = np.empty((N, NB), dtype=np.uint8)
    st = C.c_int32(status)
    mm = _model(m)
    lib().oracle_kv_merge_inplace(C.byref(mm), T, N, a, NB, C.c_int64(stride), S,
                                  sl.ctypes.data_as(C.POINTER(C.c_int32)), maxb,
                                  b.ctypes.data_as(C.POINTER(C.c_int32)), _ptr_array(pools),
                                  new_bt.ctypes.data_as(C.POINTER(C.c_int32)),
                                  live.ctypes.data_as(C.POINTER(C.c_uint8)), C.byref(st))
    return new_bt, live, st.value



# ---- Sec. 3.2, Improvement 1: padded partitions -----------------------------------------------------------------
def pages_per_tensor(rows: int, cols: int, elem_bytes: int, TP: int, page_bytes: int = 2 << 20) -> float:
    f = lib().oracle_pages_per_tensor
    f.restype = C.c_double
    return f(C.c_int64(rows), C.c_int64(cols), elem_bytes, TP, C.c_int64(page_bytes))


def padded_pitch(partition_elems: int, page_elems: int) -> int:
    f = lib().oracle_padded_pitch
    f.restype = C.c_int64
    return f(C.c_int64(partition_elems), C.c_int64(page_elems))


def padded_partition_elems(m: dict, P: int, fused_qkv=True, fused_gate_up=True) -> dict:
    """Elements of one partition of each buffer (before rounding up to pages)."""
    hid, q, kv, f = m["hidden"], m["Hq"] * m["D"] // P * m["hidden"], m["Hkv"] * m["D"] // P * m["hidden"], \
        m["I"] // P * m["hidden"]
    out = {"o": q, "down": f}
    if fused_qkv:
        out["q"] = q + 2 * kv
    else:
        out.update(q=q, k=kv, v=kv)
    if fused_gate_up:
        out["gate"] = 2 * f
    else:
        out.update(gate=f, up=f)
    return out


def empty_padded_shards(m, TP, P, page_elems, fused_qkv=True, fused_gate_up=True, fill=0xA5A5):
    """Flat uint16 buffers of P/TP padded partitions each, one dict per worker."""
    n = P // TP
    return [{name: np.full(n * padded_pitch(e, page_elems), fill, dtype=np.uint16)
             for name, e in padded_partition_elems(m, P, fused_qkv, fused_gate_up).items()} for _ in range(TP)]


def _padded_walk(logical, shards, m, TP, P, page_elems, fused_qkv, fused_gate_up, direction):
    lg = _wstruct(logical)
    mm = _model(m)
    for r in range(TP):
        sh = _wstruct(shards[r])
        lib().oracle_weights_padded_walk(C.byref(mm), TP, r, P, C.c_int64(page_elems), int(fused_qkv),
                                         int(fused_gate_up), C.byref(lg), C.byref(sh), direction)


def weights_shard_padded(logical, m, TP, P, page_elems, fused_qkv=True, fused_gate_up=True, fill=0xA5A5):
    shards = empty_padded_shards(m, TP, P, page_elems, fused_qkv, fused_gate_up, fill)
    _padded_walk(logical, shards, m, TP, P, page_elems, fused_qkv, fused_gate_up, 0)
    return shards


def weights_reconstruct_padded(shards, m, TP, P, page_elems, fused_qkv=True, fused_gate_up=True):
    logical = {n: np.zeros(s, dtype=np.uint16) for n, s in logical_shapes(m).items()}
    _padded_walk(logical, shards, m, TP, P, page_elems, fused_qkv, fused_gate_up, 1)
    return logical


def weights_transform_any(src_shards, m, a, b, fused_qkv=True, fused_gate_up=True, src_pad=None, dst_pad=None,
                          fill=0xA5A5):
    """TP a->b on one layer's weights where either side may be padded: ``*_pad`` = (P, page_elems) or None for the
    dense shards.  Reconstruct the logical tensors from the source form, shard them in the destination form."""
    if src_pad:
        logical = weights_reconstruct_padded(src_shards, m, a, src_pad[0], src_pad[1], fused_qkv, fused_gate_up)
    else:
        logical = weights_reconstruct(src_shards, m, a, fused_qkv, fused_gate_up)
    if dst_pad:
        return weights_shard_padded(logical, m, b, dst_pad[0], dst_pad[1], fused_qkv, fused_gate_up, fill)
    out = empty_shards(m, b, fused_qkv, fused_gate_up, fill)
    lg, mm = _wstruct(logical), _model(m)
    for r in range(b):
        sh = _wstruct(out[r])
        lib().oracle_weights_shard(C.byref(mm), b, r, int(fused_qkv), int(fused_gate_up), C.byref(lg), C.byref(sh))
    return out


# ---- Sec. 3.1, Improvement 1: in-place block reshaping of one instance ------------------------------------------
def kv_reshape_inplace(direction, m, T, N, a, NB, seq_lens, bt, pools, status=0, layer_stride=None, pairs_cap=None):
    """One instance, in place: ``direction`` "split" (TP=a -> TP=N*a, table over NB ids) or "merge" (TP=N*a -> TP=a,
    table over NB*N ids).  pools: list of N*a uint16 arrays, pools[w] = worker w of the TP=N*a side, worker r of the
    TP=a side is pools[r*N]; NB = blocks per layer of the TP=a side.  Rewrites the pools in place and returns
    (new_bt, pairs[n,2], n, free_mask, free_count, status)."""
    assert direction in ("split", "merge")
    sl, slp = _i32(seq_lens)
    b, bp = _i32(bt)
    assert b.ndim == 2 and b.shape[0] == len(sl) and len(pools) == N * a
    S, maxb = b.shape
    stride = pool_elems_per_layer(m, T, a, NB) if layer_stride is None else layer_stride
    if pairs_cap is None:
        pairs_cap = S * maxb
    new_bt = np.empty_like(b)
    pairs = np.full((max(pairs_cap, 1), 2), -7, dtype=np.int32)
    free_mask = np.empty(NB * N if direction == "split" else NB, dtype=np.uint8)
    n, left, st = C.c_int32(0), C.c_int32(0), C.c_int32(status)
    mm = _model(m)
    f = lib().oracle_kv_reshape_split if direction == "split" else lib().oracle_kv_reshape_merge
    f(C.byref(mm), T, N, a, NB, C.c_int64(stride), S, slp, maxb, bp, _ptr_array(pools),
      new_bt.ctypes.data_as(C.POINTER(C.c_int32)), pairs.ctypes.data_as(C.POINTER(C.c_int32)), pairs_cap,
      C.byref(n), free_mask.ctypes.data_as(C.POINTER(C.c_uint8)), C.byref(left), C.byref(st))
    return new_bt, pairs[:n.value].copy(), n.value, free_mask, left.value, st.value

"""Seeded synthetic model and KV-cache states for the TP re-layout tests and benchmark.

This module only *draws inputs*: model shapes, sequence lengths, block tables, free lists / masks, logical
tensor values and raw buffer fills.  It contains none of the re-layout's arithmetic (no head or column
partitioning, no pool addressing) and imports neither the CPU oracle nor the CUDA binding; both sides are fed
from here.

The shapes and length mixes stand in for the serving workloads the paper evaluates on (public model shapes;
its request trace is private).  No checkpoint values and no trace records are used: everything is drawn from a
counter-based generator keyed by (seed, purpose, index), so any layer can be produced on its own.
"""
from __future__ import annotations

import hashlib
import math

import numpy as np

DEFAULT_SEED = 20250919
BLOCK_TOKENS = 16


def _model(L, hidden, Hq, Hkv, D, I):
    return dict(L=L, hidden=hidden, Hq=Hq, Hkv=Hkv, D=D, I=I)


# name -> recipe.  "a"/"b" are the source and destination TP degrees.
#   lens      : how sequence lengths are drawn
#   src_free  : fraction of the source pool left free (live blocks are scattered over the whole pool)
#   dst_form  : "list" = destination free blocks given as a shuffled id list,
#               "mask" = given as a byte mask with `dst_occupied` of the pool held by foreign blocks
#   dst_slack : extra destination blocks beyond the ones needed (stay untouched)
#   kv_layers : layers of KV pools instantiated (None = all layers of the model)
CONFIGS = {
    "tiny_2to1": dict(model=_model(2, 256, 4, 4, 64, 1024), dtype="fp16", a=2, b=1, S=8,
                      lens=("uniform", 16, 256), src_free=0.25, dst_form="list", dst_slack=0.25, kv_layers=None),
    "llama2_7b_1to2": dict(model=_model(32, 4096, 32, 32, 128, 11008), dtype="bf16", a=1, b=2, S=64,
                           lens=("loguniform", 128, 4096), src_free=1 / 16, dst_form="list", dst_slack=1 / 16,
                           kv_layers=None),
    "llama2_13b_4to1": dict(model=_model(40, 5120, 40, 40, 128, 13824), dtype="bf16", a=4, b=1, S=256,
                            lens=("lognormal", 1024, 1.0, 32768), src_free=0.30, dst_form="mask",
                            dst_occupied=0.30, dst_slack=0.0, kv_layers=4),
    "llama3_8b_1to4": dict(model=_model(32, 4096, 32, 8, 128, 14336), dtype="bf16", a=1, b=4, S=128,
                           lens=("uniform", 512, 8192), src_free=0.0, dst_form="list", dst_slack=1 / 64,
                           kv_layers=None),
    "llama3_8b_2to8": dict(model=_model(32, 4096, 32, 8, 128, 14336), dtype="bf16", a=2, b=8, S=128,
                           lens=("uniform", 512, 8192), src_free=0.0, dst_form="list", dst_slack=1 / 64,
                           kv_layers=None),
    "llama3_70b_slice_8to2": dict(model=_model(8, 8192, 64, 8, 128, 28672), dtype="bf16", a=8, b=2, S=256,
                                  lens=("one_long_plus_uniform", 131072, 256, 2048), src_free=1 / 16,
                                  dst_form="list", dst_slack=1 / 16, kv_layers=None),
}


# In-place merges of N instances of TP=a into one of TP=N*a (the paper's KV micro-benchmark setting: 4 x TP1 -> TP4
# at 90 % KV-cache utilisation).  S sequences per instance; every instance has its own pool and block placement.
MERGE_CONFIGS = {
    "llama3_8b_merge_4x1to4": dict(model=_model(32, 4096, 32, 8, 128, 14336), dtype="bf16", N=4, a=1, S=48,
                                   lens=("uniform", 512, 8192), utilisation=0.9),
    # the same at 20 sequences per instance, so that a second set of pools (the out-of-place merge) also fits one GPU
    "llama3_8b_merge_4x1to4_s20": dict(model=_model(32, 4096, 32, 8, 128, 14336), dtype="bf16", N=4, a=1, S=20,
                                       lens=("uniform", 512, 8192), utilisation=0.9, weights=True),
    "tiny_merge_2x1to2": dict(model=_model(2, 256, 4, 4, 64, 1024), dtype="fp16", N=2, a=1, S=4,
                              lens=("uniform", 16, 256), utilisation=0.75),
}


def key(seed: int, purpose: str, *index: int) -> int:
    """128-bit generator key from (seed, purpose, index...)."""
    h = hashlib.blake2b(repr((int(seed), purpose, tuple(int(i) for i in index))).encode(), digest_size=16)
    return int.from_bytes(h.digest(), "little")


def rng(seed: int, purpose: str, *index: int) -> np.random.Generator:
    k = key(seed, purpose, *index)
    return np.random.Generator(np.random.Philox(key=[k & (2**64 - 1), k >> 64]))


def to_bits(x: np.ndarray, dtype: str) -> np.ndarray:
    """float32 -> 16-bit words (fp16 or bf16, round to nearest even)."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    if dtype == "fp16":
        return x.astype(np.float16).view(np.uint16)
    u = x.view(np.uint32)
    return ((u + 0x7FFF + ((u >> 16) & 1)) >> 16).astype(np.uint16)


def from_bits(w: np.ndarray, dtype: str) -> np.ndarray:
    """16-bit words -> float64."""
    w = np.ascontiguousarray(w, dtype=np.uint16)
    if dtype == "fp16":
        return w.view(np.float16).astype(np.float64)
    return (w.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def draw_seq_lens(cfg: dict, seed: int = DEFAULT_SEED, name: str = "") -> np.ndarray:
    g = rng(seed, "seq_lens", *name.encode())
    S, spec = cfg["S"], cfg["lens"]
    if spec[0] == "uniform":
        lens = g.integers(spec[1], spec[2] + 1, size=S)
    elif spec[0] == "loguniform":
        lens = np.rint(np.exp(g.uniform(math.log(spec[1]), math.log(spec[2]), size=S)))
    elif spec[0] == "lognormal":
        lens = np.clip(np.rint(spec[1] * np.exp(spec[2] * g.standard_normal(size=S))), 1, spec[3])
    elif spec[0] == "one_long_plus_uniform":
        lens = np.concatenate([[spec[1]], g.integers(spec[2], spec[3] + 1, size=S - 1)])
    else:
        raise ValueError(spec)
    return lens.astype(np.int32)


def draw_kv_state(cfg: dict, seed: int = DEFAULT_SEED, name: str = "", seq_lens=None, T: int = BLOCK_TOKENS) -> dict:
    """Sequence lengths, a scattered source block table and the destination's free blocks.

    Returns a dict with seq_lens [S], blocks_per_seq [S], n_live, NB_src, NB_dst, maxb, src_bt [S,maxb] (-1
    padded) and either dst_free_list [NB_dst'] or dst_free_mask [NB_dst] (1 = free; occupied blocks belong to
    someone else and must survive).
    """
    lens = draw_seq_lens(cfg, seed, name) if seq_lens is None else np.asarray(seq_lens, dtype=np.int32)
    nblk = (lens.astype(np.int64) + T - 1) // T
    n_live = int(nblk.sum())
    maxb = max(int(nblk.max()) if len(nblk) else 0, 1)
    NB_src = max(int(math.ceil(n_live / (1.0 - cfg.get("src_free", 0.0)))), 1)
    g = rng(seed, "src_blocks", *name.encode())
    placement = g.permutation(NB_src)[:n_live].astype(np.int32)
    src_bt = np.full((len(lens), maxb), -1, dtype=np.int32)
    k = 0
    for s, n in enumerate(nblk):
        src_bt[s, :n] = placement[k:k + n]
        k += int(n)
    st = dict(seq_lens=lens, blocks_per_seq=nblk, n_live=n_live, NB_src=NB_src, maxb=maxb, src_bt=src_bt, T=T)
    g = rng(seed, "dst_blocks", *name.encode())
    if cfg.get("dst_form", "list") == "list":
        NB_dst = max(int(math.ceil(n_live * (1.0 + cfg.get("dst_slack", 0.0)))), 1)
        st["NB_dst"] = NB_dst
        st["dst_free_list"] = g.permutation(NB_dst).astype(np.int32)
    else:
        occ = cfg.get("dst_occupied", 0.3)
        NB_dst = max(int(math.ceil(n_live * (1.0 + cfg.get("dst_slack", 0.0)) / (1.0 - occ))) + 1, 1)
        mask = np.ones(NB_dst, dtype=np.uint8)
        mask[g.permutation(NB_dst)[: NB_dst - int(math.ceil(n_live * (1.0 + cfg.get("dst_slack", 0.0))))]] = 0
        st["NB_dst"] = NB_dst
        st["dst_free_mask"] = mask
    return st


def draw_merge_state(cfg: dict, seed: int = DEFAULT_SEED, name: str = "", T: int = BLOCK_TOKENS) -> dict:
    """Tables of the N instances of a merge workload: seq_lens [N][S], src_bt [N][S][maxb] (-1 padded; each instance's
    live blocks scattered over its own pool of NB blocks), NB, maxb, n_live (live blocks summed over instances)."""
    N, S = cfg["N"], cfg["S"]
    lens = np.stack([draw_seq_lens(cfg, seed, f"{name}/{i}") for i in range(N)])
    nblk = (lens.astype(np.int64) + T - 1) // T
    maxb = max(int(nblk.max()), 1)
    NB = max(int(math.ceil(int(nblk.sum(axis=1).max()) / cfg.get("utilisation", 0.9))), 1)
    bt = np.full((N, S, maxb), -1, dtype=np.int32)
    for i in range(N):
        ids = rng(seed, "merge_blocks", i, *name.encode()).permutation(NB).astype(np.int32)
        k = 0
        for s in range(S):
            bt[i, s, :nblk[i, s]] = ids[k:k + nblk[i, s]]
            k += int(nblk[i, s])
    return dict(seq_lens=lens.astype(np.int32), src_bt=bt, NB=NB, maxb=maxb, n_live=int(nblk.sum()),
                blocks_per_seq=nblk, T=T)


def counter_words(n: int, salt: int) -> np.ndarray:
    """n 16-bit words, word i = low 16 bits of (i mod 65521)*40503 + salt: a cheap, reproducible, non-constant fill
    (one period is computed, the rest is copied)."""
    period = (np.arange(65521, dtype=np.uint32) * np.uint32(40503) + np.uint32(salt & 0xFFFF)).astype(np.uint16)
    return np.resize(period, n)


def draw_kv_logical(cfg: dict, n_tokens: int, layers, seed: int = DEFAULT_SEED, dist: str = "normal") -> np.ndarray:
    """Logical KV values for the given layers: uint16 [len(layers), n_tokens, Hkv, 2, D].

    dist "normal": N(0,1) rounded to the config's 16-bit float type; "words": uniform 16-bit words (several times
    faster to draw); "counter": a periodic counter pattern (memory-speed; for timing runs, where the values do not
    matter)."""
    m = cfg["model"]
    out = np.empty((len(layers), n_tokens, m["Hkv"], 2, m["D"]), dtype=np.uint16)
    for i, l in enumerate(layers):
        if dist == "counter":
            out[i] = counter_words(out[i].size, l).reshape(out.shape[1:])
        elif dist == "words":
            out[i] = rng(seed, "kv_words", l).integers(0, 65536, size=out.shape[1:], dtype=np.uint16)
        else:
            x = rng(seed, "kv", l).standard_normal(size=out.shape[1:], dtype=np.float32)
            out[i] = to_bits(x, cfg["dtype"])
    return out


def draw_weights_logical(cfg: dict, layer: int, seed: int = DEFAULT_SEED, std: float = 0.02,
                         dist: str = "normal") -> dict:
    """One layer's logical weights, [out,in] row-major, as uint16 words: N(0, std) rounded to the config's 16-bit
    float type, or (dist "words", for timing runs) uniform 16-bit words."""
    m = cfg["model"]
    hid, qr, kr, I = m["hidden"], m["Hq"] * m["D"], m["Hkv"] * m["D"], m["I"]
    shapes = {"q": (qr, hid), "k": (kr, hid), "v": (kr, hid), "o": (hid, qr), "gate": (I, hid), "up": (I, hid),
              "down": (hid, I)}
    out = {}
    for j, (n, s) in enumerate(shapes.items()):
        if dist == "counter":
            out[n] = counter_words(s[0] * s[1], layer * 7 + j).reshape(s)
            continue
        if dist == "words":
            out[n] = rng(seed, "w_words", layer, j).integers(0, 65536, size=s, dtype=np.uint16)
            continue
        x = rng(seed, "w", layer, j).standard_normal(size=s, dtype=np.float32) * np.float32(std)
        out[n] = to_bits(x, cfg["dtype"])
    return out


# ---- raw buffer fill (for states too large to draw through logical tensors) ----
_M1 = -7046029254386353131  # 0x9E3779B97F4A7C15 as int64
_M2 = -4658895280553007687  # 0xBF58476D1CE4E5B9
_M3 = -7723592293110705685  # 0x94D049BB133111EB


def hash_fill_(buf, seed: int, stream_id: int, chunk_words: int = 1 << 26) -> None:
    """Fill a torch uint8/int16/int64 buffer (CPU or CUDA, size a multiple of 8 bytes) with a counter hash.

    Word i of the buffer (viewed as int64) becomes mix64(seed, stream_id, i): the same bytes on any device, so
    a CPU copy of any slice can be regenerated without reading the device.
    """
    import torch

    w = buf.view(torch.int64).view(-1)
    base = (key(seed, "fill", stream_id) & (2**63 - 1))
    for lo in range(0, w.numel(), chunk_words):
        hi = min(lo + chunk_words, w.numel())
        z = torch.arange(lo, hi, dtype=torch.int64, device=w.device)
        z = (z + base) * _M1
        z = (z ^ ((z >> 30) & ((1 << 34) - 1))) * _M2
        z = (z ^ ((z >> 27) & ((1 << 37) - 1))) * _M3
        z = z ^ ((z >> 31) & ((1 << 33) - 1))
        w[lo:hi] = z

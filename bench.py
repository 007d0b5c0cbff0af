#!/usr/bin/env python
"""Benchmark of the TP a->b re-layout hot path on B200.

One step = one whole transformation of one instance: block-table rewrite, KV-cache migration and weight
re-partition (three C-ABI calls, all kernels of the library).  Prints ONE JSON line.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--config NAME] [--impl ours|reference]

N > 1 (under torchrun) runs one independent instance per GPU (the path has no exchange step on one node: every
worker's shard lives on the same GPU), so scaling is weak and the value is the sum over ranks / max time.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import workloads as wl  # noqa: E402

METRIC = "reshard GB/s (read+write)"
DEFAULT_CONFIG = "llama3_8b_1to4"
FALLBACK_HBM_GBS = 6650.0
NOMINAL_HBM_GBS = 8000.0

# DRAM bytes (read + written) per algorithmic byte of kv_reshard_pair (the default copy path), from an ncu capture of
# a one-layer slice of the workload below, scaled by the bytes of a full launch (every layer repeats the same work on
# disjoint memory).  It is a stored counter reading, not something this script measures: the line says so in
# "traffic_source", and it is only quoted for that workload with default kernel options (None = no reading for the
# current kernel).
NCU_KV_TRAFFIC_RATIO = 0.9893
NCU_KV_TRAFFIC_CONFIG = "llama3_8b_1to4"
NCU_KV_TRAFFIC_SOURCE = "ncu dram__bytes_read.sum + dram__bytes_write.sum on a 1-layer slice, scaled by units processed"


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return float(json.load(open(p))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples nvidia-smi SM clocks and throttle reasons while the timed region runs."""

    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self) -> dict:
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        self.t.join(timeout=2)
        sm = [float(r[0]) for r in self.rows if len(r) >= 7 and r[0].replace(".", "").isdigit()]
        mx = [float(r[1]) for r in self.rows if len(r) >= 7 and r[1].replace(".", "").isdigit()]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = [n for i, n in enumerate(names) if any(len(r) >= 7 and r[3 + i] == "Active" for r in self.rows)]
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": reasons, "samples": len(sm)}


def dist_setup(n_gpus: int):
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist

        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl" if n_gpus > 0 else "gloo")
    return rank, world, local


def aggregate(world: int, seconds: float, bytes_per_rank: float, device=None):
    """Whole-job time (max over ranks) and bytes (sum over ranks); identity for one process."""
    if world == 1:
        return seconds, bytes_per_rank
    import torch
    import torch.distributed as dist

    t = torch.tensor([seconds], dtype=torch.float64, device=device)
    b = torch.tensor([bytes_per_rank], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(b, op=dist.ReduceOp.SUM)
    return float(t.item()), float(b.item())


THROTTLE_REASONS = {"hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown"}


def any_rank(world: int, device, flag: bool) -> bool:
    """True if the flag is set on any rank (every rank gets the same answer)."""
    if world == 1:
        return flag
    import torch
    import torch.distributed as dist

    t = torch.tensor([1.0 if flag else 0.0], device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return bool(t.item() > 0)


def barrier(world: int):
    if world > 1:
        import torch.distributed as dist

        dist.barrier()


# ------------------------------------------------------------------------------------------------ CPU oracle leg
def oracle_sample(cfg_name: str, kv_layers=4, n_seqs=None, w_layers=4, threads=1, dist="words"):
    """A bounded sample of the workload for the CPU oracle: the first n_seqs sequences (None = all) over kv_layers
    layers of KV, and w_layers layers of weights; values are uniform 16-bit words or a counter pattern (the movement
    does not depend on them).  Returns a closure that runs one oracle a->b pass and the bytes it moves.  threads > 1:
    the oracle's own layer loop runs on that many OpenMP threads for the KV cache, and the weight layers (one oracle
    call each) are issued from as many host threads - one thread per layer, as far as there are layers."""
    from concurrent.futures import ThreadPoolExecutor

    import oracle

    oracle.build()
    oracle.set_threads(threads)
    cfg = wl.CONFIGS[cfg_name]
    m, a, b, T = dict(cfg["model"]), cfg["a"], cfg["b"], wl.BLOCK_TOKENS
    lens = wl.draw_seq_lens(cfg, name=cfg_name)[:n_seqs]
    kv_layers, w_layers = min(kv_layers, cfg.get("kv_layers") or m["L"]), min(w_layers, m["L"])
    m_kv = dict(m, L=kv_layers)
    st = wl.draw_kv_state(cfg, name=cfg_name, seq_lens=lens)
    G = int(st["blocks_per_seq"].sum()) * T
    KV = wl.draw_kv_logical(dict(cfg, model=m_kv), G, range(kv_layers), dist=dist)
    src = oracle.kv_shard(KV, m_kv, T, a, st["NB_src"], lens, st["src_bt"])
    del KV
    free = dict(free_list=st.get("dst_free_list"), free_mask=st.get("dst_free_mask"))
    dst = [np.full(kv_layers * oracle.pool_elems_per_layer(m_kv, T, b, st["NB_dst"]), 0xA5A5, np.uint16)
           for _ in range(b)]
    W = [oracle.weights_shard(wl.draw_weights_logical(cfg, l, dist=dist), m, a) for l in range(w_layers)]
    Wd = [oracle.empty_shards(m, b) for _ in range(w_layers)]
    e = 2
    kv_bytes = 2 * st["n_live"] * kv_layers * m["Hkv"] * 2 * T * m["D"] * e
    w_bytes = 2 * w_layers * e * (2 * m["Hq"] * m["D"] * m["hidden"] + 2 * m["Hkv"] * m["D"] * m["hidden"]
                                  + 3 * m["hidden"] * m["I"])

    def run():
        dst_bt, pairs, n, left, status = oracle.assign_blocks(lens, T, st["src_bt"], st["NB_src"], st["NB_dst"], **free)
        assert status == 0
        oracle.kv_transform(m_kv, T, lens, a, st["NB_src"], st["src_bt"], src, b, st["NB_dst"], dst_bt, dst)
        if threads > 1:  # the C calls release the interpreter lock: one host thread per weight layer
            with ThreadPoolExecutor(max_workers=min(threads, w_layers)) as pool:
                list(pool.map(lambda l: oracle.weights_transform(W[l], m, a, b, dst_shards=Wd[l]), range(w_layers)))
        else:
            for l in range(w_layers):
                oracle.weights_transform(W[l], m, a, b, dst_shards=Wd[l])

    desc = (f"{cfg_name}: first {len(lens)} of {cfg['S']} sequences ({st['n_live']} blocks) x {kv_layers} of "
            f"{m['L']} KV layers + {w_layers} of {m['L']} weight layers")
    return run, kv_bytes + w_bytes, desc


def oracle_merge_sample(cfg_name: str, kv_layers=1, n_seqs=16):
    """A bounded sample of a merge workload for the CPU oracle: the first n_seqs sequences of every instance over
    kv_layers layers.  Returns a closure that runs one oracle in-place merge and the bytes the merge moves."""
    import oracle

    oracle.build()
    cfg = wl.MERGE_CONFIGS[cfg_name]
    m, N, a, T = dict(cfg["model"], L=kv_layers), cfg["N"], cfg["a"], wl.BLOCK_TOKENS
    st = wl.draw_merge_state(dict(cfg, S=min(n_seqs, cfg["S"])), name=cfg_name)
    per = oracle.pool_elems_per_layer(m, T, a, st["NB"])
    g = wl.rng(wl.DEFAULT_SEED, "merge_sample")
    pools = [g.integers(0, 65536, size=kv_layers * per, dtype=np.uint16) for _ in range(N * a)]
    nbytes = 2 * st["n_live"] * kv_layers * (m["Hkv"] // N) * (N - 1) * 2 * T * m["D"] * 2

    def run():
        _, _, status = oracle.kv_merge_inplace(m, T, N, a, st["NB"], st["seq_lens"], st["src_bt"], pools)
        assert status == 0

    desc = (f"{cfg_name}: first {min(n_seqs, cfg['S'])} of {cfg['S']} sequences per instance ({st['n_live']} blocks) x "
            f"{kv_layers} of {cfg['model']['L']} layers")
    return run, nbytes, desc


def run_reference(args, rank, world):
    """The reference arm: the CPU oracle as it stands, timed on the host cores on a bounded sample per step."""
    if rank != 0:
        return
    if args.config in wl.MERGE_CONFIGS:
        run, nbytes, desc = oracle_merge_sample(args.config)
        cfg = dict(wl.MERGE_CONFIGS[args.config])
        cfg["a"], cfg["b"] = f"{cfg['N']}x{cfg['a']}", cfg["N"] * cfg["a"]
    else:
        run, nbytes, desc = oracle_sample(args.config, kv_layers=1, w_layers=2)
        cfg = wl.CONFIGS[args.config]
    for _ in range(args.warmup):
        run()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        run()
    dt = (time.perf_counter() - t0) / args.steps
    val = nbytes / dt / 1e9
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": "GB/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "u8", "data": "synthetic",
        "config": {"workload": args.config, "tp": f"{cfg['a']}->{cfg['b']}", "sample": desc},
        "cpu_baseline": {"value": val, "unit": "GB/s", "cores": 1, "kind": "oracle", "sample": desc},
        "e2e": {"value": val, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def cpu_baseline(cfg_name: str) -> dict:
    """The oracle as it stands on the host cores, on bounded samples of the workload: once on one thread, once with
    one thread per layer over all cores.  The top-level value is the all-cores one; `cores` = threads it used."""
    cfg = wl.CONFIGS[cfg_name]
    m = cfg["model"]
    st = wl.draw_kv_state(cfg, name=cfg_name)
    layer_bytes = st["n_live"] * m["Hkv"] * 2 * wl.BLOCK_TOKENS * m["D"] * 2  # live KV of one layer
    # a sample of k layers holds about 4 k copies of that on the host (sources, destinations, logical state twice)
    k1 = int(max(1, min(4, host_free_bytes() // 2 // (4 * layer_bytes)))) if host_free_bytes() else 4
    run, nbytes, desc = oracle_sample(cfg_name, kv_layers=k1, w_layers=k1)
    t0 = time.perf_counter()
    run()
    dt1 = time.perf_counter() - t0
    one = {"value": nbytes / dt1 / 1e9, "unit": "GB/s", "cores": 1, "sample": desc, "seconds": dt1}
    del run
    cores = os.cpu_count() or 1
    L_kv = cfg.get("kv_layers") or cfg["model"]["L"]
    threads = max(1, min(cores, L_kv))
    w_threads = max(1, min(threads, 8))  # weight layers in the sample (each is hundreds of MB of host memory)
    # about the same number of bytes as the one-thread sample, spread over `threads` layers: fewer sequences per layer
    n_seqs = max(1, cfg["S"] * k1 // threads)
    runN, nbytesN, descN = oracle_sample(cfg_name, kv_layers=threads, n_seqs=n_seqs, w_layers=w_threads,
                                         threads=threads, dist="counter")
    t0 = time.perf_counter()
    runN()
    dtN = time.perf_counter() - t0
    import oracle

    oracle.set_threads(1)
    allc = {"value": nbytesN / dtN / 1e9, "unit": "GB/s", "cores": threads, "host_cores": cores,
            "threads_kv": threads, "threads_weights": w_threads, "sample": descN, "seconds": dtN}
    return {"value": allc["value"], "unit": "GB/s", "cores": threads, "kind": "oracle",
            "sample": descN + f"; {threads} threads (one per KV layer), {w_threads} for the weight layers",
            "seconds": dtN, "one_thread": one, "all_cores": allc}


# ------------------------------------------------------------------------------------------------ GPU leg
KV_ORDERS = {"head": (0, 0), "token": (1, 1), "token2head": (1, 0), "head2token": (0, 1)}  # (source, destination)


def build_session(cfg_name: str, device, layers=None, kv=True, weights=True, seed=wl.DEFAULT_SEED, fill=True,
                  kv_order="head", weight_pad=0):
    import torch

    from paper_2509_19729_b200.session import Session

    cfg = wl.CONFIGS[cfg_name]
    m = dict(cfg["model"])
    kv_layers = cfg.get("kv_layers")
    if layers is not None:  # a slice of the model's layers (all tensors of those layers)
        m["L"] = layers
        kv_layers = None if kv_layers is None else min(kv_layers, layers)
    st = wl.draw_kv_state(cfg, seed=seed, name=cfg_name)
    s = Session(m, cfg["a"], cfg["b"], st["NB_src"], st["NB_dst"], cfg["S"], st["maxb"], st["n_live"],
                kv_layers=kv_layers, kv=kv, weights=weights, device=device, dst_fill=None,
                src_kv_order=KV_ORDERS[kv_order][0], dst_kv_order=KV_ORDERS[kv_order][1],
                src_weight_pad=(weight_pad, 0) if weight_pad else None,
                dst_weight_pad=(weight_pad, 0) if weight_pad else None)
    s.set_tables(st["seq_lens"], st["src_bt"], st.get("dst_free_list"), st.get("dst_free_mask"))
    if fill:
        for i, p in enumerate(s.src_pools):
            wl.hash_fill_(p, seed, 100 + i)
        for i, p in enumerate(s._wbufs[:cfg["a"]]):
            n = p.numel() // 8 * 8
            wl.hash_fill_(p[:n], seed, 200 + i)
        for p in s.dst_pools + s._wbufs[cfg["a"]:]:
            p.fill_(0xA5)
    torch.cuda.synchronize()
    return s, st


def measure_config(cfg_name: str, device, steps: int = 5, warmup: int = 3) -> dict:
    """Device time of the KV and weight calls of one benchmark configuration (default kernel options, all layers the
    configuration holds), for the per-configuration table of the bench line.  The buffers are left as allocated:
    the time of a copy does not depend on the values."""
    import torch

    s, st = build_session(cfg_name, device, fill=False)
    kv_bytes, w_bytes = s.bytes_rw(st["n_live"])
    stream = torch.cuda.current_stream()
    for _ in range(warmup):
        s.status.zero_()
        s.step()
    torch.cuda.synchronize()
    assert int(s.status.item()) == 0
    marks = []
    for _ in range(steps):
        m = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
        m[0].record(stream)
        s.rewrite_block_tables()
        m[1].record(stream)
        s.reshard_kv()
        m[2].record(stream)
        s.reshard_weights()
        m[3].record(stream)
        marks.append(m)
    torch.cuda.synchronize()
    assert int(s.status.item()) == 0
    bt_ms, kv_ms, w_ms = (statistics.mean(m[i].elapsed_time(m[i + 1]) for m in marks) for i in range(3))
    peak, _ = peaks()
    cfg = wl.CONFIGS[cfg_name]
    out = {"tp": f"{cfg['a']}->{cfg['b']}", "kv_layers": s.kv_layers, "layers": s.L, "live_blocks": st["n_live"],
           "tables_us": bt_ms * 1e3, "kv_ms": kv_ms, "kv_gbs": kv_bytes / kv_ms / 1e6, "kv_frac": kv_bytes / kv_ms / 1e6 / peak,
           "w_ms": w_ms, "w_gbs": w_bytes / w_ms / 1e6, "w_frac": w_bytes / w_ms / 1e6 / peak, "steps": steps}
    del s
    torch.cuda.empty_cache()
    return out


def build_reshape_session(cfg_name: str, device, layers=None, seed=wl.DEFAULT_SEED, fill=True, budget_gib=150.0):
    """One instance reshaped in place between TP=a and TP=b (b = N*a: split; a = N*b: merge back) with the
    configuration's sequences.  Every worker of the finer side has a pool of the coarser side's capacity, so the
    layer count is cut to what fits `budget_gib` of device memory (stated in the bench line)."""
    import torch

    import paper_2509_19729_b200 as A
    from paper_2509_19729_b200.session import ReshapeSession

    cfg = wl.CONFIGS[cfg_name]
    m = dict(cfg["model"])
    a, b = cfg["a"], cfg["b"]
    direction = "split" if b > a else "merge"
    N, coarse = max(a, b) // min(a, b), min(a, b)
    st = wl.draw_kv_state(cfg, seed=seed, name=cfg_name)
    NB = st["NB_src"]                                   # blocks of the coarser side
    per_layer = A.amoeba_layout_kv_pool_bytes(A.make_layout(m, coarse, NB)) // m["L"]
    fit = int(budget_gib * 2**30 // (per_layer * N * coarse))
    kv_layers = max(1, min(cfg.get("kv_layers") or m["L"], fit, layers or m["L"]))
    m["L"] = kv_layers
    src_bt = st["src_bt"] if direction == "split" else np.where(st["src_bt"] >= 0, st["src_bt"] * N, -1)
    s = ReshapeSession(m, N, coarse, NB, cfg["S"], st["maxb"], st["n_live"], direction=direction, device=device)
    s.set_tables(st["seq_lens"], src_bt.astype(np.int32))
    if fill:
        for i, p in enumerate(s.pools):
            wl.hash_fill_(p, seed, 600 + i)
    torch.cuda.synchronize()
    return s, st


def run_reshape(args, rank, world, local):
    """In-place block reshaping of one instance: one step = the reshaped block table + the KV migration of every
    header group that leaves its worker.  (Each step re-reads the same source segments: the old workers' memory is
    never written by a split.)"""
    import torch

    import paper_2509_19729_b200 as A

    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    cfg = wl.CONFIGS[args.config]
    s, st = build_reshape_session(args.config, device, layers=args.layers)
    for opt, val in ((A.OPT_COPY_PATH, args.copy_path), (A.OPT_CHUNK_BYTES, args.chunk), (A.OPT_STAGES, args.stages),
                     (A.OPT_CTAS_PER_SM, args.ctas_per_sm), (A.OPT_MAX_CTAS, args.max_ctas)):
        if val:
            s.set_option(opt, val)
    for item in args.opt:
        name, val = item.split("=")
        s.set_option(getattr(A, "OPT_" + name.upper()), int(val))
    nbytes = s.bytes_rw(st["n_live"])
    stream = torch.cuda.current_stream()
    ev = lambda: torch.cuda.Event(enable_timing=True)
    for _ in range(args.warmup):
        s.status.zero_()
        s.step()
    torch.cuda.synchronize()
    assert int(s.status.item()) == 0, f"device status {int(s.status.item())}"
    barrier(world)
    sampler = ClockSampler(local)
    sampler.start()
    time.sleep(0.3)
    launches0 = A.amoeba_launch_count()
    marks = []
    t_begin, t_end = ev(), ev()
    torch.cuda.synchronize()
    t_begin.record(stream)
    for _ in range(args.steps):
        m3 = [ev() for _ in range(3)]
        m3[0].record(stream)
        s.reshape_block_tables()
        m3[1].record(stream)
        s.reshape_kv()
        m3[2].record(stream)
        marks.append(m3)
    t_end.record(stream)
    torch.cuda.synchronize()
    launches = A.amoeba_launch_count() - launches0
    barrier(world)
    time.sleep(0.2)
    clocks = sampler.stop()
    assert int(s.status.item()) == 0
    sec = t_begin.elapsed_time(t_end) / 1e3 / args.steps
    bt_ms = statistics.mean(m3[0].elapsed_time(m3[1]) for m3 in marks)
    kv_ms = statistics.mean(m3[1].elapsed_time(m3[2]) for m3 in marks)
    sec_all, bytes_all = aggregate(world, sec, nbytes, device)
    if rank != 0:
        return
    peak, peak_kind = peaks()
    kv_gbs = nbytes / (kv_ms / 1e3) / 1e9
    N = max(cfg["a"], cfg["b"]) // min(cfg["a"], cfg["b"])
    full = nbytes * N // (N - 1)
    print(json.dumps({
        "metric": METRIC, "value": bytes_all / sec_all / 1e9, "unit": "GB/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": sec_all * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "u8", "data": "synthetic",
        "config": {"workload": args.config, "tp": f"{cfg['a']}->{cfg['b']} in place (one instance)",
                   "kv_layers": s.kv_layers, "layers_of_model": cfg["model"]["L"], "sequences": cfg["S"],
                   "live_blocks": st["n_live"], "block_tokens": wl.BLOCK_TOKENS, "kv_bytes_rw": nbytes,
                   "kv_bytes_rw_out_of_place": full, "weight_bytes_rw": 0,
                   "pool_bytes": sum(p.numel() for p in s.pools),
                   "note": "every worker of the finer side holds a pool of the coarser side's capacity; the layer "
                           "count is what fits one GPU",
                   "l2_policy": "no flush: every step streams far more than the 126 MB L2"},
        "phases_ms": {"reshape_block_tables": bt_ms, "reshape_kv_inplace": kv_ms},
        "phases_gbs": {"reshape_kv_inplace": kv_gbs},
        "roofline": {"kernel": "kv_reshard_pair", "bound": "hbm", "achieved": kv_gbs, "peak": peak, "unit": "GB/s",
                     "frac": kv_gbs / peak, "peak_kind": f"of {peak_kind}", "traffic": None},
        "gpu_launches": int(launches), "clocks": clocks, "e2e": None,
    }))


def run_compact(args, rank, world, local):
    """Partial swap of the weights in place (TP a -> b = N*a): every TP=a worker moves the N-th of its shards it keeps
    (--keep, default the last) to the front of its buffers.  One step = one amoeba_compact_weights_inplace call over
    all layers.  (Steps after the first move whatever the buffers then hold: the same bytes, the same addresses.)"""
    import torch

    import paper_2509_19729_b200 as A

    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    cfg = wl.CONFIGS[args.config]
    s, st = build_session(args.config, device, layers=args.layers, kv=False, fill=False)
    for item in args.opt:
        name, val = item.split("=")
        s.set_option(getattr(A, "OPT_" + name.upper()) + A.OPT_WEIGHTS_ONLY, int(val))
    N = cfg["b"] // cfg["a"]
    keep = [args.keep if args.keep is not None else N - 1] * cfg["a"]
    nbytes = A.amoeba_compact_bytes(s.plan, keep) * s.L // cfg["model"]["L"]
    stream = torch.cuda.current_stream()
    for _ in range(args.warmup):
        A.amoeba_compact_weights_inplace(s.plan, s._src_w_packed, keep, 0, s.L, s.status)
    torch.cuda.synchronize()
    assert int(s.status.item()) == 0
    barrier(world)
    sampler = ClockSampler(local)
    sampler.start()
    time.sleep(0.3)
    launches0 = A.amoeba_launch_count()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record(stream)
    for _ in range(args.steps):
        A.amoeba_compact_weights_inplace(s.plan, s._src_w_packed, keep, 0, s.L, s.status)
    t1.record(stream)
    torch.cuda.synchronize()
    launches = A.amoeba_launch_count() - launches0
    barrier(world)
    time.sleep(0.2)
    clocks = sampler.stop()
    assert int(s.status.item()) == 0
    sec_all, bytes_all = aggregate(world, t0.elapsed_time(t1) / 1e3 / args.steps, nbytes, device)
    if rank != 0:
        return
    peak, peak_kind = peaks()
    gbs = bytes_all / sec_all / 1e9
    print(json.dumps({
        "metric": METRIC, "value": gbs, "unit": "GB/s", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": sec_all * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "u8",
        "data": "synthetic",
        "config": {"workload": args.config, "tp": f"{cfg['a']}->{cfg['b']} weights compacted in place", "keep": keep,
                   "layers": s.L, "kv_bytes_rw": 0, "weight_bytes_rw": nbytes, "extra_weight_memory_bytes": 0,
                   "launches_per_call": launches / args.steps, "options": args.opt,
                   "l2_policy": "no flush: every step streams far more than the 126 MB L2"},
        "roofline": {"kernel": "w_reshard_pair", "bound": "hbm", "achieved": gbs, "peak": peak, "unit": "GB/s",
                     "frac": gbs / peak, "peak_kind": f"of {peak_kind}", "traffic": None},
        "gpu_launches": int(launches), "clocks": clocks, "e2e": None,
    }))


def run_beside(args, rank, world, local):
    """The copy beside a compute kernel (Sec. 3.1, Improvement 2: the migration runs on a side stream while the SMs it
    does not use keep computing).  The KV and weight calls of --layers layers (default 8) run with their grid capped at
    --max-ctas CTAs on one stream while a dense bf16 GEMM (torch.matmul, a library kernel: the neighbour, not the
    product) runs on another.  Reported: each alone, and each while the other one covers its whole timed region."""
    import torch

    import paper_2509_19729_b200 as A

    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    s, st = build_session(args.config, device, layers=args.layers or 8, fill=False)
    if args.max_ctas:
        s.set_option(A.OPT_MAX_CTAS, args.max_ctas)
    kv_bytes, w_bytes = s.bytes_rw(st["n_live"])
    n = 8192
    x = torch.randn(n, n, device=device, dtype=torch.bfloat16)
    y = torch.randn(n, n, device=device, dtype=torch.bfloat16)
    z = torch.empty(n, n, device=device, dtype=torch.bfloat16)
    copy_stream, gemm_stream = torch.cuda.Stream(), torch.cuda.Stream()
    s.rewrite_block_tables()
    torch.cuda.synchronize()
    ev = lambda: torch.cuda.Event(enable_timing=True)

    def copies(k):
        a, b = ev(), ev()
        with torch.cuda.stream(copy_stream):
            a.record(copy_stream)
            for _ in range(k):
                s.reshard_kv(copy_stream)
                s.reshard_weights(copy_stream)
            b.record(copy_stream)
        return a, b, k

    def gemms(k):
        a, b = ev(), ev()
        with torch.cuda.stream(gemm_stream):
            a.record(gemm_stream)
            for _ in range(k):
                torch.matmul(x, y, out=z)
            b.record(gemm_stream)
        return a, b, k

    gbs = lambda t: (kv_bytes + w_bytes) * t[2] / (t[0].elapsed_time(t[1]) / 1e3) / 1e9
    tfs = lambda t: 2.0 * n ** 3 * t[2] / (t[0].elapsed_time(t[1]) / 1e3) / 1e12
    for _ in range(2):  # warm-up of both
        copies(2), gemms(10)
        torch.cuda.synchronize()
    sampler = ClockSampler(local)
    sampler.start()
    time.sleep(0.3)
    launches0 = A.amoeba_launch_count()
    c_alone = copies(4)
    torch.cuda.synchronize()
    g_alone = gemms(40)
    torch.cuda.synchronize()
    one_copy_ms = c_alone[0].elapsed_time(c_alone[1]) / 4
    one_gemm_ms = g_alone[0].elapsed_time(g_alone[1]) / 40
    # the copy inside a longer batch of GEMMs
    k_g = int(6 * one_copy_ms / one_gemm_ms) + 20
    g_long = gemms(k_g)
    c_in = copies(3)
    torch.cuda.synchronize()
    # the GEMMs inside a longer batch of copies
    k_c = int(30 * one_gemm_ms / one_copy_ms) + 4
    c_long = copies(k_c)
    g_in = gemms(20)
    torch.cuda.synchronize()
    launches = A.amoeba_launch_count() - launches0
    time.sleep(0.2)
    clocks = sampler.stop()
    assert int(s.status.item()) == 0
    if rank != 0:
        return
    peak, peak_kind = peaks()
    cfg = wl.CONFIGS[args.config]
    print(json.dumps({
        "metric": METRIC, "value": gbs(c_in), "unit": "GB/s", "n_gpus": world, "steps": 3, "warmup": 4,
        "ms_per_step": c_in[0].elapsed_time(c_in[1]) / 3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "u8", "data": "synthetic",
        "config": {"workload": args.config, "tp": f"{cfg['a']}->{cfg['b']}", "layers": s.L,
                   "max_ctas": args.max_ctas or "all SMs", "neighbour": f"torch.matmul bf16 {n}^3 on a second stream",
                   "kv_bytes_rw": kv_bytes, "weight_bytes_rw": w_bytes,
                   "l2_policy": "no flush: every step streams far more than the 126 MB L2"},
        "copy_gbs": {"alone": gbs(c_alone), "beside_gemm": gbs(c_in)},
        "gemm_tflops": {"alone": tfs(g_alone), "beside_copy": tfs(g_in)},
        "roofline": {"kernel": "kv_reshard_pair + w_reshard_pair", "bound": "hbm", "achieved": gbs(c_in), "peak": peak,
                     "unit": "GB/s", "frac": gbs(c_in) / peak, "peak_kind": f"of {peak_kind}", "traffic": None},
        "gpu_launches": int(launches), "clocks": clocks, "e2e": None,
    }))


def build_merge_session(cfg_name: str, device, layers=None, seed=wl.DEFAULT_SEED, fill=True):
    import torch

    from paper_2509_19729_b200.session import MergeSession

    cfg = wl.MERGE_CONFIGS[cfg_name]
    m = dict(cfg["model"])
    if layers is not None:
        m["L"] = layers
    st = wl.draw_merge_state(cfg, seed=seed, name=cfg_name)
    s = MergeSession(m, cfg["N"], cfg["a"], st["NB"], cfg["S"], st["maxb"], device=device,
                     weights=bool(cfg.get("weights")))
    s.set_tables(st["seq_lens"], st["src_bt"])
    if fill:
        for i, p in enumerate(s.pools):
            wl.hash_fill_(p, seed, 300 + i)
        for i, p in enumerate(s._wbufs):
            wl.hash_fill_(p[:p.numel() // 8 * 8], seed, 500 + i)
    torch.cuda.synchronize()
    return s, st


def build_merge_copy_session(cfg_name: str, device, layers=None, seed=wl.DEFAULT_SEED, kv_order="head"):
    """The same merge workload done out of place: N source instances, one fresh set of destination pools."""
    import torch

    from paper_2509_19729_b200.session import MergeCopySession

    cfg = wl.MERGE_CONFIGS[cfg_name]
    m = dict(cfg["model"])
    if layers is not None:
        m["L"] = layers
    st = wl.draw_merge_state(cfg, seed=seed, name=cfg_name)
    NB_dst = st["n_live"] + max(st["n_live"] // 64, 1)
    free = wl.rng(seed, "merge_dst_blocks", *cfg_name.encode()).permutation(NB_dst).astype(np.int32)
    s = MergeCopySession(m, cfg["N"], cfg["a"], st["NB"], NB_dst, st["seq_lens"], st["src_bt"], free,
                         st["blocks_per_seq"].sum(axis=1), device=device,
                         src_kv_order=KV_ORDERS[kv_order][0], dst_kv_order=KV_ORDERS[kv_order][1])
    k = 0
    for inst in s.src_pools:
        for p in inst:
            wl.hash_fill_(p, seed, 400 + k)
            k += 1
    for p in s.dst_pools:
        p.fill_(0xA5)
    torch.cuda.synchronize()
    return s, st


def run_merge_copy(args, rank, world, local):
    """Out-of-place variant of the merge workload (what the merge costs without in-place block reshaping)."""
    import torch

    import paper_2509_19729_b200 as A

    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    cfg = wl.MERGE_CONFIGS[args.config]
    s, st = build_merge_copy_session(args.config, device, layers=args.layers, kv_order=args.kv_order)
    nbytes = s.bytes_rw()
    stream = torch.cuda.current_stream()
    for _ in range(args.warmup):
        s.status.zero_()
        s.step()
    torch.cuda.synchronize()
    assert int(s.status.item()) == 0
    barrier(world)
    sampler = ClockSampler(local)
    sampler.start()
    time.sleep(0.3)
    launches0 = A.amoeba_launch_count()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    t0.record(stream)
    for _ in range(args.steps):
        s.step()
    t1.record(stream)
    torch.cuda.synchronize()
    launches = A.amoeba_launch_count() - launches0
    barrier(world)
    time.sleep(0.2)
    clocks = sampler.stop()
    assert int(s.status.item()) == 0
    sec = t0.elapsed_time(t1) / 1e3 / args.steps
    sec_all, bytes_all = aggregate(world, sec, nbytes, device)
    if rank != 0:
        return
    peak, peak_kind = peaks()
    N, a = cfg["N"], cfg["a"]
    gbs = bytes_all / sec_all / 1e9
    print(json.dumps({
        "metric": METRIC, "value": gbs, "unit": "GB/s", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": sec_all * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "u8",
        "data": "synthetic",
        "config": {"workload": args.config, "tp": f"{N}x{a}->{N * a} out of place", "kv_order": args.kv_order,
                   "layers": s.kv_layers, "sequences_per_instance": cfg["S"], "live_blocks": st["n_live"],
                   "kv_bytes_rw": nbytes, "weight_bytes_rw": 0,
                   "source_pool_bytes": sum(p.numel() for inst in s.src_pools for p in inst),
                   "extra_kv_memory_bytes": sum(p.numel() for p in s.dst_pools),
                   "l2_policy": "no flush: every step streams far more than the 126 MB L2"},
        "roofline": {"kernel": "kv_reshard_pair" if args.kv_order == "head" else "kv_reshard_pair_box", "bound": "hbm",
                     "achieved": gbs, "peak": peak, "unit": "GB/s", "frac": gbs / peak, "peak_kind": f"of {peak_kind}",
                     "traffic": None},
        "gpu_launches": int(launches), "clocks": clocks, "e2e": None,
    }))


def run_merge(args, rank, world, local):
    """In-place merge workload: one step = merged block tables + the in-place KV exchange of all layers.  (A second
    step over the same tables exchanges the same segments back: every step moves the same bytes.)"""
    import torch

    import paper_2509_19729_b200 as A

    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    cfg = wl.MERGE_CONFIGS[args.config]
    s, st = build_merge_session(args.config, device, layers=args.layers)
    for opt, val in ((A.OPT_COPY_PATH, args.copy_path), (A.OPT_CHUNK_BYTES, args.chunk), (A.OPT_STAGES, args.stages),
                     (A.OPT_CTAS_PER_SM, args.ctas_per_sm)):
        if val:
            s.set_option(opt, val)
    for item in args.opt:
        name, val = item.split("=")
        s.set_option(getattr(A, "OPT_" + name.upper()), int(val))
    w_bytes = s.weight_bytes_rw()
    nbytes = s.bytes_rw(st["n_live"]) + w_bytes
    stream = torch.cuda.current_stream()
    ev = lambda: torch.cuda.Event(enable_timing=True)
    for _ in range(args.warmup):
        s.status.zero_()
        s.step()
    torch.cuda.synchronize()
    assert int(s.status.item()) == 0, f"device status {int(s.status.item())}"
    barrier(world)
    sampler = ClockSampler(local)
    sampler.start()
    time.sleep(0.3)
    launches0 = A.amoeba_launch_count()
    marks = []
    t_begin, t_end = ev(), ev()
    torch.cuda.synchronize()
    t_begin.record(stream)
    for _ in range(args.steps):
        m3 = [ev() for _ in range(4)]
        m3[3].record(stream)
        if s.inst_w:
            s.compact_weights()
        m3[0].record(stream)
        s.merge_block_tables()
        m3[1].record(stream)
        s.merge_kv()
        m3[2].record(stream)
        marks.append(m3)
    t_end.record(stream)
    torch.cuda.synchronize()
    launches = A.amoeba_launch_count() - launches0
    barrier(world)
    time.sleep(0.2)
    clocks = sampler.stop()
    assert int(s.status.item()) == 0
    sec = t_begin.elapsed_time(t_end) / 1e3 / args.steps
    bt_ms = statistics.mean(m3[0].elapsed_time(m3[1]) for m3 in marks)
    kv_ms = statistics.mean(m3[1].elapsed_time(m3[2]) for m3 in marks)
    w_ms = statistics.mean(m3[3].elapsed_time(m3[0]) for m3 in marks)
    sec_all, bytes_all = aggregate(world, sec, nbytes, device)
    pool_bytes = sum(p.numel() for p in s.pools)
    if rank != 0:
        return
    peak, peak_kind = peaks()
    kv_gbs = (nbytes - w_bytes) / (kv_ms / 1e3) / 1e9
    N, a = cfg["N"], cfg["a"]
    out = {
        "metric": METRIC, "value": bytes_all / sec_all / 1e9, "unit": "GB/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": sec_all * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "u8", "data": "synthetic",
        "config": {"workload": args.config, "tp": f"{N}x{a}->{N * a} in place", "layers": s.kv_layers,
                   "sequences_per_instance": cfg["S"], "live_blocks": st["n_live"], "pool_blocks": st["NB"],
                   "block_tokens": wl.BLOCK_TOKENS, "kv_bytes_rw": nbytes - w_bytes, "weight_bytes_rw": w_bytes,
                   "pool_bytes": pool_bytes, "extra_kv_memory_bytes": 0, "extra_weight_memory_bytes": 0,
                   "l2_policy": "no flush: every step streams far more than the 126 MB L2"},
        "phases_ms": {"compact_weights_inplace": w_ms, "merge_block_tables": bt_ms, "merge_kv_inplace": kv_ms},
        "phases_gbs": {"merge_kv_inplace": kv_gbs},
        "roofline": {"kernel": "kv_merge_pair", "bound": "hbm", "achieved": kv_gbs, "peak": peak, "unit": "GB/s",
                     "frac": kv_gbs / peak, "peak_kind": f"of {peak_kind}", "traffic": None},
        "gpu_launches": int(launches), "clocks": clocks, "e2e": None,
    }
    del s
    torch.cuda.empty_cache()
    if not args.no_cpu_baseline and world == 1:
        run, ob, desc = oracle_merge_sample(args.config, kv_layers=2, n_seqs=10**9)
        t0 = time.perf_counter()
        run()
        dt = time.perf_counter() - t0
        out["cpu_baseline"] = {"value": ob / dt / 1e9, "unit": "GB/s", "cores": 1, "kind": "oracle", "sample": desc,
                               "seconds": dt}
    print(json.dumps(out))


def host_free_bytes() -> int:
    try:
        for line in open("/proc/meminfo"):
            if line.startswith("MemAvailable"):
                return int(line.split()[1]) * 1024
    except OSError:
        pass
    return 0


def run_e2e(args, device, world):
    """The same metric through the public calls with the state in pinned HOST memory.  Every step copies the
    sources host->device, runs the three calls and copies the destinations device->host, layer by layer on three
    streams (upload of layer l+1, kernels of layer l and download of layer l-1 overlap)."""
    import torch

    cfg = wl.CONFIGS[args.config]
    L_full = cfg["model"]["L"]
    # size the layer slice so that the pinned host buffers stay within the cap
    budget = min(int(args.e2e_gib * 2**30), host_free_bytes() // (3 * max(world, 1)))  # every rank pins its own copy
    s1, st = build_session(args.config, device, layers=1, fill=False, kv_order=args.kv_order,
                           weight_pad=args.weight_pad)
    per_layer = sum(p.numel() for p in s1.src_pools + s1.dst_pools + s1._wbufs)
    del s1
    torch.cuda.empty_cache()
    layers = int(max(1, min(L_full, budget // max(per_layer, 1))))
    s, st = build_session(args.config, device, layers=layers, kv_order=args.kv_order, weight_pad=args.weight_pad)
    kvl = s.kv_layers
    a = cfg["a"]

    def by_layer(t, n):  # contiguous per-layer slices of a buffer that holds n layers
        return list(t.view(n, -1).unbind(0))

    src_dev = [by_layer(p, kvl) for p in s.src_pools]          # [rank][layer]
    dst_dev = [by_layer(p, kvl) for p in s.dst_pools]
    srcw_dev = [by_layer(p, layers) for p in s._wbufs[:a]]
    dstw_dev = [by_layer(p, layers) for p in s._wbufs[a:]]
    pin = lambda t: torch.empty(t.numel(), dtype=torch.uint8).pin_memory()
    src_host = [[pin(x) for x in r] for r in src_dev]
    dst_host = [[pin(x) for x in r] for r in dst_dev]
    srcw_host = [[pin(x) for x in r] for r in srcw_dev]
    dstw_host = [[pin(x) for x in r] for r in dstw_dev]
    for hs, ds in ((src_host, src_dev), (srcw_host, srcw_dev)):
        for hr, dr in zip(hs, ds):
            for h, d in zip(hr, dr):
                h.copy_(d)
    torch.cuda.synchronize()
    tabs_host = [torch.from_numpy(st["seq_lens"]).pin_memory(), torch.from_numpy(st["src_bt"]).pin_memory()]
    dst_bt_host = torch.empty(s.dst_bt.shape, dtype=torch.int32).pin_memory()
    status_host = torch.zeros(1, dtype=torch.int32).pin_memory()
    count = lambda hs: sum(h.numel() for r in hs for h in r)
    h2d = count(src_host) + count(srcw_host) + sum(t.numel() * 4 for t in tabs_host)
    d2h = count(dst_host) + count(dstw_host) + dst_bt_host.numel() * 4 + 4
    up, run, down = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()
    ev = lambda: torch.cuda.Event()
    done_run = [None] * layers   # previous step's kernels of layer l (they read the sources of layer l)
    done_down = [None] * layers  # previous step's download of layer l (it reads the destinations of layer l)

    def step():
        with torch.cuda.stream(up):
            s.seq_lens.copy_(tabs_host[0], non_blocking=True)
            s.src_bt.copy_(tabs_host[1], non_blocking=True)
            tabs_up = ev()
            tabs_up.record(up)
        with torch.cuda.stream(run):
            run.wait_event(tabs_up)
            s.status.zero_()
            s.rewrite_block_tables(run)
        for l in range(layers):
            with torch.cuda.stream(up):
                if done_run[l] is not None:
                    up.wait_event(done_run[l])
                for hs, ds in ((src_host, src_dev), (srcw_host, srcw_dev)):
                    for hr, dr in zip(hs, ds):
                        if l < len(dr):
                            dr[l].copy_(hr[l], non_blocking=True)
                uploaded = ev()
                uploaded.record(up)
            with torch.cuda.stream(run):
                run.wait_event(uploaded)
                if done_down[l] is not None:
                    run.wait_event(done_down[l])
                if l < kvl:
                    s.reshard_kv(run, l, l + 1)
                s.reshard_weights(run, l, l + 1)
                done_run[l] = ev()
                done_run[l].record(run)
            with torch.cuda.stream(down):
                down.wait_event(done_run[l])
                for hs, ds in ((dst_host, dst_dev), (dstw_host, dstw_dev)):
                    for hr, dr in zip(hs, ds):
                        if l < len(dr):
                            hr[l].copy_(dr[l], non_blocking=True)
                if l == layers - 1:
                    dst_bt_host.copy_(s.dst_bt, non_blocking=True)
                    status_host.copy_(s.status, non_blocking=True)
                done_down[l] = ev()
                done_down[l].record(down)

    for _ in range(2):
        step()
    torch.cuda.synchronize()
    barrier(world)
    k = max(2, min(args.steps, 5))
    t0 = time.perf_counter()
    for _ in range(k):
        step()
    torch.cuda.synchronize()  # the step's result (tables, status, destinations) is on the host
    sec = (time.perf_counter() - t0) / k
    assert int(status_host.item()) == 0
    kvb, wb = s.bytes_rw(st["n_live"])
    sec, tot = aggregate(world, sec, kvb + wb, device)
    return {"value": tot / sec / 1e9, "unit": "GB/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
            "ms_per_step": sec * 1e3,
            "sample": f"first {layers} of {L_full} layers (all sequences) held in pinned host memory; per layer: "
                      f"upload, the three calls, download, overlapped on three streams; wall clock around "
                      f"{k} steps with a device synchronize"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default=DEFAULT_CONFIG, choices=list(wl.CONFIGS) + list(wl.MERGE_CONFIGS))
    ap.add_argument("--copy-path", type=int, default=0, help="0 default, 1 vector ld/st, 2 bulk-copy ring per warp, 3 producer/consumer bulk-copy ring")
    ap.add_argument("--chunk", type=int, default=0)
    ap.add_argument("--stages", type=int, default=0)
    ap.add_argument("--ctas-per-sm", type=int, default=0)
    ap.add_argument("--kv-order", default="head", choices=list(KV_ORDERS),
                    help="KV storage order: header-centric on both sides (default), token-first on both sides, or a "
                         "conversion between them")
    ap.add_argument("--weight-pad", type=int, default=0,
                    help="P > 0: both sides hold their weights as P padded partitions per tensor (2 MiB pages)")
    ap.add_argument("--merge-mode", default="inplace", choices=["inplace", "outofplace"],
                    help="merge workloads: exchange segments in place (default) or copy every instance into fresh pools")
    ap.add_argument("--opt", action="append", default=[], metavar="NAME=VALUE",
                    help="any plan option by name (e.g. WARPS=6, LAG=3, L2_HINT=1, TENSOR_MAPS=1), repeatable")
    ap.add_argument("--max-ctas", type=int, default=0, help="cap on the copy kernels' persistent grid (0 = all SMs)")
    ap.add_argument("--layers-per-call", type=int, default=0,
                    help="k > 0: transform k layers per call (KV and weights), as when a few layers are transformed "
                         "per inference step; 0 = all layers in one call")
    ap.add_argument("--layers", type=int, default=None, help="use only the first LAYERS layers (profiling)")
    ap.add_argument("--inplace", action="store_true",
                    help="reshape the one instance in place (block reshaping) instead of copying it into fresh pools; "
                         "KV cache only, TP degrees must be multiples")
    ap.add_argument("--beside-gemm", action="store_true",
                    help="run the copy (grid capped by --max-ctas) while a dense GEMM runs on a second stream and "
                         "report both throughputs, alone and together")
    ap.add_argument("--compact-weights", action="store_true",
                    help="time the in-place partial swap of the weights (amoeba_compact_weights_inplace) instead of the "
                         "transformation; TP degrees must be multiples")
    ap.add_argument("--keep", type=int, default=None, help="--compact-weights: which N-th every worker keeps")
    ap.add_argument("--no-all-configs", action="store_true",
                    help="skip the short timing of the other benchmark configurations")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--e2e-gib", type=float, default=48.0, help="cap on pinned host memory for the e2e leg")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" and args.layers is None else args.warmup

    rank, world, local = dist_setup(args.gpus if args.impl == "ours" else 0)
    if args.impl == "reference":
        run_reference(args, rank, world)
        return

    if args.config in wl.MERGE_CONFIGS:
        (run_merge if args.merge_mode == "inplace" else run_merge_copy)(args, rank, world, local)
        return

    if args.inplace:
        run_reshape(args, rank, world, local)
        return
    if args.compact_weights:
        run_compact(args, rank, world, local)
        return
    if args.beside_gemm:
        run_beside(args, rank, world, local)
        return

    import torch

    import paper_2509_19729_b200 as A

    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    cfg = wl.CONFIGS[args.config]
    s, st = build_session(args.config, device, layers=args.layers, kv_order=args.kv_order,
                          weight_pad=args.weight_pad)
    for opt, val in ((A.OPT_COPY_PATH, args.copy_path), (A.OPT_CHUNK_BYTES, args.chunk), (A.OPT_STAGES, args.stages),
                     (A.OPT_CTAS_PER_SM, args.ctas_per_sm), (A.OPT_MAX_CTAS, args.max_ctas)):
        if val:
            s.set_option(opt, val)
    for item in args.opt:
        name, val = item.split("=")
        s.set_option(getattr(A, "OPT_" + name.upper()), int(val))
    kv_bytes, w_bytes = s.bytes_rw(st["n_live"])
    stream = torch.cuda.current_stream()

    def ev():
        return torch.cuda.Event(enable_timing=True)

    for _ in range(args.warmup):
        s.status.zero_()
        s.step()
    torch.cuda.synchronize()
    assert int(s.status.item()) == 0, f"device status {int(s.status.item())}"
    barrier(world)
    def timed_region():
        sampler = ClockSampler(local)
        sampler.start()
        time.sleep(0.3)
        marks = []
        launches0 = A.amoeba_launch_count()
        t_begin, t_end = ev(), ev()
        torch.cuda.synchronize()
        t_begin.record(stream)
        k = args.layers_per_call
        kv_ranges = [(l, min(l + k, s.kv_layers)) for l in range(0, s.kv_layers, k)] if k else [(0, s.kv_layers)]
        w_ranges = [(l, min(l + k, s.L)) for l in range(0, s.L, k)] if k else [(0, s.L)]
        for _ in range(args.steps):
            m = [ev() for _ in range(4)]
            m[0].record(stream)
            s.rewrite_block_tables()
            m[1].record(stream)
            for lo, hi in kv_ranges:
                s.reshard_kv(None, lo, hi)
            m[2].record(stream)
            for lo, hi in w_ranges:
                s.reshard_weights(None, lo, hi)
            m[3].record(stream)
            marks.append(m)
        t_end.record(stream)
        torch.cuda.synchronize()
        launches = A.amoeba_launch_count() - launches0
        barrier(world)
        time.sleep(0.2)
        clocks = sampler.stop()
        assert int(s.status.item()) == 0, f"device status {int(s.status.item())}"
        return marks, launches, clocks, t_begin.elapsed_time(t_end) / 1e3 / args.steps

    marks, launches, clocks, sec = timed_region()
    remeasured = False
    if any_rank(world, device, bool(set(clocks["reasons"]) & THROTTLE_REASONS)):
        # a slowdown was active while timing: the number does not count; measure once more
        marks, launches, clocks, sec = timed_region()
        remeasured = True
    phase = [[m[i].elapsed_time(m[i + 1]) for m in marks] for i in range(3)]
    bt_ms, kv_ms, w_ms = (statistics.mean(p) for p in phase)
    sec_all, bytes_all = aggregate(world, sec, kv_bytes + w_bytes, device)
    n_seq_layers = (s.L, s.kv_layers, int(s.info.chunk_bytes))
    del s
    torch.cuda.empty_cache()
    default_run = (args.config == DEFAULT_CONFIG and args.kv_order == "head" and args.layers is None
                   and not (args.copy_path or args.chunk or args.stages or args.ctas_per_sm or args.max_ctas or args.opt
                            or args.weight_pad or args.layers_per_call))
    all_configs = None
    if default_run and world == 1 and not args.no_all_configs:
        # the other benchmark configurations, a few steps each, same kernels and options
        all_configs = {name: measure_config(name, device) for name in wl.CONFIGS
                       if name not in (args.config, "tiny_2to1")}
    e2e = None if args.no_e2e else run_e2e(args, device, world)
    if rank != 0:
        return

    peak, peak_kind = peaks()
    traffic_known = (NCU_KV_TRAFFIC_RATIO is not None and args.config == NCU_KV_TRAFFIC_CONFIG
                     and args.kv_order == "head"
                     and not (args.copy_path or args.chunk or args.stages or args.ctas_per_sm or args.max_ctas or args.opt))
    kv_gbs = kv_bytes / (kv_ms / 1e3) / 1e9
    w_gbs = w_bytes / (w_ms / 1e3) / 1e9 if w_bytes else None
    out = {
        "metric": METRIC, "value": bytes_all / sec_all / 1e9, "unit": "GB/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": sec_all * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "u8", "data": "synthetic",
        "config": {"workload": args.config, "tp": f"{cfg['a']}->{cfg['b']}", "layers": n_seq_layers[0], "kv_layers": n_seq_layers[1],
                   "layers_per_call": args.layers_per_call or "all", "kv_order": args.kv_order, "weight_pad_parts": args.weight_pad, "sequences": cfg["S"], "live_blocks": st["n_live"], "block_tokens": wl.BLOCK_TOKENS,
                   "kv_bytes_rw": kv_bytes, "weight_bytes_rw": w_bytes,
                   "l2_policy": "no flush: every step streams far more than the 126 MB L2",
                   "max_ctas": args.max_ctas or "all SMs", "options": args.opt, "copy_path": {0: "pair (default)", 1: "ldst", 2: "bulk", 3: "pair"}[args.copy_path],
                   "chunk_bytes": n_seq_layers[2]},
        "phases_ms": {"rewrite_block_tables": bt_ms, "reshard_kv": kv_ms, "reshard_weights": w_ms,
                      "reshard_kv_min": min(phase[1]), "reshard_weights_min": min(phase[2]),
                      "reshard_kv_median": statistics.median(phase[1]),
                      "reshard_weights_median": statistics.median(phase[2])},
        "phases_gbs": {"reshard_kv": kv_gbs, "reshard_weights": w_gbs},
        "pct_of_nominal_8TBs": {"reshard_kv": 100 * kv_gbs / NOMINAL_HBM_GBS,
                                "reshard_weights": 100 * w_gbs / NOMINAL_HBM_GBS if w_gbs else None},
        "roofline": {"kernel": "kv_reshard_pair" if not args.copy_path else "kv_reshard", "bound": "hbm", "achieved": kv_gbs, "peak": peak, "unit": "GB/s",
                     "frac": kv_gbs / peak, "peak_kind": f"of {peak_kind}",
                     "traffic": NCU_KV_TRAFFIC_RATIO * kv_bytes if traffic_known else None,
                     "traffic_source": NCU_KV_TRAFFIC_SOURCE if traffic_known else None},
        "roofline_weights": None if not w_gbs else {"kernel": "w_reshard_pair" if not args.copy_path else "w_reshard", "bound": "hbm", "achieved": w_gbs,
                                                    "peak": peak, "unit": "GB/s", "frac": w_gbs / peak},
        "gpu_launches": int(launches), "clocks": clocks, "remeasured_after_slowdown": remeasured,
    }
    if all_configs is not None:
        all_configs[args.config] = {"tp": f"{cfg['a']}->{cfg['b']}", "kv_layers": n_seq_layers[1], "layers": n_seq_layers[0],
                                    "live_blocks": st["n_live"], "tables_us": bt_ms * 1e3, "kv_ms": kv_ms,
                                    "kv_gbs": kv_gbs, "kv_frac": kv_gbs / peak, "w_ms": w_ms, "w_gbs": w_gbs,
                                    "w_frac": w_gbs / peak, "steps": args.steps}
        out["all_configs"] = all_configs
    if e2e is not None:
        out["e2e"] = e2e
    if not args.no_cpu_baseline and world == 1:
        out["cpu_baseline"] = cpu_baseline(args.config)
    print(json.dumps(out))


if __name__ == "__main__":
    main()

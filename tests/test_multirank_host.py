"""Host logic of the N>1 benchmark path on CPU (gloo, world size 2): whole-job time is the max over ranks, bytes the
sum; the reference arm prints on rank 0 only.  No GPU, no data-path collective (the path runs as replicas)."""
import json
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


WORKER = r"""
import os, sys, json
sys.path.insert(0, sys.argv[1])
import torch.distributed as dist
import bench
rank, world, local = bench.dist_setup(0)          # 0 GPUs -> gloo
assert world == 2 and dist.get_backend() == "gloo"
bench.barrier(world)
sec, tot = bench.aggregate(world, 1.0 + rank, 100.0 * (rank + 1))
print(json.dumps({"rank": rank, "sec": sec, "bytes": tot}))
dist.destroy_process_group()
"""


def _launch(code_or_args, port, extra_env=None):
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port), OMP_NUM_THREADS="1", **(extra_env or {}))
        procs.append(subprocess.Popen([sys.executable, *code_or_args], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True, cwd=ROOT))
    outs = []
    for p in procs:
        out, err = p.communicate(timeout=300)
        assert p.returncode == 0, err[-2000:]
        outs.append(out)
    return outs


def test_aggregate_is_max_time_and_sum_bytes_over_ranks():
    outs = _launch(["-c", WORKER, ROOT], _free_port())
    rows = [json.loads(o.strip().splitlines()[-1]) for o in outs]
    for r in rows:
        assert r["sec"] == 2.0 and r["bytes"] == 300.0  # max(1, 2), 100 + 200


def test_reference_arm_prints_on_rank0_only():
    outs = _launch(["bench.py", "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0", "--config",
                    "tiny_2to1"], _free_port())
    line = json.loads(outs[0].strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0
    assert outs[1].strip() == ""

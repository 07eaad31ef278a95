"""The N > 1 path of bench.py on CPU: two gloo ranks (replicas only: no data-path collective exists).

What is multi-rank in the benchmark is the timing rule (max over ranks, whole-job tokens/s) and the reference arm's
"rank 0 works, the others exit 0"; both run here as real processes under torch.distributed with the gloo backend.
"""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys, json
sys.path.insert(0, {root!r})
import torch.distributed as dist
import bench
rank = int(os.environ["RANK"]); world = int(os.environ["WORLD_SIZE"])
dist.init_process_group("gloo")
# rank r pretends its K steps took (100 + 50 r) ms on the device, its end-to-end pass (120 + 10 r) ms
ms = bench.max_over_ranks([100.0 + 50.0 * rank, 120.0 + 10.0 * rank], world)
val = bench.job_tokens_per_s(8192, world, ms[0], steps=10)
dist.barrier()
if rank == 0:
    print(json.dumps(dict(ms=ms, value=val)))
dist.destroy_process_group()
"""


def _torchrun(args, env_extra=None, timeout=300):
    env = dict(os.environ)
    env.update(env_extra or {})
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr",
           "127.0.0.1", "--master-port", "29731"] + args
    return subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=timeout)


def test_two_ranks_take_the_maximum_time_and_sum_the_tokens(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER.format(root=ROOT))
    r = _torchrun([str(script)])
    assert r.returncode == 0, r.stderr[-2000:]
    line = [l for l in r.stdout.splitlines() if l.startswith("{")][-1]
    out = json.loads(line)
    assert out["ms"] == [150.0, 130.0]  # the slower rank defines both times
    assert abs(out["value"] - 2 * 8192 / (0.150 / 10)) < 1e-6  # whole job: both replicas' tokens over that time


def test_reference_arm_under_two_ranks_prints_one_line_from_rank_zero():
    r = _torchrun(["bench.py", "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0", "--workload",
                   "c1_tiny"], timeout=600)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["n_gpus"] == 2 and d["value"] > 0
    assert d["cpu_baseline"]["kind"] == "oracle" and d["e2e"]["h2d_bytes_per_step"] == 0


def test_gpus_flag_without_a_launcher_starts_the_ranks_itself():
    """`python bench.py --gpus 2` with no WORLD_SIZE in the environment re-launches itself under torch.distributed.run
    (checked with the reference arm, which needs no GPU): one JSON line from rank 0, n_gpus 2."""
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    r = subprocess.run([sys.executable, "bench.py", "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0",
                        "--workload", "c1_tiny"], cwd=ROOT, env=env, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["n_gpus"] == 2

"""The N>1 path of the benchmark is "replicas only": ranks share nothing but the timing reduction.
These CPU tests run two gloo ranks and check the max-over-ranks reduction, the whole-job value and
the reference arm's rank handling."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys, json
sys.path.insert(0, %r)
import torch, torch.distributed as dist
import bench
dist.init_process_group("gloo")
rank = dist.get_rank()
vals = bench.max_over_ranks([10.0 + rank, 5.0 - rank], dist, torch.device("cpu"))
if rank == 0:
    print(json.dumps({"vals": vals, "value": bench.whole_job_value(2e9, dist.get_world_size(), vals[0])}))
dist.destroy_process_group()
"""


def _torchrun(args, timeout=300):
    env = dict(os.environ, MASTER_ADDR="127.0.0.1")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
           "--master-addr", "127.0.0.1", "--master-port", "29533"] + args
    return subprocess.run(cmd, capture_output=True, text=True, timeout=timeout, env=env, cwd=ROOT)


def test_max_over_ranks_with_two_gloo_ranks(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER % ROOT)
    res = _torchrun([str(script)])
    assert res.returncode == 0, res.stderr[-2000:]
    line = [ln for ln in res.stdout.splitlines() if ln.startswith("{")][-1]
    out = json.loads(line)
    assert out["vals"] == [11.0, 5.0]                  # slowest rank per entry
    assert abs(out["value"] - 2 * 2e9 / 11e-3 / 1e9) < 1e-6


def test_reference_arm_prints_one_line_on_rank_zero_only():
    res = _torchrun([os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                     "--warmup", "1"])
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [ln for ln in res.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    out = json.loads(lines[0])
    assert out["impl"] == "reference" and out["n_gpus"] == 2 and out["cpu_baseline"]["kind"] == "oracle"
    assert out["e2e"]["h2d_bytes_per_step"] == 0 and out["value"] > 0

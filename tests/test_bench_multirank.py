"""Multi-rank plumbing of bench.py on CPU (gloo, world size 2): max over ranks, whole-job value,
and the rule that only rank 0 runs and prints the reference arm."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _torchrun(args, port):
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.join(ROOT, "bench.py")] + args
    env = dict(os.environ, CUDA_VISIBLE_DEVICES="", OMP_NUM_THREADS="1")
    res = subprocess.run(cmd, capture_output=True, text=True, timeout=600, cwd=ROOT, env=env)
    assert res.returncode == 0, res.stderr[-2000:]
    return [json.loads(l) for l in res.stdout.splitlines() if l.startswith("{")]


def test_two_ranks_time_is_max_and_value_is_whole_job():
    lines = _torchrun(["--selftest-dist", "--gpus", "2", "--steps", "4"], 29731)
    assert len(lines) == 1
    out = lines[0]
    assert out["n_gpus"] == 2 and out["max_ms"] == 15.0
    assert abs(out["value"] - 2 * 1000.0 * 4 / 15e-3) < 1e-6 * out["value"]


def test_reference_arm_runs_on_rank_zero_only():
    lines = _torchrun(["--impl", "reference", "--gpus", "2", "--workload", "c1", "--steps", "1", "--warmup", "0"], 29733)
    assert len(lines) == 1
    out = lines[0]
    assert out["impl"] == "reference" and out["value"] > 0 and out["cpu_baseline"]["kind"] == "oracle"
    assert out["e2e"]["h2d_bytes_per_step"] == 0

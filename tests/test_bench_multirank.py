"""bench.py with more than one rank, on CPU: replicas only, so the cross-rank logic is the max-over-ranks time, the
aggregate value, and the rule that only rank 0 of the reference arm works and prints."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _torchrun(args, port, timeout=600):
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr", "127.0.0.1",
           "--master-port", str(port)] + args
    return subprocess.run(cmd, cwd=ROOT, capture_output=True, text=True, timeout=timeout)


def test_max_over_ranks_and_aggregate_with_two_gloo_ranks():
    r = _torchrun([os.path.join("tests", "gloo_worker.py")], 29611)
    assert r.returncode == 0, r.stderr[-2000:]
    assert "GLOO_OK world=2 slowest=15.0" in r.stdout


def test_reference_arm_under_two_ranks_prints_one_line():
    r = _torchrun(["bench.py", "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0"], 29612)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [json.loads(l) for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    line = lines[0]
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["gpu_launches"] == 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["value"] > 0
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["e2e"]["d2h_bytes_per_step"] == 0

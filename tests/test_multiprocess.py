"""The N > 1 path is replicas only: no data-path collective, just a barrier and a max over ranks.
Run here as two gloo processes on CPU."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _torchrun(script_args, port):
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr",
           "127.0.0.1", "--master-port", str(port)] + script_args
    return subprocess.run(cmd, cwd=ROOT, capture_output=True, text=True, timeout=600)


def test_barrier_and_max_over_ranks_with_gloo():
    r = _torchrun([os.path.join("tests", "dist_worker.py")], 29611)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1  # rank 0 alone prints
    out = json.loads(lines[0])
    assert out["world"] == 2 and out["slowest_ms"] == 15.0
    # whole-job value = all ranks' bytes over the slowest rank's time: 2 ranks x 1 GB x 4 steps / 15 ms
    assert abs(out["value"] - 2 * 1e9 * 4 / 15.0 / 1e6) < 1e-6


def test_reference_arm_under_torchrun_prints_once_from_rank_zero():
    r = _torchrun(["bench.py", "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0", "--cfg", "0"], 29612)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    out = json.loads(lines[0])
    assert out["impl"] == "reference" and out["n_gpus"] == 2 and out["cpu_baseline"]["kind"] == "oracle"
    assert out["e2e"]["h2d_bytes_per_step"] == 0 and out["value"] > 0

"""The N > 1 path of bench.py on CPU: two gloo ranks, independent replicas, times reduced with MAX,
one JSON line from rank 0.  The path has no exchange step, so this host logic is all there is."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _torchrun(args, port):
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
           "--master-addr", "127.0.0.1", "--master-port", str(port)] + args
    return subprocess.run(cmd, capture_output=True, text=True, cwd=ROOT, timeout=600)


def test_times_are_the_slowest_ranks_and_throughput_is_the_whole_job():
    res = _torchrun([os.path.join(ROOT, "tests", "_dist_worker.py")], 29541)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [l for l in res.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    out = json.loads(lines[0])
    assert out["world"] == 2
    assert out["reduced"] == [11.0, 107.0, 119.0]
    assert abs(out["value"] - 2 * 16 * 128 / 0.107) < 1e-6


def test_reference_arm_under_two_ranks_prints_once():
    res = _torchrun([os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                     "--warmup", "0", "--batch", "1", "--config", "c3"], 29542)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [l for l in res.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    out = json.loads(lines[0])
    assert out["impl"] == "reference" and out["n_gpus"] == 2 and out["cpu_baseline"]["kind"] == "oracle"
    assert out["e2e"]["h2d_bytes_per_step"] == 0 and out["value"] > 0
    assert "32 layers" in out["config"]["workload"] and "32 x the layer time" in out["cpu_baseline"]["sample"]

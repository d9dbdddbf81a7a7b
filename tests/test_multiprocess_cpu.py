"""The N > 1 launch path on CPU (gloo, world size 2): replicas take the maximum time over
ranks, and the reference arm runs on rank 0 only."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _torchrun(args, nproc=2, port=29611):
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={nproc}",
           "--master-addr", "127.0.0.1", "--master-port", str(port)] + args
    return subprocess.run(cmd, cwd=ROOT, capture_output=True, text=True, timeout=600)


def test_max_over_ranks_with_gloo():
    script = ("import os, sys; sys.path.insert(0, %r); import bench, torch.distributed as dist; "
              "dist.init_process_group('gloo'); r = dist.get_rank(); "
              "v = bench.max_over_ranks(10.0 + 5 * r, 2, device='cpu'); "
              "print('RANK', r, v); dist.destroy_process_group()") % ROOT
    res = _torchrun(["--no-python", sys.executable, "-c", script], port=29612)
    assert res.returncode == 0, res.stderr[-2000:]
    assert res.stdout.count("15.0") == 2, res.stdout


def test_reference_arm_prints_once_under_torchrun():
    res = _torchrun([os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--workload", "tiny",
                     "--steps", "3", "--warmup", "1"], port=29613)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [l for l in res.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    rec = json.loads(lines[0])
    assert rec["impl"] == "reference" and rec["n_gpus"] == 2 and rec["cpu_baseline"]["kind"] == "oracle"
    assert rec["e2e"]["h2d_bytes_per_step"] == 0 and rec["value"] > 0

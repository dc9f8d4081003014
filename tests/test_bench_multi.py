"""The benchmark's N > 1 logic (replicas only: barrier, max-over-ranks time, whole-job value) on CPU with gloo."""
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import os, sys, json
    sys.path.insert(0, %r)
    import torch, torch.distributed as dist
    import bench
    dist.init_process_group("gloo")
    rank, world = dist.get_rank(), dist.get_world_size()
    ms, e2e = bench.max_over_ranks([10.0 + 5 * rank, 20.0 - rank], "cpu", world)
    dist.barrier()
    if rank == 0:
        print(json.dumps({"ms": ms, "e2e": e2e, "value": bench.job_value(1000, world, ms)}))
    dist.destroy_process_group()
""")


def test_replicas_max_over_ranks_and_value(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER % ROOT)
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2", "--master-addr", "127.0.0.1",
           "--master-port", "29531", str(script)]
    out = subprocess.run(cmd, capture_output=True, text=True, timeout=240, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    import json
    line = [l for l in out.stdout.splitlines() if l.startswith("{")][-1]
    d = json.loads(line)
    assert d["ms"] == 15.0 and d["e2e"] == 20.0          # the slowest rank decides
    assert abs(d["value"] - 2 * 1000 / 15e-3) < 1e-6      # both replicas' tokens over that time


def test_single_rank_passthrough():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([1.5, 2.5], "cpu", 1) == [1.5, 2.5]
    assert bench.job_value(100, 1, 10.0) == 100 / 10e-3

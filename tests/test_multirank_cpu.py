"""The N > 1 path of bench.py on CPU: two gloo ranks (replicas), slowest rank's time,
whole-job throughput, only rank 0 reports."""
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import os, sys, json
    sys.path.insert(0, %r)
    import torch.distributed as dist
    import bench
    dist.init_process_group("gloo")
    rank, world = dist.get_rank(), dist.get_world_size()
    ms = [10.0, 12.5][rank]                       # rank 1 is the slower replica
    slow = bench.max_over_ranks(ms, "cpu")
    value = bench.whole_job_value(100, slow, world)
    dist.barrier()
    if rank == 0:
        print(json.dumps({"slow": slow, "value": value, "world": world}))
    dist.destroy_process_group()
""") % ROOT


def test_two_replicas_report_the_slowest_rank(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT="29531", OMP_NUM_THREADS="1")
    out = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
                          "--master-addr", "127.0.0.1", "--master-port", "29531", str(script)],
                         env=env, capture_output=True, text=True, timeout=300)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1                         # rank 0 alone prints
    import json
    d = json.loads(lines[0])
    assert d["world"] == 2 and d["slow"] == 12.5
    assert abs(d["value"] - 2 * 100 / 12.5e-3) < 1e-6


def test_single_process_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.25) == 3.25
    assert bench.whole_job_value(128, 2.0, 1) == 64000.0

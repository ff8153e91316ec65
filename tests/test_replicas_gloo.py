"""The N > 1 host logic of bench.py (replicas only: the path has no exchange step) on CPU:
two gloo ranks take the max of their step times and the whole-job value is N x tokens / that."""
import os
import socket
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = textwrap.dedent("""
    import os, sys, json
    sys.path.insert(0, %r)
    import torch, torch.distributed as dist
    import bench
    dist.init_process_group("gloo")
    rank, world = dist.get_rank(), dist.get_world_size()
    t_local = 0.010 * (rank + 1)           # rank 1 is the slow one
    t = bench.max_over_ranks(t_local, dist, device="cpu")
    value = bench.whole_job_value(world, 32, t)
    shard = bench.replica_tag(rank, world)
    if rank == 0:
        print(json.dumps({"t": t, "value": value, "shard": shard}))
    dist.destroy_process_group()
""") % ROOT


def test_two_gloo_ranks_take_the_max_time_and_sum_the_tokens(tmp_path):
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    script = tmp_path / "child.py"
    script.write_text(CHILD)
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr", "127.0.0.1",
           "--master-port", str(port), str(script)]
    out = subprocess.run(cmd, capture_output=True, text=True, timeout=240, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    import json

    line = [l for l in out.stdout.splitlines() if l.startswith("{")][-1]
    d = json.loads(line)
    assert abs(d["t"] - 0.020) < 1e-9
    assert abs(d["value"] - 2 * 32 / 0.020) < 1e-6
    assert d["shard"] == "replica 0 of 2"

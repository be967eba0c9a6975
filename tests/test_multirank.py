"""The N > 1 path of the benchmark is replicas only (one independent sequence per rank, no data-path
collective); what ranks share is the barrier and the max-over-ranks timing.  Checked with 2 gloo ranks on CPU."""
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
    # per-rank timings: rank r reports (10 + r) ms of generation per step
    t = bench.reduce_max_over_ranks([10.0 + rank, 20.0 + rank, 30.0 - rank], device="cpu")
    value = bench.aggregate_tokens_per_s(world, 256, t[0])
    if rank == 0:
        print(json.dumps({"t": t, "value": value, "world": world}))
    dist.barrier()
""")


def test_two_gloo_ranks_take_the_max_time_and_sum_the_tokens(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER % ROOT)
    out = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
                          "--master-addr", "127.0.0.1", "--master-port", "29533", str(script)],
                         capture_output=True, text=True, timeout=240)
    assert out.returncode == 0, out.stderr[-2000:]
    import json
    line = [l for l in out.stdout.splitlines() if l.startswith("{")][-1]
    d = json.loads(line)
    assert d["world"] == 2 and d["t"] == [11.0, 21.0, 30.0]
    assert abs(d["value"] - 2 * 256 / 0.011) < 1e-6

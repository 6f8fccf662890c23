"""N > 1 plumbing of bench.py on CPU: two gloo ranks, barrier and max-over-ranks timing, whole-job
throughput from per-rank work.  The path itself has no exchange step (replicas only), so this is all
the multi-rank logic there is."""
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
    bench._dist = dist
    bench.barrier(world)
    # rank r "measured" (r + 1) * 10 ms: the job's time is the slowest rank's
    ms = bench.max_over_ranks(10.0 * (rank + 1), world, torch.device("cpu"))
    tokens = 32 * 4 * world                      # every rank decodes its own 32 sequences for 4 steps
    if rank == 0:
        print(json.dumps({"ms": ms, "value": tokens / (ms * 1e-3), "world": world}))
    dist.destroy_process_group()
""") % ROOT


def test_two_gloo_ranks_max_time_and_aggregate(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT="29611")
    out = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
                          "--master-addr", "127.0.0.1", "--master-port", "29611", str(script)],
                         capture_output=True, text=True, env=env, timeout=240)
    assert out.returncode == 0, out.stderr[-2000:]
    import json
    line = [l for l in out.stdout.splitlines() if l.startswith("{")][-1]
    res = json.loads(line)
    assert res["world"] == 2 and res["ms"] == 20.0
    assert abs(res["value"] - 32 * 4 * 2 / 0.020) < 1e-6


def test_single_rank_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5, 1, None) == 3.5
    bench.barrier(1)

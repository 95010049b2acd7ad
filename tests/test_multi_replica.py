"""The N > 1 path of the benchmark: independent replicas, whole-job throughput = all ranks' units
divided by the slowest rank's time.  Two gloo ranks on CPU (the data path has no collective)."""
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_two_ranks_aggregate_with_max_over_ranks(tmp_path):
    script = tmp_path / "ranks.py"
    script.write_text(textwrap.dedent(f"""
        import json, os, sys
        sys.path.insert(0, {ROOT!r})
        import torch.distributed as dist
        import bench
        dist.init_process_group("gloo")
        rank, world = dist.get_rank(), dist.get_world_size()
        # rank 0 took 10 ms and 40 ms, rank 1 took 30 ms and 20 ms, each for 1000 units
        mine = [10.0, 40.0] if rank == 0 else [30.0, 20.0]
        times, values = bench.aggregate_replicas(mine, 1000, world, dist)
        dist.barrier()
        if rank == 0:
            print(json.dumps(dict(times=times, values=values)))
        dist.destroy_process_group()
    """))
    env = dict(os.environ, MASTER_ADDR="127.0.0.1")
    out = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
                          "--master-addr", "127.0.0.1", "--master-port", "29731", str(script)],
                         capture_output=True, text=True, env=env, timeout=300)
    assert out.returncode == 0, out.stderr[-2000:]
    import json
    line = [l for l in out.stdout.splitlines() if l.startswith("{")][-1]
    r = json.loads(line)
    assert r["times"] == [30.0, 40.0]
    assert abs(r["values"][0] - 2000 / 0.030) < 1e-6 and abs(r["values"][1] - 2000 / 0.040) < 1e-6


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    times, values = bench.aggregate_replicas([5.0], 100, 1)
    assert times == [5.0] and values == [100 / 0.005]

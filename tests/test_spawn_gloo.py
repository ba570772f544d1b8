"""The launcher-less start of a multi-GPU run, on CPU: `bench.py --gpus N` without a launcher's
environment starts its own ranks through sharding.spawn_ranks.  Two gloo ranks stand in for two GPUs."""
import os
import sys
import textwrap

from paper_2507_17307_b200 import sharding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = textwrap.dedent("""
    import os, sys
    import torch
    import torch.distributed as dist
    sys.path.insert(0, %r)
    from paper_2507_17307_b200 import sharding
    rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
    assert os.environ["MASTER_ADDR"] == "127.0.0.1" and int(os.environ["LOCAL_RANK"]) == rank
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms, units, launches = sharding.reduce_step_stats(10.0 + rank, 4.0 + rank, 2, dist)
    if rank == 0:
        open(sys.argv[1], "w").write("%%d %%.1f %%.1f %%d" %% (world, ms, units, launches))
    dist.barrier()
    dist.destroy_process_group()
    sys.exit(int(sys.argv[2]) if rank == int(sys.argv[3]) else 0)
""") % ROOT


def test_spawn_two_ranks_rendezvous_and_reduce(tmp_path):
    out = tmp_path / "line.txt"
    script = tmp_path / "child.py"
    script.write_text(CHILD)
    rc = sharding.spawn_ranks(2, [sys.executable, str(script), str(out), "0", "0"], timeout=120)
    assert rc == 0
    assert out.read_text() == "2 11.0 9.0 4"       # slowest rank's time, totals over both ranks


def test_spawn_reports_a_failing_rank(tmp_path):
    script = tmp_path / "child.py"
    script.write_text(CHILD)
    rc = sharding.spawn_ranks(2, [sys.executable, str(script), str(tmp_path / "x.txt"), "7", "1"], timeout=120)
    assert rc == 7


def test_bench_spawns_only_without_a_launcher():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.needs_spawn(2, {}) is True
    assert bench.needs_spawn(8, {"PATH": "/bin"}) is True
    assert bench.needs_spawn(1, {}) is False
    assert bench.needs_spawn(2, {"WORLD_SIZE": "2", "RANK": "0"}) is False      # torch.distributed.run started us
    assert bench.needs_spawn(2, {"RANK": "1"}) is False

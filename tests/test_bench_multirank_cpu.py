"""The multi-rank bookkeeping of bench.py (replicas only: no data-path collective), on CPU with gloo and two ranks:
timings are reduced with a maximum over ranks and the job's throughput counts every rank's steps."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank_main(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    mine = [10.0 + rank, 4.0 - rank, 7.0]          # rank 1 is slower on the first, faster on the second
    reduced = bench.max_over_ranks(mine, torch.device("cpu"), world)
    dist.barrier()
    if rank == 0:
        out.put((reduced, bench.job_throughput(world, 100, reduced[0])))
    dist.destroy_process_group()


def test_timings_are_max_over_ranks_and_throughput_counts_all_ranks():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + (os.getpid() % 2000)
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    reduced, value = out.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert reduced == [11.0, 4.0, 7.0]
    assert abs(value - 2 * 100 / 11.0e-3) < 1e-6


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([1.5, 2.5], torch.device("cpu"), 1) == [1.5, 2.5]
    assert bench.job_throughput(1, 64, 8.0) == 8000.0


def test_gpus_flag_starts_one_rank_per_gpu(monkeypatch):
    """`python bench.py --gpus N` outside a launcher starts N ranks itself, the way the launcher would."""
    sys.path.insert(0, ROOT)
    import bench
    seen = {}

    def fake_call(cmd):
        seen["cmd"] = cmd
        return 0
    monkeypatch.setattr(bench.subprocess, "call", fake_call)
    assert bench.spawn_ranks(4, ["--gpus", "4", "--steps", "8"]) == 0
    cmd = seen["cmd"]
    assert cmd[1:4] == ["-m", "torch.distributed.run", "--nnodes=1"]
    assert "--nproc-per-node=4" in cmd
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1"
    assert int(cmd[cmd.index("--master-port") + 1]) > 0
    assert cmd[-5].endswith("bench.py") and cmd[-4:] == ["--gpus", "4", "--steps", "8"]
    # and main() takes that path only when no launcher has set the world size
    monkeypatch.delenv("WORLD_SIZE", raising=False)
    monkeypatch.setattr(sys, "argv", ["bench.py", "--gpus", "2", "--steps", "4"])
    monkeypatch.setattr(bench, "spawn_ranks", lambda n, argv: 7 if (n, argv) == (2, ["--gpus", "2", "--steps", "4"]) else 1)
    try:
        bench.main()
        raise AssertionError("main() should exit with the launcher's status")
    except SystemExit as e:
        assert e.code == 7

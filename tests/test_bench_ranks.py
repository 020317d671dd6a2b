"""Host logic of the multi-GPU bench path, on CPU: two gloo ranks time "their replica" differently,
both must continue with the slower rank's time, and the job's rate counts the units of all ranks."""
import os
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _rank_main(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        mine = [10.0 + rank, 3.0 - rank, 40.0 + 5 * rank]       # ms measured "on this rank's device"
        dist.barrier()
        got = bench.max_over_ranks(mine, world, "cpu")
        rate = bench.whole_job_rate(1000.0, world, got[2])
        out.put((rank, got, rate))
    finally:
        dist.destroy_process_group()


def test_two_ranks_take_the_slowest_time_and_add_their_units():
    world, port = 2, 29000 + os.getpid() % 2000
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_rank_main, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, got, rate in res:
        assert got == [11.0, 3.0, 45.0]                       # the maximum over the ranks, on every rank
        assert rate == pytest.approx(2 * 1000.0 / 45e-3)      # both replicas' units over the slowest time


def test_single_rank_is_the_identity():
    import bench
    assert bench.max_over_ranks([1.5, 2.5], 1, "cpu") == [1.5, 2.5]
    assert bench.whole_job_rate(10.0, 1, 5.0) == pytest.approx(2000.0)


def test_gpus_flag_without_a_launcher_starts_the_replicas(monkeypatch):
    """`bench.py --gpus 2` started as a plain process re-launches itself as two ranks (one per GPU)
    with the same arguments; under a launcher (WORLD_SIZE set) it runs as a rank instead."""
    import bench
    monkeypatch.delenv("WORLD_SIZE", raising=False)
    seen = []
    monkeypatch.setattr(bench.subprocess, "call", lambda cmd: seen.append(cmd) or 0)
    argv = ["--gpus", "2", "--steps", "4", "--warmup", "3"]
    assert bench.main(argv) == 0
    (cmd,) = seen
    assert cmd[1:3] == ["-m", "torch.distributed.run"] and "--nproc-per-node=2" in cmd and "--nnodes=1" in cmd
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1"
    assert cmd[-len(argv):] == argv and cmd[-len(argv) - 1].endswith("bench.py")
    # as a rank of a launched job the same flags do not spawn again
    monkeypatch.setenv("WORLD_SIZE", "2")
    ran = []
    monkeypatch.setattr(bench, "run_gpu", lambda args: ran.append(args.gpus))
    assert bench.main(argv) == 0 and ran == [2] and len(seen) == 1

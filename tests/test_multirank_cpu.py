"""The N > 1 path of bench.py on CPU: two gloo ranks run independent replicas; the only
communication is the barrier and the max-over-ranks of the elapsed time, and the reported value
is the sum of what all ranks processed divided by that time."""
import os
import socket
import sys

import pytest
import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, ret):
    os.environ.update({"MASTER_ADDR": "127.0.0.1", "MASTER_PORT": str(port), "RANK": str(rank),
                       "WORLD_SIZE": str(world), "LOCAL_RANK": str(rank)})
    sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
    import torch.distributed as dist
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        comm = bench.RankComm(world, device="cpu")
        comm.barrier()
        elapsed = 10.0 + 5.0 * rank           # rank 1 is the slow one
        worst = comm.max_over_ranks(elapsed)
        value = bench.aggregate_value(leaves_per_rank=256, world=world, ms_per_step=worst)
        seeds = comm.all_values(float(bench.replica_value_seed(1000, rank)))
        ret[rank] = (worst, value, seeds)
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_aggregate_like_the_bench():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    with ctx.Manager() as man:
        ret = man.dict()
        procs = [ctx.Process(target=_worker, args=(r, world, port, ret)) for r in range(world)]
        for p in procs:
            p.start()
        for p in procs:
            p.join(120)
            assert p.exitcode == 0
        for r in range(world):
            worst, value, seeds = ret[r]
            assert worst == 15.0                                  # max over ranks, same on every rank
            assert value == pytest.approx(2 * 256 / 0.015)        # all ranks' leaves / slowest time
            assert seeds[0] != seeds[1]                           # replicas draw different values


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
    import bench
    comm = bench.RankComm(1, device="cpu")
    comm.barrier()
    assert comm.max_over_ranks(3.5) == 3.5
    assert bench.aggregate_value(64, 1, 2.0) == pytest.approx(32000.0)

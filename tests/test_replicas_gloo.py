"""The multi-GPU path of bench.py on CPU: two gloo ranks.  The path has no exchange step, so N
GPUs run N independent replicas; what the ranks share is only the timing protocol (barrier,
maximum over ranks) and the whole-job throughput formula."""
import os
import socket
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        dist.barrier()
        # rank 1 is the slow replica on the device-timed leg, rank 0 on the end-to-end leg
        mine = [10.0 + 5.0 * rank, 400.0 - 100.0 * rank]
        total_ms, e2e_ms = bench.max_over_ranks(mine)
        dist.barrier()
        out[rank] = (total_ms, e2e_ms, bench.replica_throughput(1 << 30, 1, world, total_ms / 10))
    finally:
        dist.destroy_process_group()


def test_two_replicas_report_the_slowest_rank_and_the_sum_of_the_work():
    world = 2
    with mp.get_context("spawn").Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_rank_main, args=(world, _free_port(), out), nprocs=world, join=True)
        res = dict(out)
    assert res[0][:2] == res[1][:2] == (15.0, 400.0)
    # two caches of 1 GiB in 1.5 ms per step
    assert res[0][2] == pytest.approx(2 * (1 << 30) / 1.5e-3 / 1e9)


def test_single_process_needs_no_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([1.5, 2.5]) == [1.5, 2.5]
    assert bench.replica_throughput(10 ** 9, 4, 1, 1000.0) == pytest.approx(4.0)

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


def _handoff_main(rank, world, port, out):
    """Sender (rank 0) makes a card and ships its bytes; receiver (rank 1) injects its own copy."""
    sys.path.insert(0, ROOT)
    import numpy as np
    import oracle
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        L, H, d, T = 2, 2, 64, 77
        rng = np.random.default_rng(5)      # both ranks know the sender's cache, to check against
        Ks = [rng.standard_normal((H, T, d), dtype=np.float32).astype(np.float16) for _ in range(L)]
        Vs = [rng.standard_normal((H, T, d), dtype=np.float32).astype(np.float16) for _ in range(L)]
        bits = rng.choice(np.array([2, 4, 8, 16], np.uint8), size=T)
        lay = oracle.make_layout(L, H, d, T)
        size = torch.zeros(1, dtype=torch.int64)
        if rank == 0:
            st, card = oracle.card_create(lay, Ks, Vs, bits, model_id=7, sender_id=0)
            assert st == oracle.OK
            size[0] = card.size
        dist.broadcast(size, 0)
        blob = torch.from_numpy(card.copy()) if rank == 0 else torch.zeros(int(size[0]), dtype=torch.uint8)
        dist.broadcast(blob, 0)             # the handoff: the blob and nothing else
        if rank == 1:
            got = blob.numpy()
            hd = oracle.parse_header(got)
            Ko = [np.zeros((H, T, d), np.float16) for _ in range(L)]
            Vo = [np.zeros((H, T, d), np.float16) for _ in range(L)]
            assert oracle.card_inject(got, lay, Ko, Vo) == oracle.OK
            m = bits == 16
            exact = all(np.array_equal(Ko[l][:, m].view(np.uint16), Ks[l][:, m].view(np.uint16)) for l in range(L))
            err = max(float(np.abs(Ko[l].astype(np.float32) - Ks[l].astype(np.float32)).max()) for l in range(L))
            out[rank] = (hd["sender_id"], hd["model_id"], hd["total_bytes"] == got.size, exact, err)
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_a_card_handed_to_another_rank_injects_there():
    """The handoff between two processes carries one blob; the receiver needs nothing else of the
    sender (the card is position independent and names its own shape)."""
    world = 2
    with mp.get_context("spawn").Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_handoff_main, args=(world, _free_port(), out), nprocs=world, join=True)
        res = dict(out)
    sender, model, whole, exact, err = res[1]
    assert (sender, model, whole, exact) == (0, 7, True, True) and 0 < err < 2.5

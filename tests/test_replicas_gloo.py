"""The multi-GPU path is "replicas only": world_size-2 gloo processes on CPU check its bookkeeping
(max-over-ranks time, summed work), which is all that crosses ranks."""
import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank: int, world: int, port: int, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2605_23258_b200 import replicas
    assert replicas.world() == (rank, world)
    times = [10.0 + rank, 5.0 - rank, 7.0]                 # rank 1 is slower on the first, faster on the second
    mx = replicas.slowest(times)
    thr = replicas.aggregate_throughput(32768.0, 2.0 + rank)   # slowest replica: 3 ms
    dist.barrier()
    out[rank] = (mx, thr)
    dist.destroy_process_group()


def test_replica_bookkeeping_world_size_2():
    world, port = 2, _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    for rank in range(world):
        mx, thr = res[rank]
        assert mx == [11.0, 5.0, 7.0]
        assert thr == pytest.approx(2 * 32768.0 / 3e-3)


def test_single_process_is_one_replica():
    from paper_2605_23258_b200 import replicas
    assert replicas.world() == (0, 1)
    assert replicas.slowest([3.0, 4.0]) == [3.0, 4.0]
    assert replicas.aggregate_throughput(100.0, 50.0) == pytest.approx(2000.0)

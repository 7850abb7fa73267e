"""World-size-2 check (gloo, CPU) of the multi-GPU bookkeeping bench.py uses: ranks take
disjoint batches, times reduce with MAX, unit counts with SUM."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2407_15452_b200.replicas import batch_of, reduce_timing


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    times, counts = reduce_timing([10.0 + rank, 5.0 - rank], [100 * (rank + 1), 7])
    out[rank] = (times, counts, [batch_of(s, rank, world, 5) for s in range(6)])
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_reduction_and_batch_assignment():
    world = 2
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, _free_port(), out), nprocs=world, join=True)
        res = dict(out)
    for r in range(world):
        times, counts, _ = res[r]
        assert times == [11.0, 5.0] and counts == [300, 14]
    b0, b1 = res[0][2], res[1][2]
    assert b0 == [0, 2, 4, 1, 3, 0] and b1 == [1, 3, 0, 2, 4, 1]
    assert all(x != y for x, y in zip(b0, b1))          # never the same batch at the same step


def test_single_process_passthrough():
    assert reduce_timing([1.5], [3]) == ([1.5], [3])
    assert [batch_of(s, 0, 1, 3) for s in range(4)] == [0, 1, 2, 0]

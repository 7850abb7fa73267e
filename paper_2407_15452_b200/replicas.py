"""Host-side bookkeeping for running independent replicas of the path on several GPUs.

The walk + SGNS path has no exchange step between GPUs (each replica owns its tables), so the
only cross-rank work is the benchmark's: which mini-batches a rank takes, the slowest rank's
time and the summed unit counts.  Works on any torch.distributed backend (NCCL on GPUs, gloo
on CPU)."""
from __future__ import annotations

import torch
import torch.distributed as dist


def batch_of(step: int, rank: int, world: int, nb_total: int) -> int:
    """Mini-batch index a rank processes at a step: ranks take disjoint, interleaved batches."""
    return (step * world + rank) % nb_total


def reduce_timing(times, counts, device="cpu"):
    """MAX over ranks of each entry of `times`, SUM over ranks of each entry of `counts`.

    Returns (times, counts) as Python lists; with no process group it returns the inputs."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [float(t) for t in times], [int(c) for c in counts]
    t = torch.tensor([float(x) for x in times], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    c = torch.tensor([int(x) for x in counts], dtype=torch.int64, device=device)
    dist.all_reduce(c, op=dist.ReduceOp.SUM)
    return t.tolist(), c.tolist()

"""Host-side logic of the multi-GPU layout: batch-sharded replicas.

Sequences are independent, weights are small and replicate, so N ranks run N copies of the
same per-GPU workload on their own sequences with no collective on the data path.  The only
communication is for measurement: a barrier around the timed region and a max over ranks of
the device-measured times.  Works on any torch.distributed backend (nccl on GPUs, gloo in the
CPU tests)."""
from __future__ import annotations

import numpy as np
import torch
import torch.distributed as dist


def rank_batch(x: np.ndarray, rank: int) -> np.ndarray:
    """The batch of sequences rank `rank` processes: rank 0 keeps x; other ranks get the same
    token rows in a rank-seeded order (every row keeps its gate-logit margin)."""
    if rank == 0:
        return x
    B, T, M = x.shape
    perm = np.random.Generator(np.random.PCG64(1000 + rank)).permutation(B * T)
    return np.ascontiguousarray(x.reshape(B * T, M)[perm].reshape(B, T, M))


def max_over_ranks(values, device="cpu"):
    """Element-wise maximum of a list of floats over all ranks (identity without a process group)."""
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def aggregate_throughput(units_per_rank: float, world: int, seconds_slowest: float) -> float:
    """Whole-job throughput: the units all ranks processed over the slowest rank's time."""
    return world * units_per_rank / seconds_slowest

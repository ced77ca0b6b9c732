"""Host-side plumbing for running one replica of the training step per GPU.

The path itself does not shard: every rank holds the whole graph and feature table and trains on its own
seed batches; nothing is exchanged between ranks on the measured path.  What ranks do share is bookkeeping:
which batches belong to whom, and the reduction of the measurements (slowest rank's time, everybody's edges).
"""
from __future__ import annotations

import torch
import torch.distributed as dist

RANK_STRIDE = 1_000_000        # step numbers of rank r start at r * RANK_STRIDE: no two ranks draw the same batch


def first_step_of(rank: int) -> int:
    return rank * RANK_STRIDE


def reduce_measurements(times_s, counts, device=None):
    """(max over ranks of each time, sum over ranks of each count).  Works with any backend; a single
    process returns its own numbers."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [float(t) for t in times_s], [int(c) for c in counts]
    t = torch.tensor([float(x) for x in times_s], dtype=torch.float64, device=device)
    c = torch.tensor([int(x) for x in counts], dtype=torch.int64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(c, op=dist.ReduceOp.SUM)
    return [float(x) for x in t.tolist()], [int(x) for x in c.tolist()]

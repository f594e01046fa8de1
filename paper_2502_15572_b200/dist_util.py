"""Host-side plumbing for running the retrieval path on several GPUs of one node.

The path partitions by QUERY STREAM: every rank holds a replica of the
datastore and serves its own slice of the decode positions; there is no
data-path collective.  What ranks share is only the timing protocol of the
benchmark: a barrier on both sides of the timed region and the maximum of the
per-rank device times.  These helpers hold that logic so that it can be
exercised on CPU with the gloo backend.
"""
from __future__ import annotations

import os


def rank_info():
    """(rank, local_rank, world_size) from the torchrun environment (1 process = 1 GPU)."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def query_slice(n_queries: int, rank: int, world: int) -> range:
    """Indices of the query stream served by `rank`: contiguous, disjoint, covering, sizes differ by <= 1."""
    if world < 1 or not (0 <= rank < world):
        raise ValueError("bad rank/world")
    base, extra = divmod(n_queries, world)
    start = rank * base + min(rank, extra)
    return range(start, start + base + (1 if rank < extra else 0))


def max_over_ranks(values, device=None):
    """Element-wise maximum of a list of floats over all ranks (identity when not distributed)."""
    import torch
    import torch.distributed as dist
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t.tolist()]


def aggregate_throughput(units_per_rank_per_step: int, steps: int, world: int, max_ms_total: float) -> float:
    """Whole-job units/s: every rank did `steps` steps in at most `max_ms_total` milliseconds."""
    return world * units_per_rank_per_step * steps / (max_ms_total * 1e-3)

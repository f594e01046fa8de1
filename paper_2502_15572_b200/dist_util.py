"""Host-side plumbing for running the retrieval path on several GPUs of one node.

Two ways to use several GPUs:

* by QUERY STREAM (what bench.py does): every rank holds a replica of the datastore
  and serves its own slice of the decode positions; no data-path collective, only the
  benchmark's timing protocol (barrier on both sides, maximum of the per-rank times);
* by ROWS (`sharded_retrieve`): the datastore is split into contiguous row shards, one
  per rank; every rank retrieves from its shard, the small per-shard results are
  all-gathered (B * n * (8 + 4 L) bytes per rank -- latency-bound, so one collective)
  and merged on the device by `dresd_merge_shards`.

The collectives are torch.distributed calls, so the plumbing can be exercised on CPU
with the gloo backend; the merge itself is a CUDA kernel.
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


def shard_rows(N: int, rank: int, world: int) -> range:
    """Contiguous row shard of `rank` (same rule as query_slice)."""
    return query_slice(N, rank, world)


def gather_shard_results(ids, scores, tokens, row_offset: int, group=None):
    """All-gather the per-shard results.  Returns ``(ids [P][B][n], scores [P][B][n],
    tokens [P][B][n][L], offsets int64 [P])`` on the inputs' device; with one process
    the inputs come back with a leading axis of 1."""
    import torch
    import torch.distributed as dist
    off = torch.tensor([row_offset], dtype=torch.int64, device=ids.device)
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size(group) == 1:
        return ids[None], scores[None], tokens[None], off
    P = dist.get_world_size(group)

    def gather(t):
        # concatenated along axis 0 (the form every backend accepts), then split by rank
        out = torch.empty((P * t.shape[0],) + tuple(t.shape[1:]), dtype=t.dtype, device=t.device)
        dist.all_gather_into_tensor(out, t.contiguous(), group=group)
        return out.reshape((P,) + tuple(t.shape))

    return gather(ids), gather(scores), gather(tokens), gather(off).reshape(P)


def sharded_retrieve(store, row_offset: int, queries, top_n: int, draft_len: int, group=None, stream=None):
    """Retrieval over a datastore whose rows are sharded over the ranks of `group`.

    `store` holds this rank's rows, `row_offset` is the global index of its row 0.
    Every rank gets the global result (ids are global row indices)."""
    import torch
    from . import binding
    ids, scores, tokens = store.retrieve(queries, top_n, draft_len, stream=stream)
    g_ids, g_scores, g_tokens, offsets = gather_shard_results(ids, scores, tokens, row_offset, group)
    P, B = g_ids.shape[0], g_ids.shape[1]
    out = (torch.empty_like(ids), torch.empty_like(scores), torch.empty_like(tokens))
    s = (stream or torch.cuda.current_stream()).cuda_stream
    binding.dresd_merge_shards(g_ids.data_ptr(), g_scores.data_ptr(), g_tokens.data_ptr(), offsets.data_ptr(),
                               P, B, top_n, draft_len, out[0].data_ptr(), out[1].data_ptr(), out[2].data_ptr(), s)
    return out

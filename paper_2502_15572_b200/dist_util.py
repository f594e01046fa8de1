"""Host-side plumbing for running the retrieval path on several GPUs of one node.

Two ways to use several GPUs:

* by QUERY STREAM (what bench.py does): every rank holds a replica of the datastore
  and serves its own slice of the decode positions; no data-path collective, only the
  benchmark's timing protocol (barrier on both sides, maximum of the per-rank times);
* by ROWS (`sharded_retrieve`): the datastore is split into contiguous row shards, one
  per rank; every rank retrieves from its shard, the small per-shard results are
  all-gathered (B * n * (8 + 4 L) bytes per rank -- latency-bound, so ONE collective over a
  packed block, `PackedExchange` / `ShardedRetriever`) and merged on the device by
  `dresd_merge_shards_packed`.  `sharded_retrieve` is the plain form of the same step
  (three all-gathers, nothing kept between calls).

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


MAX_GLOBAL_ROWS = 2 ** 31 - 1          # merged ids are int32 row indices


def check_global_rows(offsets, rows) -> None:
    """Raises ValueError when some shard's rows would get global ids beyond int32: the merge
    kernels write ids as int32, so a sharded datastore may hold at most 2^31 - 1 rows in all."""
    for off, n in zip(offsets, rows):
        if off < 0 or n < 0 or off + n > MAX_GLOBAL_ROWS:
            raise ValueError(f"shard at row offset {off} with {n} rows passes the largest global row id "
                             f"({MAX_GLOBAL_ROWS - 1}): a sharded datastore holds at most 2^31 - 1 rows")


def _on_stream(stream):
    """Context in which torch.distributed collectives are enqueued on `stream` (torch orders a
    collective after the CURRENT stream, so kernels launched on another stream would race it)."""
    import contextlib
    import torch
    if stream is None or not torch.cuda.is_available():
        return contextlib.nullcontext()
    return torch.cuda.stream(stream)


def broadcast_array(array, src: int = 0, device="cuda", group=None):
    """A numpy array that only rank `src` holds (the others pass None) -> a tensor on `device`
    on every rank, moved by one broadcast: a replica of the datastore is generated once, not
    once per rank.  16-bit bit patterns travel as int16."""
    import numpy as np
    import torch
    import torch.distributed as dist
    multi = dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1
    rank = dist.get_rank(group) if multi else src
    meta = [None]
    if rank == src:
        a = np.ascontiguousarray(array)
        if a.dtype in (np.float16, np.uint16):
            a = a.view(np.int16)
        meta = [(tuple(a.shape), a.dtype.str)]
    if multi:
        dist.broadcast_object_list(meta, src=src, group=group)
    shape, dt = meta[0]
    # the payload travels as bytes (every backend moves uint8) and is re-viewed on arrival
    if rank == src:
        t = torch.from_numpy(a.reshape(-1).view(np.uint8)).to(device)
    else:
        t = torch.empty(int(np.prod(shape)) * np.dtype(dt).itemsize, dtype=torch.uint8, device=device)
    if multi:
        dist.broadcast(t, src=src, group=group)
    return t.view(torch.from_numpy(np.empty(0, dtype=np.dtype(dt))).dtype).reshape(shape)


def collect_rows(local_rows, first_row: int, wanted, group=None, device="cpu"):
    """Rows `wanted` (global indices, the same list on every rank) of a matrix whose rows are
    sharded over the ranks: this rank holds rows first_row .. first_row + len(local_rows) - 1
    as the numpy array `local_rows`.  Every rank gets all wanted rows, bit for bit (each row
    is contributed by its one owner and the others add zero bytes).  numpy in, numpy out."""
    import numpy as np
    import torch
    import torch.distributed as dist
    local_rows = np.ascontiguousarray(local_rows)
    wanted = np.asarray(wanted, dtype=np.int64)
    row_bytes = local_rows.shape[1] * local_rows.dtype.itemsize
    buf = np.zeros((len(wanted), row_bytes), dtype=np.uint8)
    mine = (wanted >= first_row) & (wanted < first_row + local_rows.shape[0])
    buf[mine] = local_rows[wanted[mine] - first_row].view(np.uint8).reshape(-1, row_bytes)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
        t = torch.from_numpy(buf).to(device)
        dist.all_reduce(t, op=dist.ReduceOp.SUM, group=group)
        buf = t.cpu().numpy()
    return buf.view(local_rows.dtype).reshape(len(wanted), local_rows.shape[1])


def gather_shard_results(ids, scores, tokens, row_offset: int, group=None, n_rows: int = 0):
    """All-gather the per-shard results.  Returns ``(ids [P][B][n], scores [P][B][n],
    tokens [P][B][n][L], offsets int64 [P])`` on the inputs' device; with one process
    the inputs come back with a leading axis of 1.  `n_rows` (this shard's row count), when
    given, is exchanged with the offsets and every rank checks that global ids fit int32."""
    import torch
    import torch.distributed as dist
    off = torch.tensor([row_offset], dtype=torch.int64, device=ids.device)
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size(group) == 1:
        check_global_rows([row_offset], [n_rows])
        return ids[None], scores[None], tokens[None], off
    P = dist.get_world_size(group)

    def gather(t):
        # concatenated along axis 0 (the form every backend accepts), then split by rank
        out = torch.empty((P * t.shape[0],) + tuple(t.shape[1:]), dtype=t.dtype, device=t.device)
        dist.all_gather_into_tensor(out, t.contiguous(), group=group)
        return out.reshape((P,) + tuple(t.shape))

    meta = gather(torch.tensor([[row_offset, n_rows]], dtype=torch.int64, device=ids.device)).reshape(P, 2)
    check_global_rows(meta[:, 0].tolist(), meta[:, 1].tolist())
    return gather(ids), gather(scores), gather(tokens), meta[:, 0].contiguous()


def sharded_retrieve(store, row_offset: int, queries, top_n: int, draft_len: int, group=None, stream=None):
    """Retrieval over a datastore whose rows are sharded over the ranks of `group`.

    `store` holds this rank's rows, `row_offset` is the global index of its row 0.
    Every rank gets the global result (ids are global row indices)."""
    import torch
    from . import binding
    ids, scores, tokens = store.retrieve(queries, top_n, draft_len, stream=stream)
    with _on_stream(stream):
        g_ids, g_scores, g_tokens, offsets = gather_shard_results(ids, scores, tokens, row_offset, group,
                                                                  n_rows=getattr(store, "N", 0))
    P, B = g_ids.shape[0], g_ids.shape[1]
    out = (torch.empty_like(ids), torch.empty_like(scores), torch.empty_like(tokens))
    s = (stream or torch.cuda.current_stream()).cuda_stream
    binding.dresd_merge_shards(g_ids.data_ptr(), g_scores.data_ptr(), g_tokens.data_ptr(), offsets.data_ptr(),
                               P, B, top_n, draft_len, out[0].data_ptr(), out[1].data_ptr(), out[2].data_ptr(), s)
    return out


class PackedExchange:
    """Buffers of the exchange step for a fixed (B, top_n, draft_len): this rank's results live in
    ONE block of B * n * (2 + L) 32-bit words -- ids | scores | tokens, the layout
    dresd_merge_shards_packed() reads -- so that a call needs a single all-gather; the row
    offsets of the shards are exchanged once, here.  Works on any device (CPU + gloo in the tests)."""

    def __init__(self, B: int, top_n: int, draft_len: int, row_offset: int, device, group=None, n_rows: int = 0):
        import torch
        import torch.distributed as dist
        self.group = group
        self.P = dist.get_world_size(group) if dist.is_available() and dist.is_initialized() else 1
        bn = B * top_n
        self.words = bn * (2 + draft_len)
        self.local = torch.empty(self.words, dtype=torch.int32, device=device)
        self.ids = self.local[:bn].view(B, top_n)
        self.scores = self.local[bn:2 * bn].view(torch.float32).view(B, top_n)
        self.tokens = self.local[2 * bn:].view(B, top_n, draft_len)
        off = torch.tensor([row_offset, n_rows], dtype=torch.int64, device=device)
        if self.P == 1:
            self.gathered, meta = self.local, off.view(1, 2)
        else:
            self.gathered = torch.empty(self.P * self.words, dtype=torch.int32, device=device)
            meta = torch.empty(self.P * 2, dtype=torch.int64, device=device)
            dist.all_gather_into_tensor(meta, off, group=group)
            meta = meta.view(self.P, 2)
        # every rank sees every shard's extent, so every rank raises (or none does)
        check_global_rows(meta[:, 0].tolist(), meta[:, 1].tolist())
        self.offsets = meta[:, 0].contiguous()

    def exchange(self):
        """All ranks' blocks, back to back: int32 [P * words]."""
        if self.P > 1:
            import torch.distributed as dist
            dist.all_gather_into_tensor(self.gathered, self.local, group=self.group)
        return self.gathered


class ShardedRetriever:
    """dresd_retrieve over a datastore whose rows are sharded over the ranks of `group`: the local
    call writes into the packed block, one all-gather, one merge kernel.  Buffers are kept per
    batch size; every rank gets the global result (ids are global row indices)."""

    def __init__(self, store, row_offset: int, top_n: int, draft_len: int, group=None):
        self.store, self.row_offset, self.n, self.L, self.group = store, row_offset, top_n, draft_len, group
        self._by_batch = {}

    def __call__(self, queries, stream=None):
        import torch
        from . import binding
        B = queries.shape[0]
        st = self._by_batch.get(B)
        if st is None:
            ex = PackedExchange(B, self.n, self.L, self.row_offset, queries.device, self.group,
                                n_rows=getattr(self.store, "N", 0))
            out = (torch.empty((B, self.n), dtype=torch.int32, device=queries.device),
                   torch.empty((B, self.n), dtype=torch.float32, device=queries.device),
                   torch.empty((B, self.n, self.L), dtype=torch.int32, device=queries.device))
            st = self._by_batch[B] = (ex, out)
        ex, out = st
        self.store.retrieve(queries, self.n, self.L, out=(ex.ids, ex.scores, ex.tokens), stream=stream)
        with _on_stream(stream):                       # the collective follows the kernels of `stream`
            packed = ex.exchange()
        s = (stream or torch.cuda.current_stream()).cuda_stream
        binding.dresd_merge_shards_packed(packed.data_ptr(), ex.offsets.data_ptr(), ex.P, B, self.n, self.L,
                                          out[0].data_ptr(), out[1].data_ptr(), out[2].data_ptr(), s)
        return out

"""Seeded synthetic inputs: datastores, queries and preprocessing parameters.

This module only *makes inputs*.  It holds none of the retrieval arithmetic
(no scoring, no selection, no gather) and is the one module that both the
CUDA path's tests/bench and the CPU oracle's tests may draw inputs from.

The stores stand in for the paper's datastores of reduced Llama-2 hidden
states (Section 4.2, Table 1: tens of millions of unit-length token
embeddings, each mapped to the next tokens of its position): unit-norm rows
with cluster structure, and int32 continuations with a heavy-tailed
vocabulary distribution.

Recipe (all randomness from numpy Philox, one child stream per 65,536-row
chunk, so generation is order-independent and chunk-parallel):

* centres ``M[C][d]``: N(0,1) rows, L2-normalised in float64;
* ``key_i = normalise(M[c_i] + (rho/sqrt(d)) * g_i)`` with ``c_i`` uniform in
  ``[0, C)``, ``g_i ~ N(0, I)``, ``rho = 0.5``; cast to the store dtype with
  round-to-nearest-even *after* normalising;
* ``next_tokens[i][t]``: truncated Zipf, ``P(rank r) ~ r**-1.1`` for
  ``r = 1..vocab``, token id ``r - 1``, by inverse-CDF lookup;
* queries: source row ``j_b`` uniform in ``[0, N)``;
  ``q = normalise(decode(key_j) + sigma * g)`` with per-coordinate standard
  deviation ``sigma``; cast to the store dtype.

16-bit values travel as numpy arrays of their bit patterns: ``float16`` for
``"f16"``, ``uint16`` for ``"bf16"``; ``"f32"`` is ``float32``.
"""
from __future__ import annotations

import os
from concurrent.futures import ThreadPoolExecutor

import numpy as np

CHUNK_ROWS = 65536
DTYPES = ("f32", "f16", "bf16")
DTYPE_CODE = {"f32": 0, "f16": 1, "bf16": 2}
DTYPE_BYTES = {"f32": 4, "f16": 2, "bf16": 2}


# ----------------------------------------------------------------------------
# storage-dtype casts (generator side only)
# ----------------------------------------------------------------------------
def cast_to_store(x: np.ndarray, dtype: str) -> np.ndarray:
    """Round a float array to the store dtype (round-to-nearest-even)."""
    if dtype == "f32":
        return np.ascontiguousarray(x, dtype=np.float32)
    if dtype == "f16":
        return np.ascontiguousarray(x, dtype=np.float32).astype(np.float16)
    if dtype == "bf16":
        u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
        rounded = u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))
        return (rounded >> np.uint32(16)).astype(np.uint16)
    raise ValueError(f"unknown dtype {dtype!r}")


def store_to_float32(x: np.ndarray, dtype: str) -> np.ndarray:
    """Exact widening of stored values to float32."""
    if dtype == "f32":
        return np.asarray(x, dtype=np.float32)
    if dtype == "f16":
        return np.asarray(x).view(np.float16).astype(np.float32)
    if dtype == "bf16":
        return (np.asarray(x).view(np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)
    raise ValueError(f"unknown dtype {dtype!r}")


def _store_empty(shape, dtype: str) -> np.ndarray:
    np_dt = {"f32": np.float32, "f16": np.float16, "bf16": np.uint16}[dtype]
    return np.empty(shape, dtype=np_dt)


# ----------------------------------------------------------------------------
# random streams
# ----------------------------------------------------------------------------
def _stream(seed: int, index: int) -> np.random.Generator:
    # Child `index` of the seed's SeedSequence; identical to spawn()[index]
    # without materialising the whole list.
    ss = np.random.SeedSequence(seed, spawn_key=(index,))
    return np.random.Generator(np.random.Philox(ss))


def _normalise_rows(x: np.ndarray) -> np.ndarray:
    nrm = np.sqrt(np.einsum("ij,ij->i", x, x, dtype=np.float64))
    return x / np.maximum(nrm, 1e-30)[:, None].astype(x.dtype)


def centres(seed: int, C: int, d: int) -> np.ndarray:
    """Mixture centres ``[C][d]``, float64, unit rows (stream 0 of the seed)."""
    rng = _stream(seed, 0)
    M = rng.standard_normal((C, d))
    return _normalise_rows(M)


def zipf_cdf(vocab: int, s: float = 1.1) -> np.ndarray:
    """CDF of the truncated Zipf law over ranks 1..vocab."""
    w = np.arange(1, vocab + 1, dtype=np.float64) ** (-s)
    cdf = np.cumsum(w)
    cdf /= cdf[-1]
    return cdf


def _n_threads(threads):
    if threads:
        return int(threads)
    try:
        return max(1, len(os.sched_getaffinity(0)))
    except AttributeError:  # pragma: no cover
        return max(1, os.cpu_count() or 1)


# ----------------------------------------------------------------------------
# datastore
# ----------------------------------------------------------------------------
def make_store(seed: int, N: int, d: int, C: int, dtype: str, stored_len: int,
               vocab: int = 32000, rho: float = 0.5, threads=None, rows=None):
    """Return ``(keys, next_tokens)``.

    ``keys``: ``[N][d]`` in the store dtype's container (see module doc).
    ``next_tokens``: ``[N][stored_len]`` int32 in ``[0, vocab)``.
    ``rows = (lo, hi)``: only rows lo .. hi-1 of the N-row store are made and returned
    (the same values the whole store holds there: every 65,536-row chunk has a random
    stream of its own), so that a process that holds a shard generates only its shard.
    """
    if dtype not in DTYPES:
        raise ValueError(f"unknown dtype {dtype!r}")
    r_lo, r_hi = (0, N) if rows is None else (int(rows[0]), int(rows[1]))
    if not (0 <= r_lo <= r_hi <= N):
        raise ValueError("rows must satisfy 0 <= lo <= hi <= N")
    M = centres(seed, C, d).astype(np.float32)
    cdf = zipf_cdf(vocab)
    keys = _store_empty((r_hi - r_lo, d), dtype)
    toks = np.empty((r_hi - r_lo, stored_len), dtype=np.int32)
    scale = np.float32(rho / np.sqrt(d))
    chunks = range(r_lo // CHUNK_ROWS, (r_hi + CHUNK_ROWS - 1) // CHUNK_ROWS) if r_hi > r_lo else range(0)

    def work(ci: int):
        lo = ci * CHUNK_ROWS
        hi = min(N, lo + CHUNK_ROWS)
        n_rows = hi - lo
        rng = _stream(seed, 1 + ci)
        comp = rng.integers(0, C, size=n_rows)
        g = rng.standard_normal((n_rows, d), dtype=np.float32)
        g *= scale
        g += M[comp]
        g = _normalise_rows(g)
        a, b = max(lo, r_lo), min(hi, r_hi)              # the part of the chunk that is asked for
        keys[a - r_lo:b - r_lo] = cast_to_store(g[a - lo:b - lo], dtype)
        u = rng.random((n_rows, stored_len))
        t = np.searchsorted(cdf, u, side="right")
        np.minimum(t, vocab - 1, out=t)
        toks[a - r_lo:b - r_lo] = t[a - lo:b - lo].astype(np.int32)

    nt = min(_n_threads(threads), max(1, len(chunks)))
    if nt <= 1:
        for ci in chunks:
            work(ci)
    else:
        with ThreadPoolExecutor(nt) as ex:
            list(ex.map(work, chunks))
    return keys, toks


def sort_by_first_token(keys: np.ndarray, toks: np.ndarray):
    """The same datastore with its rows in order of first stored token (stable): the layout
    dresd_store_index_first_tokens() asks for.  A permutation only."""
    order = np.argsort(toks[:, 0], kind="stable")
    return np.ascontiguousarray(keys[order]), np.ascontiguousarray(toks[order])


def make_queries(seed: int, keys: np.ndarray, dtype: str, B: int, sigma: float):
    """Queries drawn near datastore keys.  Returns ``(queries, source_rows)``.

    ``queries``: ``[B][d]`` in the store dtype's container; ``source_rows``:
    int64 ``[B]``.  The source row is usually, not always, the best match.
    """
    N, d = keys.shape
    src = query_sources(seed, N, B)
    return queries_from_rows(seed, keys[src], dtype, N, sigma), src


def query_sources(seed: int, N: int, B: int) -> np.ndarray:
    """The source rows ``make_queries(seed, keys[N], ..., B, ...)`` draws: int64 ``[B]``."""
    return _stream(seed, 0).integers(0, N, size=B).astype(np.int64)


def queries_from_rows(seed: int, source_keys: np.ndarray, dtype: str, N: int, sigma: float) -> np.ndarray:
    """The queries of ``make_queries`` given only the keys of their source rows
    (``source_keys[b] = keys[query_sources(seed, N, B)[b]]``): for processes that hold a
    shard of the rows and collect the source rows from their owners."""
    B, d = source_keys.shape
    rng = _stream(seed, 0)
    rng.integers(0, N, size=B)                           # the draw that chose the source rows
    base = store_to_float32(source_keys, dtype).astype(np.float64)
    q = base + sigma * rng.standard_normal((B, d))
    q = _normalise_rows(q)
    return cast_to_store(q.astype(np.float32), dtype)


def make_hidden_queries(seed: int, B: int, d_in: int, dtype: str,
                        scale: float = 3.0, offset: float = 0.5):
    """Raw, un-normalised hidden-state-like queries ``[B][d_in]``.

    Used to exercise z-scoring and projection: coordinates have a non-zero
    mean and a spread well away from 1 so that every preprocessing stage
    changes the result.
    """
    rng = _stream(seed, 0)
    q = offset + scale * rng.standard_normal((B, d_in))
    return cast_to_store(q.astype(np.float32), dtype)


def make_preprocess(seed: int, d_in: int, d: int, dtype: str):
    """Seeded z-score statistics and projection matrix.

    Returns ``(mean[d_in] f32, var[d_in] f32, W[d_in][d] store dtype)`` with
    ``W ~ N(0, 1/d_in)``.
    """
    rng = _stream(seed, 0)
    mean = (0.5 + 0.25 * rng.standard_normal(d_in)).astype(np.float32)
    var = (9.0 * (0.5 + rng.random(d_in))).astype(np.float32)
    W = rng.standard_normal((d_in, d)) / np.sqrt(d_in)
    return mean, var, cast_to_store(W.astype(np.float32), dtype)


# ----------------------------------------------------------------------------
# named workloads (shapes of the benchmark configurations)
# ----------------------------------------------------------------------------
WORKLOADS = {
    # name: N, d, dtype, C, B, top_n, draft_len, stored_len, sigma, seed
    "c1_tiny_f32": dict(N=100_000, d=128, dtype="f32", C=64, B=8, top_n=10,
                        draft_len=10, stored_len=10, sigma=0.05, seed=1001),
    "c2_decode_b1_f16": dict(N=10_000_000, d=256, dtype="f16", C=1024, B=1, top_n=10,
                             draft_len=10, stored_len=10, sigma=0.1, seed=1002),
    "c3_batched_bf16": dict(N=10_000_000, d=256, dtype="bf16", C=1024, B=64, top_n=32,
                            draft_len=16, stored_len=16, sigma=0.1, seed=1002),
    "c4_large_f16": dict(N=50_000_000, d=128, dtype="f16", C=4096, B=4, top_n=10,
                         draft_len=10, stored_len=10, sigma=0.1, seed=1004),
    "c5a_hidden_bf16": dict(N=4_000_000, d=4096, dtype="bf16", C=1024, B=16, top_n=10,
                            draft_len=10, stored_len=10, sigma=0.1, seed=1005),
    # shaped like the paper's own datastore (Table 1 / Section 5.2: 46.3M token embeddings reduced
    # to 64 dimensions, about 20 stored continuation tokens), 10 drafts of 10 tokens (Section 5.4)
    "paper_46m_d64_f16": dict(N=46_300_000, d=64, dtype="f16", C=4096, B=1, top_n=10,
                              draft_len=10, stored_len=20, sigma=0.1, seed=1010),
    "paper_46m_d64_f16_b16": dict(N=46_300_000, d=64, dtype="f16", C=4096, B=16, top_n=10,
                                  draft_len=10, stored_len=20, sigma=0.1, seed=1010),
    # the paper's smaller datastore (Table 1 / Section 5.6: 19M tokens, 6.49 GB on disk), same reduced width
    "paper_19m_d64_f16": dict(N=19_000_000, d=64, dtype="f16", C=4096, B=1, top_n=10,
                              draft_len=10, stored_len=20, sigma=0.1, seed=1011),
    "c5b_projected_bf16": dict(N=4_000_000, d=256, dtype="bf16", C=1024, B=16, top_n=10,
                               draft_len=10, stored_len=10, sigma=0.1, seed=1006,
                               d_in=4096, proj_seed=1007),
}


def make_workload(name: str, N: int | None = None, threads=None):
    """Build a named workload (optionally with fewer rows).  Returns a dict."""
    cfg = dict(WORKLOADS[name])
    if N is not None:
        cfg["N"] = int(N)
    keys, toks = make_store(cfg["seed"], cfg["N"], cfg["d"], cfg["C"], cfg["dtype"],
                            cfg["stored_len"], threads=threads)
    out = dict(cfg, name=name, keys=keys, next_tokens=toks)
    if "d_in" in cfg:
        mean, var, W = make_preprocess(cfg["proj_seed"], cfg["d_in"], cfg["d"], cfg["dtype"])
        out.update(W=W)
        out["queries"] = make_hidden_queries(cfg["seed"] + 100, cfg["B"], cfg["d_in"],
                                             cfg["dtype"], scale=1.0, offset=0.0)
        out["source_rows"] = None
    else:
        q, src = make_queries(cfg["seed"] + 100, keys, cfg["dtype"], cfg["B"], cfg["sigma"])
        out["queries"] = q
        out["source_rows"] = src
    return out

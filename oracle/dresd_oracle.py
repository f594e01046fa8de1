"""ctypes front end of the brute-force C oracle (``dresd_oracle.c``).

TEST INFRASTRUCTURE: argument marshalling only; all arithmetic is in the C
file, which restates Algorithm 1 steps 4-7 / Eq. 1-3 / Section 3.5 of the
paper in float64 with a full sort.  Arrays of 16-bit values are passed as
their bit patterns (numpy ``float16`` for f16, ``uint16`` for bf16).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "dresd_oracle.c")
_LIB = os.path.join(_HERE, "libdresd_oracle.so")
_DTYPE_CODE = {"f32": 0, "f16": 1, "bf16": 2}
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc if the shared object is missing or stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-fPIC", "-shared", "-fopenmp", "-std=gnu11",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        c = ctypes
        lib.dresd_oracle_decode.restype = c.c_double
        lib.dresd_oracle_decode.argtypes = [c.c_uint32, c.c_int]
        lib.dresd_oracle_preprocess.restype = c.c_int
        lib.dresd_oracle_preprocess.argtypes = [
            c.c_void_p, c.c_int, c.c_int, c.c_int, c.c_void_p, c.c_void_p, c.c_double,
            c.c_void_p, c.c_int, c.c_void_p, c.c_double, c.c_void_p]
        lib.dresd_oracle_fit_zscore.restype = c.c_int
        lib.dresd_oracle_fit_zscore.argtypes = [c.c_void_p, c.c_int64, c.c_int, c.c_int, c.c_void_p, c.c_void_p]
        lib.dresd_oracle_e4m3_decode.restype = c.c_double
        lib.dresd_oracle_e4m3_decode.argtypes = [c.c_uint32]
        lib.dresd_oracle_e4m3_encode.restype = c.c_uint32
        lib.dresd_oracle_e4m3_encode.argtypes = [c.c_double]
        lib.dresd_oracle_quantised_scores.restype = c.c_int
        lib.dresd_oracle_quantised_scores.argtypes = [c.c_void_p, c.c_int64, c.c_int, c.c_int, c.c_void_p,
                                                     c.c_void_p, c.c_int]
        lib.dresd_oracle_scores.restype = c.c_int
        lib.dresd_oracle_scores.argtypes = [c.c_void_p, c.c_int64, c.c_int, c.c_int,
                                            c.c_void_p, c.c_void_p, c.c_int]
        lib.dresd_oracle_retrieve.restype = c.c_int
        lib.dresd_oracle_retrieve.argtypes = [
            c.c_void_p, c.c_void_p, c.c_int64, c.c_int, c.c_int, c.c_int,
            c.c_void_p, c.c_int, c.c_int,
            c.c_void_p, c.c_void_p, c.c_double, c.c_void_p, c.c_void_p, c.c_double,
            c.c_int, c.c_int, c.c_void_p,
            c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p, c.c_int]
        _lib = lib
    return _lib


def _store_array(x, dtype: str) -> np.ndarray:
    want = {"f32": np.float32, "f16": np.float16, "bf16": np.uint16}[dtype]
    a = np.asarray(x)
    if a.dtype != want:
        if dtype == "f32":
            a = a.astype(np.float32)
        else:
            raise TypeError(f"{dtype} arrays must be passed as {want.__name__} bit patterns")
    return np.ascontiguousarray(a)


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _f32_or_none(a):
    return None if a is None else np.ascontiguousarray(a, dtype=np.float32)


def default_threads() -> int:
    try:
        return max(1, len(os.sched_getaffinity(0)))
    except AttributeError:  # pragma: no cover
        return max(1, os.cpu_count() or 1)


def decode(bits: int, dtype: str) -> float:
    """Exact value of one stored bit pattern."""
    return float(_load().dresd_oracle_decode(int(bits) & 0xFFFFFFFF, _DTYPE_CODE[dtype]))


def preprocess(queries, dtype: str, mean=None, var=None, eps_z: float = 1e-5,
               W=None, pca_mean=None, eps_n: float = 1e-12) -> np.ndarray:
    """Eq. 1 -> projection -> Eq. 2.  Returns the unit queries, float64 ``[B][d]``."""
    q = _store_array(queries, dtype)
    B, d_in = q.shape
    mean, var, pca_mean = _f32_or_none(mean), _f32_or_none(var), _f32_or_none(pca_mean)
    if W is not None:
        W = _store_array(W, dtype)
        if W.shape[0] != d_in:
            raise ValueError("W must be [d_in][d]")
        d = W.shape[1]
    else:
        d = d_in
    out = np.empty((B, d), dtype=np.float64)
    rc = _load().dresd_oracle_preprocess(_ptr(q), B, d_in, _DTYPE_CODE[dtype], _ptr(mean),
                                         _ptr(var), eps_z, _ptr(W), d, _ptr(pca_mean),
                                         eps_n, _ptr(out))
    if rc != 0:
        raise ValueError("oracle preprocess: bad arguments")
    return out


def fit_zscore(sample, dtype: str):
    """Statistics of Eq. 1 (Section 3.2) from a sample ``[N][d_in]`` of stored embeddings:
    ``(mean, var)`` float64 ``[d_in]``, var = population variance."""
    v = _store_array(sample, dtype)
    N, d_in = v.shape
    mean = np.empty(d_in, dtype=np.float64)
    var = np.empty(d_in, dtype=np.float64)
    rc = _load().dresd_oracle_fit_zscore(_ptr(v), N, d_in, _DTYPE_CODE[dtype], _ptr(mean), _ptr(var))
    if rc != 0:
        raise ValueError("oracle fit_zscore: bad arguments")
    return mean, var


def scores(keys, dtype: str, qhat, threads: int = 1) -> np.ndarray:
    """Inner product of one float64 unit query with every stored key: ``[N]`` float64."""
    k = _store_array(keys, dtype)
    N, d = k.shape
    qh = np.ascontiguousarray(qhat, dtype=np.float64)
    if qh.shape != (d,):
        raise ValueError("qhat must be [d]")
    s = np.empty(N, dtype=np.float64)
    rc = _load().dresd_oracle_scores(_ptr(k), N, d, _DTYPE_CODE[dtype], _ptr(qh), _ptr(s), threads)
    if rc != 0:
        raise ValueError("oracle scores: bad arguments")
    return s


@dataclass
class OracleResult:
    ids: np.ndarray          # int32 [B][top_n]
    scores: np.ndarray       # float64 [B][top_n]
    tokens: np.ndarray       # int32 [B][top_n][draft_len]
    full_scores: np.ndarray | None  # float64 [B][N] when requested


def retrieve(keys, next_tokens, dtype: str, queries, top_n: int, draft_len: int,
             mean=None, var=None, eps_z: float = 1e-5, W=None, pca_mean=None,
             eps_n: float = 1e-12, want_full_scores: bool = False,
             threads: int = 1, first_token=None) -> OracleResult:
    """One whole draft-model call, brute force (see the C file's header).

    ``first_token``: optional int32 ``[B]``; query b only considers keys whose first
    stored token equals ``first_token[b]`` (-1 = no filter).  Missing neighbours come
    back as id -1, score -inf, tokens -1.
    """
    k = _store_array(keys, dtype)
    N, d = k.shape
    nt = np.ascontiguousarray(next_tokens, dtype=np.int32)
    if nt.ndim != 2 or nt.shape[0] != N:
        raise ValueError("next_tokens must be [N][stored_len]")
    q = _store_array(queries, dtype)
    B, d_in = q.shape
    mean, var, pca_mean = _f32_or_none(mean), _f32_or_none(var), _f32_or_none(pca_mean)
    if W is not None:
        W = _store_array(W, dtype)
        if W.shape != (d_in, d):
            raise ValueError("W must be [d_in][d]")
    elif d_in != d:
        raise ValueError("queries must have the key dimension when there is no projection")
    ids = np.empty((B, top_n), dtype=np.int32)
    sc = np.empty((B, top_n), dtype=np.float64)
    tok = np.empty((B, top_n, draft_len), dtype=np.int32)
    full = np.empty((B, N), dtype=np.float64) if want_full_scores else None
    ft = None
    if first_token is not None:
        ft = np.ascontiguousarray(first_token, dtype=np.int32)
        if ft.shape != (B,):
            raise ValueError("first_token must be [B]")
    rc = _load().dresd_oracle_retrieve(
        _ptr(k), _ptr(nt), N, d, _DTYPE_CODE[dtype], nt.shape[1],
        _ptr(q), B, d_in, _ptr(mean), _ptr(var), eps_z, _ptr(W), _ptr(pca_mean), eps_n,
        top_n, draft_len, _ptr(ft), _ptr(ids), _ptr(sc), _ptr(tok), _ptr(full), threads)
    if rc != 0:
        raise ValueError("oracle retrieve: bad arguments")
    return OracleResult(ids, sc, tok, full)


def drafts_prepare(tokens, ids, eos_id: int):
    """Section 3.6 / Fig. 3: EOS-padded n x L draft matrices and their validity flags."""
    tok = np.ascontiguousarray(tokens, dtype=np.int32)
    idx = np.ascontiguousarray(ids, dtype=np.int32)
    B, n, L = tok.shape
    drafts = np.empty_like(tok)
    valid = np.empty((B, n), dtype=np.int32)
    lib = _load()
    lib.dresd_oracle_drafts_prepare.restype = ctypes.c_int
    lib.dresd_oracle_drafts_prepare.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_int,
                                                ctypes.c_int, ctypes.c_int32, ctypes.c_void_p, ctypes.c_void_p]
    if lib.dresd_oracle_drafts_prepare(_ptr(tok), _ptr(idx), B, n, L, eos_id, _ptr(drafts), _ptr(valid)) != 0:
        raise ValueError("oracle drafts_prepare: bad arguments")
    return drafts, valid


def drafts_accept(drafts, valid, llm_tokens):
    """Section 3.6: longest exactly matching draft prefix plus the LLM's own next token."""
    d = np.ascontiguousarray(drafts, dtype=np.int32)
    v = np.ascontiguousarray(valid, dtype=np.int32)
    m = np.ascontiguousarray(llm_tokens, dtype=np.int32)
    B, n, L = d.shape
    if m.shape != (B, n, L + 1):
        raise ValueError("llm_tokens must be [B][n][L+1]")
    best = np.empty(B, dtype=np.int32)
    length = np.empty(B, dtype=np.int32)
    out = np.empty((B, L + 1), dtype=np.int32)
    lib = _load()
    lib.dresd_oracle_drafts_accept.restype = ctypes.c_int
    lib.dresd_oracle_drafts_accept.argtypes = [ctypes.c_void_p] * 3 + [ctypes.c_int] * 3 + [ctypes.c_void_p] * 3
    if lib.dresd_oracle_drafts_accept(_ptr(d), _ptr(v), _ptr(m), B, n, L, _ptr(best), _ptr(length), _ptr(out)) != 0:
        raise ValueError("oracle drafts_accept: bad arguments")
    return best, length, out


def e4m3_decode(code: int) -> float:
    """Value of one E4M3 code (0..255); the two NaN codes give nan."""
    return float(_load().dresd_oracle_e4m3_decode(int(code) & 0xFF))


def e4m3_encode(x: float) -> int:
    """E4M3 code of x: round to nearest, ties to even, saturating at +-448."""
    return int(_load().dresd_oracle_e4m3_encode(float(x)))


def quantised_scores(keys, dtype: str, qhat, threads: int = 1) -> np.ndarray:
    """Approximate scores of one float64 unit query against the 8-bit copy of every key."""
    k = _store_array(keys, dtype)
    N, d = k.shape
    qh = np.ascontiguousarray(qhat, dtype=np.float64)
    if qh.shape != (d,):
        raise ValueError("qhat must be [d]")
    out = np.empty(N, dtype=np.float64)
    rc = _load().dresd_oracle_quantised_scores(_ptr(k), N, d, _DTYPE_CODE[dtype], _ptr(qh), _ptr(out), threads)
    if rc != 0:
        raise ValueError("oracle quantised_scores: bad arguments")
    return out


def retrieve_quantised(keys, next_tokens, dtype: str, queries, top_n: int, draft_len: int, candidates: int,
                       mean=None, var=None, eps_z: float = 1e-5, W=None, pca_mean=None, threads: int = 1,
                       first_token=None):
    """Candidates by approximate (8-bit) score, exact re-ranking, value lookup.

    For each query: the `candidates` rows with the largest approximate score (ties to the
    lower row) are scored exactly; the `top_n` best of them (score descending, row
    ascending) are returned with their stored tokens.  Returns ``(ids, scores, tokens,
    approx, exact)`` with approx / exact the full float64 score vectors ``[B][N]``."""
    toks = np.ascontiguousarray(next_tokens, dtype=np.int32)
    N = toks.shape[0]
    if not (1 <= top_n <= candidates <= N) or not (1 <= draft_len <= toks.shape[1]):
        raise ValueError("need 1 <= top_n <= candidates <= N and 1 <= draft_len <= stored_len")
    qhat = preprocess(queries, dtype, mean=mean, var=var, eps_z=eps_z, W=W, pca_mean=pca_mean)
    B = qhat.shape[0]
    ids = np.empty((B, top_n), dtype=np.int32)
    sc = np.empty((B, top_n), dtype=np.float64)
    tok = np.empty((B, top_n, draft_len), dtype=np.int32)
    approx = np.empty((B, N), dtype=np.float64)
    exact = np.empty((B, N), dtype=np.float64)
    rows = np.arange(N)
    for b in range(B):
        approx[b] = quantised_scores(keys, dtype, qhat[b], threads)
        exact[b] = scores(keys, dtype, qhat[b], threads)
        pool = rows
        if first_token is not None and int(first_token[b]) >= 0:
            pool = rows[toks[:, 0] == int(first_token[b])]
        cand = pool[np.lexsort((pool, -approx[b][pool]))][:candidates]   # approx descending, row ascending
        order = cand[np.lexsort((cand, -exact[b][cand]))][:top_n]    # exact descending, row ascending
        k = len(order)
        ids[b], sc[b], tok[b] = -1, -np.inf, -1
        ids[b, :k] = order
        sc[b, :k] = exact[b][order]
        tok[b, :k] = toks[order, :draft_len]
    return ids, sc, tok, approx, exact

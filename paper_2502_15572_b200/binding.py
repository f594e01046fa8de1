"""Thin ctypes binding of ``libdresd.so`` (see ``include/dresd.h``).

Argument marshalling only: every step of the retrieval path runs in the CUDA
kernels behind the C ABI.  There is no CPU fallback -- if the library is
missing or a call fails, a :class:`DresdError` is raised.

Functions carry the C names (``dresd_store_create`` ...); :class:`Store` wraps
them for torch tensors (used for device memory and streams only).
"""
from __future__ import annotations

import ctypes
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libdresd.so")
LIB_DEBUG_PATH = os.path.join(_HERE, "libdresd_debug.so")    # loaded instead when DRESD_DEBUG=1 (bounds-checked build)

DRESD_F32, DRESD_F16, DRESD_BF16 = 0, 1, 2
DTYPE_CODE = {"f32": DRESD_F32, "f16": DRESD_F16, "bf16": DRESD_BF16}
DRESD_OK = 0
STATUS_NAME = {0: "DRESD_OK", -1: "DRESD_ERR_INVALID", -2: "DRESD_ERR_UNSUPPORTED",
               -3: "DRESD_ERR_ALLOC", -4: "DRESD_ERR_CUDA", -5: "DRESD_ERR_TIMEOUT",
               -6: "DRESD_ERR_INTERNAL"}
MAX_BATCH, MAX_TOP_N, MAX_DIM = 64, 32, 4096

EXPORTS = (
    "dresd_store_create", "dresd_store_set_preprocess", "dresd_retrieve", "dresd_retrieve_host",
    "dresd_preprocess", "dresd_store_status", "dresd_store_set_option",
    "dresd_store_profile_read", "dresd_store_last_launches", "dresd_store_last_key_passes",
    "dresd_last_error",
    "dresd_store_destroy", "dresd_retrieve_noalloc", "dresd_store_enable_first_token_filter",
    "dresd_retrieve_filtered", "dresd_drafts_prepare", "dresd_drafts_accept",
    "dresd_merge_shards", "dresd_build_keys", "dresd_fit_zscore", "dresd_set_global_option", "dresd_quantise_keys", "dresd_store_attach_quantised",
    "dresd_retrieve_quantised", "dresd_store_index_first_tokens", "dresd_merge_shards_packed",
    "dresd_noalloc_status", "dresd_debug_build", "dresd_store_debug_selftest",
)


class DresdError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"{STATUS_NAME.get(status, status)}: {message}")
        self.status = status
        self.message = message


_lib = None


def load(path: str | None = None) -> ctypes.CDLL:
    """Load the CUDA library; raises if it has not been built."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    p = path or (LIB_DEBUG_PATH if os.environ.get("DRESD_DEBUG") == "1" else LIB_PATH)
    if not os.path.exists(p):
        raise DresdError(-4, f"{p} not found: build it with `python -m paper_2502_15572_b200.build` "
                             "(there is no CPU fallback)")
    lib = ctypes.CDLL(p)
    c = ctypes
    vp, i32, i64, f32 = c.c_void_p, c.c_int, c.c_int64, c.c_float
    lib.dresd_store_create.restype = i32
    lib.dresd_store_create.argtypes = [vp, vp, i64, i32, i32, i32, c.POINTER(vp)]
    lib.dresd_store_set_preprocess.restype = i32
    lib.dresd_store_set_preprocess.argtypes = [vp, i32, vp, vp, f32, vp, vp]
    lib.dresd_retrieve.restype = i32
    lib.dresd_retrieve.argtypes = [vp, vp, i32, i32, i32, vp, vp, vp, vp]
    lib.dresd_retrieve_host.restype = i32
    lib.dresd_retrieve_host.argtypes = [vp, vp, i32, i32, i32, vp, vp, vp, vp]
    lib.dresd_preprocess.restype = i32
    lib.dresd_preprocess.argtypes = [vp, vp, i32, vp, vp]
    lib.dresd_store_status.restype = i32
    lib.dresd_store_status.argtypes = [vp]
    lib.dresd_store_set_option.restype = i32
    lib.dresd_store_set_option.argtypes = [vp, c.c_char_p, i32]
    lib.dresd_store_profile_read.restype = i32
    lib.dresd_store_profile_read.argtypes = [vp, c.POINTER(c.c_double), c.POINTER(c.c_int)]
    lib.dresd_store_last_launches.restype = i32
    lib.dresd_store_last_launches.argtypes = [vp]
    lib.dresd_store_last_key_passes.restype = c.c_double
    lib.dresd_store_last_key_passes.argtypes = [vp]
    lib.dresd_last_error.restype = c.c_char_p
    lib.dresd_last_error.argtypes = []
    lib.dresd_store_destroy.restype = None
    lib.dresd_store_destroy.argtypes = [vp]
    lib.dresd_store_enable_first_token_filter.restype = i32
    lib.dresd_store_enable_first_token_filter.argtypes = [vp, vp]
    lib.dresd_store_index_first_tokens.restype = i32
    lib.dresd_store_index_first_tokens.argtypes = [vp, vp]
    lib.dresd_retrieve_filtered.restype = i32
    lib.dresd_retrieve_filtered.argtypes = [vp, vp, vp, i32, i32, i32, vp, vp, vp, vp]
    lib.dresd_drafts_prepare.restype = i32
    lib.dresd_drafts_prepare.argtypes = [vp, vp, i32, i32, i32, i32, vp, vp, vp]
    lib.dresd_drafts_accept.restype = i32
    lib.dresd_drafts_accept.argtypes = [vp, vp, vp, i32, i32, i32, vp, vp, vp, vp]
    lib.dresd_merge_shards.restype = i32
    lib.dresd_merge_shards.argtypes = [vp, vp, vp, vp, i32, i32, i32, i32, vp, vp, vp, vp]
    lib.dresd_merge_shards_packed.restype = i32
    lib.dresd_merge_shards_packed.argtypes = [vp, vp, i32, i32, i32, i32, vp, vp, vp, vp]
    lib.dresd_build_keys.restype = i32
    lib.dresd_build_keys.argtypes = [vp, i64, i32, i32, vp, vp, f32, vp, i32, vp, vp, vp]
    lib.dresd_quantise_keys.restype = i32
    lib.dresd_quantise_keys.argtypes = [vp, i64, i32, i32, vp, vp]
    lib.dresd_store_attach_quantised.restype = i32
    lib.dresd_store_attach_quantised.argtypes = [vp, vp]
    lib.dresd_retrieve_quantised.restype = i32
    lib.dresd_retrieve_quantised.argtypes = [vp, vp, vp, i32, i32, i32, i32, vp, vp, vp, vp]
    lib.dresd_set_global_option.restype = i32
    lib.dresd_set_global_option.argtypes = [ctypes.c_char_p, i32]
    lib.dresd_fit_zscore.restype = i32
    lib.dresd_fit_zscore.argtypes = [vp, i64, i32, i32, vp, vp, vp]
    lib.dresd_retrieve_noalloc.restype = i32
    lib.dresd_retrieve_noalloc.argtypes = [vp, vp, i64, i32, i32, i32, vp, i32, i32, i32, vp, vp, vp, vp]
    lib.dresd_noalloc_status.restype = i32
    lib.dresd_noalloc_status.argtypes = [vp]
    lib.dresd_debug_build.restype = i32
    lib.dresd_debug_build.argtypes = []
    lib.dresd_store_debug_selftest.restype = i32
    lib.dresd_store_debug_selftest.argtypes = [vp, vp]
    if path is None:
        _lib = lib
    return lib


def dresd_last_error() -> str:
    return load().dresd_last_error().decode()


def _check(status: int) -> None:
    if status != DRESD_OK:
        raise DresdError(status, dresd_last_error())


# ---- the C calls, by name, on raw addresses -----------------------------------
def dresd_store_create(keys_ptr: int, next_tokens_ptr: int, N: int, d: int, dtype: int,
                       stored_len: int) -> int:
    h = ctypes.c_void_p()
    _check(load().dresd_store_create(keys_ptr, next_tokens_ptr, N, d, dtype, stored_len, ctypes.byref(h)))
    return h.value


def dresd_store_set_preprocess(store: int, d_in: int, mean_ptr, var_ptr, eps_z: float, W_ptr,
                               pca_mean_ptr) -> None:
    _check(load().dresd_store_set_preprocess(store, d_in, mean_ptr, var_ptr, eps_z, W_ptr, pca_mean_ptr))


def dresd_retrieve(store: int, queries_ptr: int, B: int, top_n: int, draft_len: int, out_ids_ptr: int,
                   out_scores_ptr: int, out_tokens_ptr: int, stream: int = 0) -> None:
    _check(load().dresd_retrieve(store, queries_ptr, B, top_n, draft_len, out_ids_ptr, out_scores_ptr,
                                 out_tokens_ptr, stream))


def dresd_store_enable_first_token_filter(store: int, stream: int = 0) -> None:
    _check(load().dresd_store_enable_first_token_filter(store, stream))


def dresd_store_index_first_tokens(store: int, stream: int = 0) -> None:
    _check(load().dresd_store_index_first_tokens(store, stream))


def dresd_retrieve_filtered(store: int, queries_ptr: int, first_tokens_ptr, B: int, top_n: int, draft_len: int,
                            out_ids_ptr: int, out_scores_ptr: int, out_tokens_ptr: int, stream: int = 0) -> None:
    _check(load().dresd_retrieve_filtered(store, queries_ptr, first_tokens_ptr, B, top_n, draft_len,
                                          out_ids_ptr, out_scores_ptr, out_tokens_ptr, stream))


def dresd_drafts_prepare(tokens_ptr: int, ids_ptr: int, B: int, n: int, L: int, eos_id: int,
                         out_drafts_ptr: int, out_valid_ptr: int, stream: int = 0) -> None:
    _check(load().dresd_drafts_prepare(tokens_ptr, ids_ptr, B, n, L, eos_id, out_drafts_ptr, out_valid_ptr, stream))


def dresd_drafts_accept(drafts_ptr: int, valid_ptr: int, llm_ptr: int, B: int, n: int, L: int,
                        out_best_ptr: int, out_len_ptr: int, out_tokens_ptr: int, stream: int = 0) -> None:
    _check(load().dresd_drafts_accept(drafts_ptr, valid_ptr, llm_ptr, B, n, L, out_best_ptr, out_len_ptr,
                                      out_tokens_ptr, stream))


def dresd_merge_shards_packed(packed_ptr: int, offsets_ptr: int, P: int, B: int, top_n: int, draft_len: int,
                              out_ids_ptr: int, out_scores_ptr: int, out_tokens_ptr: int, stream: int = 0) -> None:
    _check(load().dresd_merge_shards_packed(packed_ptr, offsets_ptr, P, B, top_n, draft_len, out_ids_ptr,
                                            out_scores_ptr, out_tokens_ptr, stream))


def dresd_merge_shards(ids_ptr: int, scores_ptr: int, tokens_ptr: int, offsets_ptr: int, P: int, B: int,
                       top_n: int, draft_len: int, out_ids_ptr: int, out_scores_ptr: int, out_tokens_ptr: int,
                       stream: int = 0) -> None:
    _check(load().dresd_merge_shards(ids_ptr, scores_ptr, tokens_ptr, offsets_ptr, P, B, top_n, draft_len,
                                     out_ids_ptr, out_scores_ptr, out_tokens_ptr, stream))


def dresd_build_keys(hidden_ptr: int, N: int, d_in: int, dtype: int, mean_ptr, var_ptr, eps_z: float, W_ptr: int,
                     d: int, pca_mean_ptr, out_keys_ptr: int, stream: int = 0) -> None:
    """Eq. 1 -> v W -> Eq. 2 over N rows of hidden states: builds the datastore's key matrix."""
    _check(load().dresd_build_keys(hidden_ptr, N, d_in, dtype, mean_ptr, var_ptr, eps_z, W_ptr, d, pca_mean_ptr,
                                   out_keys_ptr, stream))


def dresd_quantise_keys(keys_ptr: int, N: int, d: int, dtype: int, out_q8_ptr: int, stream: int = 0) -> None:
    _check(load().dresd_quantise_keys(keys_ptr, N, d, dtype, out_q8_ptr, stream))


def dresd_store_attach_quantised(store: int, keys_q8_ptr: int) -> None:
    _check(load().dresd_store_attach_quantised(store, keys_q8_ptr))


def dresd_retrieve_quantised(store: int, queries_ptr: int, first_tokens_ptr, B: int, top_n: int, draft_len: int,
                             candidates: int, out_ids_ptr: int, out_scores_ptr: int, out_tokens_ptr: int,
                             stream: int = 0) -> None:
    _check(load().dresd_retrieve_quantised(store, queries_ptr, first_tokens_ptr, B, top_n, draft_len, candidates,
                                           out_ids_ptr, out_scores_ptr, out_tokens_ptr, stream))


def dresd_set_global_option(name: str, value: int) -> None:
    _check(load().dresd_set_global_option(name.encode(), int(value)))


def dresd_fit_zscore(sample_ptr: int, N: int, d_in: int, dtype: int, out_mean_ptr: int, out_var_ptr: int,
                     stream: int = 0) -> None:
    """E[V] and population Var[V] of Eq. 1 from a sample of N stored embeddings."""
    _check(load().dresd_fit_zscore(sample_ptr, N, d_in, dtype, out_mean_ptr, out_var_ptr, stream))


def dresd_retrieve_host(store: int, queries_ptr: int, B: int, top_n: int, draft_len: int,
                        out_ids_ptr: int, out_scores_ptr: int, out_tokens_ptr: int, stream: int = 0) -> None:
    _check(load().dresd_retrieve_host(store, queries_ptr, B, top_n, draft_len, out_ids_ptr,
                                      out_scores_ptr, out_tokens_ptr, stream))


def dresd_preprocess(store: int, queries_ptr: int, B: int, out_qhat_ptr: int, stream: int = 0) -> None:
    _check(load().dresd_preprocess(store, queries_ptr, B, out_qhat_ptr, stream))


def dresd_store_status(store: int) -> None:
    _check(load().dresd_store_status(store))


def dresd_store_set_option(store: int, name: str, value: int) -> None:
    _check(load().dresd_store_set_option(store, name.encode(), value))


def dresd_store_profile_read(store: int):
    """Returns ``(scan_ms_total, calls)``."""
    ms, n = ctypes.c_double(0.0), ctypes.c_int(0)
    _check(load().dresd_store_profile_read(store, ctypes.byref(ms), ctypes.byref(n)))
    return ms.value, n.value


def dresd_store_last_launches(store: int) -> int:
    return int(load().dresd_store_last_launches(store))


def dresd_store_last_key_passes(store: int) -> float:
    return float(load().dresd_store_last_key_passes(store))


def dresd_store_destroy(store: int) -> None:
    load().dresd_store_destroy(store)


def dresd_retrieve_noalloc(keys_ptr: int, next_tokens_ptr: int, N: int, d: int, dtype: int,
                           stored_len: int, queries_ptr: int, B: int, top_n: int, draft_len: int,
                           out_ids_ptr: int, out_scores_ptr: int, out_tokens_ptr: int, stream: int = 0) -> None:
    """Retrieval without any device allocation (static in-library workspace, B <= 8).

    For hosts that may not call cudaMalloc when a draft is needed; see the
    header for the limits and the rule that calls must not overlap on the GPU.
    """
    _check(load().dresd_retrieve_noalloc(keys_ptr, next_tokens_ptr, N, d, dtype, stored_len, queries_ptr,
                                         B, top_n, draft_len, out_ids_ptr, out_scores_ptr, out_tokens_ptr,
                                         stream))


def dresd_debug_build() -> int:
    """1 when the loaded library is the bounds-checked debug build."""
    return int(load().dresd_debug_build())


def dresd_store_debug_selftest(store: int, stream: int = 0) -> None:
    _check(load().dresd_store_debug_selftest(store, stream))


def dresd_noalloc_status(stream: int = 0) -> None:
    """Waits for `stream`; raises DRESD_ERR_TIMEOUT if a device-side wait of the last
    dresd_retrieve_noalloc() call expired."""
    _check(load().dresd_noalloc_status(stream))


# ---- torch convenience ----------------------------------------------------------
def _torch():
    import torch
    return torch


def to_device(array, dtype: str, device="cuda"):
    """Upload a numpy array holding store-dtype values (bit patterns for 16-bit)."""
    import numpy as np
    torch = _torch()
    a = np.ascontiguousarray(array)
    if dtype == "bf16":
        return torch.from_numpy(a.view(np.int16)).to(device).view(torch.bfloat16)
    if dtype == "f16":
        return torch.from_numpy(a.view(np.float16)).to(device)
    return torch.from_numpy(a.astype(np.float32, copy=False)).to(device)


class Store:
    """A datastore on the current CUDA device; tensors passed in are borrowed."""

    def __init__(self, keys, next_tokens, dtype: str):
        torch = _torch()
        want = {"f32": torch.float32, "f16": torch.float16, "bf16": torch.bfloat16}[dtype]
        if not keys.is_cuda or not next_tokens.is_cuda:
            raise DresdError(-1, "keys and next_tokens must be CUDA tensors (there is no CPU path)")
        if keys.dtype != want or next_tokens.dtype != torch.int32:
            raise DresdError(-1, f"keys must be {want}, next_tokens int32")
        if not keys.is_contiguous() or not next_tokens.is_contiguous():
            raise DresdError(-1, "keys and next_tokens must be contiguous")
        self.dtype = dtype
        self.torch_dtype = want
        self.keys, self.next_tokens = keys, next_tokens       # keep alive
        self.N, self.d = keys.shape
        self.stored_len = next_tokens.shape[1]
        self.d_in = self.d
        self._pre = None
        self.handle = dresd_store_create(keys.data_ptr(), next_tokens.data_ptr(), self.N, self.d,
                                         DTYPE_CODE[dtype], self.stored_len)

    def set_preprocess(self, d_in, mean=None, var=None, eps_z=1e-5, W=None, pca_mean=None):
        self._pre = (mean, var, W, pca_mean)                  # keep alive
        ptr = lambda t: None if t is None else t.data_ptr()
        dresd_store_set_preprocess(self.handle, d_in, ptr(mean), ptr(var), eps_z, ptr(W), ptr(pca_mean))
        self.d_in = d_in

    def set_option(self, name: str, value: int):
        dresd_store_set_option(self.handle, name, value)

    def retrieve(self, queries, top_n: int, draft_len: int, out=None, stream=None):
        """Returns ``(ids [B][n] int32, scores [B][n] f32, tokens [B][n][L] int32)`` on the device."""
        torch = _torch()
        B = queries.shape[0]
        if out is None:
            dev = queries.device
            out = (torch.empty((B, top_n), dtype=torch.int32, device=dev),
                   torch.empty((B, top_n), dtype=torch.float32, device=dev),
                   torch.empty((B, top_n, draft_len), dtype=torch.int32, device=dev))
        ids, scores, tokens = out
        s = (stream or torch.cuda.current_stream()).cuda_stream
        dresd_retrieve(self.handle, queries.data_ptr(), B, top_n, draft_len, ids.data_ptr(),
                       scores.data_ptr(), tokens.data_ptr(), s)
        return ids, scores, tokens

    def enable_first_token_filter(self, stream=None):
        s = (stream or _torch().cuda.current_stream()).cuda_stream
        dresd_store_enable_first_token_filter(self.handle, s)

    def index_first_tokens(self, stream=None):
        """For a store whose rows are sorted by first stored token: filtered calls then scan only
        the rows of the queries' tokens."""
        s = (stream or _torch().cuda.current_stream()).cuda_stream
        dresd_store_index_first_tokens(self.handle, s)

    def retrieve_filtered(self, queries, first_tokens, top_n: int, draft_len: int, out=None, stream=None):
        """Like retrieve(), restricted per query to keys whose first stored token is first_tokens[b]."""
        torch = _torch()
        B = queries.shape[0]
        if out is None:
            dev = queries.device
            out = (torch.empty((B, top_n), dtype=torch.int32, device=dev),
                   torch.empty((B, top_n), dtype=torch.float32, device=dev),
                   torch.empty((B, top_n, draft_len), dtype=torch.int32, device=dev))
        ids, scores, tokens = out
        s = (stream or torch.cuda.current_stream()).cuda_stream
        dresd_retrieve_filtered(self.handle, queries.data_ptr(),
                                None if first_tokens is None else first_tokens.data_ptr(), B, top_n, draft_len,
                                ids.data_ptr(), scores.data_ptr(), tokens.data_ptr(), s)
        return ids, scores, tokens

    def attach_quantised(self, stream=None):
        """Build the 8-bit (E4M3) copy of the keys on the device and attach it; returns the copy."""
        torch = _torch()
        s = (stream or torch.cuda.current_stream()).cuda_stream
        q8 = torch.empty((self.N, self.d), dtype=torch.uint8, device=self.keys.device)
        dresd_quantise_keys(self.keys.data_ptr(), self.N, self.d, DTYPE_CODE[self.dtype], q8.data_ptr(), s)
        dresd_store_attach_quantised(self.handle, q8.data_ptr())
        self.keys_q8 = q8                                # keep the borrowed buffer alive
        return q8

    def retrieve_quantised(self, queries, top_n: int, draft_len: int, candidates: int, out=None, stream=None,
                           first_tokens=None):
        """Candidates by 8-bit approximate score, exact re-ranking of `candidates` rows per query;
        first_tokens (int32 device tensor [B], -1 = any) restricts the candidates per query."""
        torch = _torch()
        B = queries.shape[0]
        if out is None:
            dev = queries.device
            out = (torch.empty((B, top_n), dtype=torch.int32, device=dev),
                   torch.empty((B, top_n), dtype=torch.float32, device=dev),
                   torch.empty((B, top_n, draft_len), dtype=torch.int32, device=dev))
        ids, scores, tokens = out
        s = (stream or torch.cuda.current_stream()).cuda_stream
        dresd_retrieve_quantised(self.handle, queries.data_ptr(),
                                 None if first_tokens is None else first_tokens.data_ptr(), B, top_n, draft_len,
                                 candidates, ids.data_ptr(), scores.data_ptr(), tokens.data_ptr(), s)
        return ids, scores, tokens

    def retrieve_host(self, queries, top_n: int, draft_len: int, out, stream=None):
        """Host (pinned) tensors in and out; blocks until the results are on the host."""
        torch = _torch()
        ids, scores, tokens = out
        s = (stream or torch.cuda.current_stream()).cuda_stream
        dresd_retrieve_host(self.handle, queries.data_ptr(), queries.shape[0], top_n, draft_len,
                            ids.data_ptr(), scores.data_ptr(), tokens.data_ptr(), s)
        return ids, scores, tokens

    def preprocess(self, queries, stream=None):
        torch = _torch()
        B = queries.shape[0]
        out = torch.empty((B, self.d), dtype=torch.float32, device=queries.device)
        s = (stream or torch.cuda.current_stream()).cuda_stream
        dresd_preprocess(self.handle, queries.data_ptr(), B, out.data_ptr(), s)
        return out

    def status(self):
        dresd_store_status(self.handle)

    def profile_read(self):
        return dresd_store_profile_read(self.handle)

    def last_key_passes(self) -> float:
        return dresd_store_last_key_passes(self.handle)

    def last_launches(self) -> int:
        return dresd_store_last_launches(self.handle)

    def close(self):
        if getattr(self, "handle", None):
            dresd_store_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

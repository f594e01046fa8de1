"""Stores sorted by first stored token (Section 3.5: only drafts that start with x_{t+1} are
kept): with the token index a filtered call scans the rows of the queries' tokens only.  The
result must be the filtered full scan's, bit for bit, and the oracle's."""
import numpy as np
import pytest

import oracle
from paper_2502_15572_b200 import binding, synth
from tests import checker
from tests.gpu_util import gpu_store

pytestmark = pytest.mark.gpu


def _sorted_store(seed, N, d, dtype, L, vocab, missing=None):
    keys, toks = synth.make_store(seed, N, d, 16, dtype, L, vocab=vocab)
    if missing is not None:                          # a token inside the range that no row stores
        toks[toks[:, 0] == missing, 0] = missing + 1
    return synth.sort_by_first_token(keys, toks)


def _tokens(rng, B, vocab, missing):
    ft = rng.integers(0, vocab, size=B).astype(np.int32)
    if B > 2:
        ft[2] = ft[0]                                # two queries share a window
    if B > 3:
        ft[3] = vocab + 3                            # beyond the largest stored token
    if B > 4 and missing is not None:
        ft[4] = missing                              # inside the range, but no rows
    if B > 6:
        ft[6] = (ft[5] + 1) % vocab                  # neighbouring windows meet inside a tile
    return ft


@pytest.mark.parametrize("dtype,d,B,n,L,N,vocab", [
    ("f16", 256, 1, 10, 10, 40009, 50),
    ("bf16", 64, 16, 10, 4, 50021, 12),              # 512-row tiles, every token asked for
    ("f16", 128, 40, 10, 4, 40009, 3000),            # windows of ~13 rows: dozens per tile
    ("bf16", 256, 64, 32, 4, 30011, 12),             # the batch that otherwise runs with the keys as N
    ("f16", 64, 5, 5, 2, 50021, 50),
    ("bf16", 192, 9, 16, 3, 20011, 7),
    ("f16", 32, 7, 10, 2, 50022, 50),                # two keys per row: a window edge may fall inside a row
    ("bf16", 32, 16, 5, 2, 50022, 3000),
    ("f16", 64, 48, 10, 2, 50021, 50),               # one column per query, windows
])
def test_windows_equal_filtered_full_scan_and_oracle(dtype, d, B, n, L, N, vocab):
    import torch
    missing = 5 if vocab > 6 else None
    keys, toks = _sorted_store(9900 + d + B, N, d, dtype, L, vocab, missing)
    q, _ = synth.make_queries(9901 + d + B, keys, dtype, B, 0.1)
    ft = _tokens(np.random.default_rng(9902 + d + B), B, vocab, missing)
    dq, dft = binding.to_device(q, dtype), torch.from_numpy(ft).cuda()
    st = gpu_store(keys, toks, dtype)
    try:
        st.index_first_tokens()
        st.index_first_tokens()                      # idempotent
        win = st.retrieve_filtered(dq, dft, n, L)
        torch.cuda.synchronize()
        st.status()
        st.set_option("first_token_windows", 0)
        full = st.retrieve_filtered(dq, dft, n, L)
        torch.cuda.synchronize()
        st.set_option("first_token_windows", 1)
        for a, b in zip(win, full):
            assert torch.equal(a, b)
        # one query without a token: the call scans everything, the result is again the same
        ft2 = ft.copy()
        ft2[0] = -1
        dft2 = torch.from_numpy(ft2).cuda()
        mixed = st.retrieve_filtered(dq, dft2, n, L)
        st.set_option("first_token_windows", 0)
        mixed_full = st.retrieve_filtered(dq, dft2, n, L)
        torch.cuda.synchronize()
        for a, b in zip(mixed, mixed_full):
            assert torch.equal(a, b)
    finally:
        st.close()
    ids, sc, tok = (x.cpu().numpy() for x in win)
    o = oracle.retrieve(keys, toks, dtype, q, n, L, first_token=ft, want_full_scores=True,
                        threads=oracle.dresd_oracle.default_threads())
    for b in range(B):
        try:
            checker.check_query_filtered(o.full_scores[b], toks, ids[b], sc[b], tok[b], dtype, n, L, int(ft[b]))
        except AssertionError as e:
            raise AssertionError(f"query {b} (first token {ft[b]}): {e}") from None
        assert np.array_equal(o.ids[b] == -1, ids[b] == -1)
    if B > 3:
        assert np.all(ids[3] == -1)                  # nobody stores that token
    if B > 4 and missing is not None:
        assert np.all(ids[4] == -1)


def test_index_rejects_an_unsorted_store_and_leaves_it_usable():
    import torch
    keys, toks = synth.make_store(9950, 5000, 64, 4, "f16", 2, vocab=20)
    st = gpu_store(keys, toks, "f16")
    try:
        with pytest.raises(binding.DresdError) as e:
            st.index_first_tokens()
        assert e.value.status == -1 and "sorted" in e.value.message
        ft = torch.from_numpy(toks[:3, 0].astype(np.int32)).cuda()
        ids, _, tok = st.retrieve_filtered(binding.to_device(keys[:3], "f16"), ft, 1, 2)
        torch.cuda.synchronize()
        assert np.array_equal(tok.cpu().numpy()[:, 0, 0], toks[:3, 0])
    finally:
        st.close()


@pytest.mark.parametrize("dtype,d,B,N,vocab", [("f16", 64, 7, 30011, 40), ("bf16", 64, 20, 30011, 9), ("bf16", 256, 6, 40009, 40)])
def test_quantised_search_over_windows_equals_the_full_filtered_search(dtype, d, B, N, vocab):
    """8-bit copy, d = 64 in packed rows (two keys and two first tokens per 128-byte row, N odd:
    window edges fall between the two keys of a row) and d = 256."""
    import torch
    n, L, m = 6, 3, 24
    keys, toks = _sorted_store(9960 + d + B, N, d, dtype, L, vocab, missing=5)
    q, _ = synth.make_queries(9961 + d + B, keys, dtype, B, 0.1)
    ft = _tokens(np.random.default_rng(9962 + d + B), B, vocab, 5)
    ft[-1] = int(toks[N - 1, 0])                      # the window that holds the odd last key
    dq, dft = binding.to_device(q, dtype), torch.from_numpy(ft).cuda()
    st = gpu_store(keys, toks, dtype)
    try:
        st.attach_quantised()
        st.index_first_tokens()
        win = st.retrieve_quantised(dq, n, L, m, first_tokens=dft)
        torch.cuda.synchronize()
        st.status()
        st.set_option("first_token_windows", 0)
        full = st.retrieve_quantised(dq, n, L, m, first_tokens=dft)
        torch.cuda.synchronize()
        for a, b in zip(win, full):
            assert torch.equal(a, b)
    finally:
        st.close()
    ids = win[0].cpu().numpy()
    for b in range(B):
        rows = np.flatnonzero(toks[:, 0] == ft[b])
        k = min(n, len(rows))
        assert np.all(np.isin(ids[b, :k], rows)) and np.all(ids[b, k:] == -1)


def test_calls_whose_windows_are_empty_or_shared():
    """No row at all for the call's tokens (no CTA has a tile), and all queries naming one token."""
    import torch
    keys, toks = _sorted_store(9980, 20011, 64, "f16", 3, 30, missing=5)
    st = gpu_store(keys, toks, "f16")
    try:
        st.index_first_tokens()
        q = binding.to_device(keys[:4], "f16")
        for ft in ([5], [1000], [5, 1000, 5, 31]):
            d = torch.tensor(ft, dtype=torch.int32, device="cuda")
            ids, sc, tok = st.retrieve_filtered(q[:len(ft)], d, 4, 3)
            torch.cuda.synchronize()
            assert torch.all(ids == -1) and torch.all(torch.isinf(sc)) and torch.all(tok == -1)
        t0 = int(toks[0, 0])
        d = torch.full((4,), t0, dtype=torch.int32, device="cuda")
        ids, _, _ = st.retrieve_filtered(q, d, 4, 3)
        torch.cuda.synchronize()
        ids = ids.cpu().numpy()
        rows = np.flatnonzero(toks[:, 0] == t0)
        assert np.all(np.isin(ids, rows))
        for b in range(4):                            # rows 0..3 start with t0 (sorted): each query finds its own key
            assert np.array_equal(keys[ids[b, 0]], keys[b]) or toks[b, 0] != t0
        st.status()
    finally:
        st.close()

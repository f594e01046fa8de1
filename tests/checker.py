"""Comparison of a retrieval result with the oracle's, element by element.

The rule (per query; ``s`` = the oracle's float64 score of every row, ``o`` =
the oracle's order, ``n`` = top_n):

* ids are distinct and in range;
* every returned score is within ``tol`` of the oracle's score of the row it
  names, and within ``tol`` of the oracle's score at that rank;
* every row scoring more than ``band`` above the oracle's n-th score is
  present, and nothing scoring more than ``band`` below it is returned;
* returned scores do not increase down the list, and the id at a rank is the
  oracle's id wherever the oracle's score at that rank is separated from its
  neighbours by more than twice the kernel's accumulation error ``eps_acc``
  (inside such a near-tie cluster any order is valid);
* tokens are bit-exact copies of the stored continuation of the returned id.

``tol`` is 2e-3 for 16-bit keys and 1e-5 for fp32 keys; ``band`` is 2e-3.

``eps_acc`` is stated for unit-length keys.  The accumulation error of an inner
product is proportional to the sum of |q_j k_ij|, which the key's length bounds
(the query has unit length), so for stores whose keys are not unit vectors the
caller passes ``key_scale`` = the largest key norm and ``eps_acc`` is multiplied
by it (never below 1).  ``tol`` and ``band`` stay absolute.
"""
from __future__ import annotations

import numpy as np

TOL = {"f32": 1e-5, "f16": 2e-3, "bf16": 2e-3}
BAND = 2e-3
# accumulation error of the CUDA path: fp32 FMA with four partial sums (fp32
# keys) / fp32 tensor-core accumulation of a two-term query split (16-bit).
EPS_ACC = {"f32": 5e-6, "f16": 1e-5, "bf16": 1e-5}


def oracle_order(full_scores: np.ndarray, k: int) -> np.ndarray:
    """First k rows in (score desc, id asc) order of one query's float64 scores."""
    N = full_scores.shape[0]
    k = min(k, N)
    if k < N:
        part = np.argpartition(-full_scores, k - 1)[:k]
        kth = full_scores[part].min()
        cand = np.nonzero(full_scores >= kth)[0]
    else:
        cand = np.arange(N)
    order = cand[np.lexsort((cand, -full_scores[cand]))]
    return order[:k]


def check_query(s: np.ndarray, next_tokens: np.ndarray, g_ids, g_scores, g_tokens, dtype: str,
                top_n: int, draft_len: int, oracle_ids=None, key_scale: float = 1.0):
    """Raises AssertionError with a description on the first violation.

    Returns the number of ranks whose id equals the oracle's.
    """
    N = s.shape[0]
    tol, band, eps = TOL[dtype], BAND, EPS_ACC[dtype] * max(1.0, float(key_scale))
    g_ids = np.asarray(g_ids).astype(np.int64)
    g_scores = np.asarray(g_scores).astype(np.float64)
    g_tokens = np.asarray(g_tokens)
    o = oracle_order(s, top_n + 1)
    if oracle_ids is not None:                      # the C oracle's own full sort must agree
        assert np.array_equal(o[:top_n], np.asarray(oracle_ids)[:top_n]), "oracle order mismatch"
    assert g_ids.shape == (top_n,) and g_scores.shape == (top_n,)
    assert g_tokens.shape == (top_n, draft_len)
    assert np.all((g_ids >= 0) & (g_ids < N)), f"id out of range: {g_ids}"
    assert len(set(g_ids.tolist())) == top_n, f"duplicate ids: {g_ids}"
    err_own = np.abs(g_scores - s[g_ids])
    assert np.all(err_own <= tol), f"score vs oracle score of the same row: max err {err_own.max():.3e}"
    err_rank = np.abs(g_scores - s[o[:top_n]])
    assert np.all(err_rank <= tol), f"score vs oracle score at the same rank: max err {err_rank.max():.3e}"
    nth = s[o[top_n - 1]]
    must = np.nonzero(s > nth + band)[0]
    missing = set(must.tolist()) - set(g_ids.tolist())
    assert not missing, f"rows clearly inside the top-n are missing: {sorted(missing)[:5]}"
    assert np.all(s[g_ids] >= nth - band), "a returned row scores clearly below the n-th best"
    assert np.all(np.diff(g_scores) <= 0), "returned scores increase down the list"
    so = s[o]
    exact = int(np.sum(g_ids == o[:top_n]))
    # Clusters of consecutive oracle ranks whose scores are chained by gaps <= 2*eps.
    # Rank n (the first row left out) takes part so that a tie across the cut is seen.
    a = 0
    while a < top_n:
        b = a
        while b + 1 < len(so) and so[b] - so[b + 1] <= 2 * eps:
            b += 1
        if b == a:
            assert g_ids[a] == o[a], (f"rank {a}: id {g_ids[a]} != oracle {o[a]} although the oracle "
                                      f"score is separated by more than {2 * eps:.1e}")
        elif b < top_n:                              # cluster strictly inside the list: same set
            assert set(g_ids[a:b + 1].tolist()) == set(o[a:b + 1].tolist()), \
                f"ranks {a}..{b}: ids {g_ids[a:b + 1]} are not a permutation of the oracle's near-tie {o[a:b + 1]}"
        else:                                        # cluster crosses the cut: any near-tie row is valid
            got = s[g_ids[a:top_n]]
            assert np.all(got <= so[a] + 2 * eps) and np.all(got >= so[-1] - 2 * eps), \
                f"ranks {a}..{top_n - 1}: ids {g_ids[a:top_n]} are not near-ties of the oracle's {o[a:]}"
        a = b + 1
    want_tok = next_tokens[g_ids][:, :draft_len]
    assert np.array_equal(g_tokens, want_tok), "tokens are not the stored continuation of the returned ids"
    return exact


def check_batch(full_scores, next_tokens, ids, scores, tokens, dtype, top_n, draft_len, oracle_ids=None,
                key_scale: float = 1.0):
    """All queries of a batch; returns the fraction of ranks identical to the oracle."""
    B = full_scores.shape[0]
    exact = 0
    for b in range(B):
        try:
            exact += check_query(full_scores[b], next_tokens, ids[b], scores[b], tokens[b], dtype,
                                 top_n, draft_len, None if oracle_ids is None else oracle_ids[b], key_scale)
        except AssertionError as e:
            raise AssertionError(f"query {b}: {e}") from None
    return exact / float(B * top_n)


def check_query_filtered(s, next_tokens, g_ids, g_scores, g_tokens, dtype, top_n, draft_len, first_token):
    """First-token filter: the result must be the top-n of the rows whose first stored
    token is `first_token` (all rows when it is negative), padded with id -1 / -inf / -1."""
    g_ids = np.asarray(g_ids).astype(np.int64)
    rows = np.arange(s.shape[0]) if first_token < 0 else np.nonzero(next_tokens[:, 0] == first_token)[0]
    k = min(top_n, len(rows))
    assert np.all(g_ids[k:] == -1), f"expected {top_n - k} padding ids, got {g_ids[k:]}"
    assert np.all(np.isneginf(np.asarray(g_scores)[k:])) and np.all(np.asarray(g_tokens)[k:] == -1)
    if k == 0:
        return 0
    pos = np.searchsorted(rows, g_ids[:k])
    assert np.all(pos < len(rows)) and np.all(rows[np.minimum(pos, len(rows) - 1)] == g_ids[:k]), \
        f"a returned row does not start with token {first_token}: {g_ids[:k]}"
    return check_query(s[rows], next_tokens[rows], pos, np.asarray(g_scores)[:k], np.asarray(g_tokens)[:k],
                       dtype, k, draft_len)

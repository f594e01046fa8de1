"""Parity at the benchmark's full sizes, in the launch configuration bench.py times.

The oracle needs several seconds per query on a 10M-row datastore, so full-size
runs are checked on a SAMPLE of the queries element by element (the same checker
as the small cases), and on ALL queries via properties that hold at any size:
ids distinct and in range, scores non-increasing, tokens equal to the stored
continuation of the returned id, and every returned score equal to the oracle's
score of that row (computed row by row for the returned ids only).
"""
import numpy as np
import pytest

import oracle
from paper_2502_15572_b200 import binding, synth
from tests import checker
from tests.gpu_util import gpu_store

pytestmark = pytest.mark.gpu


def _row_scores(keys, dtype, qhat, ids):
    """Oracle scores of selected rows only (float64, exact decode)."""
    return oracle.scores(keys[ids], dtype, qhat)


def _properties(keys, toks, dtype, q, ids, sc, tok, n, L):
    N = keys.shape[0]
    tol = checker.TOL[dtype]
    qh = oracle.preprocess(q, dtype)
    for b in range(q.shape[0]):
        assert np.all((ids[b] >= 0) & (ids[b] < N)) and len(set(ids[b].tolist())) == n
        assert np.all(np.diff(sc[b]) <= 0)
        assert np.array_equal(tok[b], toks[ids[b]][:, :L])
        want = _row_scores(keys, dtype, qh[b], ids[b])
        assert np.max(np.abs(want - sc[b])) <= tol


_CACHE = {}


def _workload(name):
    """The named workload; the last one made stays in memory for the next test that asks for it."""
    if name not in _CACHE:
        _CACHE.clear()
        _CACHE[name] = synth.make_workload(name)
    return _CACHE[name]


def _sampled_parity(w, sample, q=None):
    import torch
    keys, toks, dtype = w["keys"], w["next_tokens"], w["dtype"]
    n, L, B = w["top_n"], w["draft_len"], w["B"]
    q = w["queries"] if q is None else q
    st = gpu_store(keys, toks, dtype)
    dq = binding.to_device(q, dtype)
    outs = []
    for j in range(0, q.shape[0], B):                      # batches exactly as bench.py issues them
        ids, sc, tok = st.retrieve(dq[j:j + B], n, L)
        outs.append((ids.cpu().numpy(), sc.cpu().numpy(), tok.cpu().numpy()))
    torch.cuda.synchronize()
    st.status()
    st.close()
    ids = np.concatenate([o[0] for o in outs])
    sc = np.concatenate([o[1] for o in outs])
    tok = np.concatenate([o[2] for o in outs])
    _properties(keys, toks, dtype, q, ids, sc, tok, n, L)
    o = oracle.retrieve(keys, toks, dtype, q[sample], n, L, want_full_scores=True,
                        threads=oracle.dresd_oracle.default_threads())
    rate = checker.check_batch(o.full_scores, toks, ids[sample], sc[sample], tok[sample], dtype, n, L,
                               oracle_ids=o.ids)
    return rate


def test_config2_decode_batch1_full_size():
    """10M x 256 fp16, single queries: 64 calls checked by properties, 3 against the oracle."""
    w = _workload("c2_decode_b1_f16")
    q, _ = synth.make_queries(w["seed"] + 100, w["keys"], "f16", 64, w["sigma"])
    rate = _sampled_parity(w, sample=[0, 17, 63], q=q)
    assert rate >= 0.9


def test_config2_quantised_full_size():
    """10M x 256 fp16, single queries through the quantised search (8-bit candidates, exact
    re-ranking of 32), as `bench.py --quantised 32` issues them: 32 calls checked by
    properties (rows distinct and in range, exact scores in order, stored tokens), 3 against
    the oracle's statement of the same rules, and the recall of the exact path's rows."""
    import torch
    w = _workload("c2_decode_b1_f16")
    keys, toks, dtype, n, L, m = w["keys"], w["next_tokens"], "f16", w["top_n"], w["draft_len"], 32
    q, _ = synth.make_queries(w["seed"] + 200, keys, dtype, 32, w["sigma"])
    st = gpu_store(keys, toks, dtype)
    try:
        st.attach_quantised()
        dq = binding.to_device(q, dtype)
        outs, exact_ids = [], []
        for j in range(q.shape[0]):
            o = st.retrieve_quantised(dq[j:j + 1], n, L, m)
            outs.append([t.cpu().numpy() for t in o])
            exact_ids.append(st.retrieve(dq[j:j + 1], n, L)[0].cpu().numpy())
        torch.cuda.synchronize()
        st.status()
    finally:
        st.close()
    ids = np.concatenate([o[0] for o in outs])
    sc = np.concatenate([o[1] for o in outs])
    tok = np.concatenate([o[2] for o in outs])
    _properties(keys, toks, dtype, q, ids, sc, tok, n, L)
    recall = np.mean([len(set(a.tolist()) & set(b[0].tolist())) / n for a, b in zip(ids, exact_ids)])
    assert recall >= 0.95
    sample = [0, 13, 31]
    _, _, _, approx, exact = oracle.retrieve_quantised(keys, toks, dtype, q[sample], n, L, m,
                                                       threads=oracle.dresd_oracle.default_threads())
    for k, b in enumerate(sample):
        cut = np.sort(approx[k])[-m]
        got = ids[b]
        assert np.all(approx[k][got] >= cut - 5e-4)
        safe = np.flatnonzero(approx[k] >= cut + 5e-4)
        nth = exact[k][got[-1]]
        assert not [i for i in safe if exact[k][i] > nth + 2e-5 and i not in set(got.tolist())]


def test_config3_batched_full_size():
    """10M x 256 bf16, one batch of 64 (tensor-core kernel with its probe pass): 3 queries against the oracle."""
    w = synth.make_workload("c3_batched_bf16")
    rate = _sampled_parity(w, sample=[0, 31, 63])
    assert rate >= 0.9


def test_config4_large_full_size():
    """50M x 128 fp16 (12.8 GB of keys, the largest row count of the configurations), one batch
    of 4 as bench.py issues it: all 4 queries by properties and against the oracle's full result."""
    _CACHE.clear()
    w = synth.make_workload("c4_large_f16")
    rate = _sampled_parity(w, sample=[0, 1, 2, 3])
    assert rate >= 0.9


def test_config5a_unreduced_full_size():
    """4M x 4096 bf16 (32.8 GB of keys, 8 KB rows: the query operand travels with every key slab,
    64 slabs per row, the largest byte offsets of the configurations), one batch of 16, no
    projection: all 16 queries by properties, 4 of them against the oracle's full result."""
    _CACHE.clear()
    w = synth.make_workload("c5a_hidden_bf16")
    rate = _sampled_parity(w, sample=[0, 5, 10, 15])
    assert rate >= 0.9


def test_config5b_projected_full_size():
    """4M x 256 bf16 with the 4096 -> 256 projection, batch 16: all 16 queries against the oracle."""
    import torch
    w = synth.make_workload("c5b_projected_bf16")
    keys, toks, dtype, n, L = w["keys"], w["next_tokens"], w["dtype"], w["top_n"], w["draft_len"]
    st = gpu_store(keys, toks, dtype)
    dW = binding.to_device(w["W"], dtype)
    st.set_preprocess(w["d_in"], W=dW)
    ids, sc, tok = st.retrieve(binding.to_device(w["queries"], dtype), n, L)
    torch.cuda.synchronize()
    st.status()
    ids, sc, tok = ids.cpu().numpy(), sc.cpu().numpy(), tok.cpu().numpy()
    st.close()
    o = oracle.retrieve(keys, toks, dtype, w["queries"], n, L, W=w["W"], want_full_scores=True,
                        threads=oracle.dresd_oracle.default_threads())
    rate = checker.check_batch(o.full_scores, toks, ids, sc, tok, dtype, n, L, oracle_ids=o.ids)
    assert rate >= 0.9


def test_paper_shaped_sorted_store_full_size():
    """46.3M x 64 fp16 with its rows sorted by first stored token, as
    `bench.py --workload paper_46m_d64_f16 --first-token-filter --sorted-store` issues them:
    24 single-query calls and 2 calls of 16, each scanning only its tokens' rows.  Every call
    must equal the filtered scan of the whole store bit for bit; all rows carry the wanted
    token, distinct, scores in order and equal to the oracle's score of the row, tokens the
    stored ones; 2 queries element by element against the oracle's filtered search."""
    import torch
    _CACHE.clear()
    w = synth.make_workload("paper_46m_d64_f16")
    dtype, n, L = "f16", w["top_n"], w["draft_len"]
    q, src = synth.make_queries(w["seed"] + 300, w["keys"], dtype, 56, w["sigma"])
    ft = np.ascontiguousarray(w["next_tokens"][src, 0]).astype(np.int32)
    keys, toks = synth.sort_by_first_token(w["keys"], w["next_tokens"])
    del w
    st = gpu_store(keys, toks, dtype)
    try:
        st.index_first_tokens()
        dq, dft = binding.to_device(q, dtype), torch.from_numpy(ft).cuda()
        calls = [(j, j + 1) for j in range(24)] + [(24, 40), (40, 56)]
        outs = []
        for a, b in calls:
            st.set_option("first_token_windows", 1)
            win = [t.clone() for t in st.retrieve_filtered(dq[a:b], dft[a:b], n, L)]
            st.set_option("first_token_windows", 0)
            full = st.retrieve_filtered(dq[a:b], dft[a:b], n, L)
            torch.cuda.synchronize()
            for x, y in zip(win, full):
                assert torch.equal(x, y)
            outs.append([t.cpu().numpy() for t in win])
        st.status()
    finally:
        st.close()
    ids = np.concatenate([o[0] for o in outs])
    sc = np.concatenate([o[1] for o in outs])
    tok = np.concatenate([o[2] for o in outs])
    qh = oracle.preprocess(q, dtype)
    for b in range(q.shape[0]):
        k = int(np.sum(ids[b] >= 0))
        assert k == min(n, int(np.sum(toks[:, 0] == ft[b]))) and np.all(ids[b, k:] == -1)
        got = ids[b, :k]
        assert len(set(got.tolist())) == k and np.all(toks[got, 0] == ft[b])
        assert np.all(np.diff(sc[b, :k]) <= 0) and np.array_equal(tok[b, :k], toks[got][:, :L])
        assert np.max(np.abs(_row_scores(keys, dtype, qh[b], got) - sc[b, :k])) <= checker.TOL[dtype]
    sample = [3, 30]
    o = oracle.retrieve(keys, toks, dtype, q[sample], n, L, first_token=ft[sample], want_full_scores=True,
                        threads=oracle.dresd_oracle.default_threads())
    for k, b in enumerate(sample):
        checker.check_query_filtered(o.full_scores[k], toks, ids[b], sc[b], tok[b], dtype, n, L, int(ft[b]))

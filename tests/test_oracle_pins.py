"""Pins for the CPU oracle: hand cases, closed forms, brute force, invariants.

Everything here runs without a GPU.  The oracle is checked against values
worked out by hand from the paper's formulas (tests/golden/hand_cases.json),
against closed forms that the mathematics fixes, against an independent
float64 numpy formulation on small inputs, and against the invariants of
exact nearest-neighbour search.
"""
import json
import os

import numpy as np
import pytest

import oracle
from paper_2502_15572_b200 import synth

HERE = os.path.dirname(os.path.abspath(__file__))
with open(os.path.join(HERE, "golden", "hand_cases.json")) as f:
    GOLDEN = json.load(f)


def _tokens(N, L):
    return (100 * np.arange(N, dtype=np.int32)[:, None] + np.arange(L, dtype=np.int32)[None, :])


# --------------------------------------------------------------------------
# bit decoders
# --------------------------------------------------------------------------
@pytest.mark.parametrize("bits,dtype,value", [
    (0x3C00, "f16", 1.0), (0x0001, "f16", 2.0 ** -24), (0x7BFF, "f16", 65504.0),
    (0xC000, "f16", -2.0), (0x3555, "f16", 0.333251953125), (0x0400, "f16", 2.0 ** -14),
    (0x8000, "f16", 0.0),
    (0x3F80, "bf16", 1.0), (0x4049, "bf16", 3.140625), (0xBF00, "bf16", -0.5),
    (0x0080, "bf16", 2.0 ** -126), (0x0001, "bf16", 2.0 ** -133),
    (0x3F800000, "f32", 1.0), (0xC0490FDB, "f32", float(np.float32(-3.14159274))),
])
def test_decode_known_patterns(bits, dtype, value):
    assert oracle.decode(bits, dtype) == value


def test_decode_all_16bit_patterns_match_ieee():
    bits = np.arange(65536, dtype=np.uint32)
    want16 = bits.astype(np.uint16).view(np.float16).astype(np.float64)
    wantbf = (bits << np.uint32(16)).view(np.float32).astype(np.float64)
    for b in range(0, 65536, 1):
        g16 = oracle.decode(b, "f16")
        gbf = oracle.decode(b, "bf16")
        for got, want in ((g16, want16[b]), (gbf, wantbf[b])):
            if np.isnan(want):
                assert np.isnan(got)
            else:
                assert got == want and np.signbit(got) == np.signbit(want)


# --------------------------------------------------------------------------
# preprocessing: Eq. 1 -> projection -> Eq. 2
# --------------------------------------------------------------------------
@pytest.mark.parametrize("case", GOLDEN["preprocess"], ids=lambda c: c["cite"])
def test_preprocess_hand_cases(case):
    v = np.array([case["v"]], dtype=np.float32)
    W = None if case["W"] is None else np.array(case["W"], dtype=np.float32)
    got = oracle.preprocess(v, "f32", mean=case["mean"], var=case["var"], eps_z=case["eps_z"],
                            W=W, pca_mean=case["pca_mean"])
    np.testing.assert_allclose(got[0], case["qhat"], atol=1.5e-6, rtol=0)


def test_preprocess_closed_forms():
    rng = np.random.default_rng(5)
    v = rng.standard_normal((6, 40)).astype(np.float32)
    q = oracle.preprocess(v, "f32")
    # unit length
    np.testing.assert_allclose(np.linalg.norm(q, axis=1), 1.0, atol=1e-14)
    # scale invariance (powers of two keep the scaled input exactly representable)
    q4 = oracle.preprocess((4.0 * v).astype(np.float32), "f32")
    np.testing.assert_allclose(q4, q, atol=1e-15)
    # direction is preserved
    v64 = v.astype(np.float64)
    np.testing.assert_allclose(q, v64 / np.linalg.norm(v64, axis=1, keepdims=True), atol=1e-15)
    # identity projection changes nothing
    qi = oracle.preprocess(v, "f32", W=np.eye(40, dtype=np.float32))
    np.testing.assert_allclose(qi, q, atol=1e-15)
    # a permutation matrix permutes coordinates
    perm = rng.permutation(40)
    P = np.zeros((40, 40), dtype=np.float32)
    P[perm, np.arange(40)] = 1.0            # (vP)[c] = v[perm[c]]
    qp = oracle.preprocess(v, "f32", W=P)
    np.testing.assert_allclose(qp, q[:, perm], atol=1e-15)


def test_preprocess_epsilon_guards():
    z = np.zeros((1, 8), dtype=np.float32)
    assert np.all(oracle.preprocess(z, "f32") == 0.0)             # 0 / max(0, eps) = 0
    tiny = np.zeros((1, 4), dtype=np.float32)
    tiny[0, 0] = 1e-20
    got = oracle.preprocess(tiny, "f32", eps_n=1e-12)
    assert got[0, 0] == pytest.approx(float(np.float32(1e-20)) / 1e-12, rel=1e-12)
    got = oracle.preprocess(tiny, "f32", eps_n=1e-30)
    assert got[0, 0] == pytest.approx(1.0, rel=1e-12)


@pytest.mark.parametrize("dtype", ["f32", "f16", "bf16"])
def test_preprocess_matches_numpy_float64(dtype):
    d_in, d, B = 96, 24, 5
    mean, var, W = synth.make_preprocess(11, d_in, d, dtype)
    q = synth.make_hidden_queries(12, B, d_in, dtype)
    pm = (0.1 * np.arange(d_in)).astype(np.float32)
    got = oracle.preprocess(q, dtype, mean=mean, var=var, eps_z=1e-5, W=W, pca_mean=pm)
    q64 = synth.store_to_float32(q, dtype).astype(np.float64)
    W64 = synth.store_to_float32(W, dtype).astype(np.float64)
    z = (q64 - mean.astype(np.float64)) / np.sqrt(var.astype(np.float64) + 1e-5)
    vl = (z - pm.astype(np.float64)) @ W64
    want = vl / np.maximum(np.linalg.norm(vl, axis=1, keepdims=True), 1e-12)
    np.testing.assert_allclose(got, want, atol=1e-13)


# --------------------------------------------------------------------------
# scoring + selection + lookup
# --------------------------------------------------------------------------
@pytest.mark.parametrize("case", GOLDEN["retrieve"], ids=lambda c: c["derivation"][:30])
def test_retrieve_hand_cases(case):
    keys = np.array(case["keys"], dtype=np.float32)
    toks = _tokens(len(keys), 3)
    r = oracle.retrieve(keys, toks, "f32", np.array([case["query"]], dtype=np.float32),
                        top_n=case["top_n"], draft_len=2)
    assert r.ids[0].tolist() == case["ids"]
    np.testing.assert_allclose(r.scores[0], case["scores"], atol=1.5e-6, rtol=0)
    assert r.tokens[0].tolist() == [[100 * i, 100 * i + 1] for i in case["ids"]]


def test_identity_keys():
    d = 16
    keys = np.eye(d, dtype=np.float32)
    toks = _tokens(d, 4)
    for j in (0, 5, 15):
        q = np.zeros((1, d), dtype=np.float32)
        q[0, j] = 3.0
        r = oracle.retrieve(keys, toks, "f32", q, top_n=4, draft_len=4)
        others = [i for i in range(d) if i != j][:3]
        assert r.ids[0].tolist() == [j] + others
        assert r.scores[0].tolist() == [1.0, 0.0, 0.0, 0.0]
        assert r.tokens[0, 0].tolist() == [100 * j + t for t in range(4)]


def test_zero_query_returns_lowest_ids():
    keys, toks = synth.make_store(3, 50, 8, 4, "f32", 3)
    r = oracle.retrieve(keys, toks, "f32", np.zeros((1, 8), dtype=np.float32), top_n=5, draft_len=3)
    assert r.ids[0].tolist() == [0, 1, 2, 3, 4]
    assert np.all(r.scores == 0.0)


@pytest.mark.parametrize("dtype", ["f32", "f16", "bf16"])
def test_matches_independent_numpy_bruteforce(dtype):
    N, d, B, n, L = 700, 24, 6, 9, 5
    keys, toks = synth.make_store(21, N, d, 8, dtype, 7)
    q, _ = synth.make_queries(22, keys, dtype, B, 0.1)
    r = oracle.retrieve(keys, toks, dtype, q, top_n=n, draft_len=L, want_full_scores=True)
    K = synth.store_to_float32(keys, dtype).astype(np.float64)
    Q = synth.store_to_float32(q, dtype).astype(np.float64)
    Q = Q / np.linalg.norm(Q, axis=1, keepdims=True)
    S = Q @ K.T
    np.testing.assert_allclose(r.full_scores, S, atol=1e-14)
    for b in range(B):
        order = np.argsort(-S[b], kind="stable")[:n]
        assert r.ids[b].tolist() == order.tolist()
        np.testing.assert_allclose(r.scores[b], S[b, order], atol=1e-14)
        assert np.array_equal(r.tokens[b], toks[order][:, :L])
        assert np.all(np.diff(r.scores[b]) <= 0)


def test_self_retrieval_and_mrr():
    # Eq. 4: with exact search over distinct unit keys every key finds itself first.
    for dtype, tol in (("f32", 1e-6), ("f16", 2.0 ** -10), ("bf16", 2.0 ** -7)):
        keys, toks = synth.make_store(31, 400, 32, 6, dtype, 4)
        idx = np.arange(0, 400, 13)
        r = oracle.retrieve(keys, toks, dtype, keys[idx], top_n=3, draft_len=4,
                            want_full_scores=True)
        rr = []
        for b, i in enumerate(idx):
            rank = 1 + int(np.sum(r.full_scores[b] > r.full_scores[b, i]))
            rr.append(1.0 / rank)
        assert np.mean(rr) == 1.0
        assert r.ids[:, 0].tolist() == idx.tolist()
        K = synth.store_to_float32(keys, dtype).astype(np.float64)
        np.testing.assert_allclose(r.scores[:, 0], np.linalg.norm(K[idx], axis=1), atol=1e-14)
        np.testing.assert_allclose(r.scores[:, 0], 1.0, atol=tol)


def test_cauchy_schwarz_bound():
    keys, toks = synth.make_store(41, 300, 16, 4, "f16", 2)
    q, _ = synth.make_queries(42, keys, "f16", 3, 0.3)
    r = oracle.retrieve(keys, toks, "f16", q, top_n=1, draft_len=1, want_full_scores=True)
    K = synth.store_to_float32(keys, "f16").astype(np.float64)
    assert np.all(np.abs(r.full_scores) <= np.linalg.norm(K, axis=1)[None, :] + 1e-14)


def test_permutation_invariance():
    N = 500
    keys, toks = synth.make_store(51, N, 16, 5, "f32", 6)
    q, _ = synth.make_queries(52, keys, "f32", 4, 0.1)
    r0 = oracle.retrieve(keys, toks, "f32", q, top_n=8, draft_len=6)
    perm = np.random.default_rng(53).permutation(N)     # new row p holds old row perm[p]
    r1 = oracle.retrieve(keys[perm], toks[perm], "f32", q, top_n=8, draft_len=6)
    assert np.array_equal(perm[r1.ids], r0.ids)
    assert np.array_equal(r1.scores, r0.scores)         # per-row arithmetic is position-free
    assert np.array_equal(r1.tokens, r0.tokens)


def test_shard_merge_equals_whole():
    N, n = 600, 7
    keys, toks = synth.make_store(61, N, 16, 5, "bf16", 5)
    q, _ = synth.make_queries(62, keys, "bf16", 3, 0.1)
    whole = oracle.retrieve(keys, toks, "bf16", q, top_n=n, draft_len=5)
    cut = 233
    a = oracle.retrieve(keys[:cut], toks[:cut], "bf16", q, top_n=n, draft_len=5)
    b = oracle.retrieve(keys[cut:], toks[cut:], "bf16", q, top_n=n, draft_len=5)
    for i in range(3):
        ids = np.concatenate([a.ids[i], b.ids[i] + cut])
        sc = np.concatenate([a.scores[i], b.scores[i]])
        tk = np.concatenate([a.tokens[i], b.tokens[i]])
        order = np.lexsort((ids, -sc))[:n]
        assert np.array_equal(ids[order], whole.ids[i])
        assert np.array_equal(sc[order], whole.scores[i])
        assert np.array_equal(tk[order], whole.tokens[i])


def test_prefix_properties_and_duplicates():
    N = 300
    keys, toks = synth.make_store(71, N, 16, 5, "f32", 8)
    keys[200] = keys[17]                      # exact duplicate rows: lower id first, adjacent
    q = keys[17:18].copy()
    big = oracle.retrieve(keys, toks, "f32", q, top_n=12, draft_len=8)
    small = oracle.retrieve(keys, toks, "f32", q, top_n=5, draft_len=3)
    assert np.array_equal(big.ids[:, :5], small.ids)
    assert np.array_equal(big.tokens[:, :5, :3], small.tokens)
    assert big.ids[0, :2].tolist() == [17, 200]
    assert big.scores[0, 0] == big.scores[0, 1]


def test_batch_equals_single_queries():
    keys, toks = synth.make_store(81, 256, 16, 4, "f16", 4)
    q, _ = synth.make_queries(82, keys, "f16", 5, 0.1)
    allq = oracle.retrieve(keys, toks, "f16", q, top_n=6, draft_len=4)
    for b in range(5):
        one = oracle.retrieve(keys, toks, "f16", q[b:b + 1], top_n=6, draft_len=4)
        assert np.array_equal(one.ids[0], allq.ids[b])
        assert np.array_equal(one.scores[0], allq.scores[b])


def test_row_threads_do_not_change_scores():
    keys, _ = synth.make_store(91, 5000, 32, 4, "bf16", 1)
    qh = oracle.preprocess(keys[:1], "bf16")[0]
    assert np.array_equal(oracle.scores(keys, "bf16", qh, threads=1),
                          oracle.scores(keys, "bf16", qh, threads=4))


def test_projected_retrieval_end_to_end_matches_two_steps():
    d_in, d, N = 48, 16, 200
    keys, toks = synth.make_store(101, N, d, 4, "bf16", 3)
    mean, var, W = synth.make_preprocess(102, d_in, d, "bf16")
    q = synth.make_hidden_queries(103, 3, d_in, "bf16")
    r = oracle.retrieve(keys, toks, "bf16", q, top_n=4, draft_len=3, mean=mean, var=var, W=W,
                        want_full_scores=True)
    qh = oracle.preprocess(q, "bf16", mean=mean, var=var, W=W)
    for b in range(3):
        assert np.array_equal(r.full_scores[b], oracle.scores(keys, "bf16", qh[b]))


def test_bad_arguments_raise():
    keys, toks = synth.make_store(111, 20, 8, 2, "f32", 4)
    q = keys[:1]
    with pytest.raises(ValueError):
        oracle.retrieve(keys, toks, "f32", q, top_n=21, draft_len=2)
    with pytest.raises(ValueError):
        oracle.retrieve(keys, toks, "f32", q, top_n=0, draft_len=2)
    with pytest.raises(ValueError):
        oracle.retrieve(keys, toks, "f32", q, top_n=2, draft_len=5)
    with pytest.raises(ValueError):
        oracle.retrieve(keys, toks, "f32", q[:, :4], top_n=2, draft_len=2)


# --------------------------------------------------------------------------
# first-token filter (Sections 3.1 / 3.5)
# --------------------------------------------------------------------------
def test_first_token_filter_hand_case():
    # keys k0..k3 as in the golden cases; unit query (1,0) scores (1, 0, 0.6, -1).
    keys = np.array([[1.0, 0.0], [0.0, 1.0], [0.6, 0.8], [-1.0, 0.0]], dtype=np.float32)
    toks = np.array([[7, 1], [5, 2], [5, 3], [5, 4]], dtype=np.int32)
    q = np.array([[2.0, 0.0]], dtype=np.float32)
    r = oracle.retrieve(keys, toks, "f32", q, top_n=3, draft_len=2, first_token=[5])
    assert r.ids[0].tolist() == [2, 1, 3]                       # k0 starts with 7: ruled out
    np.testing.assert_allclose(r.scores[0], [0.6, 0.0, -1.0], atol=1e-7)
    assert r.tokens[0].tolist() == [[5, 3], [5, 2], [5, 4]]
    r = oracle.retrieve(keys, toks, "f32", q, top_n=3, draft_len=2, first_token=[7])
    assert r.ids[0].tolist() == [0, -1, -1]                     # one match only: padded
    assert r.scores[0, 0] == 1.0 and np.all(np.isneginf(r.scores[0, 1:]))
    assert r.tokens[0].tolist() == [[7, 1], [-1, -1], [-1, -1]]
    r = oracle.retrieve(keys, toks, "f32", q, top_n=3, draft_len=2, first_token=[-1])
    assert r.ids[0].tolist() == [0, 2, 1]                       # -1 = no filter


def test_first_token_filter_equals_search_of_the_matching_subset():
    N, d, B, n = 800, 16, 5, 6
    keys, toks = synth.make_store(131, N, d, 6, "f16", 4, vocab=7)
    q, _ = synth.make_queries(132, keys, "f16", B, 0.1)
    ft = np.array([0, 1, 2, 6, -1], dtype=np.int32)
    got = oracle.retrieve(keys, toks, "f16", q, top_n=n, draft_len=4, first_token=ft)
    for b in range(B):
        rows = np.arange(N) if ft[b] < 0 else np.nonzero(toks[:, 0] == ft[b])[0]
        k = min(n, len(rows))
        sub = oracle.retrieve(keys[rows], toks[rows], "f16", q[b:b + 1], top_n=k, draft_len=4)
        assert np.array_equal(got.ids[b, :k], rows[sub.ids[0]])
        assert np.array_equal(got.scores[b, :k], sub.scores[0])
        assert np.array_equal(got.tokens[b, :k], sub.tokens[0])
        assert np.all(got.ids[b, k:] == -1) and np.all(np.isneginf(got.scores[b, k:]))
        if ft[b] >= 0:
            assert np.all(got.tokens[b, :k, 0] == ft[b])


# --------------------------------------------------------------------------
# statistics of Eq. 1 (Section 3.2): E[V], Var[V] from a sample
# --------------------------------------------------------------------------
def _as_store(a, dtype):
    return synth.cast_to_store(np.asarray(a, dtype=np.float32), dtype)


@pytest.mark.parametrize("case", GOLDEN["fit_zscore"], ids=lambda c: c["cite"])
def test_fit_zscore_hand_cases(case):
    for dtype in case.get("dtypes", ["f32", "f16", "bf16"]):
        mean, var = oracle.fit_zscore(_as_store(case["V"], dtype), dtype)
        np.testing.assert_allclose(mean, case["mean"], rtol=0, atol=1e-12)
        np.testing.assert_allclose(var, case["var"], rtol=1e-12, atol=1e-12)


def test_fit_zscore_closed_forms():
    # 0..N-1 in one column: mean (N-1)/2, population variance (N^2-1)/12
    N = 1000
    V = np.stack([np.arange(N), 3.0 - 2.0 * np.arange(N)], axis=1).astype(np.float32)
    mean, var = oracle.fit_zscore(V, "f32")
    np.testing.assert_allclose(mean, [(N - 1) / 2, 3.0 - (N - 1)], rtol=1e-14)
    np.testing.assert_allclose(var, [(N * N - 1) / 12, 4 * (N * N - 1) / 12], rtol=1e-13)
    # +-1 alternating: mean 0, variance 1; a constant shift moves the mean only
    pm = np.where(np.arange(64) % 2 == 0, 1.0, -1.0).astype(np.float32)[:, None]
    for shift in (0.0, 512.0):
        mean, var = oracle.fit_zscore(_as_store(pm + shift, "f16"), "f16")
        assert mean[0] == shift and var[0] == 1.0


def test_fit_zscore_then_eq1_standardises_the_sample():
    """Feeding the fitted statistics to Eq. 1 gives the sample mean 0 and variance
    Var/(Var + eps) per dimension: the definition the statistics exist for."""
    rng = np.random.default_rng(77)
    V = (rng.normal(size=(500, 6)) * np.array([0.1, 1, 5, 20, 1, 1]) + np.array([0, 3, -7, 40, 0, 0])).astype(np.float32)
    Vs = _as_store(V, "bf16")
    mean, var = oracle.fit_zscore(Vs, "bf16")
    x = synth.store_to_float32(Vs, "bf16").astype(np.float64)
    eps = 1e-5
    z = (x - mean) / np.sqrt(var + eps)
    np.testing.assert_allclose(z.mean(axis=0), 0.0, atol=1e-12)
    np.testing.assert_allclose((z * z).mean(axis=0), var / (var + eps), rtol=1e-12)
    # row order and duplication of the whole sample change nothing
    m2, v2 = oracle.fit_zscore(np.concatenate([Vs[::-1], Vs]), "bf16")
    np.testing.assert_allclose(m2, mean, rtol=1e-13, atol=1e-13)
    np.testing.assert_allclose(v2, var, rtol=1e-12)


def test_fit_zscore_bad_arguments():
    with pytest.raises(ValueError):
        oracle.fit_zscore(np.zeros((0, 4), dtype=np.float32), "f32")


# --------------------------------------------------------------------------
# quantised candidate search: E4M3 codes, approximate scores, re-ranking
# --------------------------------------------------------------------------
def test_e4m3_decode_all_codes_match_the_format_definition():
    """1 sign, 4 exponent bits (bias 7), 3 mantissa bits; exponent 0 is subnormal; only
    S.1111.111 is NaN (the format has no infinities), so the largest finite value is 448."""
    for code in range(256):
        s, e, m = code >> 7, (code >> 3) & 15, code & 7
        got = oracle.e4m3_decode(code)
        if e == 15 and m == 7:
            assert np.isnan(got)
            continue
        want = (m / 8.0) * 2.0 ** -6 if e == 0 else (1 + m / 8.0) * 2.0 ** (e - 7)
        assert got == (-want if s else want)
    assert oracle.e4m3_decode(0x7E) == 448.0 and oracle.e4m3_decode(0x01) == 2.0 ** -9
    assert oracle.e4m3_decode(0x38) == 1.0 and oracle.e4m3_decode(0xB8) == -1.0


def test_e4m3_encode_known_values_ties_and_saturation():
    enc, dec = oracle.e4m3_encode, oracle.e4m3_decode
    for code in range(256):                              # every finite code encodes back to itself
        if (code & 0x7F) != 0x7F:
            assert enc(dec(code)) == code
    assert enc(1.0) == 0x38 and enc(-2.0) == 0xC0 and enc(448.0) == 0x7E
    assert enc(1e6) == 0x7E and enc(-1e6) == 0xFE and enc(449.0) == 0x7E      # saturating, never NaN
    assert enc(float("nan")) & 0x7F == 0x7F
    # ties go to the even mantissa: 1.0625 is halfway between 1.0 (m=0) and 1.125 (m=1)
    assert enc(1.0625) == 0x38 and enc(1.1875) == 0x3A        # 1.1875: between 1.125 (m=1) and 1.25 (m=2)
    assert enc(1.0626) == 0x39 and enc(1.0624) == 0x38
    # below half of the smallest subnormal (2^-10) -> 0; exactly half -> 0 (even); just above -> 2^-9
    assert enc(2.0 ** -10) == 0x00 and enc(2.0 ** -10 * 1.001) == 0x01 and enc(2.0 ** -11) == 0x00
    # monotone
    xs = np.linspace(-500, 500, 20001)
    codes = np.array([dec(enc(x)) for x in xs])
    assert np.all(np.diff(codes) >= 0)


def test_e4m3_encode_matches_an_independent_library_conversion():
    torch = pytest.importorskip("torch")
    if not hasattr(torch, "float8_e4m3fn"):
        pytest.skip("this torch has no float8_e4m3fn")
    rng = np.random.default_rng(5)
    x = np.concatenate([rng.normal(size=4000) * 20, rng.normal(size=2000) * 0.01, rng.uniform(-448, 448, 2000),
                        np.array([0.0, 448.0, -448.0, 2.0 ** -9, 2.0 ** -10 * 3])]).astype(np.float32)
    want = torch.from_numpy(x).to(torch.float8_e4m3fn).to(torch.float32).numpy()
    got = np.array([oracle.e4m3_decode(oracle.e4m3_encode(float(v))) for v in x], dtype=np.float32)
    assert np.array_equal(got, want)


def test_quantised_scores_hand_case_and_exactly_representable_inputs():
    # keys and query whose 256-fold multiples are E4M3 values: the approximate score is the exact one
    keys = np.array([[0.5, 0.25, 0.0, -0.125], [1.0, 0.0, 0.0, 0.0], [0.0, -0.75, 0.5, 0.5]], dtype=np.float32)
    q = np.array([0.5, -0.5, 0.25, 0.0])
    a = oracle.quantised_scores(keys, "f32", q)
    np.testing.assert_allclose(a, keys.astype(np.float64) @ q, rtol=0, atol=1e-15)
    # hand case with rounding: k = 0.3 -> 76.8 -> e4m3 80 (grid step 8 above 64); q = 0.3:
    # h1 = 80, residual -3.2 -> 16 * -3.2 = -51.2 -> e4m3 -52 (step 4 above 32) -> q ~ 80 - 52/16 = 76.75
    a = oracle.quantised_scores(np.array([[0.3]], dtype=np.float32), "f32", np.array([0.3]))
    np.testing.assert_allclose(a, [76.75 * 80 / 65536], rtol=1e-12)


def test_quantised_scores_are_close_to_exact_and_reranking_recovers_the_neighbours():
    dtype, N, d = "bf16", 6000, 64
    keys, toks = synth.make_store(910, N, d, 8, dtype, 3)
    q, _ = synth.make_queries(911, keys, dtype, 4, 0.1)
    ids, sc, tok, approx, exact = oracle.retrieve_quantised(keys, toks, dtype, q, 5, 3, 40)
    # error model: keys carry 3 mantissa bits (relative error <= 2^-4 per element), the query two terms
    assert np.max(np.abs(approx - exact)) < 0.02
    ref = oracle.retrieve(keys, toks, dtype, q, 5, 3)
    assert np.mean(ids == ref.ids) >= 0.9                   # recall of the exact neighbours on this easy store
    # with every row a candidate the result IS the exact one
    ids_all, sc_all, tok_all, _, _ = oracle.retrieve_quantised(keys, toks, dtype, q, 5, 3, N)
    assert np.array_equal(ids_all, ref.ids) and np.array_equal(tok_all, ref.tokens)
    np.testing.assert_allclose(sc_all, ref.scores, rtol=0, atol=1e-12)
    # the returned rows are candidates, sorted by exact score, tokens copied verbatim
    for b in range(4):
        cut = np.sort(approx[b])[-40]
        assert np.all(approx[b][ids[b]] >= cut)
        assert np.all(np.diff(sc[b]) <= 0)
        assert np.array_equal(tok[b], toks[ids[b], :3])


def test_quantised_first_token_filter_equals_search_of_the_matching_subset():
    dtype, N, d = "f16", 3000, 64
    keys, toks = synth.make_store(920, N, d, 8, dtype, 3)
    q, _ = synth.make_queries(921, keys, dtype, 3, 0.1)
    vals, counts = np.unique(toks[:, 0], return_counts=True)
    common = int(vals[np.argmax(counts)])
    rare = int(vals[np.argmin(counts)])                       # fewer matches than top_n: padding
    ft = np.array([common, -1, rare], dtype=np.int32)
    ids, sc, tok, approx, exact = oracle.retrieve_quantised(keys, toks, dtype, q, 4, 3, 8, first_token=ft)
    for b, want in enumerate(ft):
        sub = np.arange(N) if want < 0 else np.flatnonzero(toks[:, 0] == want)
        m = min(8, len(sub))
        r = oracle.retrieve_quantised(keys[sub], toks[sub], dtype, q[b:b + 1], min(4, len(sub)), 3, m)
        k = min(4, len(sub))
        assert np.array_equal(ids[b, :k], sub[r[0][0]])
        np.testing.assert_allclose(sc[b, :k], r[1][0], rtol=0, atol=1e-12)
        assert np.array_equal(tok[b, :k], r[2][0])
        assert np.all(ids[b, k:] == -1) and np.all(sc[b, k:] == -np.inf) and np.all(tok[b, k:] == -1)
    assert np.sum(toks[:, 0] == rare) < 4                      # the padding case really occurred


def test_quantised_scores_match_an_independent_formulation():
    """The same three rules written with a library's E4M3 conversion and a float64 matmul."""
    torch = pytest.importorskip("torch")
    if not hasattr(torch, "float8_e4m3fn"):
        pytest.skip("this torch has no float8_e4m3fn")
    rng = np.random.default_rng(31)
    N, d = 500, 48
    keys = rng.normal(size=(N, d)).astype(np.float32)
    keys /= np.linalg.norm(keys, axis=1, keepdims=True)
    k16 = keys.astype(np.float16)                               # the store: fp16 bit patterns
    q = rng.normal(size=d).astype(np.float32)
    q /= np.linalg.norm(q)                                      # float32 values, handed over exactly
    f8 = lambda x: torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).to(torch.float8_e4m3fn).to(torch.float32).numpy().astype(np.float64)
    k8 = f8(k16.astype(np.float32) * 256.0)
    q256 = q.astype(np.float64) * 256.0
    h1 = f8(q256)
    h2 = f8((q256 - h1) * 16.0)
    want = k8 @ (h1 + h2 / 16.0) / 65536.0
    got = oracle.quantised_scores(k16, "f16", q.astype(np.float64))
    np.testing.assert_allclose(got, want, rtol=0, atol=1e-13)

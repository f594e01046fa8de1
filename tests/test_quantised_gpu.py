"""Quantised candidate search (8-bit E4M3 keys, approximate scores on the tensor cores, exact
re-ranking) against the oracle's statement of the same rules.

What is unique is compared exactly: the key codes byte for byte, and the final rows wherever
the candidate cut is not within rounding of a tie.  The GPU sums the exact 8-bit products in
fp32 and takes the unit query in fp32, the oracle in float64, so a row whose approximate score
is within DELTA of the m-th best may fall on either side of the cut."""
import numpy as np
import pytest

import oracle
from paper_2502_15572_b200 import binding, synth
from tests.gpu_util import gpu_store

pytestmark = pytest.mark.gpu

# Approximate scores: sums of <= 2 d exact products accumulated in fp32 (relative 2^-24 each),
# plus, rarely, one query element whose fp32 value rounds to the neighbouring 8-bit code
# (one 8-bit step of one term: <= 2^-4 |q_j k_ij|, about 3e-4 at d >= 64 for unit vectors).
DELTA = 5e-4
SCORE_TOL = 2e-3            # final scores, as for the exact path on 16-bit keys
EPS_ACC = 1e-5              # exact scores closer than this may swap


def _codes(keys, dtype):
    x = synth.store_to_float32(keys, dtype).astype(np.float64) * 256.0
    flat = np.array([oracle.e4m3_encode(v) for v in np.unique(x)], dtype=np.uint8)
    lut = dict(zip(np.unique(x).tolist(), flat.tolist()))
    return np.vectorize(lut.get, otypes=[np.uint8])(x)


def test_key_quantiser_matches_the_oracle_codes_byte_for_byte():
    import torch
    for dtype in ("f16", "bf16"):
        keys, toks = synth.make_store(8000, 3001, 64, 8, dtype, 2)
        # add values that saturate, underflow and sit on ties
        special = np.array([2.0, -3.0, 1.75, 2.0 ** -18, -2.0 ** -17, 0.0, 1.0625 / 256, 0.5], dtype=np.float32)
        keys = keys.copy()
        keys[0, :8] = synth.cast_to_store(special[None, :], dtype)[0]
        dk = binding.to_device(keys, dtype)
        q8 = torch.empty((keys.shape[0], keys.shape[1]), dtype=torch.uint8, device="cuda")
        binding.dresd_quantise_keys(dk.data_ptr(), keys.shape[0], keys.shape[1], binding.DTYPE_CODE[dtype],
                                    q8.data_ptr(), torch.cuda.current_stream().cuda_stream)
        torch.cuda.synchronize()
        want = _codes(keys, dtype)
        got = q8.cpu().numpy()
        # -0.0 and +0.0 are the same value; compare values where the code differs only in the sign of zero
        diff = got != want
        assert np.all((got[diff] & 0x7F) == 0) and np.all((want[diff] & 0x7F) == 0)


def _check_against_oracle(keys, toks, dtype, q, n, L, m, pre=None):
    import torch
    pre = pre or {}
    st = gpu_store(keys, toks, dtype)
    try:
        if pre:
            dev = {k: (None if pre.get(k) is None else torch.from_numpy(np.asarray(pre[k], dtype=np.float32)).cuda())
                   for k in ("mean", "var", "pca_mean")}
            W = None if pre.get("W") is None else binding.to_device(pre["W"], dtype)
            st.set_preprocess(q.shape[1], dev["mean"], dev["var"], pre.get("eps_z", 1e-5), W, dev["pca_mean"])
        st.attach_quantised()
        ids, sc, tok = st.retrieve_quantised(binding.to_device(q, dtype), n, L, m)
        torch.cuda.synchronize()
        st.status()
        ids, sc, tok = ids.cpu().numpy(), sc.cpu().numpy(), tok.cpu().numpy()
        again = st.retrieve_quantised(binding.to_device(q, dtype), n, L, m)
        torch.cuda.synchronize()
        assert np.array_equal(again[0].cpu().numpy(), ids) and np.array_equal(again[1].cpu().numpy(), sc)
    finally:
        st.close()
    o_ids, o_sc, o_tok, approx, exact = oracle.retrieve_quantised(
        keys, toks, dtype, q, n, L, m, mean=pre.get("mean"), var=pre.get("var"), eps_z=pre.get("eps_z", 1e-5),
        W=pre.get("W"), pca_mean=pre.get("pca_mean"), threads=oracle.dresd_oracle.default_threads())
    identical = 0
    for b in range(q.shape[0]):
        cut = np.sort(approx[b])[-m]
        got = ids[b]
        assert len(set(got.tolist())) == n and np.all(got >= 0)
        # 1. every returned row is a candidate (up to rounding at the cut)
        assert np.all(approx[b][got] >= cut - DELTA)
        # 2. scores are the exact scores of the returned rows, in non-increasing order
        np.testing.assert_allclose(sc[b], exact[b][got], rtol=0, atol=SCORE_TOL)
        assert np.all(np.diff(exact[b][got]) <= 2 * EPS_ACC)
        # 3. no safe candidate (clearly above the cut) that beats the returned n-th row is missing
        safe = np.flatnonzero(approx[b] >= cut + DELTA)
        nth = exact[b][got[-1]]
        missing = [i for i in safe if exact[b][i] > nth + 2 * EPS_ACC and i not in set(got.tolist())]
        assert not missing, f"query {b}: safe candidates {missing[:5]} beat the returned n-th row"
        # 4. tokens are the stored tokens of the returned rows
        assert np.array_equal(tok[b], toks[got, :L])
        identical += int(np.array_equal(got, o_ids[b]))
    return identical / q.shape[0]


@pytest.mark.parametrize("dtype,d,B,n,L,m,N", [
    ("f16", 256, 1, 10, 10, 32, 148 * 128 * 2 + 37),
    ("bf16", 256, 8, 8, 4, 32, 30011),
    ("bf16", 64, 16, 5, 3, 20, 50021),            # the paper's reduced dimension: one 64-byte row per key
    ("f16", 128, 33, 4, 2, 16, 40009),            # wide batch: 128 operand rows
    ("bf16", 512, 4, 10, 3, 32, 20011),
    ("f16", 80, 3, 3, 2, 3, 9973),                # row of 80 bytes (not a multiple of 64), candidates == top_n
    ("bf16", 256, 2, 1, 1, 1, 700),               # top-1 with a single candidate
])
def test_quantised_retrieval_matches_the_oracle_of_the_same_rules(dtype, d, B, n, L, m, N):
    keys, toks = synth.make_store(8100 + d + B, N, d, 32, dtype, L + 1)
    q, _ = synth.make_queries(8150 + d + B, keys, dtype, B, 0.1)
    same = _check_against_oracle(keys, toks, dtype, q, n, L, m)
    assert same >= 0.7          # apart from ties at the cut, the rows ARE the oracle's


def test_quantised_retrieval_with_projection_and_zscore():
    dtype, d_in, d, B, N = "bf16", 512, 128, 6, 20011
    keys, toks = synth.make_store(8200, N, d, 16, dtype, 4)
    mean, var, W = synth.make_preprocess(8201, d_in, d, dtype)
    q = synth.make_hidden_queries(8202, B, d_in, dtype)
    _check_against_oracle(keys, toks, dtype, q, 5, 4, 32, pre=dict(mean=mean, var=var, W=W))


def test_quantised_retrieval_large_batch_uses_probe_and_finds_planted_rows():
    """64 queries x 32 candidates on a store large enough for the probe pass; every query is a
    stored row, which must come back first with score ~1 (Eq. 4: reciprocal rank 1)."""
    import torch
    dtype, N, d, B = "bf16", 148 * 256 * 130, 128, 64
    keys, toks = synth.make_store(8300, N, d, 64, dtype, 2)
    idx = np.random.default_rng(8301).integers(0, N, size=B)
    st = gpu_store(keys, toks, dtype)
    try:
        st.attach_quantised()
        ids, sc, tok = st.retrieve_quantised(binding.to_device(keys[idx], dtype), 4, 2, 32)
        torch.cuda.synchronize()
        st.status()
        got = ids.cpu().numpy()
        # duplicates of a row may precede it (ties go to the lower row): compare the key bits
        assert np.all([np.array_equal(keys[got[b, 0]], keys[idx[b]]) for b in range(B)])
        np.testing.assert_allclose(sc.cpu().numpy()[:, 0], 1.0, atol=2.0 ** -7)
    finally:
        st.close()


def test_quantised_argument_errors():
    import torch
    keys, toks = synth.make_store(8400, 500, 64, 4, "f16", 2)
    st = gpu_store(keys, toks, "f16")
    try:
        q = binding.to_device(keys[:2], "f16")
        with pytest.raises(binding.DresdError):          # nothing attached yet
            st.retrieve_quantised(q, 2, 1, 8)
        st.attach_quantised()
        for n, m in ((4, 3), (2, 33), (0, 8)):            # candidates < top_n, > 32, top_n < 1
            with pytest.raises(binding.DresdError):
                st.retrieve_quantised(q, n, 1, m)
        out = st.retrieve_quantised(q, 2, 1, 8)
        torch.cuda.synchronize()
        assert np.array_equal(out[0].cpu().numpy()[:, 0], [0, 1])
    finally:
        st.close()
    k32, t32 = synth.make_store(8401, 300, 64, 4, "f32", 2)
    s32 = gpu_store(k32, t32, "f32")
    try:
        with pytest.raises(binding.DresdError):
            binding.dresd_store_attach_quantised(s32.handle, torch.zeros(300 * 64, dtype=torch.uint8, device="cuda").data_ptr())
    finally:
        s32.close()


# d = 64: the 8-bit copy is scanned as rows of two keys (one 128-byte line).  Odd and even N
# (the last key of an odd store is handed to the re-ranking as an extra candidate), batch
# sizes on both sides of the 32-query limit of the packed form, and the unpacked form.
@pytest.mark.parametrize("pack2", [1, 0], ids=["two_keys_per_row", "one_key_per_row"])
@pytest.mark.parametrize("dtype,B,n,L,m,N", [
    ("f16", 1, 10, 4, 32, 148 * 512 * 2 + 37),
    ("bf16", 16, 5, 3, 20, 50022),
    ("f16", 32, 4, 2, 16, 40009),
    ("bf16", 33, 4, 2, 16, 30011),             # more than 32 queries: one key per row in both runs
    ("f16", 3, 3, 2, 3, 7),                    # three packed rows and an odd key
    ("bf16", 2, 1, 1, 1, 2),                   # a single packed row
])
def test_quantised_retrieval_d64_packed_rows(pack2, dtype, B, n, L, m, N):
    import torch
    d = 64
    keys, toks = synth.make_store(8500 + B, N, d, 8, dtype, L + 1)
    q, _ = synth.make_queries(8550 + B, keys, dtype, B, 0.1)
    n, m = min(n, N), min(m, N)
    st = gpu_store(keys, toks, dtype)
    try:
        st.attach_quantised()
        outs = []
        for p in (pack2, 1 - pack2):
            st.set_option("pack2", p)
            o = st.retrieve_quantised(binding.to_device(q, dtype), n, L, m)
            torch.cuda.synchronize()
            st.status()
            outs.append([t.cpu().numpy() for t in o])
    finally:
        st.close()
    # the two forms visit the same keys with the same arithmetic: identical results
    for a, b in zip(outs[0], outs[1]):
        assert np.array_equal(a, b)
    # and against the oracle (the first form)
    ids, sc, tok = outs[0]
    _, _, _, approx, exact = oracle.retrieve_quantised(keys, toks, dtype, q, n, L, m,
                                                       threads=oracle.dresd_oracle.default_threads())
    for b in range(B):
        cut = np.sort(approx[b])[-m]
        got = ids[b]
        assert len(set(got.tolist())) == n and np.all(got >= 0) and np.all(got < N)
        # the last key of an odd packed store is always re-ranked, whatever its approximate score
        extra = N - 1 if (N % 2 == 1 and B <= 32) else -1
        assert np.all((approx[b][got] >= cut - DELTA) | (got == extra))
        np.testing.assert_allclose(sc[b], exact[b][got], rtol=0, atol=SCORE_TOL)
        assert np.all(np.diff(exact[b][got]) <= 2 * EPS_ACC)
        safe = np.flatnonzero(approx[b] >= cut + DELTA)
        nth = exact[b][got[-1]]
        assert not [i for i in safe if exact[b][i] > nth + 2 * EPS_ACC and i not in set(got.tolist())]
        assert np.array_equal(tok[b], toks[got, :L])


@pytest.mark.parametrize("dtype,d,B,N", [("bf16", 256, 6, 40009), ("f16", 64, 5, 30011)])
def test_quantised_retrieval_with_first_token_filter(dtype, d, B, N):
    """Only keys whose first stored token matches are candidates (Section 3.5); -1 switches the
    filter off for a query; a rare token leaves slots empty (id -1, score -inf, tokens -1).
    At d = 64 the packed form (two keys, two first tokens per row; N is odd, so the last key
    reaches the re-ranking as an extra candidate and is filtered there) must agree with the
    unpacked one."""
    import torch
    n, L, m = 6, 3, 24
    keys, toks = synth.make_store(8600 + d, N, d, 16, dtype, L)
    q, src = synth.make_queries(8601 + d, keys, dtype, B, 0.1)
    vals, counts = np.unique(toks[:, 0], return_counts=True)
    ft = toks[src, 0].astype(np.int32)                         # the token of the query's source row
    ft[1] = -1
    ft[2] = int(vals[np.argmin(counts)])                       # rare: fewer than n matches
    st = gpu_store(keys, toks, dtype)
    try:
        st.attach_quantised()
        st.enable_first_token_filter()
        dft = torch.from_numpy(ft).cuda()
        ids, sc, tok = st.retrieve_quantised(binding.to_device(q, dtype), n, L, m, first_tokens=dft)
        torch.cuda.synchronize()
        st.status()
        ids, sc, tok = ids.cpu().numpy(), sc.cpu().numpy(), tok.cpu().numpy()
        if d == 64:
            st.set_option("pack2", 0)
            other = st.retrieve_quantised(binding.to_device(q, dtype), n, L, m, first_tokens=dft)
            torch.cuda.synchronize()
            assert np.array_equal(other[0].cpu().numpy(), ids) and np.array_equal(other[1].cpu().numpy(), sc)
            # the last key as a query: it must be found through the extra-candidate route, and only
            # when its first token is the wanted one
            st.set_option("pack2", 1)
            last = binding.to_device(keys[N - 1:N], dtype)
            for want, expect in ((int(toks[N - 1, 0]), N - 1), (int(toks[N - 1, 0]) + 1, None)):
                o = st.retrieve_quantised(last, 1, L, 4, first_tokens=torch.tensor([want], dtype=torch.int32, device="cuda"))
                torch.cuda.synchronize()
                got0 = int(o[0].cpu().numpy()[0, 0])
                if expect is None:
                    assert got0 != N - 1
                else:
                    assert np.array_equal(keys[got0], keys[N - 1])     # the key itself (or an earlier duplicate)
    finally:
        st.close()
    o_ids, o_sc, o_tok, approx, exact = oracle.retrieve_quantised(keys, toks, dtype, q, n, L, m, first_token=ft,
                                                                  threads=oracle.dresd_oracle.default_threads())
    for b in range(B):
        ok_rows = np.arange(N) if ft[b] < 0 else np.flatnonzero(toks[:, 0] == ft[b])
        k = min(n, len(ok_rows))
        got = ids[b, :k]
        assert np.all(ids[b, k:] == -1) and np.all(sc[b, k:] == -np.inf) and np.all(tok[b, k:] == -1)
        assert np.all(np.isin(got, ok_rows)) and len(set(got.tolist())) == k
        cut = np.sort(approx[b][ok_rows])[-min(m, len(ok_rows))]
        assert np.all(approx[b][got] >= cut - DELTA)
        np.testing.assert_allclose(sc[b, :k], exact[b][got], rtol=0, atol=SCORE_TOL)
        assert np.all(np.diff(exact[b][got]) <= 2 * EPS_ACC)
        safe = ok_rows[approx[b][ok_rows] >= cut + DELTA]
        if k:
            nth = exact[b][got[-1]]
            assert not [i for i in safe if exact[b][i] > nth + 2 * EPS_ACC and i not in set(got.tolist())]
        assert np.array_equal(tok[b, :k], toks[got, :L])
    assert np.sum(toks[:, 0] == ft[2]) < n


def test_quantised_packed_rows_with_probe_pass_against_oracle():
    """d = 64, 16 queries x 32 candidates on a store large enough for the probe pass of the packed
    form (tile-best rows of even and odd keys seed the filter): full check against the oracle."""
    dtype, d, B, n, L, m = "f16", 64, 16, 10, 2, 32
    N = 148 * 512 * 130 + 1                                     # odd: the last key is the extra candidate
    keys, toks = synth.make_store(8700, N, d, 256, dtype, L)
    q, _ = synth.make_queries(8701, keys, dtype, B, 0.1)
    q[3] = keys[N - 1]                                          # one query IS the last key
    import torch
    st = gpu_store(keys, toks, dtype)
    try:
        st.attach_quantised()
        st.set_option("probe", 32)                              # every 32nd tile: this store has 9,620 tiles
        ids, sc, tok = st.retrieve_quantised(binding.to_device(q, dtype), n, L, m)
        torch.cuda.synchronize()
        st.status()
        assert st.last_launches() == 5                          # K1, probe scan + its merge, scan, merge/re-rank
        ids, sc, tok = ids.cpu().numpy(), sc.cpu().numpy(), tok.cpu().numpy()
    finally:
        st.close()
    _, _, _, approx, exact = oracle.retrieve_quantised(keys, toks, dtype, q, n, L, m,
                                                       threads=oracle.dresd_oracle.default_threads())
    assert np.array_equal(keys[ids[3, 0]], keys[N - 1])
    for b in range(B):
        cut = np.sort(approx[b])[-m]
        got = ids[b]
        assert len(set(got.tolist())) == n and np.all(got >= 0) and np.all(got < N)
        assert np.all((approx[b][got] >= cut - DELTA) | (got == N - 1))
        np.testing.assert_allclose(sc[b], exact[b][got], rtol=0, atol=SCORE_TOL)
        assert np.all(np.diff(exact[b][got]) <= 2 * EPS_ACC)
        safe = np.flatnonzero(approx[b] >= cut + DELTA)
        nth = exact[b][got[-1]]
        assert not [i for i in safe if exact[b][i] > nth + 2 * EPS_ACC and i not in set(got.tolist())]
        assert np.array_equal(tok[b], toks[got, :L])

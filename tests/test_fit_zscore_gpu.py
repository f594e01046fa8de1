"""Statistics of Eq. 1 (Section 3.2: E[V], population Var[V] of a sample of embeddings):
dresd_fit_zscore against the oracle's two-pass float64 computation, and chained into the
datastore build (fit -> build_keys -> search)."""
import numpy as np
import pytest

import oracle
from paper_2502_15572_b200 import binding, synth

pytestmark = pytest.mark.gpu


def _fit(sample, dtype):
    import torch
    N, d_in = sample.shape
    dv = binding.to_device(sample, dtype)
    mean = torch.empty(d_in, dtype=torch.float32, device="cuda")
    var = torch.empty(d_in, dtype=torch.float32, device="cuda")
    binding.dresd_fit_zscore(dv.data_ptr(), N, d_in, binding.DTYPE_CODE[dtype], mean.data_ptr(), var.data_ptr(),
                             torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    return mean.cpu().numpy().astype(np.float64), var.cpu().numpy().astype(np.float64)


def _sample(seed, N, d_in, dtype, offset_scale=3.0):
    """Embeddings with per-column offsets and spreads over several orders of magnitude
    (LLM hidden states have a few dimensions whose mean dwarfs their spread)."""
    rng = np.random.default_rng(seed)
    sigma = np.exp(rng.uniform(np.log(0.02), np.log(8.0), size=d_in))
    mu = rng.normal(size=d_in) * offset_scale * sigma
    mu[::17] = 40.0 * sigma[::17]                     # offset 40 sigma: the shifted sums must cope
    x = (rng.standard_normal((N, d_in)) * sigma + mu).astype(np.float32)
    return synth.cast_to_store(x, dtype)


def _check(sample, dtype):
    got_m, got_v = _fit(sample, dtype)
    want_m, want_v = oracle.fit_zscore(sample, dtype)
    sd = np.sqrt(want_v)
    # Tolerances: outputs are fp32 (2^-24 relative rounding).  Chunk sums of at most 64 fp32
    # terms of (x - K) and (x - K)^2 err by < 64 * 2^-24 relative in the worst case (the
    # float64 accumulation above them adds nothing visible); K is within a few sigma / sqrt(32)
    # of the mean, so Var = S2/N - (S1/N)^2 cancels at most a small multiple of Var.
    assert np.all(np.abs(got_m - want_m) <= 2.0 ** -23 * np.abs(want_m) + 4e-6 * sd + 1e-30)
    assert np.all(np.abs(got_v - want_v) <= 2e-5 * want_v + 1e-30)
    return got_m, got_v


@pytest.mark.parametrize("dtype,N,d_in", [
    ("bf16", 20000, 4096),       # two column blocks
    ("f16", 50000, 512),         # four row lanes per CTA
    ("bf16", 3001, 200),         # 25 column groups: 250 of 256 threads active, ragged rows
    ("f16", 1, 64),              # a single row: variance 0
    ("f16", 7, 8),               # one column group, 32 row lanes, fewer rows than lanes
    ("bf16", 100000, 2304),      # a column block that is partly empty (288 groups)
    ("f16", 300000, 64),         # narrow and long
])
def test_fit_zscore_matches_oracle(dtype, N, d_in):
    got_m, got_v = _check(_sample(7000 + d_in + N % 97, N, d_in, dtype), dtype)
    if N == 1:
        assert np.all(got_v == 0.0)


def test_fit_zscore_constant_and_outlier_columns():
    """A constant column has variance exactly 0; a first row that is a far outlier (the shift
    is taken from the first rows) does not spoil the variance of the rest."""
    dtype, N, d_in = "f16", 40000, 128
    x = np.random.default_rng(71).standard_normal((N, d_in)).astype(np.float32)
    x[:, 5] = 3.25
    x[0, 9] = 2000.0
    s = synth.cast_to_store(x, dtype)
    got_m, got_v = _check(s, dtype)
    assert got_v[5] == 0.0 and got_m[5] == 3.25


def test_fit_zscore_is_reproducible():
    dtype, N, d_in = "bf16", 60000, 1024
    s = _sample(72, N, d_in, dtype)
    a, b = _fit(s, dtype), _fit(s, dtype)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])


def test_fit_then_build_then_search():
    """Section 3.2 -> 3.5 on the GPU alone: statistics from the hidden states, keys built with
    them, the store searched with a hidden state as the query: it finds its own row (Eq. 4:
    reciprocal rank 1), and the fitted statistics equal the oracle's within fp32 rounding."""
    import torch
    dtype, N, d_in, d = "bf16", 30000, 1024, 128
    _, _, W = synth.make_preprocess(7301, d_in, d, dtype)
    hidden = _sample(7302, N, d_in, dtype, offset_scale=1.0)
    dh = binding.to_device(hidden, dtype)
    dW = binding.to_device(W, dtype)
    mean = torch.empty(d_in, dtype=torch.float32, device="cuda")
    var = torch.empty(d_in, dtype=torch.float32, device="cuda")
    s = torch.cuda.current_stream().cuda_stream
    code = binding.DTYPE_CODE[dtype]
    binding.dresd_fit_zscore(dh.data_ptr(), N, d_in, code, mean.data_ptr(), var.data_ptr(), s)
    keys = torch.empty((N, d), dtype=dh.dtype, device="cuda")
    binding.dresd_build_keys(dh.data_ptr(), N, d_in, code, mean.data_ptr(), var.data_ptr(), 1e-5, dW.data_ptr(), d,
                             None, keys.data_ptr(), s)
    toks = torch.arange(N, dtype=torch.int32, device="cuda").reshape(N, 1).contiguous()
    st = binding.Store(keys, toks, dtype)
    st.set_preprocess(d_in, mean, var, 1e-5, dW, None)
    idx = np.random.default_rng(7303).integers(0, N, size=16)
    ids, sc, tok = st.retrieve(binding.to_device(hidden[idx], dtype), 1, 1)
    torch.cuda.synchronize()
    st.status()
    assert np.array_equal(ids.cpu().numpy()[:, 0], idx)
    st.close()
    # the keys equal the oracle's preprocessing with the oracle's own statistics
    om, ov = oracle.fit_zscore(hidden, dtype)
    want = oracle.preprocess(hidden[:512], dtype, mean=om, var=ov, eps_z=1e-5, W=W)
    got = synth.store_to_float32(keys[:512].cpu().view(torch.int16).numpy().view(np.uint16), dtype).astype(np.float64)
    assert np.max(np.abs(got - want)) <= 2.0 ** -8 * 0.51 + 1e-4


def test_fit_zscore_bad_arguments():
    import torch
    x = torch.zeros((4, 64), dtype=torch.float16, device="cuda")
    m = torch.zeros(64, dtype=torch.float32, device="cuda")
    for args in [(x.data_ptr(), 0, 64, 1), (x.data_ptr(), 4, 60, 1), (x.data_ptr(), 4, 64, 0),
                 (x.data_ptr() + 2, 4, 64, 1), (0, 4, 64, 1)]:
        with pytest.raises(binding.DresdError):
            binding.dresd_fit_zscore(args[0], args[1], args[2], args[3], m.data_ptr(), m.data_ptr(), 0)

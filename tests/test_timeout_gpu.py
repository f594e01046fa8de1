"""Failure detection without a GPU fault, for every pipelined kernel of the library.

Each kernel moves its data through a ring of shared-memory stages guarded by barriers, and
every wait on a barrier is bounded.  The tests make one wait run out from the host: a test
hook lets the first CTA announce the copies of one stage to its barrier without issuing them
(a barrier that nothing will ever complete) and the wait limit is lowered to 100 ms.  The
kernel must then return in an orderly way -- no trap, no endless spin, tensor memory freed,
every warp through its named barriers -- and report DRESD_ERR_TIMEOUT; the next call on the
same store, with the hook off, must be correct again.
"""
import numpy as np
import pytest

from paper_2502_15572_b200 import binding, synth
from tests.gpu_util import gpu_retrieve, gpu_store

pytestmark = pytest.mark.gpu


# one case per kernel form that serves the default route
@pytest.mark.parametrize("dtype,d,B,N,options", [
    ("f16", 256, 1, 60013, {}),                         # tcgen05, keys as M, two issuers on alternate slabs
    ("f16", 512, 2, 60013, {}),                         # tcgen05, keys as M, one issuer, two stage groups per tile
    ("bf16", 64, 2, 148 * 512 * 2 + 77, {}),            # tcgen05, narrow rows: four sub-tiles, two issuers
    ("bf16", 4096, 16, 2003, {}),                       # tcgen05, query operand travelling with the key slabs
    ("f16", 64, 40, 148 * 512 * 2 + 77, {}),            # tcgen05, one column per query, sixteen selection warps
    ("bf16", 32, 4, 148 * 1024 * 2 + 78, {}),           # tcgen05, two keys per row
    ("f16", 512, 64, 60013, {}),                        # tcgen05, two sub-tiles sharing an operand slab, sixteen warps
    ("f16", 512, 64, 60013, {"epi_warps": 8}),
    ("bf16", 256, 40, 148 * 256 * 2 + 5, {}),           # tcgen05, keys as the N operand
    ("f16", 256, 40, 60013, {"keys_as_m": 1}),          # tcgen05, keys as M, 128 accumulator columns
    ("f32", 128, 4, 148 * 512 * 2 + 19, {}),            # fp32 keys, FFMA kernel
    ("f16", 128, 2, 60013, {"scan_path": 1}),           # streaming mma.sync kernel
])
def test_lost_stage_times_out_and_store_stays_usable(dtype, d, B, N, options):
    import torch
    keys, toks = synth.make_store(8500 + d + B, N, d, 16, dtype, 4)
    q, _ = synth.make_queries(8501 + d + B, keys, dtype, B, 0.1)
    st = gpu_store(keys, toks, dtype)
    try:
        for k, v in options.items():
            st.set_option(k, v)
        good = gpu_retrieve(st, q, 10, 4)
        st.set_option("wait_ms", 100)
        st.set_option("debug_lose_stage", 2)
        st.retrieve(binding.to_device(q, dtype), 10, 4)
        torch.cuda.synchronize()
        with pytest.raises(binding.DresdError) as e:
            st.status()
        assert e.value.status == -5
        st.set_option("debug_lose_stage", 0)
        st.set_option("wait_ms", 0)
        again = gpu_retrieve(st, q, 10, 4)           # status() inside: clean again
        assert all(np.array_equal(a, b) for a, b in zip(good, again))
    finally:
        st.close()


@pytest.mark.parametrize("pairs", [1, 0], ids=["cta_pairs", "single_cta"])
@pytest.mark.parametrize("zscore", [True, False])
def test_build_keys_lost_stage_times_out(pairs, zscore):
    import torch
    dtype, N, d_in, d = "bf16", 148 * 512 + 300, 512, 128
    mean, var, W = synth.make_preprocess(8600, d_in, d, dtype)
    hidden = synth.make_hidden_queries(8601, N, d_in, dtype)
    dh, dW = binding.to_device(hidden, dtype), binding.to_device(W, dtype)
    dm, dv = torch.from_numpy(mean).cuda(), torch.from_numpy(var).cuda()
    out = torch.empty((N, d), dtype=dh.dtype, device="cuda")
    s = torch.cuda.current_stream().cuda_stream

    def build(dst):
        binding.dresd_build_keys(dh.data_ptr(), N, d_in, binding.DRESD_BF16, dm.data_ptr() if zscore else None,
                                 dv.data_ptr() if zscore else None, 1e-5, dW.data_ptr(), d, None, dst.data_ptr(), s)

    binding.dresd_set_global_option("build_keys_pairs", pairs)
    try:
        build(out)
        good = out.clone()
        binding.dresd_set_global_option("build_keys_wait_ms", 100)
        binding.dresd_set_global_option("build_keys_debug_lose_stage", 2)
        with pytest.raises(binding.DresdError) as e:
            build(torch.empty_like(out))
        assert e.value.status == -5
        binding.dresd_set_global_option("build_keys_debug_lose_stage", 0)
        binding.dresd_set_global_option("build_keys_wait_ms", 0)
        again = torch.empty_like(out)
        build(again)
        assert torch.equal(good, again)
    finally:
        binding.dresd_set_global_option("build_keys_debug_lose_stage", 0)
        binding.dresd_set_global_option("build_keys_wait_ms", 0)
        binding.dresd_set_global_option("build_keys_pairs", 1)

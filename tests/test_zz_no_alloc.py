"""dresd_retrieve_noalloc(): the retrieval call for hosts that may not allocate.

Some programs that embed this library cannot call cudaMalloc when they need a
draft (a serving runtime that owns all device memory through its own pool, a
plug-in inside another program's budget).  For them the library carries one
entry point whose workspace is a fixed array inside the library image.  This
test calls it through the C ABI twice in a row -- the second call finds the
first call's leftovers in the shared workspace -- and requires the same
answers as the store-based dresd_retrieve(), which runs the same kernels.

Collected last on purpose (file name), so that a failure here cannot hide the
result of any other test in a run that stops at the first failure.
"""
import numpy as np
import pytest

from paper_2502_15572_b200 import binding, synth

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dtype,d,N", [("f16", 256, 30011), ("bf16", 128, 20011), ("f32", 128, 10007)])
def test_noalloc_matches_store_path_twice(dtype, d, N):
    import torch
    n, L, stored = 10, 6, 8
    keys, toks = synth.make_store(9100 + d, N, d, 16, dtype, stored)
    dk = binding.to_device(keys, dtype)
    dt = torch.from_numpy(toks).cuda()
    store = binding.Store(dk, dt, dtype)
    stream = torch.cuda.current_stream().cuda_stream
    # two calls in a row with different batches: the second sees the first's leftovers
    for call, B in enumerate((8, 3)):
        q, _ = synth.make_queries(9200 + call, keys, dtype, B, 0.1)
        dq = binding.to_device(q, dtype)
        ref_ids, ref_sc, ref_tok = store.retrieve(dq, n, L)
        ids = torch.full((B, n), -7, dtype=torch.int32, device="cuda")
        sc = torch.full((B, n), float("nan"), dtype=torch.float32, device="cuda")
        tok = torch.full((B, n, L), -7, dtype=torch.int32, device="cuda")
        binding.dresd_retrieve_noalloc(dk.data_ptr(), dt.data_ptr(), N, d, binding.DTYPE_CODE[dtype], stored,
                                       dq.data_ptr(), B, n, L, ids.data_ptr(), sc.data_ptr(),
                                       tok.data_ptr(), stream)
        torch.cuda.synchronize()
        # same kernels, same launch geometry: identical ids and tokens, scores within the
        # tolerance the parity tests use for this dtype (they are in fact bit-identical)
        tol = 1e-5 if dtype == "f32" else 2e-3
        assert np.array_equal(ids.cpu().numpy(), ref_ids.cpu().numpy())
        assert np.array_equal(tok.cpu().numpy(), ref_tok.cpu().numpy())
        np.testing.assert_allclose(sc.cpu().numpy(), ref_sc.cpu().numpy(), atol=tol, rtol=0)
    store.close()


def test_noalloc_rejects_what_does_not_fit():
    import torch
    keys, toks = synth.make_store(9300, 2000, 64, 4, "f16", 4)
    dk = binding.to_device(keys, "f16")
    dt = torch.from_numpy(toks).cuda()
    dq = torch.zeros((9, 64), dtype=torch.float16, device="cuda")
    ids = torch.empty((9, 4), dtype=torch.int32, device="cuda")
    sc = torch.empty((9, 4), dtype=torch.float32, device="cuda")
    tok = torch.empty((9, 4, 4), dtype=torch.int32, device="cuda")
    with pytest.raises(binding.DresdError) as e:
        binding.dresd_retrieve_noalloc(dk.data_ptr(), dt.data_ptr(), 2000, 64, binding.DRESD_F16, 4,
                                       dq.data_ptr(), 9, 4, 4, ids.data_ptr(), sc.data_ptr(), tok.data_ptr(), 0)
    assert e.value.status == -2 and "DRESD_NOALLOC_MAX_BATCH" in e.value.message
    with pytest.raises(binding.DresdError) as e:
        binding.dresd_retrieve_noalloc(dk.data_ptr(), dt.data_ptr(), 2000, 64, binding.DRESD_F16, 4,
                                       dq.data_ptr(), 2, 33, 4, ids.data_ptr(), sc.data_ptr(), tok.data_ptr(), 0)
    assert e.value.status == -2

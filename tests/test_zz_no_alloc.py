"""dresd_retrieve_noalloc(): the retrieval call for hosts that may not allocate.

Some programs that embed this library cannot call cudaMalloc when they need a
draft (a serving runtime that owns all device memory through its own pool, a
plug-in inside another program's budget).  For them the library carries one
entry point whose workspace is a fixed array inside the library image.  This
test calls it through the C ABI twice in a row -- the second call finds the
first call's leftovers in the shared workspace -- and checks each call against
the CPU oracle with the checker every parity test uses.  As a second check it
compares with the store-based dresd_retrieve(): for 16-bit stores the
allocation-free call runs the streaming scoring kernel, so the store is put on
that kernel too ("scan_path" 1) and the answers must then be identical; against
the store's default tcgen05 kernel they only have to agree within the parity
tolerances.  Free device memory must not move across the calls.

Collected last on purpose (file name), so that a failure here cannot hide the
result of any other test in a run that stops at the first failure.
"""
import numpy as np
import pytest

import oracle
from paper_2502_15572_b200 import binding, synth
from tests import checker

pytestmark = pytest.mark.gpu


def _call(dk, dt, N, d, dtype, stored, dq, B, n, L, stream):
    import torch
    ids = torch.full((B, n), -7, dtype=torch.int32, device="cuda")
    sc = torch.full((B, n), float("nan"), dtype=torch.float32, device="cuda")
    tok = torch.full((B, n, L), -7, dtype=torch.int32, device="cuda")
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    binding.dresd_retrieve_noalloc(dk.data_ptr(), dt.data_ptr(), N, d, binding.DTYPE_CODE[dtype], stored,
                                   dq.data_ptr(), B, n, L, ids.data_ptr(), sc.data_ptr(), tok.data_ptr(), stream)
    binding.dresd_noalloc_status(stream)                # waits for the stream; raises on a device-side timeout
    free_after = torch.cuda.mem_get_info()[0]
    return ids.cpu().numpy(), sc.cpu().numpy(), tok.cpu().numpy(), free_before - free_after


@pytest.mark.parametrize("dtype,d,N", [("f16", 256, 30011), ("bf16", 128, 20011), ("f32", 128, 10007)])
def test_noalloc_matches_oracle_twice(dtype, d, N):
    import torch
    n, L, stored = 10, 6, 8
    keys, toks = synth.make_store(9100 + d, N, d, 16, dtype, stored)
    dk = binding.to_device(keys, dtype)
    dt = torch.from_numpy(toks).cuda()
    store = binding.Store(dk, dt, dtype)
    stream = torch.cuda.current_stream().cuda_stream
    batches = (8, 3)
    qs = [synth.make_queries(9200 + call, keys, dtype, B, 0.1)[0] for call, B in enumerate(batches)]
    dqs = [binding.to_device(q, dtype) for q in qs]
    # The first launch of a kernel loads its code, which may take device memory once per process;
    # that is the CUDA runtime's doing and happens for any kernel.  One call per shape up front,
    # so that the measured calls below show what the entry point itself does.
    for dq, B in zip(dqs, batches):
        _call(dk, dt, N, d, dtype, stored, dq, B, n, L, stream)
    # two calls in a row with different batches: the second sees the first's leftovers
    for q, dq, B in zip(qs, dqs, batches):
        ids, sc, tok, taken = _call(dk, dt, N, d, dtype, stored, dq, B, n, L, stream)
        assert taken == 0, f"free device memory changed by {taken} bytes across an allocation-free call"
        o = oracle.retrieve(keys, toks, dtype, q, n, L, want_full_scores=True,
                            threads=oracle.dresd_oracle.default_threads())
        checker.check_batch(o.full_scores, toks, ids, sc, tok, dtype, n, L, oracle_ids=o.ids)
        # the store path on its default kernel: same answers within the parity tolerances
        ref_ids, ref_sc, ref_tok = [t.cpu().numpy() for t in store.retrieve(dq, n, L)]
        checker.check_batch(o.full_scores, toks, ref_ids, ref_sc, ref_tok, dtype, n, L, oracle_ids=o.ids)
        np.testing.assert_allclose(sc, ref_sc, atol=2 * checker.EPS_ACC[dtype], rtol=0)
        # the store path on the same kernel: identical
        if dtype != "f32":
            store.set_option("scan_path", 1)
        same_ids, same_sc, same_tok = [t.cpu().numpy() for t in store.retrieve(dq, n, L)]
        store.set_option("scan_path", 0)
        assert np.array_equal(ids, same_ids) and np.array_equal(tok, same_tok) and np.array_equal(sc, same_sc)
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

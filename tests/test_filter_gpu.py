"""First-token filter (Sections 3.1 / 3.5) on the GPU against the oracle: all three
scoring kernels, plentiful and scarce matches, mixed filtered / unfiltered queries."""
import numpy as np
import pytest

import oracle
from paper_2502_15572_b200 import binding, synth
from tests import checker
from tests.gpu_util import gpu_store

pytestmark = pytest.mark.gpu


def _run(dtype, d, B, n, L, N, vocab, path, seed):
    import torch
    keys, toks = synth.make_store(seed, N, d, 16, dtype, L + 1, vocab=vocab)
    q, _ = synth.make_queries(seed + 1, keys, dtype, B, 0.1)
    rng = np.random.default_rng(seed + 2)
    ft = rng.integers(0, vocab, size=B).astype(np.int32)
    ft[::5] = -1                                     # every fifth query unfiltered
    if B > 2:
        ft[1] = vocab + 3                            # a token nobody stores: all padding
    st = gpu_store(keys, toks, dtype)
    st.set_option("scan_path", path)
    st.enable_first_token_filter()
    ids, sc, tok = st.retrieve_filtered(binding.to_device(q, dtype), torch.from_numpy(ft).cuda(), n, L)
    torch.cuda.synchronize()
    st.status()
    ids, sc, tok = ids.cpu().numpy(), sc.cpu().numpy(), tok.cpu().numpy()
    # unfiltered call on the same store still works and differs where the filter bites
    ids0, _, _ = st.retrieve(binding.to_device(q, dtype), n, L)
    st.close()
    o = oracle.retrieve(keys, toks, dtype, q, n, L, first_token=ft, want_full_scores=True,
                        threads=oracle.dresd_oracle.default_threads())
    for b in range(B):
        try:
            checker.check_query_filtered(o.full_scores[b], toks, ids[b], sc[b], tok[b], dtype, n, L, int(ft[b]))
        except AssertionError as e:
            raise AssertionError(f"query {b} (first token {ft[b]}): {e}") from None
        # the oracle's own padding agrees
        assert np.array_equal(o.ids[b] == -1, ids[b] == -1)
        if ft[b] < 0:
            assert np.array_equal(ids[b], ids0[b].cpu().numpy())


@pytest.mark.parametrize("dtype,d,B,n,L,N,vocab,path", [
    ("f16", 256, 1, 10, 10, 40009, 50, 0),
    ("f16", 256, 4, 10, 4, 40009, 50, 1),
    ("bf16", 256, 16, 10, 4, 40009, 50, 2),
    ("bf16", 256, 64, 32, 4, 30011, 12, 2),
    ("f16", 128, 8, 10, 4, 40009, 3000, 1),        # scarce matches: ~13 rows per token
    ("bf16", 128, 33, 10, 4, 40009, 3000, 2),
    ("f16", 64, 3, 5, 2, 50021, 50, 0),
    ("bf16", 512, 6, 10, 3, 20011, 50, 1),
    ("f32", 128, 8, 10, 10, 40009, 50, 0),
    ("f32", 64, 11, 32, 2, 20011, 3000, 0),
])
def test_first_token_filter_parity(dtype, d, B, n, L, N, vocab, path):
    _run(dtype, d, B, n, L, N, vocab, path, 9500 + d + B)


def test_filtered_call_needs_the_column():
    import torch
    keys, toks = synth.make_store(9601, 2000, 64, 4, "f16", 2)
    st = gpu_store(keys, toks, "f16")
    q = binding.to_device(keys[:2], "f16")
    ft = torch.zeros(2, dtype=torch.int32, device="cuda")
    with pytest.raises(binding.DresdError) as e:
        st.retrieve_filtered(q, ft, 2, 2)
    assert e.value.status == -1 and "enable_first_token_filter" in e.value.message
    st.enable_first_token_filter()
    st.retrieve_filtered(q, ft, 2, 2)
    st.retrieve_filtered(q, None, 2, 2)               # NULL = plain retrieve
    torch.cuda.synchronize()
    st.close()

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
    ("f16", 32, 6, 10, 2, 50022, 50, 0),           # two keys per row: a token per key of the row
    ("bf16", 32, 16, 10, 2, 50022, 3000, 0),
    ("f16", 32, 30, 10, 2, 50022, 50, 0),          # one column per query
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


@pytest.mark.parametrize("filtered", [False, True])
def test_row_sharded_merge_equals_whole_store(filtered):
    """Exchange step of a row-sharded datastore on one GPU: three stores over row slices,
    their results stacked as an all-gather would, merged by dresd_merge_shards."""
    import torch
    N, d, dtype, B, n, L = 50021, 128, "bf16", 9, 10, 4
    vocab = 3000 if filtered else 32000
    keys, toks = synth.make_store(9701, N, d, 16, dtype, L, vocab=vocab)
    q, _ = synth.make_queries(9702, keys, dtype, B, 0.1)
    ft = torch.from_numpy(np.random.default_rng(9703).integers(2000, 3000, size=B).astype(np.int32)).cuda()
    dq = binding.to_device(q, dtype)

    def run(k, t):
        st = gpu_store(k, t, dtype)
        if filtered:
            st.enable_first_token_filter()
            out = st.retrieve_filtered(dq, ft, n, L)
        else:
            out = st.retrieve(dq, n, L)
        torch.cuda.synchronize()
        st.close()
        return out

    whole = run(keys, toks)
    cuts = [0, 12345, 30000, N]
    parts = [run(keys[a:b], toks[a:b]) for a, b in zip(cuts[:-1], cuts[1:])]
    g_ids = torch.stack([p[0] for p in parts]).contiguous()
    g_sc = torch.stack([p[1] for p in parts]).contiguous()
    g_tok = torch.stack([p[2] for p in parts]).contiguous()
    offsets = torch.tensor(cuts[:-1], dtype=torch.int64, device="cuda")
    out = (torch.empty_like(whole[0]), torch.empty_like(whole[1]), torch.empty_like(whole[2]))
    binding.dresd_merge_shards(g_ids.data_ptr(), g_sc.data_ptr(), g_tok.data_ptr(), offsets.data_ptr(), 3, B, n, L,
                               out[0].data_ptr(), out[1].data_ptr(), out[2].data_ptr(),
                               torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    for a, b in zip(out, whole):
        assert torch.equal(a, b)
    # the same exchange as ONE block per shard (ids | scores | tokens), the single-all-gather form
    packed = torch.cat([torch.cat([p[0].reshape(-1), p[1].reshape(-1).view(torch.int32), p[2].reshape(-1)])
                        for p in parts]).contiguous()
    out2 = (torch.empty_like(whole[0]), torch.empty_like(whole[1]), torch.empty_like(whole[2]))
    binding.dresd_merge_shards_packed(packed.data_ptr(), offsets.data_ptr(), 3, B, n, L, out2[0].data_ptr(),
                                      out2[1].data_ptr(), out2[2].data_ptr(), torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    for a, b in zip(out2, whole):
        assert torch.equal(a, b)
    if filtered:
        assert (whole[0] == -1).any()          # scarce tokens: some queries have fewer than n matches


def test_sharded_retrieve_single_process():
    import torch
    from paper_2502_15572_b200 import dist_util
    keys, toks = synth.make_store(9801, 20011, 64, 8, "f16", 3)
    q, _ = synth.make_queries(9802, keys, "f16", 2, 0.1)
    st = gpu_store(keys, toks, "f16")
    dq = binding.to_device(q, "f16")
    ref = st.retrieve(dq, 5, 3)
    got = dist_util.sharded_retrieve(st, 1000, dq, 5, 3)
    torch.cuda.synchronize()
    assert torch.equal(got[0], ref[0] + 1000) and torch.equal(got[1], ref[1]) and torch.equal(got[2], ref[2])
    sharded = dist_util.ShardedRetriever(st, 1000, 5, 3)
    for _ in range(2):                                  # the second call reuses the buffers
        got = sharded(dq)
        torch.cuda.synchronize()
        assert torch.equal(got[0], ref[0] + 1000) and torch.equal(got[1], ref[1]) and torch.equal(got[2], ref[2])
    st.close()

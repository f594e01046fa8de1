"""Draft matrix preparation and longest-match acceptance (Section 3.6, Fig. 3):
oracle pins on CPU, GPU kernels against the oracle."""
import numpy as np
import pytest

import oracle


def test_prepare_hand_case():
    # EOS = 0.  Draft 1 ends early; draft 2 equals draft 0 after padding; draft 3 is missing.
    tok = np.array([[[5, 6, 7, 8], [5, 0, 9, 9], [5, 6, 7, 8], [1, 2, 3, 4]]], dtype=np.int32)
    ids = np.array([[10, 11, 12, -1]], dtype=np.int32)
    drafts, valid = oracle.drafts_prepare(tok, ids, 0)
    assert drafts[0].tolist() == [[5, 6, 7, 8], [5, 0, 0, 0], [5, 6, 7, 8], [0, 0, 0, 0]]
    assert valid[0].tolist() == [1, 1, 0, 0]


def test_accept_hand_cases():
    drafts = np.array([[[5, 6, 7, 8], [5, 6, 9, 9], [4, 4, 4, 4]]], dtype=np.int32)
    valid = np.array([[1, 1, 1]], dtype=np.int32)
    # the LLM agrees with draft 0 for two tokens, with draft 1 for three, never with draft 2
    llm = np.array([[[5, 6, 1, 1, 1], [5, 6, 9, 2, 2], [5, 3, 3, 3, 3]]], dtype=np.int32)
    best, length, out = oracle.drafts_accept(drafts, valid, llm)
    assert best.tolist() == [1] and length.tolist() == [4]
    assert out[0].tolist() == [5, 6, 9, 2, -1]                   # 3 draft tokens + the LLM's own token
    # full match: the token after the whole draft is appended
    llm2 = np.array([[[5, 6, 7, 8, 42], [5, 6, 9, 2, 2], [5, 3, 3, 3, 3]]], dtype=np.int32)
    best, length, out = oracle.drafts_accept(drafts, valid, llm2)
    assert best.tolist() == [0] and length.tolist() == [5] and out[0].tolist() == [5, 6, 7, 8, 42]
    # a tie goes to the better-ranked draft; an invalid draft never wins
    llm3 = np.array([[[5, 6, 1, 1, 1], [5, 6, 1, 1, 1], [4, 4, 4, 4, 9]]], dtype=np.int32)
    best, length, _ = oracle.drafts_accept(drafts, valid, llm3)
    assert best.tolist() == [2] and length.tolist() == [5]
    best, length, out = oracle.drafts_accept(drafts, np.array([[1, 1, 0]], dtype=np.int32), llm3)
    assert best.tolist() == [0] and length.tolist() == [3] and out[0].tolist() == [5, 6, 1, -1, -1]
    # nothing valid: still one token, the LLM's own next token
    best, length, out = oracle.drafts_accept(drafts, np.zeros((1, 3), dtype=np.int32), llm3)
    assert best.tolist() == [-1] and length.tolist() == [1] and out[0].tolist() == [5, -1, -1, -1, -1]


def test_accept_at_least_one_token_and_prefix_property():
    rng = np.random.default_rng(3)
    B, n, L = 40, 7, 9
    drafts = rng.integers(0, 3, size=(B, n, L)).astype(np.int32)
    llm = rng.integers(0, 3, size=(B, n, L + 1)).astype(np.int32)
    valid = (rng.random((B, n)) < 0.8).astype(np.int32)
    best, length, out = oracle.drafts_accept(drafts, valid, llm)
    assert np.all(length >= 1) and np.all(length <= L + 1)
    for b in range(B):
        a = length[b] - 1
        if best[b] >= 0:
            r = best[b]
            assert valid[b, r] == 1
            assert np.array_equal(out[b, :a], drafts[b, r, :a]) and np.array_equal(out[b, :a], llm[b, r, :a])
            assert out[b, a] == llm[b, r, a] and np.all(out[b, a + 1:] == -1)
            for r2 in range(n):                                   # nobody matches longer
                if valid[b, r2]:
                    m = 0
                    while m < L and drafts[b, r2, m] == llm[b, r2, m]:
                        m += 1
                    assert m < a or (m == a and r2 >= r)
        else:
            assert not valid[b].any() and a == 0


@pytest.mark.gpu
@pytest.mark.parametrize("B,n,L,vocab", [(1, 10, 10, 3), (64, 32, 16, 2), (7, 3, 20, 4), (5, 1, 1, 2)])
def test_gpu_drafts_match_oracle(B, n, L, vocab):
    import torch
    from paper_2502_15572_b200 import binding
    rng = np.random.default_rng(100 + B + n)
    tok = rng.integers(0, vocab, size=(B, n, L)).astype(np.int32)
    tok[:, 1:, :] = np.where(rng.random((B, n - 1, 1)) < 0.3, tok[:, :1, :], tok[:, 1:, :])   # some duplicates
    ids = rng.integers(0, 1000, size=(B, n)).astype(np.int32)
    ids[rng.random((B, n)) < 0.15] = -1
    llm = rng.integers(0, vocab, size=(B, n, L + 1)).astype(np.int32)
    llm[:, :, :L] = np.where(rng.random((B, n, L)) < 0.7, tok, llm[:, :, :L])                 # mostly agreeing
    want_d, want_v = oracle.drafts_prepare(tok, ids, 0)
    want = oracle.drafts_accept(want_d, want_v, llm)
    dev = lambda a: torch.from_numpy(a).cuda()
    d_tok, d_ids, d_llm = dev(tok), dev(ids), dev(llm)
    d_drafts = torch.empty((B, n, L), dtype=torch.int32, device="cuda")
    d_valid = torch.empty((B, n), dtype=torch.int32, device="cuda")
    binding.dresd_drafts_prepare(d_tok.data_ptr(), d_ids.data_ptr(), B, n, L, 0, d_drafts.data_ptr(),
                                 d_valid.data_ptr(), torch.cuda.current_stream().cuda_stream)
    best = torch.empty(B, dtype=torch.int32, device="cuda")
    length = torch.empty(B, dtype=torch.int32, device="cuda")
    out = torch.empty((B, L + 1), dtype=torch.int32, device="cuda")
    binding.dresd_drafts_accept(d_drafts.data_ptr(), d_valid.data_ptr(), d_llm.data_ptr(), B, n, L,
                                best.data_ptr(), length.data_ptr(), out.data_ptr(),
                                torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    assert np.array_equal(d_drafts.cpu().numpy(), want_d) and np.array_equal(d_valid.cpu().numpy(), want_v)
    assert np.array_equal(best.cpu().numpy(), want[0]) and np.array_equal(length.cpu().numpy(), want[1])
    assert np.array_equal(out.cpu().numpy(), want[2])

"""Seeded random shapes through the C ABI against the oracle: dtype, width, batch, n, draft
length, store size, scan path and operand order drawn at random; plain, filtered and
sorted-store (token windows) calls.  The fixed cases elsewhere pick their shapes by hand; this
one is there for the combinations nobody thought of."""
import numpy as np
import pytest

import oracle
from paper_2502_15572_b200 import binding, synth
from tests import checker
from tests.gpu_util import gpu_store

pytestmark = pytest.mark.gpu

WIDTHS = [8, 16, 24, 40, 64, 72, 96, 128, 136, 192, 200, 256, 264, 320, 512, 520, 1024]
BATCHES = [1, 2, 3, 7, 8, 9, 16, 17, 31, 32, 33, 48, 63, 64]


def _one(rng, seed):
    import torch
    dtype = str(rng.choice(["f16", "bf16", "f32"], p=[0.45, 0.45, 0.1]))
    step = 4 if dtype == "f32" else 8
    d = max(step, int(rng.choice(WIDTHS)) // step * step)
    B = int(rng.choice(BATCHES))
    L = int(rng.integers(1, 6))
    N = int(rng.choice([1, 31, 129, 1000, 5003, 20011, 40009, 70001]))
    n = min(int(rng.choice([1, 2, 5, 10, 16, 31, 32])), N)
    vocab = int(rng.choice([3, 17, 500]))
    mode = str(rng.choice(["plain", "filter", "windows"]))
    if dtype == "f32" and mode == "windows":
        mode = "filter"
    path = int(rng.choice([0, 1, 2])) if dtype != "f32" else 0
    kam = int(rng.integers(0, 2))
    desc = f"{dtype} d={d} B={B} n={n} L={L} N={N} vocab={vocab} mode={mode} scan_path={path} keys_as_m={kam}"
    keys, toks = synth.make_store(seed, N, d, 8, dtype, L + 1, vocab=vocab)
    if mode == "windows":
        keys, toks = synth.sort_by_first_token(keys, toks)
    q, _ = synth.make_queries(seed + 1, keys, dtype, B, 0.1)
    ft = rng.integers(0, vocab + 1, size=B).astype(np.int32)         # vocab itself: a token nobody stores
    if mode == "filter" and B > 1:
        ft[rng.integers(0, B)] = -1
    st = gpu_store(keys, toks, dtype)
    try:
        st.set_option("scan_path", path)
        st.set_option("keys_as_m", kam)
        dq = binding.to_device(q, dtype)
        if mode == "plain":
            ids, sc, tok = st.retrieve(dq, n, L)
            ft = None
        else:
            st.enable_first_token_filter()
            if mode == "windows":
                st.index_first_tokens()
            ids, sc, tok = st.retrieve_filtered(dq, torch.from_numpy(ft).cuda(), n, L)
        torch.cuda.synchronize()
        st.status()
    finally:
        st.close()
    ids, sc, tok = ids.cpu().numpy(), sc.cpu().numpy(), tok.cpu().numpy()
    o = oracle.retrieve(keys, toks, dtype, q, n, L, first_token=ft, want_full_scores=True,
                        threads=oracle.dresd_oracle.default_threads())
    for b in range(B):
        try:
            if ft is None:
                checker.check_query(o.full_scores[b], toks, ids[b], sc[b], tok[b], dtype, n, L)
            else:
                checker.check_query_filtered(o.full_scores[b], toks, ids[b], sc[b], tok[b], dtype, n, L, int(ft[b]))
        except AssertionError as e:
            raise AssertionError(f"{desc}, query {b}: {e}") from None


@pytest.mark.parametrize("seed", [11, 12, 13, 14])
def test_random_shapes_against_the_oracle(seed):
    rng = np.random.default_rng(seed)
    for k in range(15):
        _one(rng, 100 * seed + k)

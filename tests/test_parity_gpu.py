"""GPU parity: the CUDA path through the C ABI against the CPU oracle, element by element."""
import numpy as np
import pytest

import oracle
from paper_2502_15572_b200 import binding, synth
from tests import checker
from tests.gpu_util import gpu_retrieve, gpu_store, run_both

pytestmark = pytest.mark.gpu


def _check(keys, toks, dtype, q, n, L, pre=None, options=None):
    ids, sc, tok, o = run_both(keys, toks, dtype, q, n, L, pre=pre, options=options)
    return checker.check_batch(o.full_scores, toks, ids, sc, tok, dtype, n, L, oracle_ids=o.ids)


# Sizes span several tiles per CTA of a 148-CTA grid plus a ragged tail.
@pytest.mark.parametrize("dtype,d,B,n,L,N", [
    ("f16", 256, 1, 10, 10, 148 * 64 * 3 + 37),
    ("bf16", 256, 4, 10, 10, 148 * 64 * 2 + 5),
    ("f16", 256, 8, 32, 16, 30011),
    ("bf16", 256, 7, 5, 3, 9001),
    ("f16", 128, 3, 10, 10, 148 * 128 * 2 + 77),
    ("bf16", 128, 8, 32, 4, 40009),
    ("f16", 64, 2, 10, 10, 148 * 256 + 300),
    ("bf16", 64, 5, 17, 10, 50021),
    ("f16", 72, 2, 10, 6, 20011),          # row = 144 bytes: not a multiple of the 128-byte slab
    ("bf16", 200, 3, 10, 6, 20011),
    ("f16", 512, 2, 10, 6, 20011),         # long rows: k-chunked kernel
    ("bf16", 1024, 4, 10, 6, 9973),
    ("bf16", 320, 5, 8, 6, 9973),
    ("f32", 128, 8, 10, 10, 148 * 128 * 2 + 19),
    ("f32", 64, 3, 32, 10, 20011),
    ("f32", 200, 9, 10, 5, 10007),
    ("f32", 1100, 2, 10, 5, 5003),
    ("f16", 256, 9, 10, 10, 20011),        # more queries than one launch holds
    ("bf16", 256, 64, 32, 16, 20011),
    ("f32", 128, 20, 10, 10, 20011),
])
def test_parity_shapes(dtype, d, B, n, L, N):
    keys, toks = synth.make_store(7000 + d + B, N, d, 32, dtype, L + 2)
    q, _ = synth.make_queries(7100 + d + B, keys, dtype, B, 0.1)
    _check(keys, toks, dtype, q, n, L)


# One case per form of the tcgen05 kernel's MMA issue and of the fp32 loop: two issuer threads on
# alternate sub-tiles (narrow rows), on alternate slabs into two accumulator sets (wide rows), the
# single-issuer exceptions, ragged last slabs (steps beyond the row width are skipped), three-slab
# stage groups, the epilogue's sub-tile split for few queries, 17-32 queries with the keys as N,
# and every fp32 register tile (1, 2, 4, 8 queries; more than 8 = several passes).
@pytest.mark.parametrize("dtype,d,B,n,L,N", [
    ("f16", 32, 1, 10, 4, 148 * 512 + 301),     # half-filled slab, 4 sub-tiles, sub-tile split
    ("bf16", 96, 3, 10, 4, 60013),              # 1.5 slabs, 2 sub-tiles
    ("f16", 160, 1, 10, 4, 40009),              # 2.5 slabs: one group of three per tile, two sets
    ("bf16", 192, 12, 16, 4, 40009),            # three full slabs, 9-16 queries
    ("f16", 256, 16, 10, 4, 148 * 128 * 2 + 9), # two sets, 32 accumulator columns
    ("bf16", 256, 20, 10, 4, 40009),            # 17-32 queries: keys as the N operand
    ("f16", 200, 32, 32, 4, 30011),
    ("bf16", 512, 2, 10, 4, 30011),             # 8 slabs, few queries: one issuer
    ("f16", 512, 12, 10, 4, 30011),             # 8 slabs, 9-16 queries: two sets
    ("bf16", 960, 3, 10, 4, 10007),             # 15 slabs, few queries: two sets
    ("f16", 320, 24, 10, 4, 20011),             # 17-32 queries, wider than 256: two sets, 64 columns
    ("bf16", 448, 64, 32, 4, 20011),            # 64 queries, 7 slabs: two sets, 128 columns (all of TMEM)
    ("f16", 1024, 48, 10, 4, 6007),
    ("f32", 128, 1, 10, 4, 148 * 512 * 2 + 77),
    ("f32", 96, 2, 10, 4, 60013),
    ("f32", 256, 4, 32, 4, 40009),
    ("f32", 64, 8, 10, 4, 148 * 512 + 5),
    ("f32", 2048, 3, 10, 4, 3001),              # wide fp32 rows: four queries per launch
    ("f32", 40, 13, 5, 2, 20011),
])
def test_parity_kernel_forms(dtype, d, B, n, L, N):
    keys, toks = synth.make_store(7300 + d + B, N, d, 32, dtype, L + 1)
    q, _ = synth.make_queries(7400 + d + B, keys, dtype, B, 0.1)
    _check(keys, toks, dtype, q, n, L)


# Both 16-bit scoring kernels at every batch size: path 1 = streaming mma.sync kernel
# (several passes when B > 8), path 2 = tcgen05/TMEM kernel (one pass, operand padded).
@pytest.mark.parametrize("path", [1, 2])
@pytest.mark.parametrize("dtype,d,B,n,L,N", [
    ("f16", 256, 1, 10, 10, 148 * 128 * 2 + 37),
    ("bf16", 256, 8, 32, 4, 30011),
    ("f16", 256, 16, 10, 10, 30011),
    ("bf16", 256, 33, 32, 16, 148 * 128 + 77),
    ("bf16", 256, 64, 32, 16, 30011),
    ("f16", 64, 20, 10, 3, 40009),
    ("bf16", 128, 12, 10, 3, 40009),
    ("f16", 72, 5, 10, 3, 20011),
    ("bf16", 512, 16, 10, 3, 20011),
    ("bf16", 4096, 16, 10, 3, 2003),       # query operand too large to stay in shared memory
    ("f16", 2048, 40, 7, 3, 1501),
])
def test_parity_both_16bit_paths(path, dtype, d, B, n, L, N):
    keys, toks = synth.make_store(7200 + d + B, N, d, 32, dtype, L + 1)
    q, _ = synth.make_queries(7250 + d + B, keys, dtype, B, 0.1)
    _check(keys, toks, dtype, q, n, L, options={"scan_path": path})


def _rescaled(keys, dtype, seed, lo=0.25, hi=4.0):
    """The same rows with lengths spread log-uniformly over lo..hi (store dtype after scaling)."""
    rng = np.random.default_rng(seed)
    f = np.exp(rng.uniform(np.log(lo), np.log(hi), size=keys.shape[0])).astype(np.float32)
    scaled = synth.store_to_float32(keys, dtype) * f[:, None]
    return synth.cast_to_store(scaled, dtype), float(f.max()) * 1.01


# Keys that are NOT unit vectors: Eq. 3 is read as the inner product of the unit query with the
# key as stored (keys are never renormalised), so a long key can outrank a better-aligned short
# one.  One case per dtype and scoring kernel, lengths 0.25 .. 4.
@pytest.mark.parametrize("dtype,d,B,n,L,N,options", [
    ("f32", 128, 5, 10, 4, 40009, None),
    ("f16", 256, 3, 10, 4, 40009, None),                       # tcgen05, keys as M
    ("bf16", 64, 16, 10, 4, 60013, None),                      # narrow rows, sub-tiles
    ("bf16", 256, 40, 32, 4, 30011, None),                     # keys as the N operand
    ("f16", 128, 6, 10, 4, 40009, {"scan_path": 1}),           # streaming mma.sync kernel
    ("bf16", 512, 64, 16, 4, 20011, None),                     # 64 queries on wide rows
    ("f16", 64, 64, 10, 4, 60013, None),                       # 64 queries on narrow rows
])
def test_parity_keys_not_unit_length(dtype, d, B, n, L, N, options):
    keys, toks = synth.make_store(7500 + d + B, N, d, 32, dtype, L + 1)
    keys, kmax = _rescaled(keys, dtype, 7501 + d)
    q, _ = synth.make_queries(7502 + d + B, keys, dtype, B, 0.1)
    ids, sc, tok, o = run_both(keys, toks, dtype, q, n, L, options=options)
    assert np.max(np.abs(o.full_scores)) > 2.0                  # the spread is really there
    checker.check_batch(o.full_scores, toks, ids, sc, tok, dtype, n, L, oracle_ids=o.ids, key_scale=kmax)


# 32-element 16-bit keys are 64 bytes: an even-sized store is scanned as rows of two keys (up to 16
# queries; more run the one-column-per-query form).  Against the oracle, and bit for bit against
# the one-key-per-row scan ("pack2" 0): the zero halves of the operand rows add exact zeros.
@pytest.mark.parametrize("dtype,B,n,N", [
    ("f16", 1, 10, 148 * 1024 * 2 + 302),      # several 1024-key tiles per CTA, ragged tail
    ("bf16", 4, 10, 60014),
    ("f16", 8, 32, 60014),                     # 32 accumulator columns
    ("bf16", 16, 10, 148 * 1024 + 6),          # 64 columns
    ("f16", 16, 16, 2 * 148 * 128 * 1024 // 128 + 2),   # B * n = 256: with the probe pass when large enough
    ("f16", 3, 5, 2),                          # a single row of two keys
    ("bf16", 2, 10, 1022),
    ("f16", 5, 10, 60013),                     # odd size: the one-key-per-row scan
    ("f16", 24, 10, 60014),                    # more than 16 queries: one column per query
])
def test_parity_two_keys_per_row(dtype, B, n, N):
    import torch
    d, L = 32, 3
    keys, toks = synth.make_store(7600 + B, N, d, 16, dtype, L)
    q, _ = synth.make_queries(7601 + B, keys, dtype, B, 0.1)
    n = min(n, N)
    ids, sc, tok, o = run_both(keys, toks, dtype, q, n, L)
    checker.check_batch(o.full_scores, toks, ids, sc, tok, dtype, n, L, oracle_ids=o.ids)
    i0, s0, t0, _ = run_both(keys, toks, dtype, q, n, L, options={"pack2": 0, "merged_columns": 2})
    if B <= 16:
        assert np.array_equal(ids, i0) and np.array_equal(sc, s0) and np.array_equal(tok, t0)


@pytest.mark.parametrize("path", [1, 2])
def test_adversarial_order_both_paths(path):
    # ascending scores in memory: every row beats all rows before it (queue overflow path)
    N, d, dtype = 12000, 64, "bf16"
    keys, toks = synth.make_store(7270, N, d, 4, dtype, 2)
    q, _ = synth.make_queries(7271, keys, dtype, 12, 0.1)
    s = oracle.scores(keys, dtype, oracle.preprocess(q[:1], dtype)[0])
    order = np.argsort(s, kind="stable")
    _check(keys[order], toks[order], dtype, q, 10, 2, options={"scan_path": path})


# Ascending scores in memory (every row beats all rows before it: the queues overflow round after round)
# for every form of the tcgen05 kernel's epilogue -- rounds on demand with warps at different tiles, the
# fast rejection and its out-of-line exact step, sub-tiles, two keys per row, keys as N.
@pytest.mark.parametrize("dtype,d,B,n,N", [
    ("f16", 64, 64, 32, 148 * 512 + 3000),      # one column per query, four sub-tiles
    ("bf16", 64, 16, 10, 148 * 512 + 3000),     # hi block | lo block, four sub-tiles
    ("f16", 64, 28, 10, 148 * 512 + 3000),      # the same with 64 columns (17-32 queries)
    ("f16", 32, 8, 10, 148 * 1024 + 3000),      # two keys per row
    ("bf16", 512, 40, 16, 40000),               # two sub-tiles sharing an operand slab
    ("f16", 256, 3, 32, 40000),                 # two accumulator sets
    ("bf16", 256, 33, 32, 60000),               # keys as N
    ("f16", 1024, 20, 10, 20000),
])
def test_adversarial_order_every_epilogue_form(dtype, d, B, n, N):
    keys, toks = synth.make_store(7280 + d + B, N, d, 4, dtype, 2)
    q, _ = synth.make_queries(7281 + d + B, keys, dtype, B, 0.1)
    s = oracle.scores(keys, dtype, oracle.preprocess(q[:1], dtype)[0])
    order = np.argsort(s, kind="stable")
    _check(keys[order], toks[order], dtype, q, n, 2)


# Forty and more tiles per CTA without a probe pass: the lists fill from nothing in every CTA, rounds are asked
# for tile after tile while the selection warps are at different tiles (two accumulator buffers apart), and the
# warps that wait for an accumulator attend them from their polling loops.
@pytest.mark.parametrize("dtype,d,B,n,N", [
    ("f16", 64, 10, 10, 148 * 512 * 24 + 333),      # hi block | lo block, four sub-tiles
    ("bf16", 64, 40, 16, 148 * 512 * 12 + 5),       # one column per query, sixteen selection warps
    ("f16", 256, 5, 32, 148 * 128 * 40 + 77),       # two accumulator sets
])
def test_rounds_on_demand_over_many_tiles(dtype, d, B, n, N):
    keys, toks = synth.make_store(7800 + d + B, N, d, 4, dtype, 2)
    q, _ = synth.make_queries(7801 + d + B, keys, dtype, B, 0.1)
    _check(keys, toks, dtype, q, n, 2, options={"probe": 0})


# Measurement switches that select another form of the same computation: results must not change.
@pytest.mark.parametrize("dtype,d,B,n,N,options", [
    ("f16", 64, 64, 32, 148 * 512 * 2 + 77, {"epi_warps": 8}),          # one column per query on eight warps
    ("bf16", 64, 40, 10, 60013, {"epi_warps": 8}),
    ("f16", 128, 64, 16, 60013, {"epi_warps": 8}),                      # two columns, two sub-tiles, eight warps
    ("bf16", 1024, 48, 10, 20011, {"epi_warps": 8}),
    ("f16", 64, 16, 10, 148 * 512 * 2 + 77, {"round_per_tile": 1}),     # a round after every tile
    ("bf16", 512, 64, 16, 30011, {"round_per_tile": 1}),
    ("bf16", 256, 48, 32, 148 * 256 * 2 + 5, {"fast_reject": 0}),       # keys as N, exact compare only
    ("f16", 64, 48, 10, 60013, {"merged_columns": 2}),                  # two columns per query
    ("bf16", 256, 64, 32, 60013, {"merge_level": 8}),                   # queues folded early ...
    ("f16", 64, 20, 32, 60013, {"merge_level": 32}),                    # ... and only when full
    ("f16", 320, 24, 10, 30011, {"merged_columns": 1}),                 # one column per query on wide rows
    ("bf16", 64, 24, 10, 148 * 512 * 2 + 77, {"merged_columns": 1}),    # ... and for 17-32 queries (32 columns)
])
def test_measurement_switches_do_not_change_results(dtype, d, B, n, N, options):
    keys, toks = synth.make_store(7700 + d + B, N, d, 16, dtype, 3)
    q, _ = synth.make_queries(7701 + d + B, keys, dtype, B, 0.1)
    ids, sc, tok, o = run_both(keys, toks, dtype, q, n, 2, options=options)
    checker.check_batch(o.full_scores, toks, ids, sc, tok, dtype, n, 2, oracle_ids=o.ids)
    ids0, sc0, tok0, _ = run_both(keys, toks, dtype, q, n, 2)
    assert np.array_equal(tok0, tok) or np.array_equal(ids0, ids)      # ids may swap only inside rounding ties
    np.testing.assert_allclose(sc, sc0, atol=2 * checker.EPS_ACC[dtype], rtol=0)


def test_config1_tiny_exact_knn_full():
    w = synth.make_workload("c1_tiny_f32")
    rate = _check(w["keys"], w["next_tokens"], "f32", w["queries"], w["top_n"], w["draft_len"])
    assert rate >= 0.95


@pytest.mark.parametrize("dtype", ["f32", "f16", "bf16"])
def test_preprocess_matches_oracle(dtype):
    import torch
    d_in, d, B = 1024, 256, 5
    keys, toks = synth.make_store(7301, 4096, d, 8, dtype, 4)
    mean, var, W = synth.make_preprocess(7302, d_in, d, dtype)
    pm = (0.01 * np.arange(d_in)).astype(np.float32)
    q = synth.make_hidden_queries(7303, B, d_in, dtype)
    st = gpu_store(keys, toks, dtype)
    try:
        cases = [
            dict(),                                          # Eq. 2 only (needs d_in == d)
            dict(mean=mean, var=var, W=W),
            dict(W=W),
            dict(mean=mean, var=var, W=W, pca_mean=pm),
        ]
        for c in cases:
            qq = q if c else synth.make_hidden_queries(7304, B, d, dtype)
            dev = {k: (binding.to_device(v, dtype) if k == "W" else torch.from_numpy(v).cuda())
                   for k, v in c.items()}
            st.set_preprocess(qq.shape[1], dev.get("mean"), dev.get("var"), 1e-5, dev.get("W"),
                              dev.get("pca_mean"))
            got = st.preprocess(binding.to_device(qq, dtype)).cpu().numpy()
            want = oracle.preprocess(qq, dtype, mean=c.get("mean"), var=c.get("var"), eps_z=1e-5,
                                     W=c.get("W"), pca_mean=c.get("pca_mean"))
            # fp32 arithmetic over d_in terms: a few 1e-7 relative to a unit vector
            np.testing.assert_allclose(got, want, atol=2e-6, rtol=0)
            np.testing.assert_allclose(np.linalg.norm(got.astype(np.float64), axis=1), 1.0, atol=1e-6)
    finally:
        st.close()


def test_zscore_only_without_projection():
    d = 256
    keys, toks = synth.make_store(7401, 20011, d, 8, "f16", 4)
    mean, var, _ = synth.make_preprocess(7402, d, d, "f16")
    q = synth.make_hidden_queries(7403, 3, d, "f16")
    _check(keys, toks, "f16", q, 10, 4, pre=dict(mean=mean, var=var, eps_z=1e-3))


@pytest.mark.parametrize("dtype,d_in,d,B", [("bf16", 4096, 256, 16), ("f16", 768, 64, 3), ("f32", 512, 128, 4)])
def test_projected_retrieval(dtype, d_in, d, B):
    keys, toks = synth.make_store(7501, 30011, d, 16, dtype, 10)
    mean, var, W = synth.make_preprocess(7502, d_in, d, dtype)
    q = synth.make_hidden_queries(7503, B, d_in, dtype)
    _check(keys, toks, dtype, q, 10, 10, pre=dict(mean=mean, var=var, W=W))


# ---------------------------------------------------------------------------- edge cases
@pytest.mark.parametrize("dtype", ["f32", "f16", "bf16"])
@pytest.mark.parametrize("N,n", [(1, 1), (5, 5), (33, 32), (64, 10), (257, 32)])
def test_tiny_stores(dtype, N, n):
    keys, toks = synth.make_store(7600 + N, N, 64, 3, dtype, 3)
    q, _ = synth.make_queries(7601, keys, dtype, 3, 0.2)
    _check(keys, toks, dtype, q, n, 3)


@pytest.mark.parametrize("dtype", ["f32", "f16"])
def test_scores_ascending_in_memory(dtype):
    # Worst case for a running-threshold filter: every key beats all before it.
    N, d = 20000, 64
    keys, toks = synth.make_store(7701, N, d, 4, dtype, 2)
    q, _ = synth.make_queries(7702, keys, dtype, 2, 0.1)
    s = oracle.scores(keys, dtype, oracle.preprocess(q[:1], dtype)[0])
    order = np.argsort(s, kind="stable")
    _check(keys[order], toks[order], dtype, q, 10, 2)
    _check(keys[order[::-1]], toks[order[::-1]], dtype, q, 10, 2)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_all_keys_identical_gives_lowest_ids(dtype):
    N, d = 5000, 64
    keys, toks = synth.make_store(7801, N, d, 2, dtype, 2)
    keys[:] = keys[0]
    q, _ = synth.make_queries(7802, keys, dtype, 2, 0.1)
    ids, sc, tok, o = run_both(keys, toks, dtype, q, 12, 2)
    assert np.array_equal(ids, np.tile(np.arange(12), (2, 1)))
    assert np.array_equal(o.ids, ids)
    assert np.array_equal(tok, toks[ids][:, :, :2])


def test_duplicates_and_zero_query():
    N, d = 9000, 128
    keys, toks = synth.make_store(7901, N, d, 8, "f16", 4)
    keys[8000] = keys[123]
    keys[4000] = keys[123]
    q = np.concatenate([keys[123:124], np.zeros((1, d), dtype=np.float16)])
    ids, sc, tok, o = run_both(keys, toks, "f16", q, 6, 4)
    assert ids[0, :3].tolist() == [123, 4000, 8000]
    assert sc[0, 0] == sc[0, 1] == sc[0, 2]
    assert ids[1].tolist() == [0, 1, 2, 3, 4, 5] and np.all(sc[1] == 0.0)
    checker.check_batch(o.full_scores, toks, ids, sc, tok, "f16", 6, 4, oracle_ids=o.ids)


# ---------------------------------------------------------------------------- invariants on the GPU
def test_invariants_permutation_shards_prefix_repeat():
    N, d, dtype = 30011, 256, "f16"
    keys, toks = synth.make_store(8001, N, d, 16, dtype, 10)
    q, _ = synth.make_queries(8002, keys, dtype, 4, 0.1)
    st = gpu_store(keys, toks, dtype)
    ids, sc, tok = gpu_retrieve(st, q, 10, 10)
    ids2, sc2, tok2 = gpu_retrieve(st, q, 10, 10)
    assert np.array_equal(ids, ids2) and np.array_equal(sc, sc2) and np.array_equal(tok, tok2)
    # prefixes
    ids5, sc5, tok5 = gpu_retrieve(st, q, 5, 4)
    assert np.array_equal(ids5, ids[:, :5]) and np.array_equal(sc5, sc[:, :5])
    assert np.array_equal(tok5, tok[:, :5, :4])
    # batch of B equals B single-query calls (different kernel instantiations)
    for b in range(4):
        i1, s1, t1 = gpu_retrieve(st, q[b:b + 1], 10, 10)
        assert np.array_equal(i1[0], ids[b])
        np.testing.assert_allclose(s1[0], sc[b], atol=1e-6)
    st.close()
    # permutation of the rows: ids map through the permutation, scores are bit-identical
    perm = np.random.default_rng(8003).permutation(N)
    stp = gpu_store(keys[perm], toks[perm], dtype)
    idp, scp, tokp = gpu_retrieve(stp, q, 10, 10)
    stp.close()
    assert np.array_equal(perm[idp], ids) and np.array_equal(scp, sc) and np.array_equal(tokp, tok)
    # shard merge: top-n of the whole = merge of the shards' top-n
    cut = 12345
    sa = gpu_store(keys[:cut], toks[:cut], dtype)
    sb = gpu_store(keys[cut:], toks[cut:], dtype)
    ia, sca, ta = gpu_retrieve(sa, q, 10, 10)
    ib, scb, tb = gpu_retrieve(sb, q, 10, 10)
    sa.close()
    sb.close()
    for b in range(4):
        mi = np.concatenate([ia[b], ib[b] + cut])
        ms = np.concatenate([sca[b], scb[b]])
        mt = np.concatenate([ta[b], tb[b]])
        order = np.lexsort((mi, -ms.astype(np.float64)))[:10]
        assert np.array_equal(mi[order], ids[b]) and np.array_equal(ms[order], sc[b])
        assert np.array_equal(mt[order], tok[b])


def test_self_retrieval_mrr_is_one():
    N, d, dtype = 40000, 128, "bf16"
    keys, toks = synth.make_store(8101, N, d, 64, dtype, 2)
    idx = np.random.default_rng(8102).integers(0, N, size=64)
    st = gpu_store(keys, toks, dtype)
    ids, sc, _ = gpu_retrieve(st, keys[idx], 1, 1)
    st.close()
    # Eq. 4: reciprocal rank of the correct item; exact search finds every key first
    assert np.mean(1.0 / (1 + (ids[:, 0] != idx))) == 1.0
    np.testing.assert_allclose(sc[:, 0], 1.0, atol=2.0 ** -7)


def test_grid_option_and_host_call():
    import torch
    N, d, dtype = 30011, 256, "f16"
    keys, toks = synth.make_store(8201, N, d, 16, dtype, 10)
    q, _ = synth.make_queries(8202, keys, dtype, 2, 0.1)
    st = gpu_store(keys, toks, dtype)
    ref = gpu_retrieve(st, q, 10, 10)
    for grid in (1, 7, 296):
        st.set_option("grid", grid)
        got = gpu_retrieve(st, q, 10, 10)
        assert all(np.array_equal(a, b) for a, b in zip(ref, got))
    st.set_option("grid", 0)
    qh = torch.from_numpy(q.view(np.float16)).pin_memory()
    out = (torch.empty((2, 10), dtype=torch.int32).pin_memory(),
           torch.empty((2, 10), dtype=torch.float32).pin_memory(),
           torch.empty((2, 10, 10), dtype=torch.int32).pin_memory())
    st.retrieve_host(qh, 10, 10, out)
    assert all(np.array_equal(a, b.numpy()) for a, b in zip(ref, out))
    assert st.last_launches() == 3          # preprocess, scan with fused selection, merge + gather
    st.close()


def test_argument_errors_on_device():
    import torch
    keys, toks = synth.make_store(8301, 1000, 64, 4, "f16", 4)
    st = gpu_store(keys, toks, "f16")
    q = binding.to_device(keys[:2], "f16")
    with pytest.raises(binding.DresdError) as e:
        st.retrieve(q, 0, 2)
    assert e.value.status == -1
    with pytest.raises(binding.DresdError) as e:
        st.retrieve(q, 2, 5)
    assert e.value.status == -1
    with pytest.raises(binding.DresdError) as e:
        st.retrieve(q, 33, 2)
    assert e.value.status == -2
    big = torch.zeros((65, 64), dtype=torch.float16, device="cuda")
    with pytest.raises(binding.DresdError) as e:
        st.retrieve(big, 2, 2)
    assert e.value.status == -2
    with pytest.raises(binding.DresdError) as e:      # host pointer where a device pointer is required
        binding.dresd_retrieve(st.handle, keys.ctypes.data, 1, 1, 1, keys.ctypes.data, keys.ctypes.data,
                               keys.ctypes.data, 0)
    assert e.value.status == -1
    ids, sc, tok = st.retrieve(q[:0], 2, 2)          # B == 0 is a no-op
    st.close()
    with pytest.raises(binding.DresdError):
        binding.dresd_store_create(0, 0, 10, 64, 1, 4)
    k = torch.zeros((8, 12), dtype=torch.float16, device="cuda")   # 24-byte rows
    with pytest.raises(binding.DresdError) as e:
        binding.Store(k, torch.zeros((8, 2), dtype=torch.int32, device="cuda"), "f16")
    assert e.value.status == -1


def test_bounded_wait_reports_timeout_and_store_stays_usable():
    """Failure detection without a GPU fault: one CTA never receives one pipeline stage
    (a barrier that nothing completes); every wait on it runs out after 100 ms, the
    kernel returns in an orderly way, the status word says TIMEOUT, and the next call
    on the same store is correct again."""
    N, d, dtype = 60013, 128, "f16"
    keys, toks = synth.make_store(8401, N, d, 16, dtype, 4)
    q, _ = synth.make_queries(8402, keys, dtype, 2, 0.1)
    st = gpu_store(keys, toks, dtype)
    st.set_option("scan_path", 1)
    good = gpu_retrieve(st, q, 10, 4)
    st.set_option("wait_ms", 100)
    st.set_option("debug_lose_stage", 2)
    import torch
    st.retrieve(binding.to_device(q, dtype), 10, 4)
    torch.cuda.synchronize()
    with pytest.raises(binding.DresdError) as e:
        st.status()
    assert e.value.status == -5
    st.set_option("debug_lose_stage", 0)
    st.set_option("wait_ms", 0)
    again = gpu_retrieve(st, q, 10, 4)               # status() inside: clean again
    assert all(np.array_equal(a, b) for a, b in zip(good, again))
    st.close()


# 33-64 queries on rows of 129-256 elements run the tcgen05 kernel with the operand roles
# swapped (queries = M operand, keys = N = 256 operand).  Both forms against the oracle.
@pytest.mark.parametrize("keys_as_m", [0, 1], ids=["keys_as_n", "keys_as_m"])
@pytest.mark.parametrize("dtype,d,B,n,L,N", [
    ("bf16", 256, 64, 32, 16, 148 * 256 * 3 + 77),     # several tiles per CTA, ragged tail
    ("f16", 256, 33, 10, 4, 256 * 7 + 1),              # fewer tiles than CTAs, one key in the last tile
    ("bf16", 192, 48, 32, 3, 40009),                   # three slabs per row
    ("f16", 136, 64, 5, 3, 20011),                     # row = 272 bytes, last slab mostly padding
    ("bf16", 256, 40, 32, 2, 100),                     # a single partial tile
    ("f16", 200, 57, 1, 1, 33333),                     # top-1
])
def test_parity_wide_batches_both_operand_orders(keys_as_m, dtype, d, B, n, L, N):
    keys, toks = synth.make_store(7400 + d + B, N, d, 32, dtype, L + 1)
    q, _ = synth.make_queries(7450 + d + B, keys, dtype, B, 0.1)
    _check(keys, toks, dtype, q, n, L, options={"keys_as_m": keys_as_m})


def test_wide_batch_adversarial_order_and_agreement_of_both_forms():
    """Ascending scores in memory (every key beats all before it: queue overflow and resume),
    checked against the oracle; then the two operand orders must return the same rows, with
    scores equal to fp32 rounding."""
    N, d, dtype, B, n = 30000, 256, "bf16", 64, 32
    keys, toks = synth.make_store(7470, N, d, 4, dtype, 2)
    q, _ = synth.make_queries(7471, keys, dtype, B, 0.1)
    s = oracle.scores(keys, dtype, oracle.preprocess(q[:1], dtype)[0])
    order = np.argsort(s, kind="stable")
    keys, toks = keys[order], toks[order]
    _check(keys, toks, dtype, q, n, 2, options={"keys_as_m": 0})
    st = gpu_store(keys, toks, dtype)
    try:
        outs = []
        for form in (0, 1):
            st.set_option("keys_as_m", form)
            outs.append(gpu_retrieve(st, q, n, 2))
        np.testing.assert_allclose(outs[0][1], outs[1][1], rtol=0, atol=2e-6)
        same = np.mean(outs[0][0] == outs[1][0])
        assert same >= 0.99                               # near-ties may swap within fp32 rounding
    finally:
        st.close()


def test_retrieve_can_be_captured_in_a_cuda_graph_and_replayed():
    """dresd_retrieve enqueues kernels only (no allocation, no host synchronisation), so a
    serving loop can capture it once and replay it: the replay must use the CURRENT contents
    of the query buffer and give the same result as a direct call."""
    import torch
    dtype, N, d, B, n, L = "f16", 60011, 256, 4, 10, 5
    keys, toks = synth.make_store(7600, N, d, 16, dtype, L)
    q1, _ = synth.make_queries(7601, keys, dtype, B, 0.1)
    q2, _ = synth.make_queries(7602, keys, dtype, B, 0.1)
    st = gpu_store(keys, toks, dtype)
    try:
        want1 = gpu_retrieve(st, q1, n, L)
        want2 = gpu_retrieve(st, q2, n, L)
        qbuf = binding.to_device(q1, dtype)
        ids = torch.empty((B, n), dtype=torch.int32, device="cuda")
        sc = torch.empty((B, n), dtype=torch.float32, device="cuda")
        tok = torch.empty((B, n, L), dtype=torch.int32, device="cuda")
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            for _ in range(2):          # warm-up outside the capture (function attributes, lazy loading)
                binding.dresd_retrieve(st.handle, qbuf.data_ptr(), B, n, L, ids.data_ptr(), sc.data_ptr(),
                                       tok.data_ptr(), side.cuda_stream)
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            binding.dresd_retrieve(st.handle, qbuf.data_ptr(), B, n, L, ids.data_ptr(), sc.data_ptr(),
                                   tok.data_ptr(), torch.cuda.current_stream().cuda_stream)
        for q, want in ((q1, want1), (q2, want2), (q1, want1)):
            qbuf.copy_(binding.to_device(q, dtype))
            g.replay()
            torch.cuda.synchronize()
            st.status()
            assert np.array_equal(ids.cpu().numpy(), want[0])
            assert np.array_equal(sc.cpu().numpy(), want[1])
            assert np.array_equal(tok.cpu().numpy(), want[2])
    finally:
        st.close()


@pytest.mark.parametrize("dtype,d,B", [("f16", 256, 2), ("bf16", 256, 40), ("f32", 128, 3), ("f16", 64, 1)])
def test_non_finite_inputs_neither_hang_nor_fault(dtype, d, B):
    """NaN keys never enter a result (a comparison with NaN is false); the other rows are ranked
    as if the NaN rows scored nothing; a NaN query selects nothing at all.  The calls return, the
    health word stays clean and the store remains usable."""
    import torch
    N, n, L = 30011, 10, 3
    keys, toks = synth.make_store(7700 + d, N, d, 16, dtype, L)
    q, _ = synth.make_queries(7701 + d, keys, dtype, B, 0.1)
    bad = np.array([0, 5, 777, 12345, N - 1])
    poisoned = keys.copy()
    nan_bits = {"f16": np.float16(np.nan), "f32": np.float32(np.nan)}.get(dtype)
    if dtype == "bf16":
        poisoned[bad, 3] = np.uint16(0x7FC0)
    else:
        poisoned[bad, 3] = nan_bits
    zeroed = keys.copy()
    zeroed[bad] = 0                                     # a zero row scores 0, far below the neighbours
    st = gpu_store(poisoned, toks, dtype)
    try:
        ids, sc, tok = gpu_retrieve(st, q, n, L)
        assert not np.isin(ids, bad).any() and np.all(ids >= 0) and np.all(np.isfinite(sc))
        o = oracle.retrieve(zeroed, toks, dtype, q, n, L, want_full_scores=True)
        checker.check_batch(o.full_scores, toks, ids, sc, tok, dtype, n, L, oracle_ids=o.ids)
        qn = q.copy()
        if dtype == "bf16":
            qn[:, 0] = np.uint16(0x7FC0)
        else:
            qn[:, 0] = nan_bits
        ids2, sc2, tok2 = gpu_retrieve(st, qn, n, L)    # gpu_retrieve checks the health word
        assert np.all(ids2 == -1) and np.all(sc2 == -np.inf) and np.all(tok2 == -1)
        ids3, _, _ = gpu_retrieve(st, q, n, L)          # and the store still answers
        assert np.array_equal(ids3, ids)
    finally:
        st.close()


# The corners of the supported envelope: the widest rows with the widest batch (query operand
# streamed with the keys), the narrowest rows the loader accepts (16 bytes), the longest lists.
@pytest.mark.parametrize("dtype,d,B,n,L,N", [
    ("bf16", 4096, 64, 32, 2, 1501),
    ("f16", 8, 1, 1, 1, 100),
    ("f16", 8, 64, 32, 1, 5000),
    ("f32", 4096, 8, 32, 2, 1201),
    ("f32", 4, 9, 3, 1, 777),
    ("bf16", 264, 64, 32, 1, 30011),           # five slabs: the 33-64 query kernel hands over to the other form
])
def test_parity_envelope_corners(dtype, d, B, n, L, N):
    keys, toks = synth.make_store(7800 + d + B, N, d, 8, dtype, L)
    q, _ = synth.make_queries(7850 + d + B, keys, dtype, B, 0.1)
    _check(keys, toks, dtype, q, n, L)


def test_host_call_with_pinned_and_with_pageable_buffers():
    """Pinned buffers are read and written by the kernels directly; pageable ones go through
    staging copies.  Same results either way, equal to the device-buffer call."""
    import torch
    dtype, N, d, B, n, L = "f16", 40009, 128, 5, 10, 4
    keys, toks = synth.make_store(7900, N, d, 16, dtype, L)
    q, _ = synth.make_queries(7901, keys, dtype, B, 0.1)
    st = gpu_store(keys, toks, dtype)
    try:
        ref = gpu_retrieve(st, q, n, L)
        for pinned in (True, False):
            qh = torch.from_numpy(q.copy())
            outs = [torch.full((B, n), -7, dtype=torch.int32), torch.full((B, n), -7.0, dtype=torch.float32),
                    torch.full((B, n, L), -7, dtype=torch.int32)]
            if pinned:
                qh = qh.pin_memory()
                outs = [o.pin_memory() for o in outs]
            assert qh.is_pinned() == pinned
            st.retrieve_host(qh, n, L, tuple(outs))
            for a, b in zip(ref, outs):
                assert np.array_equal(a, b.numpy())
    finally:
        st.close()

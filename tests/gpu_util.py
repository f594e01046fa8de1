"""Helpers for the GPU parity tests: run the CUDA path and the oracle on the same inputs."""
from __future__ import annotations

import numpy as np

import oracle
from paper_2502_15572_b200 import binding


def gpu_store(keys, toks, dtype):
    import torch
    k = binding.to_device(keys, dtype)
    t = torch.from_numpy(np.ascontiguousarray(toks)).cuda()
    return binding.Store(k, t, dtype)


def gpu_retrieve(store, queries, top_n, draft_len):
    """Upload queries (numpy, store dtype), run dresd_retrieve, return numpy (ids, scores, tokens)."""
    import torch
    q = binding.to_device(queries, store.dtype)
    ids, sc, tok = store.retrieve(q, top_n, draft_len)
    torch.cuda.synchronize()
    store.status()
    return ids.cpu().numpy(), sc.cpu().numpy(), tok.cpu().numpy()


def run_both(keys, toks, dtype, queries, top_n, draft_len, pre=None, options=None, threads=None):
    """Returns ``(gpu_ids, gpu_scores, gpu_tokens, oracle_result)``; pre = dict(mean,var,eps_z,W,pca_mean)."""
    import torch
    pre = pre or {}
    st = gpu_store(keys, toks, dtype)
    try:
        if pre:
            dev = {}
            for name in ("mean", "var", "pca_mean"):
                v = pre.get(name)
                dev[name] = None if v is None else torch.from_numpy(np.asarray(v, dtype=np.float32)).cuda()
            W = pre.get("W")
            dev["W"] = None if W is None else binding.to_device(W, dtype)
            st.set_preprocess(queries.shape[1], dev["mean"], dev["var"], pre.get("eps_z", 1e-5),
                              dev["W"], dev["pca_mean"])
        for k, v in (options or {}).items():
            st.set_option(k, v)
        g = gpu_retrieve(st, queries, top_n, draft_len)
    finally:
        st.close()
    o = oracle.retrieve(keys, toks, dtype, queries, top_n, draft_len,
                        mean=pre.get("mean"), var=pre.get("var"), eps_z=pre.get("eps_z", 1e-5),
                        W=pre.get("W"), pca_mean=pre.get("pca_mean"), want_full_scores=True,
                        threads=threads or oracle.dresd_oracle.default_threads())
    return g[0], g[1], g[2], o

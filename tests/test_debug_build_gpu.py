"""The bounds-checked debug build (libdresd_debug.so, -DDRESD_DEBUG_BOUNDS).

No memory checker can be run on the GPUs this library is tested on, so the library carries its own
checks: in the debug build every global index and pipeline-ring slot the kernels form is tested where
it is formed, and a violation is reported through the status word instead of being dereferenced.
The tests run a cross-section of the kernels (every scoring kernel, ragged sizes, filter, windows,
quantised search, projection) in a child process with DRESD_DEBUG=1: results must match the oracle
and no check may fire.  A self-test fails one check on purpose -- without attempting the access --
to show that a violation would be seen.
"""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r'''
import sys
import numpy as np
import torch
import oracle
from paper_2502_15572_b200 import binding, build as lib_build, synth
from tests import checker
from tests.gpu_util import gpu_store, run_both

lib_build.build(debug=True)
assert binding.dresd_debug_build() == 1, "the release library was loaded"

# the reporting path: check 7 fails on purpose, the access is skipped, the status names the site
keys, toks = synth.make_store(1, 2000, 64, 4, "f16", 2)
st = gpu_store(keys, toks, "f16")
binding.dresd_store_debug_selftest(st.handle, 0)
try:
    st.status()
    raise SystemExit("the failed check was not reported")
except binding.DresdError as e:
    assert e.status == -6 and "check 7" in e.message, (e.status, e.message)
st.status()                                   # the word is cleared: clean again
st.close()

cases = [  # dtype, d, B, n, L, N, options
    ("f16", 256, 1, 10, 4, 148 * 128 * 2 + 37, {}),
    ("bf16", 64, 5, 10, 3, 50021, {}),
    ("f16", 32, 3, 10, 2, 60014, {}),                  # two keys per row
    ("bf16", 64, 40, 10, 2, 60013, {}),                # one column per query
    ("bf16", 256, 40, 32, 2, 148 * 256 + 5, {}),       # keys as N
    ("f16", 512, 64, 10, 2, 20011, {}),                # two sub-tiles sharing an operand slab
    ("bf16", 4096, 16, 10, 2, 2003, {}),               # travelling query operand
    ("f16", 128, 6, 10, 2, 40009, {"scan_path": 1}),   # streaming kernel
    ("f32", 128, 8, 10, 2, 148 * 512 + 19, {}),
    ("f16", 256, 3, 5, 2, 1, {}),                      # one row
    ("bf16", 256, 64, 32, 2, 33, {}),
]
for dtype, d, B, n, L, N, opt in cases:
    keys, toks = synth.make_store(100 + d + B, N, d, 16, dtype, L + 1)
    q, _ = synth.make_queries(101 + d + B, keys, dtype, B, 0.1)
    n = min(n, N)
    ids, sc, tok, o = run_both(keys, toks, dtype, q, n, L, options=opt)     # status() inside: no check fired
    checker.check_batch(o.full_scores, toks, ids, sc, tok, dtype, n, L, oracle_ids=o.ids)

# first-token filter, token windows and the quantised search on a sorted store
dtype, d, B, n, L, N = "f16", 64, 9, 5, 2, 50021
keys, toks = synth.make_store(300, N, d, 16, dtype, L + 1, vocab=50)
keys, toks = synth.sort_by_first_token(keys, toks)
q, src = synth.make_queries(301, keys, dtype, B, 0.1)
ft = np.ascontiguousarray(toks[src, 0]).astype(np.int32)
st = gpu_store(keys, toks, dtype)
st.index_first_tokens()
st.attach_quantised()
dq, dft = binding.to_device(q, dtype), torch.from_numpy(ft).cuda()
win = [t.cpu().numpy() for t in st.retrieve_filtered(dq, dft, n, L)]
st.set_option("first_token_windows", 0)
full = [t.cpu().numpy() for t in st.retrieve_filtered(dq, dft, n, L)]
qz = [t.cpu().numpy() for t in st.retrieve_quantised(dq, n, L, 32, first_tokens=dft)]
torch.cuda.synchronize()
st.status()
st.close()
assert all(np.array_equal(a, b) for a, b in zip(win, full))
o = oracle.retrieve(keys, toks, dtype, q, n, L, first_token=ft, want_full_scores=True, threads=4)
for b in range(B):
    checker.check_query_filtered(o.full_scores[b], toks, win[0][b], win[1][b], win[2][b], dtype, n, L, int(ft[b]))
    assert np.all((qz[0][b] < 0) | (toks[np.maximum(qz[0][b], 0), 0] == ft[b]))
print("debug build ok")
'''


@pytest.mark.gpu
def test_kernels_under_the_bounds_checked_build():
    env = dict(os.environ, DRESD_DEBUG="1", PYTHONPATH=ROOT + os.pathsep + os.environ.get("PYTHONPATH", ""))
    r = subprocess.run([sys.executable, "-c", CHILD], capture_output=True, text=True, env=env, cwd=ROOT, timeout=900)
    assert r.returncode == 0 and "debug build ok" in r.stdout, (r.stdout[-2000:], r.stderr[-3000:])


def test_debug_library_builds_and_exports_the_same_symbols():
    """CPU: the debug build compiles for sm_100a, loads, and exports every entry point of the release build."""
    import ctypes
    from paper_2502_15572_b200 import binding, build as lib_build
    path = lib_build.build(debug=True)
    lib = ctypes.CDLL(path)
    for name in binding.EXPORTS:
        assert hasattr(lib, name), name
    lib.dresd_debug_build.restype = ctypes.c_int
    assert lib.dresd_debug_build() == 1
    assert binding.dresd_debug_build() == (1 if os.environ.get("DRESD_DEBUG") == "1" else 0)

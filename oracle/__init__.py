"""CPU oracle for the DReSD retrieval path: test infrastructure only.

Only tests, the smoke check and the benchmark's CPU-baseline leg may import
this package.  It never imports the CUDA package.
"""
from .dresd_oracle import (  # noqa: F401
    build,
    decode,
    preprocess,
    fit_zscore,
    scores,
    retrieve,
    OracleResult,
    drafts_prepare,
    drafts_accept,
    e4m3_decode,
    e4m3_encode,
    quantised_scores,
    retrieve_quantised,
)

"""CPU oracle (test infrastructure only): see oracle.py and calidrop_oracle.c."""
from .oracle import (  # noqa: F401
    build_oracle,
    calibrate_given_indices,
    compress,
    decode,
    full_attention,
    max_threads,
    pool_votes,
    topk,
)

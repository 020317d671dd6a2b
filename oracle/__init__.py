"""CPU oracle (test infrastructure only): see oracle.py and calidrop_oracle.c."""
from .oracle import (  # noqa: F401
    accumulated_attention,
    build_oracle,
    calibrate_given_indices,
    compress,
    decode,
    full_attention,
    max_threads,
    pool_votes,
    select_from_scores,
    streaming_indices,
    topk,
)

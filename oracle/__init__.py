"""CPU oracle for the verify / prune / accept step.  TEST INFRASTRUCTURE ONLY.

A plain, slow, fp64 numpy restatement of what the hot path computes, written
from the paper's definitions (Sec. 2.2 for the accept rule and residual
resampling; Eq. 2 and Eq. 3 for the variation score and Top-K; Sec. 4.2 for
what the draft context keeps; textbook scaled-dot-product attention for the
verification pass, which the paper uses unchanged; Algorithm 1 and the appendix
on the parallel pipeline for the Pre-/Post-verify mode machine).

It shares no code with the CUDA path and must never be imported by it: only
the tests, the smoke check and the bench's CPU-baseline leg may call it.
Every function here is pinned by CPU tests to something other than itself
(brute force on tiny inputs, closed forms, library routines, distributional
tests); none is "parity unpinned".
"""
from .attention import bf16_bits_to_f64, verify_attn  # noqa: F401
from .uvprune import (variation_score, select_topk, gather_rows, cosine_similarity, similarity_sum,  # noqa: F401
                      similarity_variation)
from .accept import softmax64, spec_accept, window_size, window_size_rounded  # noqa: F401
from .pipeline import Schedule, parallel_decode, simulate_iid  # noqa: F401

"""B200-native verify / prune / accept hot path of ParallelVLM's draft-then-verify loop.

`binding` marshals torch tensors into the C ABI of libpvlm.so (include/pvlm.h);
`workloads` draws the seeded synthetic inputs; `build` compiles the library.
"""
from . import workloads  # noqa: F401
from .binding import (PvlmError, lib, spec_accept, uvprune_select_gather, uvprune_similarity, verify_attn)  # noqa: F401

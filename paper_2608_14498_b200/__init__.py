"""B200-native prefix/suffix scoring kernels (sm_100a) behind a small C ABI.

``prefix_attn``, ``suffix_attn`` and ``token_logprobs`` marshal arguments into the shared library
built from ``csrc/``; every step of the scoring path runs in those CUDA kernels.  There is no CPU
or eager fallback: a missing library or a non-sm_100 device is an error.
"""
from .binding import (  # noqa: F401
    RpxError,
    attn_backward,
    attn_backward_workspace_bytes,
    chunk_attn,
    get_lm_head_pairing,
    get_sm_budget,
    library_path,
    load_library,
    prefix_attn,
    prefix_attn_workspace_bytes,
    selftest_bounded_wait,
    set_lm_head_pairing,
    set_sm_budget,
    status_string,
    suffix_attn,
    suffix_attn_workspace_bytes,
    token_logprobs,
    token_logprobs_backward,
    token_logprobs_backward_workspace_bytes,
    token_logprobs_merge,
    token_logprobs_shard,
    token_logprobs_static,
    token_logprobs_workspace_bytes,
    version,
)

"""B200-native segment-level causal attention: thin Python binding over the C-ABI library.

Every step of the path runs in the CUDA kernels of ``libsegattn.so``; this package only
marshals arguments.  PyTorch supplies device memory and streams.
"""
from .binding import (SegAttnError, Prefill, count_pairs, gather_context, gather_context_rope, launch_count, lib, params_for, poll_status,
                      profile_kernels, retrieval_select, rope_apply, rope_table, seg_attn_bwd, seg_attn_bwd_static, seg_attn_fwd, seg_attn_step_host, selftest_wait_timeout, workspace_bytes)

__all__ = ["SegAttnError", "Prefill", "count_pairs", "gather_context", "gather_context_rope", "launch_count", "lib", "params_for", "poll_status",
           "profile_kernels", "retrieval_select", "rope_apply", "rope_table", "seg_attn_bwd", "seg_attn_bwd_static", "seg_attn_fwd", "seg_attn_step_host", "selftest_wait_timeout", "workspace_bytes"]

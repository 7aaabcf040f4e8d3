"""B200-native speculative-decoding rollout step: ctypes binding of the libgm CUDA library.

The package holds the CUDA sources (csrc/), the in-tree build (build.py) and a thin binding
(binding.py) whose functions carry the names of the C ABI in include/gm.h.  There is no CPU
fallback: every entry point raises if libgm.so is not built or no sm_100 device is present.
"""
from .binding import (  # noqa: F401
    Context, State, GmError, lib, pack_weights, random_packed_weights,
    gm_draft, gm_verify, gm_accept, gm_spec_step, gm_spec_step_host, gm_draw, gm_prefill, gm_rollout_begin, gm_rollout_step, gm_rollout_run, Rollout, gm_pages_reset, gm_pages_reserve, gm_pages_release, gm_pages_free_count, gm_capture_hidden, gm_head_prefill, gm_reconstruct, gm_head_state_grad, gm_head_ffn_backward, gm_attention_backward, gm_head_attn_backward, gm_head_update_backward, gm_head_update_step, head_grad_buffers, gm_head_input_backward, gm_adamw_step, gm_overlap, gm_dca_loss, gm_dca_grad, gm_set_top_p, gm_nucleus, gm_gemm, gm_gemm_swiglu, gm_attention, gm_attention_noalloc, gm_record_begin, gm_record_end, gm_spec_step_rec, Record,
    gm_profile, gm_profile_read, gm_chain_trace, gm_chain_trace_read, gm_selftest_wait_expiry, gm_launch_count, gm_last_status, gm_strerror,
    GM_OK, GM_ERR_INVALID_ARG, GM_ERR_UNSUPPORTED, GM_ERR_KV_CAPACITY, GM_ERR_CUDA,
    GM_ERR_DEVICE_TIMEOUT, GM_ERR_BAD_PAGE, GM_ERR_NO_EXTENSION, GM_ERR_SCRATCH_LIMIT, GM_ERR_OVERRUN, GM_NOALLOC_SCRATCH_BYTES, GM_NOALLOC_MAX_BATCH, GM_FLAG_SIMPLE_GEMM, GM_FLAG_SAMPLER_CLUSTER, GM_FLAG_SAMPLER_STREAM, GM_FLAG_SAMPLER_FLOW, GM_FLAG_GRAPH,
    GM_KC_GEMM, GM_KC_ATTENTION, GM_KC_ELEMENTWISE, GM_KC_SAMPLER, GM_KC_RECORD, EXPORTS,
)

"""B200-native Fork-dLLM confidence pass: a C-ABI CUDA library (csrc/, include/fork_dllm.h) and a
thin ctypes binding with the same entry-point names."""
from .binding import (  # noqa: F401
    FORK_BF16, FORK_DEV_TIMEOUT, FORK_DEV_WINDOW_CLAMPED, FORK_ERR_CUDA, FORK_ERR_INVALID_ARG, FORK_ERR_MAX_STEPS,
    FORK_ERR_PROVIDER, FORK_ERR_WORKSPACE, FORK_F32, FORK_OK, FORK_ROW_BAD_TOKEN, FORK_ROW_NONFINITE,
    FORK_TUNE_CTAS_PER_SM, FORK_TUNE_L2_EVICT_FIRST, FORK_TUNE_MIN_UNITS, FORK_TUNE_LOOP_AHEAD, FORK_TUNE_LATE_CTA, FORK_TUNE_ONE_KERNEL, FORK_TUNE_PDL, FORK_TUNE_STAGES, FORK_TUNE_VARIANT, ForkError, ForkState, fork_decode_loop,
    fork_device_status, fork_kernel_launches, fork_mask_handovers, fork_logits_fn, fork_logprob, fork_logprob_args, fork_set_tuning,
    FORK_FALLBACK_LEFTMOST, FORK_FALLBACK_MAX_CONF, FORK_FALLBACK_MAX_ENTROPY, FORK_FALLBACK_MIN_CONF,
    FORK_FALLBACK_RANDOM, fork_select_top_entropy, fork_grpo_loss, fork_grpo_args, fork_logprob_backward, fork_grpo_fused, fork_grpo_fused_args,
    fork_logprob_bwd_args, fork_vp_reduce, fork_vp_reduce_peers, fork_vp_select, fork_step_vocab_parallel, gather_rank_major, vocab_shards,
    fork_status_string, fork_step, fork_step_args, fork_step_static, fork_step_fused_head, fork_decode_loop_fused_head, fork_head_args, FORK_STATIC_SCRATCH_BYTES, fork_workspace_bytes, lib, make_step_args,
)

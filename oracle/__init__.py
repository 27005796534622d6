"""CPU oracle for the pruned-GRPO hot path (DPPO).

TEST INFRASTRUCTURE ONLY.  This package is a plain, slow, float64 restatement
of what the paper defines.  It is imported by the tests, by the smoke check and
by the benchmark's CPU-baseline / reference legs; the product path never calls
it.  It shares no code, tables or constants with the CUDA library.

Parity status: every public function below is pinned by at least one test that
does not go through the function itself (closed forms, invariants, brute
force, published known-answer vectors); none is "parity unpinned".
"""
from .philox import philox4x32_10, uniform53
from .dppo_oracle import (
    group_advantages,
    completion_candidates,
    prompt_candidates,
    draw_uniforms,
    prune_masks,
    rescale,
    prune_and_rescale,
    history_epochs,
    pack_prompts,
    bf16_bits_to_f64,
    f64_to_bf16_bits,
    token_logprob,
    sequence_log_ratio,
    token_terms,
    grpo_loss,
    lmhead_grpo_loss,
)

__all__ = [
    "philox4x32_10", "uniform53",
    "group_advantages", "completion_candidates", "prompt_candidates",
    "draw_uniforms", "prune_masks", "rescale", "prune_and_rescale", "history_epochs",
    "pack_prompts", "bf16_bits_to_f64", "f64_to_bf16_bits",
    "token_logprob", "sequence_log_ratio", "token_terms", "grpo_loss", "lmhead_grpo_loss",
]

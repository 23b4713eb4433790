"""CPU oracle for the MLPMoE forward path (test infrastructure, not product code).

Only the test suite, the smoke check and the benchmark's CPU-baseline leg may
import this package.  It shares no code with the CUDA library.
"""
from .mlpmoe_oracle import (  # noqa: F401
    branch_offsets,
    silu,
    branch_forward,
    mlpmoe_forward,
    mlpmoe_forward_h_bf16,
    routed_forward,
    fade_schedule,
    fade_position,
    fade_mask,
    fade,
    neuron_scores,
    fade_structured_count,
    fade_structured,
    prune_alpha,
    first_k_keep,
    nnz_per_branch,
    live_neurons,
    surviving_set,
    mlpmoe_forward_skiplist,
    round_to_bf16,
    rmsnorm,
    stack_forward,
)

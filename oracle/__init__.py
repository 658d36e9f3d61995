"""CPU float64 oracle for one CAST draft-and-verify step.

TEST INFRASTRUCTURE ONLY.  Nothing here is part of the product path: only the
tests, the smoke check and the benchmark's CPU-baseline leg may import it.  It
shares no code with the CUDA library and never receives values computed by it.
"""
from .cast_oracle import (  # noqa: F401
    CostTable,
    OracleConfig,
    CastOracle,
    select_grid,
    alg1_select_max_valid_index,
    alg1_is_stable,
    topk_children,
    log_sum_exp,
    tree_attention,
    greedy_accept,
    stochastic_accept,
    compact_kv,
    ancestor_masks,
)

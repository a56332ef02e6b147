"""CPU oracle of the unified-memory-pool hot path -- TEST INFRASTRUCTURE.

Only tests, the smoke check and the benchmark's CPU-baseline leg may import
this package.  It never imports the CUDA library or its binding.
"""
from .flowpool_oracle import (  # noqa: F401
    OraclePool, OraclePlan, PlanConfig, PoolConfig, build_oracle, lib,
    plan_from_lengths, bestfit_segment_tree, balance, f32_to_bf16_rne, cost_int, STATUS,
)

"""Float64 CPU oracle for the SAKI per-position routing path.

TEST INFRASTRUCTURE ONLY.  Nothing in the product path may import this
package: only the tests, the smoke check and the benchmark's CPU-baseline
leg do.  It shares no code with the CUDA library.
"""
from .saki_oracle import (  # noqa: F401
    STAGE_PROPOSE, STAGE_ACCEPT, STAGE_RESIDUAL, STAGE_BONUS,
    ST_SATURATED, ST_EPS_ZERO, ST_MASKED, ST_NONFINITE, ST_BAD_ID,
    ST_TIMEOUT, ST_NOT_COMPUTED,
    philox4x32_10, uniform_from_word, scalar_uniform,
    log_softmax, bridge_stats, solve_lambda, bridge_distribution,
    total_variation, inverse_cdf_draw, round_to_bf16,
    route_row, route, sample_proposal_row, sample_proposal, spec_verify,
    bwd_from_meta_row, bwd_from_meta,
    STAGE_SELECT, SELECT_RANDOM, SELECT_TV_WEIGHTED, select_tm,
    lmhead_lse,
)

"""B200-native SAKI per-position routing: thin Python binding over the C-ABI
library built from csrc/.  Importing the package does not load the CUDA
library; the first call does, and raises if it is missing (no CPU fallback)."""
from .binding import (  # noqa: F401
    load_library, lmhead_lse, vshard_in, vshard_partial, vshard_combine, vshard_combine_host, VSHARD_PARTIALS, VSHARD_STATE, route_fwd, route_fwd_bwd, route_fwd_bwd_noalloc, route_bwd_from_meta, select_tm, SELECT_RANDOM, SELECT_TV_WEIGHTED, alloc_outputs, route_host, spec_verify, sample_proposal,
    check, set_kernel, last_kernel, redo_count, set_spec_early_out, spec_positions_routed, solve_evaluations, set_wait_limit, set_phase_clock, phase_cycles, PHASES, launch_count, last_error, version, SakiError,
)

"""The row-per-SM kernel's phase clock: off by default, changes no result, and its sums add up."""
import pytest
import torch

import paper_2609_36601_b200 as P
from paper_2609_36601_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def test_phase_clock_counts_rows_and_leaves_results_alone():
    w = synth.Workload("clock", 300, 32000, "bf16", 0.05, 1.0, True, 77, 5)
    d = synth.generate(w, DEV)
    prev_k = P.set_kernel(3)
    try:
        out0, g0 = P.route_fwd_bwd(d["s"], d["t"], d["proposal"], w.eps, seed=w.seed)
        off = P.phase_cycles()
        assert all(v == 0 for v in off.values())          # the clock is off unless asked for
        prev = P.set_phase_clock(True)
        assert prev is False
        out1, g1 = P.route_fwd_bwd(d["s"], d["t"], d["proposal"], w.eps, seed=w.seed)
        on = P.phase_cycles()
        P.set_phase_clock(False)
        out2 = P.route_fwd(d["s"], d["t"], d["proposal"], w.eps, seed=w.seed)
        assert all(v == 0 for v in P.phase_cycles().values())
    finally:
        P.set_phase_clock(False)
        P.set_kernel(prev_k)
    assert on["rows"] == w.N
    for k in ("lse", "solve", "final", "lse_scalar", "solve_scalar"):
        assert on[k] > 0, k
    # the three passes dominate a row of 32000 elements, and a row takes 10k to 200k cycles
    passes = on["lse"] + on["solve"] + on["final"]
    total = sum(v for k, v in on.items() if k != "rows")
    assert 0.3 * total < passes < total
    assert 1e4 < total / w.N < 2e5
    for k in out0:
        assert torch.equal(out0[k], out1[k]), k
    assert torch.equal(g0, g1)
    for k in out2:
        assert torch.equal(out0[k], out2[k]), k

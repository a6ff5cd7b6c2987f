"""The give-up path of the row-per-SM kernel's bounded wait, exercised without withholding anything: the
wait limit is set to a few cycles, so the wait for a row's bulk copy runs out although the copy is on its
way.  The kernel must return, a row is either flagged TIMEOUT with zero outputs or routed correctly,
saki_check counts the flagged rows, and the next ordinary call is unaffected."""
import numpy as np
import pytest
import torch

import paper_2609_36601_b200 as P
from paper_2609_36601_b200 import binding, synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.mark.parametrize("V,N", [(2048, 64), (32000, 700), (151936, 320)])
def test_expired_wait_flags_rows_and_leaves_the_library_usable(V, N):
    w = synth.Workload("limit", N, V, "bf16", 0.1, 1.5, True, 4100 + V % 97, 9)
    d = synth.generate(w, DEV)
    prev_k = P.set_kernel(3)
    P.check()                                       # clears what earlier tests may have left
    try:
        ref, g_ref = P.route_fwd_bwd(d["s"], d["t"], d["proposal"], w.eps, seed=w.seed)
        torch.cuda.synchronize()
        assert P.last_kernel() == 3 and P.check() == 0
        # the rows out of L2 again, so that the first copies of the limited call come from memory
        flush = torch.empty(320 << 20, dtype=torch.uint8, device=DEV)
        flush.fill_(1)
        torch.cuda.synchronize()
        assert P.set_wait_limit(2) == 0
        out, g = P.route_fwd_bwd(d["s"], d["t"], d["proposal"], w.eps, seed=w.seed)
        assert P.set_wait_limit(0) == 2
        n_flagged = P.check()                       # synchronises: the kernel came back
        again, g_again = P.route_fwd_bwd(d["s"], d["t"], d["proposal"], w.eps, seed=w.seed)
        torch.cuda.synchronize()
        assert P.check() == 0
    finally:
        P.set_wait_limit(0)
        P.set_kernel(prev_k)
    st = out["row_status"].cpu().numpy().astype(np.uint32)
    late = (st & binding.ROW_TIMEOUT) != 0
    assert late.sum() >= 1, "no wait ran out: the limit did not reach the kernel"
    assert n_flagged == int(late.sum())
    lt = torch.as_tensor(late, device=DEV)
    # flagged rows: nothing but the status
    assert np.all(st[late] == binding.ROW_TIMEOUT)
    assert torch.all(out["token"][lt] == -1) and torch.all(out["corrected"][lt] == 0)
    for k in ("lambda", "kl", "tv", "accept_prob", "loss", "logp_x", "logq_y"):
        assert torch.all(out[k][lt] == 0), k
    assert torch.all(g[lt] == 0)
    # the others: exactly what the undisturbed call gives
    for k in out:
        assert torch.equal(out[k][~lt], ref[k][~lt]), k
    assert torch.equal(g[~lt], g_ref[~lt])
    # and the call after it is undisturbed
    for k in again:
        assert torch.equal(again[k], ref[k]), k
    assert torch.equal(g_again, g_ref)

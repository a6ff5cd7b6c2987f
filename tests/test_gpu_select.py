"""Parity of saki_select_tm (placement controls of the paper's ablation) with the oracle, and the two
ablation flows composed from the library's calls."""
import numpy as np
import pytest
import torch

import oracle as O
import paper_2609_36601_b200 as P
from paper_2609_36601_b200 import synth
from parity import to_np64

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _case(lens, seed, p_zero_tv=0.3):
    rng = np.random.default_rng(seed)
    seq = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    N = int(seq[-1])
    C = (rng.random(N) < 0.25).astype(np.uint8)
    tv = (rng.random(N) * (rng.random(N) >= p_zero_tv)).astype(np.float32)
    mask = (rng.random(N) < 0.85).astype(np.uint8)
    st = np.where(rng.random(N) < 0.05, 64, 0).astype(np.int32)
    return seq, C, tv, mask, st


@pytest.mark.parametrize("mode", [P.SELECT_RANDOM, P.SELECT_TV_WEIGHTED])
@pytest.mark.parametrize("lens", [[5, 0, 1, 300, 17, 2048, 63], [9000, 3, 4097], [1] * 40])
def test_selection_matches_oracle(mode, lens):
    seq, C, tv, mask, st = _case(lens, 100 + len(lens))
    t = lambda a: torch.as_tensor(a, device=DEV)
    sel, m = P.select_tm(t(seq), t(C), t(tv), mode, seed=11, row_offset=1 << 20, mask=t(mask), rollout_status=t(st))
    torch.cuda.synchronize()
    rsel, rm, margin = O.select_tm(seq, C, tv, mode, seed=11, row_offset=1 << 20, mask=mask,
                                   rollout_status=st.astype(np.uint32))
    assert np.array_equal(m.cpu().numpy(), rm)
    sel = sel.cpu().numpy()
    for b in range(len(lens)):
        lo, hi = seq[b], seq[b + 1]
        assert sel[lo:hi].sum() == rm[b]
        if margin[b] >= 1e-12:      # the device's log may differ from numpy's in the last bit
            assert np.array_equal(sel[lo:hi], rsel[lo:hi]), b


def test_too_few_positive_tv_is_filled_uniformly():
    tv = np.zeros(600, dtype=np.float32)
    tv[[7, 300]] = [0.3, 0.1]
    C = np.zeros(600, dtype=np.uint8)
    C[:9] = 1
    seq = np.array([0, 600], dtype=np.int64)
    t = lambda a: torch.as_tensor(a, device=DEV)
    sel, m = P.select_tm(t(seq), t(C), t(tv), P.SELECT_TV_WEIGHTED, seed=5)
    rsel, rm, _ = O.select_tm(seq, C, tv, O.SELECT_TV_WEIGHTED, seed=5)
    assert int(m[0]) == 9 and np.array_equal(sel.cpu().numpy(), rsel) and rsel[7] == 1 and rsel[300] == 1


def test_ablation_flows_compose():
    """TV-Weighted-TM and teacher-sampled supervision, composed from routing, selection / sampling and
    the metadata-driven backward, against the same composition of the oracle's functions."""
    w = synth.Workload("t", 96, 4096, "bf16", 0.1, 1.5, True, 61, 17)
    d = synth.generate(w, DEV)
    out = P.route_fwd(d["s"], d["t"], d["proposal"], w.eps, seed=w.seed)
    seq = torch.tensor([0, 40, 41, 96], dtype=torch.int64, device=DEV)
    sel, m = P.select_tm(seq, out["corrected"], out["tv"], P.SELECT_TV_WEIGHTED, seed=9, rollout_status=out["row_status"])
    # positions the control does not choose keep RKL supervision on the trajectory's own token y (the
    # committed one: a correction's residual draw, else the proposal), with the advantage taken at y
    adv = out["logT_y"] - out["logp_y"]
    mo, g = P.route_bwd_from_meta(d["s"], sel, out["token"], out["teacher_top1"], adv, rollout_status=out["row_status"])
    torch.cuda.synchronize()
    s64 = to_np64(d["s"])
    rsel, rm, margin = O.select_tm(seq.cpu().numpy(), out["corrected"].cpu().numpy(), out["tv"].cpu().numpy(),
                                   O.SELECT_TV_WEIGHTED, seed=9, rollout_status=out["row_status"].cpu().numpy())
    assert np.all(margin >= 1e-12) and np.array_equal(sel.cpu().numpy(), rsel)
    ref = O.bwd_from_meta(s64, rsel, out["token"].cpu().numpy(), out["teacher_top1"].cpu().numpy(),
                          adv.cpu().numpy().astype(np.float64), rollout_status=out["row_status"].cpu().numpy(),
                          grad_dtype="bf16")
    assert np.allclose(mo["loss"].cpu().numpy(), ref["loss"], rtol=1e-4, atol=1e-5)
    assert np.max(np.abs(to_np64(g) - ref["grad"])) <= 4e-3
    # teacher-sampled supervision: the target is a draw from T (Gumbel-max under another seed)
    vt = P.sample_proposal(d["t"], 1.0, seed=w.seed + 1000)
    vt_ref, gaps = O.sample_proposal(to_np64(d["t"]), 1.0, seed=w.seed + 1000)
    ok = gaps >= 1e-6
    assert np.array_equal(vt.cpu().numpy()[ok], vt_ref[ok])
    adv = out["logT_x"] - out["logp_x"]
    mo2, g2 = P.route_bwd_from_meta(d["s"], out["corrected"], d["proposal"], vt, adv, rollout_status=out["row_status"])
    torch.cuda.synchronize()
    ref2 = O.bwd_from_meta(s64, out["corrected"].cpu().numpy(), d["proposal"].cpu().numpy(), vt.cpu().numpy(),
                           adv.cpu().numpy().astype(np.float64), rollout_status=out["row_status"].cpu().numpy(),
                           grad_dtype="bf16")
    assert np.allclose(mo2["loss"].cpu().numpy(), ref2["loss"], rtol=1e-4, atol=1e-5)
    assert np.max(np.abs(to_np64(g2) - ref2["grad"])) <= 4e-3


def test_bad_arguments():
    seq = torch.tensor([0, 4], dtype=torch.int64, device=DEV)
    C = torch.zeros(4, dtype=torch.uint8, device=DEV)
    with pytest.raises(P.SakiError):
        P.select_tm(seq, C, None, P.SELECT_TV_WEIGHTED)
    with pytest.raises(P.SakiError):
        P.select_tm(seq, C, None, 7)
    sel, m = P.select_tm(seq, C, None, P.SELECT_RANDOM)
    assert int(sel.sum()) == 0 and int(m[0]) == 0

"""Block verification with early out (Section 3.5: positions behind a sequence's first rejection are
discarded).  The row-per-SM kernel hands out positions in position-major order and passes over those
whose sequence is known to have stopped; every output must be the one the call gives when it routes all
positions and resolves afterwards, and the positions routed must cover the ones verification needs (a
position whose predecessor was still undecided when it was handed out is routed without need: with many
sequences per SM that is rare; with fewer than two per SM the library routes every position in static
order instead)."""
import numpy as np
import pytest
import torch

import oracle as O
import paper_2609_36601_b200 as P
from paper_2609_36601_b200 import synth
from parity import force_second_tier, to_np64

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _case(B, K, V, eps=0.2, sigma=1.5, gen_seed=91, seed=21):
    w = synth.Workload("t", B * (K + 1), V, "bf16", eps, sigma, True, gen_seed, seed, K=K)
    d = synth.generate(w, DEV)
    s3, t3 = d["s"].view(B, K + 1, V), d["t"].view(B, K + 1, V)
    draft = d["proposal"].view(B, K + 1)[:, :K].contiguous()
    return w, d, s3, t3, draft


def _both(s3, t3, draft, eps, seed):
    out = {}
    prev = P.set_spec_early_out(True)
    try:
        for on in (False, True):
            P.set_spec_early_out(on)
            r = P.spec_verify(s3, t3, draft, eps, seed=seed)
            torch.cuda.synchronize()
            assert P.last_kernel() == 3
            out[on] = (r, P.spec_positions_routed())
            P.check()
    finally:
        P.set_spec_early_out(prev)
    return out


def _same(a, b):
    for k in ("n_accept", "next_token", "next_is_correction"):
        assert torch.equal(a[k], b[k]), k
    for k in a["per_pos"]:
        if k == "loss":                      # block verification does not write it
            continue
        x, y = a["per_pos"][k], b["per_pos"][k]
        assert torch.equal(x, y), k          # bit-identical, floats included


def _sms():
    return torch.cuda.get_device_properties(0).multi_processor_count


@pytest.mark.parametrize("B,K,V", [(300, 6, 4096), (640, 16, 2048), (1500, 1, 2048), (7, 16, 8192), (149, 1, 2048), (1, 5, 32000)])
def test_outputs_do_not_depend_on_early_out(B, K, V):
    w, d, s3, t3, draft = _case(B, K, V)
    out = _both(s3, t3, draft, w.eps, w.seed)
    _same(out[True][0], out[False][0])
    n_acc = out[True][0]["n_accept"].cpu().numpy()
    st = out[True][0]["per_pos"]["row_status"].view(B, K + 1).cpu().numpy()
    assert out[False][1] == 0
    # a sequence needs its first n_accept + 1 positions (all K + 1 if every draft token was accepted)
    needed = int(np.minimum(n_acc + 1, K + 1).sum())
    if B < 2 * _sms():
        assert out[True][1] == 0           # few sequences: every position routed, in static order
        return
    assert needed <= out[True][1] <= B * (K + 1)
    if B >= 4 * _sms():
        assert out[True][1] <= needed + (B * (K + 1) - needed) // 4, (needed, out[True][1])   # most of the rest is skipped
    for b in range(B):
        assert np.all(st[b, n_acc[b] + 1:] == P.binding.ROW_NOT_COMPUTED)
        assert np.all(st[b, :n_acc[b] + 1] & P.binding.ROW_NOT_COMPUTED == 0)


def test_early_out_against_the_oracle():
    B, K, V = 2 * _sms() + 5, 5, 4096
    w, d, s3, t3, draft = _case(B, K, V, eps=0.1, gen_seed=92, seed=22)
    res = P.spec_verify(s3, t3, draft, w.eps, seed=w.seed)
    torch.cuda.synchronize()
    assert P.last_kernel() == 3 and 0 < P.spec_positions_routed() < B * (K + 1)
    ref = O.spec_verify(to_np64(s3), to_np64(t3), draft.cpu().numpy(), w.eps, seed=w.seed)
    ok = ref["margin"] >= 1e-6
    assert np.array_equal(res["n_accept"].cpu().numpy()[ok], ref["n_accept"][ok])
    assert np.array_equal(res["next_token"].cpu().numpy()[ok], ref["next_token"][ok])
    assert np.array_equal(res["next_is_correction"].cpu().numpy()[ok], ref["next_is_correction"][ok])


def test_flagged_and_second_tier_positions_inside_sequences():
    B, K, V = 2 * _sms() + 4, 4, 8192
    w, d, s3, t3, draft = _case(B, K, V, gen_seed=93, seed=23)
    s3[3, 1, 17] = float("nan")            # flagged position: verification of sequence 3 stops there
    s3[9, 0, 5] = float("inf")
    draft[20, 2] = -1                      # bad draft id
    force_second_tier(d, [5 * (K + 1) + 0, 5 * (K + 1) + 1, 30 * (K + 1) + K, 41 * (K + 1) + 2])
    out = _both(s3, t3, draft, w.eps, w.seed)
    _same(out[True][0], out[False][0])
    assert P.redo_count() >= 1
    res = out[True][0]
    ref = O.spec_verify(to_np64(s3), to_np64(t3), draft.cpu().numpy(), w.eps, seed=w.seed)
    ok = ref["margin"] >= 1e-6
    assert np.array_equal(res["n_accept"].cpu().numpy()[ok], ref["n_accept"][ok])
    assert np.array_equal(res["next_token"].cpu().numpy()[ok], ref["next_token"][ok])
    n_acc = res["n_accept"].cpu().numpy()
    assert n_acc[3] <= 1 and n_acc[9] == 0 and n_acc[20] <= 2
    # positions that went to the second tier do not end their sequence by themselves: the walk goes on
    # behind them, so at least the needed positions were routed
    assert out[True][1] >= int(np.minimum(n_acc + 1, K + 1).sum())


def test_strided_sequences_and_a_second_stream():
    B, K, V = 2 * _sms() + 14, 3, 2048
    w, d, s3, t3, draft = _case(B, K, V, gen_seed=94, seed=24)
    pad_s = torch.zeros((B, K + 3, V + 64), dtype=torch.bfloat16, device=DEV)
    pad_t = torch.zeros_like(pad_s)
    pad_s[:, 1:K + 2, :V] = s3
    pad_t[:, 1:K + 2, :V] = t3
    a = P.spec_verify(s3, t3, draft, w.eps, seed=w.seed)
    st = torch.cuda.Stream()
    st.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(st):
        b = P.spec_verify(pad_s[:, 1:K + 2, :V], pad_t[:, 1:K + 2, :V], draft, w.eps, seed=w.seed, stream=st)
    torch.cuda.synchronize()
    _same(a, b)
    assert P.spec_positions_routed(st) > 0

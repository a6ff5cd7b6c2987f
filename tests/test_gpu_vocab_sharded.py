"""Vocabulary-sharded routing on the GPU: the rows' columns cut into 2, 8 and uneven slices, every slice
reduced by its own kernel calls (one rank after the other on the one device: the same calls, in the same
order, that one rank per GPU makes around its all-gather), against the float64 oracle on the whole rows and
against the unsharded call.  Both families of slice kernels: the float32 ones (bf16 slices on 16-byte
boundaries, eps >= 0.02; the default) and the float64 ones (everything else, and under set_kernel(1))."""
import numpy as np
import pytest
import torch

import oracle as O
import paper_2609_36601_b200 as P
from paper_2609_36601_b200 import synth
from paper_2609_36601_b200.vshard import route_vocab_sharded_local, split_columns
from parity import compare_rows, grad_check, oracle_inputs, to_np64

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _slices(d, cuts):
    return [(d["s"][:, a:a + n], d["t"][:, a:a + n], a) for a, n in cuts]


def _special_rows(d, w):
    mask = torch.ones(w.N, dtype=torch.uint8, device=DEV)
    mask[3] = 0
    d["proposal"][5] = w.V + 1                                    # bad id
    d["s"][6, w.V // 2 + 11] = float("nan")                        # non-finite, in the second half of the row
    d["t"][8] = (d["s"][8].float() + 0.01).to(d["t"].dtype)        # teacher = student up to a constant: lambda = 1
    return mask


@pytest.mark.parametrize("tier", ["f32", "f64"])
@pytest.mark.parametrize("V,world", [(151936, 2), (151936, 8), (32000, 3), (1000, 7)])
def test_sliced_rows_match_the_oracle_and_the_unsharded_call(V, world, tier):
    w = synth.Workload("vs", 40, V, "bf16", 0.1, 1.5, True, 900 + world, 40 + world)
    d = synth.generate(w, DEV)
    mask = _special_rows(d, w)
    cuts = split_columns(V, world)
    if world == 7:                                               # uneven, with an empty slice in the middle
        cuts = [(0, 100), (100, 0), (100, 250), (350, 1), (351, 349), (700, 299), (999, 1)]
    prev = P.set_kernel(1 if tier == "f64" else 0)
    try:
        out, gs, waves = route_vocab_sharded_local(_slices(d, cuts), V, d["proposal"], w.eps, w.temperature, w.seed, mask=mask,
                                                   grad_scale=0.5)
        torch.cuda.synchronize()
    finally:
        P.set_kernel(prev)
    g = torch.cat(gs, dim=1)
    assert 1 <= waves <= 6
    s64, t64 = oracle_inputs(d)
    ref = O.route(s64, t64, d["proposal"].cpu().numpy(), w.eps, w.temperature, w.seed, 0, mask=mask.cpu().numpy(),
                  grad_scale=0.5, want_grad=True, grad_dtype=w.dtype)
    n_exempt = compare_rows(out, ref)
    assert n_exempt <= 2
    same = out["corrected"].cpu().numpy() == ref["corrected"]
    live = same & (ref["status"] & (8 | 16) == 0)
    tok = np.where(ref["corrected"] == 1, ref["teacher_top1"], ref["token"])
    grad_check(to_np64(g)[live], ref["grad"][live], w.dtype, tok[live])
    assert torch.all(g[5] == 0) and torch.all(g[6] == 0) and torch.all(g[3] == 0)      # flagged and masked rows
    # float64 all the way: far inside the tolerance on lambda (1e-5), which is what the float32 kernels are held to
    tol = 1e-6 if tier == "f64" else 1e-5
    assert np.max(np.abs(out["lambda"].cpu().numpy() - ref["lam"])) <= tol
    st = ref["status"]
    assert st[3] & 4 and st[5] == 16 and st[6] == 8 and st[8] & 1
    # the unsharded float64 kernel on the same rows: same flags and ids, floats to float32 rounding
    prev = P.set_kernel(1)
    try:
        whole, g_whole = P.route_fwd_bwd(d["s"], d["t"], d["proposal"], w.eps, w.temperature, w.seed, mask=mask, grad_scale=0.5)
        torch.cuda.synchronize()
    finally:
        P.set_kernel(prev)
    ok = torch.as_tensor(np.minimum(ref["margin_accept"], ref["margin_draw"]) >= 1e-6, device=DEV)
    for k in ("corrected", "token", "teacher_top1", "row_status"):
        assert torch.equal(out[k][ok], whole[k][ok]), k
    for k in ("lambda", "tv", "kl", "accept_prob", "loss", "logp_x", "logq_y"):
        assert float((out[k] - whole[k]).abs().max()) <= tol * (1 + float(whole[k].abs().max())), k
    print(f"\n[parity] vocabulary-sharded V={V} world={world} {tier} slice kernels: {waves} evaluation waves, margin-exempt "
          f"{n_exempt}, corrected {int(ref['corrected'].sum())} of {w.N}, max |dlambda| "
          f"{np.max(np.abs(out['lambda'].cpu().numpy() - ref['lam'])):.2e}")


@pytest.mark.parametrize("eps", [0.0, 5.0])
def test_endpoints_need_no_evaluation_wave(eps):
    w = synth.Workload("vs", 16, 8192, "bf16", eps, 1.0, True, 77, 9)
    d = synth.generate(w, DEV)
    out, gs, waves = route_vocab_sharded_local(_slices(d, split_columns(w.V, 4)), w.V, d["proposal"], eps, seed=w.seed)
    torch.cuda.synchronize()
    s64, t64 = oracle_inputs(d)
    ref = O.route(s64, t64, d["proposal"].cpu().numpy(), eps, 1.0, w.seed, want_grad=True, grad_dtype=w.dtype)
    compare_rows(out, ref)
    if eps == 0.0:
        assert waves == 0 and int(out["corrected"].sum()) == 0
    else:
        assert np.all(ref["lam"] == 1.0) and waves == 0
    grad_check(to_np64(torch.cat(gs, dim=1)), ref["grad"], w.dtype, np.where(ref["corrected"] == 1, ref["teacher_top1"], ref["token"]))


@pytest.mark.parametrize("eps", [1e-4, 2e-3, 0.02, 0.1, 3.0])
def test_hard_rows_in_slices(eps):
    """Rows that stress the numerics (near one-hot students and teachers, large magnitudes and offsets, a flat row,
    disjoint peaks) cut into four slices: radii below 0.02 are reduced in float64 altogether; from 0.02 on the
    float32 slice kernels are at work and the combine hands the rows they cannot resolve to the float64 ones."""
    V, N = 4096, 10
    gen = torch.Generator(device=DEV).manual_seed(5)
    s = 2.0 * torch.randn((N, V), generator=gen, device=DEV)
    t = s + 1.5 * torch.randn((N, V), generator=gen, device=DEV)
    s[0, 17] += 40.0
    t[1, 99] += 40.0
    s[2] *= 12.0; t[2] *= 12.0
    t[3] = s[3]
    s[4] = 0.0; t[4] = 0.0; t[4, 5] = 3.0
    s[5] += 300.0; t[5] -= 250.0
    s[6, 7] = 80.0; t[6, 9] = 80.0
    s[7, 100] += 25.0; t[7, 100] += 24.0; t[7, 200] += 18.0       # both nearly one-hot on the same token
    s[8] = 0.0; t[8] = 0.0; s[8, 300] = 17.5; t[8, 300] = 11.8    # p = 0.9999, T = 0.97 on one token: a very flat KL(q_beta || p)
    s, t = s.to(torch.bfloat16), t.to(torch.bfloat16)
    x = torch.tensor([17, 3, 5, 8, 0, 11, 7, 100, 300, 3], dtype=torch.int32, device=DEV)
    d = dict(s=s, t=t, proposal=x)
    state = []
    out, gs, waves = route_vocab_sharded_local(_slices(d, split_columns(V, 4)), V, x, eps, seed=31, state_out=state)
    torch.cuda.synchronize()
    s64, t64 = oracle_inputs(d)
    ref = O.route(s64, t64, x.cpu().numpy(), eps, 1.0, 31, want_grad=True, grad_dtype="bf16")
    n_exempt = compare_rows(out, ref)
    same = out["corrected"].cpu().numpy() == ref["corrected"]
    grad_check(to_np64(torch.cat(gs, dim=1))[same], ref["grad"][same], "bf16",
               np.where(ref["corrected"] == 1, ref["teacher_top1"], ref["token"])[same])
    n64 = int((state[0][:, 30] != 0).sum().item())
    if eps < 0.02:
        assert n64 == 0                    # no row is marked: the whole call runs on the float64 kernels
    if eps == 0.02:
        assert state[0][8, 30] != 0        # the flat row is handed over
    print(f"\n[parity] hard rows in 4 slices, eps={eps}: {waves} waves, {n64} of {N} rows handed to the float64 slice "
          f"kernels, margin-exempt {n_exempt}, max |dlambda| {np.max(np.abs(out['lambda'].cpu().numpy() - ref['lam'])):.2e}")


@pytest.mark.parametrize("dtype,temperature,eps", [("bf16", 0.7, 0.1), ("bf16", 1.6, 0.03), ("f32", 0.9, 0.1)])
def test_temperature_and_dtype_in_slices(dtype, temperature, eps):
    """Temperatures other than 1 (they scale both logit rows, the moments of the logit difference and the gradient)
    on the float32 slice kernels, and fp32 logits, which the float64 kernels take."""
    V = 8192 if dtype == "bf16" else 1024
    w = synth.Workload("vs", 48, V, dtype, eps, 1.5, dtype == "bf16", 1200, 61, temperature=temperature)
    d = synth.generate(w, DEV)
    out, gs, waves = route_vocab_sharded_local(_slices(d, split_columns(V, 4)), V, d["proposal"], eps, temperature, w.seed,
                                               grad_scale=0.25)
    torch.cuda.synchronize()
    s64, t64 = oracle_inputs(d)
    ref = O.route(s64, t64, d["proposal"].cpu().numpy(), eps, temperature, w.seed, grad_scale=0.25, want_grad=True,
                  grad_dtype=dtype)
    n_exempt = compare_rows(out, ref)
    assert n_exempt <= 2
    same = out["corrected"].cpu().numpy() == ref["corrected"]
    grad_check(to_np64(torch.cat(gs, dim=1))[same], ref["grad"][same], dtype,
               np.where(ref["corrected"] == 1, ref["teacher_top1"], ref["token"])[same])

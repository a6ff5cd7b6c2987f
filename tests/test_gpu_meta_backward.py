"""Parity of saki_route_bwd_from_meta (the trainer's step, Section 3.5) with the float64 oracle."""
import numpy as np
import pytest
import torch

import oracle as O
import paper_2609_36601_b200 as P
from paper_2609_36601_b200 import synth
from parity import grad_check, to_np64

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _meta(n, V, seed, p_corr=0.3):
    g = torch.Generator(device="cpu").manual_seed(seed)
    C = (torch.rand(n, generator=g) < p_corr).to(torch.uint8)
    x = torch.randint(0, V, (n,), generator=g, dtype=torch.int32)
    vs = torch.randint(0, V, (n,), generator=g, dtype=torch.int32)
    A = torch.randn(n, generator=g)
    return C, x, vs, A


def _check(s, C, x, vs, A, tau=1.0, mask=None, status=None, scale=1.0, rows=None, expect_kernel=None):
    dev = lambda v: None if v is None else v.to(DEV)
    out, g = P.route_bwd_from_meta(s, dev(C), dev(x), dev(vs), dev(A), temperature=tau, mask=dev(mask),
                                   rollout_status=dev(status), grad_scale=scale)
    torch.cuda.synchronize()
    if expect_kernel is not None:
        assert P.last_kernel() == expect_kernel
    n = s.shape[0]
    rr = list(range(n)) if rows is None else list(rows)
    dtype = "bf16" if s.dtype == torch.bfloat16 else "f32"
    idx = torch.as_tensor(rr, device=DEV)
    ref = O.bwd_from_meta(to_np64(s[idx]), C.numpy()[rr], x.numpy()[rr], vs.numpy()[rr], A.numpy().astype(np.float64)[rr],
                          tau, None if mask is None else mask.numpy()[rr],
                          None if status is None else status.numpy()[rr], scale, dtype)
    st = out["row_status"].cpu().numpy().astype(np.uint32)[rr]
    assert np.array_equal(st, ref["status"])
    loss, lp = out["loss"].cpu().numpy()[rr], out["logp_tok"].cpu().numpy()[rr]
    # log pi(tok) from a float32 log-sum-exp: 1e-5 (1 + |ref|); the loss is coef * that
    assert np.all(np.abs(lp - ref["logp_tok"]) <= 1e-5 * (1 + np.abs(ref["logp_tok"])))
    coef = np.where(C.numpy()[rr] == 1, 1.0, A.numpy()[rr])
    assert np.all(np.abs(loss - ref["loss"]) <= 1e-4 * np.abs(ref["loss"]) + 1e-5 * np.abs(coef) + 1e-7)
    gg = to_np64(g[idx])
    tok = np.where(C.numpy()[rr] == 1, vs.numpy()[rr], x.numpy()[rr])
    ok = ref["status"] == 0
    if ok.any():
        grad_check(gg[ok], ref["grad"][ok], dtype, tok[ok])
    assert np.all(gg[~ok] == 0)
    return out, g, ref


@pytest.mark.parametrize("V,N", [(2048, 7), (32000, 300), (50048, 20), (106496, 160), (106752, 160), (151936, 320),
                                 (200000, 150)])
def test_streaming_kernel_shapes(V, N):
    """Fully resident rows, the largest resident V, the smallest streamed one, the benchmark's V, and a
    larger one; more rows than blocks where memory allows, so that rows follow each other in a block."""
    w = synth.Workload("t", N, V, "bf16", 0.1, 1.5, True, 300 + N, 50)
    s = synth.generate(w, DEV)["s"]
    C, x, vs, A = _meta(N, V, 7 + N)
    rows = range(0, N, max(1, N // 12))
    _check(s, C, x, vs, A, tau=0.9, scale=0.37, rows=rows, expect_kernel=4)


@pytest.mark.parametrize("V,N,dtype", [(1000, 9, torch.bfloat16), (4099, 5, torch.bfloat16), (33, 7, torch.float32),
                                        (2, 4, torch.float32), (5000, 6, torch.float32)])
def test_general_kernel_shapes(V, N, dtype):
    g = torch.Generator(device=DEV).manual_seed(V)
    s = (2.0 * torch.randn((N, V), generator=g, device=DEV)).to(dtype)
    C, x, vs, A = _meta(N, V, 11 + V)
    _check(s, C, x, vs, A, tau=1.3, scale=0.5, expect_kernel=1)


def test_flags_masks_and_strides():
    N, V = 12, 4096
    g = torch.Generator(device=DEV).manual_seed(5)
    buf = (2.0 * torch.randn((N, V + 64), generator=g, device=DEV)).to(torch.bfloat16)
    s = buf[:, :V]                                   # row stride V + 64
    C, x, vs, A = _meta(N, V, 3)
    C[:6] = torch.tensor([0, 1, 0, 1, 0, 0], dtype=torch.uint8)
    s[0, 77] = float("nan")
    vs[1] = V
    x[2] = -1
    A[4] = float("inf")
    status = torch.zeros(N, dtype=torch.int32)
    status[3] = 64
    mask = torch.ones(N, dtype=torch.uint8)
    mask[5] = 0
    P.check()
    out, grad, ref = _check(s, C, x, vs, A, mask=mask, status=status, expect_kernel=4)
    assert list(ref["status"][:6]) == [8, 16, 16, 64, 8, 4]
    assert P.check() == 4            # the NONFINITE and BAD_ID rows
    prev = P.set_kernel(1)
    try:
        _check(s, C, x, vs, A, mask=mask, status=status, expect_kernel=1)
    finally:
        P.set_kernel(prev)


def test_unchanged_logits_reproduce_the_routing_call():
    """Metadata of a routing call fed back with the same logits: same loss, same gradient (bit for bit
    on the bf16 gradient except where the two float32 paths round a value differently)."""
    w = synth.Workload("t", 200, 32000, "bf16", 0.1, 1.5, True, 77, 51)
    d = synth.generate(w, DEV)
    out, g = P.route_fwd_bwd(d["s"], d["t"], d["proposal"], w.eps, seed=w.seed, grad_scale=0.25)
    A = out["logT_x"] - out["logp_x"]
    m, gm = P.route_bwd_from_meta(d["s"], out["corrected"], d["proposal"], out["teacher_top1"], A,
                                  rollout_status=out["row_status"], grad_scale=0.25)
    torch.cuda.synchronize()
    assert torch.allclose(m["loss"], out["loss"], rtol=1e-4, atol=1e-6)
    diff = (gm.float() - g.float()).abs()
    assert float(diff.max()) <= 2e-3 * 0.25
    assert float((diff > 0).float().mean()) < 1e-3


def test_wide_range_rows_take_the_float64_kernel():
    N, V = 6, 40000
    g = torch.Generator(device=DEV).manual_seed(9)
    s = torch.full((N, V), -400.0, device=DEV) + 0.5 * torch.randn((N, V), generator=g, device=DEV)
    # the streaming kernel deals the row's steps of 256 elements out in order to its warps (16 per block up to
    # V = 98304, 32 beyond): steps // W each, one more to the first steps % W
    W = 16 if V <= 98304 else 32
    q, rem = divmod((V + 255) // 256, W)
    for i in range(N):                     # peaks away from the first 256 logits of a warp's segment
        wi = (5 * i) % W
        start = 256 * (q * wi + min(wi, rem))
        pos = (torch.randint(400, 256 * q - 50, (30,), generator=g, device=DEV) + start).clamp(max=V - 1)
        s[i, pos] = 2.0 * torch.randn((30,), generator=g, device=DEV)
    s = s.to(torch.bfloat16)
    C, x, vs, A = _meta(N, V, 13)
    _check(s, C, x, vs, A, expect_kernel=4)
    assert P.redo_count() == N


def test_bad_arguments():
    s = torch.zeros((2, 128), dtype=torch.bfloat16, device=DEV)
    C, x, vs, A = (v.to(DEV) for v in _meta(2, 128, 1))
    with pytest.raises(P.SakiError) as ei:
        P.route_bwd_from_meta(s, C, x, vs, A, temperature=0.0)
    assert ei.value.code == 1
    with pytest.raises(P.SakiError):
        P.route_bwd_from_meta(s, C, x, vs, A, grad_scale=float("nan"))
    z = torch.zeros((0, 128), dtype=torch.bfloat16, device=DEV)
    e = torch.zeros(0, device=DEV)
    out, g = P.route_bwd_from_meta(z, e.to(torch.uint8), e.to(torch.int32), e.to(torch.int32), e)
    assert g.shape == (0, 128)

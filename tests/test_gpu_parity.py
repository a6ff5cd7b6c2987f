"""Parity of the CUDA path (through the C ABI) with the float64 oracle."""
import numpy as np
import pytest
import torch

import oracle as O
import paper_2609_36601_b200 as P
from paper_2609_36601_b200 import synth
from parity import compare_rows, force_second_tier, grad_check, oracle_inputs, to_np64, warp_segments

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
KERNELS = {"general": 1, "cluster": 2, "auto": 0}


@pytest.fixture(params=list(KERNELS))
def kernel(request):
    prev = P.set_kernel(KERNELS[request.param])
    yield request.param
    P.set_kernel(prev)


def _route_oracle(d, w, rows=None, mask=None, want_grad=True, row_offset=0, grad_scale=1.0, eps=None):
    s64, t64 = oracle_inputs(d)
    x = d["proposal"].cpu().numpy()
    return O.route(s64, t64, x, w.eps if eps is None else eps, w.temperature, w.seed, row_offset, mask=mask,
                   grad_scale=grad_scale, want_grad=want_grad, grad_dtype=w.dtype, rows=rows)


def _check_fwd_bwd(d, w, rows=None, mask=None, row_offset=0, grad_scale=1.0, eps=None):
    e = w.eps if eps is None else eps
    m = None if mask is None else torch.as_tensor(mask, dtype=torch.uint8, device=DEV)
    out_f = P.route_fwd(d["s"], d["t"], d["proposal"], e, w.temperature, w.seed, row_offset, mask=m)
    out, g = P.route_fwd_bwd(d["s"], d["t"], d["proposal"], e, w.temperature, w.seed, row_offset, mask=m,
                             grad_scale=grad_scale)
    torch.cuda.synchronize()
    for k in out:   # forward-only and forward+backward agree bit for bit
        assert torch.equal(out[k], out_f[k]), k
    ref = _route_oracle(d, w, rows, mask, True, row_offset, grad_scale, eps)
    n_exempt = compare_rows(out, ref, rows)
    rr = np.arange(len(d["proposal"])) if rows is None else np.asarray(list(rows))
    gg = to_np64(g)[rr]
    same = (out["corrected"].cpu().numpy()[rr] == ref["corrected"])
    tok = np.where(ref["corrected"] == 1, ref["teacher_top1"], ref["token"])[same]
    stats = grad_check(gg[same], ref["grad"][same], w.dtype, tok)
    return out, ref, n_exempt, stats


def test_cfg1_tiny_fp32_all_rows(kernel):
    w = synth.WORKLOADS["cfg1"]
    d = synth.generate(w, DEV)
    # the proposal utility agrees with the oracle's Gumbel-max (outside the margin)
    x_gpu = P.sample_proposal(d["s"], w.temperature, w.seed).cpu().numpy()
    x_ref, gaps = O.sample_proposal(to_np64(d["s"]), w.temperature, w.seed)
    assert np.array_equal(x_gpu[gaps >= 1e-6], x_ref[gaps >= 1e-6])
    d["proposal"] = torch.as_tensor(x_ref, device=DEV)
    out, ref, n_exempt, stats = _check_fwd_bwd(d, w)
    assert n_exempt <= 2
    assert 0.15 < np.median(ref["tv"]) < 0.2237      # Pinsker cap sqrt(eps/2)


@pytest.mark.parametrize("V,N,dtype", [(1000, 9, "bf16"), (4099, 5, "bf16"), (33, 7, "f32"), (2, 4, "f32"),
                                        (20000, 3, "bf16")])
def test_ragged_shapes(kernel, V, N, dtype):
    w = synth.Workload("t", N, V, dtype, 0.1, 1.5, V > 100, 77, 9, temperature=0.9)
    d = synth.generate(w, DEV)
    _check_fwd_bwd(d, w, row_offset=(1 << 33) + 5, grad_scale=0.125)


@pytest.mark.parametrize("V,N,eps,sigma", [(2048, 5, 0.1, 1.5), (32000, 24, 0.05, 1.0), (50048, 10, 0.1, 1.5),
                                           (151936, 12, 0.1, 1.5), (163840, 3, 0.01, 2.0), (151936, 6, 1.0, 0.5)])
@pytest.mark.parametrize("which", [2, 3])
def test_fast_kernel_shapes(V, N, eps, sigma, which):
    """The two bf16 hot-path kernels: the cluster kernel at every cluster size (1, 2, 4, 8 blocks
    per row) and the row-per-SM kernel with and without a part of the row left in L2."""
    prev = P.set_kernel(which)
    try:
        w = synth.Workload("t", N, V, "bf16", eps, sigma, True, 90 + N, 21)
        d = synth.generate(w, DEV)
        _check_fwd_bwd(d, w, row_offset=7)
        assert P.last_kernel() == which
        if V <= 50048:      # more rows than blocks: every block routes several rows back to back
            w = synth.Workload("t", 400, V, "bf16", eps, sigma, True, 91 + N, 22)
            d = synth.generate(w, DEV)
            _check_fwd_bwd(d, w, rows=range(0, 400, 7))
    finally:
        P.set_kernel(prev)


@pytest.mark.parametrize("V", [53384, 56000, 75008, 262144])
def test_rowsm_streamed_shapes(V):
    """Row-per-SM kernel, rows that no longer fit in shared memory: 14 steps per warp (the shortest
    streamed part), a ragged last step, and the largest V it serves; two rows per block, so the ring
    of streamed steps runs over from a row's last pass into the next row and ends after the last."""
    prev = P.set_kernel(3)
    try:
        w = synth.Workload("t", 300, V, "bf16", 0.1, 1.5, True, 131, 41)
        d = synth.generate(w, DEV)
        _check_fwd_bwd(d, w, rows=range(0, 300, 23), row_offset=3)
        assert P.last_kernel() == 3
    finally:
        P.set_kernel(prev)


@pytest.mark.parametrize("V", [13320, 14344, 26808, 49152])
def test_rowsm_streamed_shapes_four_blocks_per_sm(V):
    """The same for the instance with four blocks of four warps per SM (rows up to 49152 elements): one warp
    of four with a streamed part, the shortest streamed part with a ragged last step, an odd number of streamed
    steps, the longest row it serves; more rows than blocks, so the ring runs over into the next row."""
    prev = P.set_kernel(3)
    try:
        w = synth.Workload("t", 700, V, "bf16", 0.1, 1.5, True, 137, 43)
        d = synth.generate(w, DEV)
        _check_fwd_bwd(d, w, rows=range(0, 700, 41), row_offset=3)
        assert P.last_kernel() == 3
    finally:
        P.set_kernel(prev)


def test_strided_rows_and_mask(kernel):
    w = synth.Workload("t", 12, 3000, "bf16", 0.05, 1.0, True, 78, 10)
    d = synth.generate(w, DEV)
    pad = torch.zeros((12, 3000 + 72), dtype=torch.bfloat16, device=DEV)
    for k in ("s", "t"):
        buf = pad.clone()
        buf[:, :3000] = d[k]
        d[k] = buf[:, :3000]            # row stride 3072
    mask = np.array([1, 0] * 6, dtype=np.uint8)
    out, ref, _, _ = _check_fwd_bwd(d, w, mask=mask)
    assert np.all(out["loss"].cpu().numpy()[mask == 0] == 0)


def test_eps_zero_and_saturation(kernel):
    w = synth.Workload("t", 16, 2048, "bf16", 0.0, 0.5, True, 79, 11)
    d = synth.generate(w, DEV)
    out, ref, _, _ = _check_fwd_bwd(d, w, eps=0.0)
    assert torch.all(out["corrected"] == 0) and torch.all(out["lambda"] == 0)
    assert torch.all((out["row_status"] & 2) != 0)
    out, ref, _, _ = _check_fwd_bwd(d, w, eps=5.0)
    assert torch.all(out["lambda"] == 1) and torch.all((out["row_status"] & 1) != 0)
    out, ref, _, _ = _check_fwd_bwd(d, w, eps=0.3)
    sat = (ref["status"] & 1) != 0
    assert 0 < sat.sum() < 16, "want a mix of saturated and interior rows"


def test_flagged_rows(kernel):
    w = synth.Workload("t", 6, 1500, "bf16", 0.1, 1.5, True, 80, 12)
    d = synth.generate(w, DEV)
    d["s"][1, 700] = float("nan")
    d["t"][2, 3] = float("inf")
    d["t"][3, 1499] = float("-inf")
    d["proposal"][4] = 1500
    d["proposal"][5] = -1
    P.check()
    out, ref, _, _ = _check_fwd_bwd(d, w)
    st = out["row_status"].cpu().numpy()
    assert list(st[1:]) == [8, 8, 8, 16, 16] and st[0] == 0
    assert torch.all(out["token"][1:] == -1)
    assert P.check() == 10          # 5 rows x (fwd + fwd_bwd)
    assert P.check() == 0


def test_empty_and_bad_arguments():
    z = torch.zeros((0, 128), dtype=torch.bfloat16, device=DEV)
    out, g = P.route_fwd_bwd(z, z, torch.zeros(0, dtype=torch.int32, device=DEV), 0.1)
    assert g.shape == (0, 128)
    s = torch.zeros((2, 128), dtype=torch.bfloat16, device=DEV)
    x = torch.zeros(2, dtype=torch.int32, device=DEV)
    for kw in (dict(eps=-1.0), dict(eps=float("nan")), dict(eps=0.1, temperature=0.0)):
        with pytest.raises(P.SakiError) as ei:
            P.route_fwd(s, s, x, **kw)
        assert ei.value.code == 1
    with pytest.raises(P.SakiError):
        P.route_fwd(s[:, :1], s[:, :1], x, 0.1)     # V < 2


def test_determinism_and_chunk_invariance(kernel):
    w = synth.Workload("t", 40, 5000, "bf16", 0.1, 1.5, True, 81, 13)
    d = synth.generate(w, DEV)
    a, ga = P.route_fwd_bwd(d["s"], d["t"], d["proposal"], w.eps, seed=w.seed)
    b, gb = P.route_fwd_bwd(d["s"], d["t"], d["proposal"], w.eps, seed=w.seed)
    c, gc = P.route_fwd_bwd(d["s"][17:], d["t"][17:], d["proposal"][17:], w.eps, seed=w.seed, row_offset=17)
    torch.cuda.synchronize()
    for k in a:
        assert torch.equal(a[k], b[k]) and torch.equal(a[k][17:], c[k]), k
    assert torch.equal(ga, gb) and torch.equal(ga[17:], gc)


def test_rows_alone_and_inside_a_larger_call_when_the_kernel_changes_with_the_size():
    """Automatic dispatch serves a call of at most 32 long rows with the cluster kernel and a larger one with
    the row-per-SM kernel.  The two agree with the oracle, and therefore with each other, to the tolerances,
    not to the bit: flags and ids wherever the oracle's decision is outside the margin, floats to 2e-5."""
    w = synth.Workload("piece", 40, 151936, "bf16", 0.1, 1.5, True, 83, 15)
    d = synth.generate(w, DEV)
    lo, hi = 14, 26                                   # 12 rows
    prev = P.set_kernel(0)
    try:
        big, g_big = P.route_fwd_bwd(d["s"], d["t"], d["proposal"], w.eps, seed=w.seed)
        k_big = P.last_kernel()
        piece, g_piece = P.route_fwd_bwd(d["s"][lo:hi], d["t"][lo:hi], d["proposal"][lo:hi], w.eps, seed=w.seed,
                                         row_offset=lo)
        k_piece = P.last_kernel()
        # pinned to one kernel, the piece is bit-identical to the rows inside the large call
        P.set_kernel(3)
        pinned, g_pinned = P.route_fwd_bwd(d["s"][lo:hi], d["t"][lo:hi], d["proposal"][lo:hi], w.eps, seed=w.seed,
                                           row_offset=lo)
        torch.cuda.synchronize()
    finally:
        P.set_kernel(prev)
    assert (k_big, k_piece) == (3, 2)
    for k in big:
        assert torch.equal(big[k][lo:hi], pinned[k]), k
    assert torch.equal(g_big[lo:hi], g_pinned)
    rows = list(range(lo, hi))
    ref = _route_oracle(d, w, rows)
    n1 = compare_rows(big, ref, rows)
    ref_piece = dict(ref)
    n2 = compare_rows(piece, ref_piece)
    ok = np.minimum(ref["margin_accept"], ref["margin_draw"]) >= 1e-6
    okt = torch.as_tensor(ok, device=DEV)
    for k in ("corrected", "token", "teacher_top1", "row_status"):
        assert torch.equal(big[k][lo:hi][okt], piece[k][okt]), k
    for k in ("lambda", "tv", "kl", "accept_prob"):
        assert float((big[k][lo:hi] - piece[k]).abs().max()) <= 2e-5, k
    same = okt & (big["corrected"][lo:hi] == piece["corrected"])
    dg = (g_big[lo:hi][same].float() - g_piece[same].float()).abs()
    assert float(dg.max()) <= 4e-3
    print(f"\n[parity] piece vs whole, V=151936: margin-exempt {n1}/{n2} of 12; gradient entries that differ "
          f"{int((dg > 0).sum())} of {dg.numel()}, max {float(dg.max()):.2e}")


def test_spec_verify_small(kernel):
    B, K, V = 48, 4, 3000
    w = synth.Workload("t", B * (K + 1), V, "bf16", 0.2, 1.5, True, 82, 14, K=K)
    d = synth.generate(w, DEV)
    s3, t3 = d["s"].view(B, K + 1, V), d["t"].view(B, K + 1, V)
    draft = d["proposal"].view(B, K + 1)[:, :K].contiguous()
    draft[5, 1] = V + 3                    # a bad id stops verification of that sequence
    res = P.spec_verify(s3, t3, draft, w.eps, seed=w.seed, seq_offset=3)
    torch.cuda.synchronize()
    ref = O.spec_verify(to_np64(s3), to_np64(t3), draft.cpu().numpy(), w.eps, seed=w.seed, seq_offset=3)
    ok = ref["margin"] >= 1e-6
    assert np.array_equal(res["n_accept"].cpu().numpy()[ok], ref["n_accept"][ok])
    assert np.array_equal(res["next_token"].cpu().numpy()[ok], ref["next_token"][ok])
    assert np.array_equal(res["next_is_correction"].cpu().numpy()[ok], ref["next_is_correction"][ok])
    assert len(set(ref["n_accept"])) >= 3
    per = {k: v.cpu().numpy().reshape(B, K + 1) for k, v in res["per_pos"].items()}
    for b in np.nonzero(ok)[0]:
        for j in range(K + 1):
            r = ref["per_pos"][b][j]
            assert per["row_status"][b, j] == r["status"], (b, j)
            assert per["token"][b, j] == r["token"] and per["corrected"][b, j] == r["corrected"]
            for name, key in (("lambda", "lam"), ("tv", "tv"), ("kl", "kl"), ("accept_prob", "accept_prob")):
                assert abs(per[name][b, j] - r[key]) <= 1e-5, (name, b, j)
            for name in ("logp_y", "logq_y", "logT_y", "logp_x", "logq_x"):
                assert abs(per[name][b, j] - r[name]) <= 1e-5 * (1 + abs(r[name])), (name, b, j)
    assert ref["n_accept"][5] <= 1 and res["next_token"][5].item() == ref["next_token"][5]


def test_proposal_utility_bf16():
    w = synth.Workload("t", 64, 7001, "bf16", 0.1, 1.5, True, 83, 15, temperature=0.8)
    d = synth.generate(w, DEV)
    x_gpu = P.sample_proposal(d["s"], w.temperature, w.seed, row_offset=11).cpu().numpy()
    x_ref, gaps = O.sample_proposal(to_np64(d["s"]), w.temperature, w.seed, row_offset=11)
    assert np.array_equal(x_gpu[gaps >= 1e-6], x_ref[gaps >= 1e-6])


def test_host_entry_matches_device_entry(kernel):
    w = synth.Workload("t", 700, 2500, "bf16", 0.1, 1.5, True, 84, 16)
    d = synth.generate(w, DEV)
    out, g = P.route_fwd_bwd(d["s"], d["t"], d["proposal"], w.eps, seed=w.seed, grad_scale=0.5)
    hs, ht = d["s"].cpu().pin_memory(), d["t"].cpu().pin_memory()
    hout, hg = P.route_host(hs, ht, d["proposal"].cpu(), w.eps, seed=w.seed, grad_scale=0.5)
    torch.cuda.synchronize()
    for k in out:
        assert torch.equal(out[k].cpu(), hout[k]), k
    assert torch.equal(g.cpu(), hg)


@pytest.mark.parametrize("which", [1, 2, 3])
def test_hard_rows(which):
    """Rows that stress the numerics: near one-hot students and teachers, very small and very large
    radii, large logit magnitudes, teacher equal to the student, a flat row."""
    prev = P.set_kernel(which)
    try:
        V, N = 4096, 10
        gen = torch.Generator(device=DEV).manual_seed(5)
        s = 2.0 * torch.randn((N, V), generator=gen, device=DEV)
        t = s + 1.5 * torch.randn((N, V), generator=gen, device=DEV)
        s[0, 17] += 40.0                       # student nearly one-hot
        t[1, 99] += 40.0                       # teacher nearly one-hot
        s[2] *= 12.0; t[2] *= 12.0             # logits of magnitude ~100
        t[3] = s[3]                            # teacher == student: saturated at once
        s[4] = 0.0; t[4] = 0.0; t[4, 5] = 3.0  # flat student
        s[5] += 300.0; t[5] -= 250.0           # large common offsets
        s[6, 7] = 80.0; t[6, 9] = 80.0         # disjoint peaks: KL(T||p) huge
        s, t = s.to(torch.bfloat16), t.to(torch.bfloat16)
        x = torch.tensor([17, 3, 5, 8, 0, 11, 7, 1, 2, 3], dtype=torch.int32, device=DEV)
        w = synth.Workload("t", N, V, "bf16", 0.1, 1.5, False, 0, 31)
        redone = {}
        for eps in (1e-6, 1e-4, 4e-4, 2e-3, 0.02, 0.1, 3.0):
            _check_fwd_bwd(dict(s=s, t=t, proposal=x, mask=None), w, eps=eps)
            redone[eps] = P.redo_count()
            if eps < 5e-3 and which != 3:
                assert P.last_kernel() == 1      # radii below 5e-3 are beyond the cluster kernel's float32 sums
            else:
                assert P.last_kernel() == which  # the row-per-SM kernel takes every radius (KL by quadrature)
    finally:
        P.set_kernel(prev)


@pytest.mark.parametrize("gap", [30.0, 60.0, 120.0, 400.0])
def test_wide_range_rows(gap):
    """Rows whose mass sits on a few positions far above a low plateau.  The row-per-SM kernel fixes the
    exponent shifts of its first pass from the first 256 logits of each warp's segment: with the plateau
    `gap` below the peaks its sums grow by up to e^gap, and beyond ~88 nats they overflow, which must
    hand the row to the float64 kernel, not flag or corrupt it."""
    prev = P.set_kernel(3)
    try:
        V, N = 40000, 12
        gen = torch.Generator(device=DEV).manual_seed(77)
        s = torch.full((N, V), -gap, device=DEV) + 0.5 * torch.randn((N, V), generator=gen, device=DEV)
        t = s + 0.5 * torch.randn((N, V), generator=gen, device=DEV)
        for i in range(N):
            # peaks away from the first 256 logits of a warp's segment
            segs = warp_segments(V)
            start, nsteps = segs[i % len(segs)]
            pos = (torch.randint(400, 256 * nsteps - 100, (40,), generator=gen, device=DEV) + start).clamp(max=V - 1)
            s[i, pos] = 2.0 * torch.randn((40,), generator=gen, device=DEV)
            t[i, pos] = s[i, pos] + 1.5 * torch.randn((40,), generator=gen, device=DEV)
        s, t = s.to(torch.bfloat16), t.to(torch.bfloat16)
        x = torch.argmax(s, dim=1).to(torch.int32)
        w = synth.Workload("t", N, V, "bf16", 0.1, 1.5, False, 0, 35)
        _check_fwd_bwd(dict(s=s, t=t, proposal=x, mask=None), w, eps=0.1)
        assert P.last_kernel() == 3
        if gap > 100.0:
            assert P.redo_count() == N      # every row overflowed in float32 and was routed in float64
        elif gap < 50.0:
            assert P.redo_count() == 0
    finally:
        P.set_kernel(prev)


@pytest.mark.parametrize("eps", [1e-6, 1e-4, 2e-3, 4.9e-3, 0.015])
def test_small_radii_on_the_row_per_sm_kernel(eps):
    """Radii of the paper's late schedule (eps -> 0): the row-per-SM kernel forms KL by quadrature of its
    slope there, which keeps lambda accurate relatively, not just absolutely."""
    prev = P.set_kernel(3)
    try:
        w = synth.Workload("t", 400, 32000, "bf16", eps, 1.0, True, 1002, 2)
        d = synth.generate(w, DEV)
        rows = range(0, 400, 9)
        out, ref, _, _ = _check_fwd_bwd(d, w, rows=rows, row_offset=5)
        assert P.last_kernel() == 3
        assert P.redo_count() <= 20
        lam = out["lambda"].cpu().numpy()[list(rows)].astype(np.float64)
        # below 5e-3 every row is settled by the quadrature or by the float64 kernel: held to a tenth of the
        # tolerance on lambda (1e-5)
        assert np.max(np.abs(lam - ref["lam"])) <= (1e-6 if eps < 5e-3 else 1e-5)
    finally:
        P.set_kernel(prev)


@pytest.mark.parametrize("V,eps,sigma,temperature,gen_seed", [(143368, 0.0058, 2.08, 0.7, 1000), (143368, 0.0058, 2.08, 0.7, 1001),
                                                            (158896, 0.0144, 0.83, 0.7, 5024), (49144, 0.0398, 2.0, 1.0, 1005)])
def test_nearly_one_hot_rows_at_small_radii(V, eps, sigma, temperature, gen_seed):
    """Rows found by comparing the bf16 kernels with the float64 kernel on random workloads: a nearly one-hot
    student, so that KL(q_beta || p) is very flat and lambda is large although the radius is small.  The float32
    value of KL is off by more than its usual bound there and the one-panel quadrature is wrong although its two
    rules agree; such rows must come out within the tolerance all the same (by the two-panel quadrature or the
    float64 kernel).  Every row against the float64 kernel, the ones that used to fail against the oracle."""
    w = synth.Workload("t", 400, V, "bf16", eps, sigma, True, gen_seed, gen_seed - 923, temperature=temperature)
    d = synth.generate(w, DEV)
    out = P.route_fwd(d["s"], d["t"], d["proposal"], eps, temperature, w.seed)
    assert P.last_kernel() == 3
    prev = P.set_kernel(1)
    try:
        ref = P.route_fwd(d["s"], d["t"], d["proposal"], eps, temperature, w.seed)
        torch.cuda.synchronize()
    finally:
        P.set_kernel(prev)
    dl = (out["lambda"] - ref["lambda"]).abs()
    assert float(dl.max()) <= 1e-5, (float(dl.max()), int(dl.argmax()))
    assert float((out["tv"] - ref["tv"]).abs().max()) <= 1e-5
    # the flattest rows (largest lambda) against the oracle itself
    rows = torch.topk(ref["lambda"], 3).indices.cpu().numpy()
    s64, t64 = oracle_inputs(d)
    for r in rows:
        o = O.route(s64[r:r + 1], t64[r:r + 1], d["proposal"][r:r + 1].cpu().numpy(), eps, temperature, w.seed, row_offset=int(r))
        assert abs(float(out["lambda"][r]) - o["lam"][0]) <= 1e-5, (int(r), float(out["lambda"][r]), o["lam"][0])


def test_calls_on_two_streams_do_not_share_scratch():
    """The row list of the two-tier routing is kept per stream: two calls whose kernels may overlap on
    the GPU give what each gives alone."""
    prev = P.set_kernel(0)
    try:
        ws = [synth.Workload("a", 1500, 32000, "bf16", 0.005, 1.0, True, 1002, 2),
              synth.Workload("b", 1200, 8192, "bf16", 0.005, 0.5, True, 99, 18)]
        ds = [synth.generate(w, DEV) for w in ws]
        force_second_tier(ds[0], [5, 6, 900, 1499])
        force_second_tier(ds[1], [0, 77, 1199])
        alone = []
        for w, d in zip(ws, ds):
            alone.append(P.route_fwd_bwd(d["s"], d["t"], d["proposal"], w.eps, seed=w.seed))
            torch.cuda.synchronize()
            assert P.redo_count() > 0, "the workloads should put rows on the list"
        streams = [torch.cuda.Stream(device=DEV) for _ in ws]
        for rep in range(3):
            res = []
            for w, d, st in zip(ws, ds, streams):
                with torch.cuda.stream(st):
                    res.append(P.route_fwd_bwd(d["s"], d["t"], d["proposal"], w.eps, seed=w.seed, stream=st))
            torch.cuda.synchronize()
            for (o, g), (ro, rg) in zip(res, alone):
                for k in o:
                    assert torch.equal(o[k], ro[k]), (rep, k)
                assert torch.equal(g, rg), rep
    finally:
        P.set_kernel(prev)


def test_spec_verify_k_limits():
    V = 2048
    for K in (1, 16):
        B = 6
        w = synth.Workload("t", B * (K + 1), V, "bf16", 0.05, 1.0, True, 60 + K, 33, K=K)
        d = synth.generate(w, DEV)
        s3, t3 = d["s"].view(B, K + 1, V), d["t"].view(B, K + 1, V)
        draft = d["proposal"].view(B, K + 1)[:, :K].contiguous()
        res = P.spec_verify(s3, t3, draft, w.eps, seed=w.seed)
        ref = O.spec_verify(to_np64(s3), to_np64(t3), draft.cpu().numpy(), w.eps, seed=w.seed)
        ok = ref["margin"] >= 1e-6
        assert np.array_equal(res["n_accept"].cpu().numpy()[ok], ref["n_accept"][ok])
        assert np.array_equal(res["next_token"].cpu().numpy()[ok], ref["next_token"][ok])
    with pytest.raises(P.SakiError):
        bad = torch.zeros((2, 18, V), dtype=torch.bfloat16, device=DEV)
        P.spec_verify(bad, bad, torch.zeros((2, 17), dtype=torch.int32, device=DEV), 0.1)


def test_evaluation_pass_counter():
    """The row-per-SM kernel counts its evaluation passes: none at eps = 0, about one per unsaturated row otherwise."""
    w = synth.shrink(synth.WORKLOADS["cfg2"], 600)
    d = synth.generate(w, DEV)
    out = P.route_fwd(d["s"], d["t"], d["proposal"], 0.0, seed=w.seed)
    assert P.last_kernel() == 3 and P.solve_evaluations() == 0
    out = P.route_fwd(d["s"], d["t"], d["proposal"], w.eps, seed=w.seed)
    n_solved = int(((out["row_status"] & 1) == 0).sum().item())
    assert n_solved <= P.solve_evaluations() <= int(1.2 * n_solved)
    prev = P.set_kernel(1)
    try:
        P.route_fwd(d["s"], d["t"], d["proposal"], w.eps, seed=w.seed)
        assert P.solve_evaluations() == 0      # another kernel served the call
    finally:
        P.set_kernel(prev)


def test_small_batches_of_long_rows_take_the_cluster_kernel():
    """Automatic dispatch: up to 32 rows with V >= 65536 go one row per cluster (lower latency for a decoding
    step of a small batch); more rows, shorter rows or a radius the cluster kernel cannot resolve do not."""
    prev = P.set_kernel(0)
    try:
        w = synth.Workload("t", 12, 65536, "bf16", 0.1, 1.5, True, 611, 41)
        d = synth.generate(w, DEV)
        _check_fwd_bwd(d, w)
        assert P.last_kernel() == 2
        _check_fwd_bwd(d, w, eps=1e-3)               # below the cluster kernel's smallest radius
        assert P.last_kernel() == 3
        w2 = synth.Workload("t", 33, 65536, "bf16", 0.1, 1.5, True, 612, 42)
        d2 = synth.generate(w2, DEV)
        P.route_fwd(d2["s"], d2["t"], d2["proposal"], w2.eps, seed=w2.seed)
        assert P.last_kernel() == 3
        w3 = synth.Workload("t", 12, 32000, "bf16", 0.1, 1.5, True, 613, 43)
        d3 = synth.generate(w3, DEV)
        P.route_fwd(d3["s"], d3["t"], d3["proposal"], w3.eps, seed=w3.seed)
        assert P.last_kernel() == 3
        # a block verification of few positions goes the same way
        B, K, V = 4, 6, 65536
        w4 = synth.Workload("t", B * (K + 1), V, "bf16", 0.2, 1.5, True, 614, 44, K=K)
        d4 = synth.generate(w4, DEV)
        s3, t3 = d4["s"].view(B, K + 1, V), d4["t"].view(B, K + 1, V)
        draft = d4["proposal"].view(B, K + 1)[:, :K].contiguous()
        res = P.spec_verify(s3, t3, draft, w4.eps, seed=w4.seed)
        torch.cuda.synchronize()
        assert P.last_kernel() == 2
        ref = O.spec_verify(to_np64(s3), to_np64(t3), draft.cpu().numpy(), w4.eps, seed=w4.seed)
        ok = ref["margin"] >= 1e-6
        assert np.array_equal(res["n_accept"].cpu().numpy()[ok], ref["n_accept"][ok])
        assert np.array_equal(res["next_token"].cpu().numpy()[ok], ref["next_token"][ok])
    finally:
        P.set_kernel(prev)

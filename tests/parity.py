"""Element-by-element comparison of the CUDA path with the float64 oracle.

Tolerances (written here so that the tests state them):
  flags and ids       bit-exact, except rows whose oracle decision margin is
                      below 1e-6 (|u - accept_prob| for the acceptance test;
                      distance of the inverse-CDF target from the nearer cell
                      edge as a fraction of the total for the draws), which are
                      counted and returned
  lambda, TV          |delta| <= 1e-5
  other fp32 scalars  |delta| <= 1e-5 (kl, accept_prob) or 1e-5 (1+|ref|) (log-probs)
  loss                |delta| <= 1e-4 |ref| + 1e-6 (1 + |k1| + |log p(x)|), k1 = log p(x) - log T(x): the loss is
                      k1 log p(x), and a log-sum-exp taken from float32 sums resolves each factor to ~1e-7;
                      rows that need the absolute term are counted, and must have |loss| < 0.25
  gradient, fp32      |delta| <= 1e-6 + 2e-6 |ref|
  gradient, bf16      |delta| <= 2e-3 where |g_ref| < 1; elsewhere within one
                      bf16 ulp of the oracle's rounded value; and relative
                      error <= 2^-7 on entries with |g_ref| >= 1e-30 (small
                      entries must not be flushed to zero), except the supervised
                      token's entry coef (p - 1), which cancels when p is near 1
"""
import math

import numpy as np
import torch

import oracle as O

MARGIN = 1e-6


def to_np64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to("cpu").to(torch.float64).numpy()


def bf16_ulp(x):
    x = np.abs(np.asarray(x, dtype=np.float64))
    _, e = np.frexp(np.maximum(x, 2.0 ** -126))
    return np.ldexp(1.0, (e - 1) - 7)


def grad_check(g_gpu: np.ndarray, g_ref: np.ndarray, dtype: str, tok=None):
    """g_ref is the oracle gradient already rounded to the output dtype.  `tok[i]` is the supervised
    token of row i: that entry is coef (p - 1), a difference that cancels when p is close to 1, so it is
    held to the absolute bound only (the relative bound exists to keep small-p entries from being
    flushed to zero, which does not apply to it)."""
    d = np.abs(g_gpu - g_ref)
    if dtype == "f32":
        tol = 1e-6 + 2e-6 * np.abs(g_ref)
        assert np.all(d <= tol), f"fp32 gradient error {d.max():.3e}"
        return dict(max_abs=float(d.max()), n_ulp=0)
    small = np.abs(g_ref) < 1.0
    assert np.all(d[small] <= 2e-3), f"bf16 gradient max-abs error {d[small].max():.3e}"
    big_ok = d[~small] <= bf16_ulp(g_ref[~small]) * 1.0000001
    assert np.all(big_ok), "bf16 gradient entry with |g|>=1 off by more than one ulp"
    nz = np.abs(g_ref) >= 1e-30
    n_tok_abs_only = 0
    if tok is not None:
        ti, tj = np.arange(len(tok)), np.asarray(tok)
        at_tok = nz[ti, tj]
        n_tok_abs_only = int(np.count_nonzero(d[ti, tj][at_tok] > 2.0 ** -7 * 1.0000001 * np.abs(g_ref[ti, tj][at_tok])))
        nz[ti, tj] = False
    rel = d[nz] / np.abs(g_ref[nz])
    assert np.all(rel <= 2.0 ** -7 * 1.0000001), f"bf16 gradient relative error {rel.max():.3e}"
    return dict(max_abs=float(d[small].max()) if small.any() else 0.0,
                n_ulp=int(np.count_nonzero(g_gpu != g_ref)),
                n_tok_abs_only=n_tok_abs_only)   # supervised-token entries held by the absolute bound alone


LOSS_FLOOR_MAX = 0.25   # a row that meets the loss bound only through its absolute floor has a loss this small


def compare_rows(gpu: dict, ref: dict, rows=None, check_loss=True, report=None):
    """gpu: dict of torch tensors (all rows); ref: oracle dict over `rows`.
    Returns the number of margin-exempt rows.  `report` (a dict) receives the counts a reader of the test
    output wants: rows compared, margin-exempt rows by decision, rows whose loss error exceeds the pure
    relative bound (they pass by the absolute floor, and only if their loss is below LOSS_FLOOR_MAX), and
    the largest errors."""
    n_total = len(gpu["token"])
    rows = np.arange(n_total) if rows is None else np.asarray(list(rows))
    g = {k: v.detach().cpu().numpy()[rows] for k, v in gpu.items() if isinstance(v, torch.Tensor)}
    exempt = (np.minimum(ref["margin_accept"], ref["margin_draw"]) < MARGIN)
    ok = ~exempt
    assert np.array_equal(g["teacher_top1"], ref["teacher_top1"]), "teacher argmax differs"
    assert np.array_equal(g["row_status"].astype(np.uint32), ref["status"]), \
        f"row status differs: {g['row_status'][:8]} vs {ref['status'][:8]}"
    assert np.array_equal(g["corrected"][ok], ref["corrected"][ok]), "accept/correct flags differ"
    assert np.array_equal(g["token"][ok], ref["token"][ok]), \
        f"committed tokens differ at rows {rows[ok][g['token'][ok] != ref['token'][ok]][:5]}"
    for name, key, tol in (("lambda", "lam", 1e-5), ("tv", "tv", 1e-5), ("kl", "kl", 1e-5),
                           ("accept_prob", "accept_prob", 1e-5)):
        d = np.abs(g[name].astype(np.float64) - ref[key])
        assert np.all(d <= tol), f"{name}: max error {d.max():.3e}"
    same = ok & (g["corrected"] == ref["corrected"]) & (g["token"] == ref["token"])
    for name in ("logp_x", "logq_x", "logT_x", "logp_y", "logq_y", "logT_y"):
        d = np.abs(g[name].astype(np.float64) - ref[name])[same]
        assert np.all(d <= 1e-5 * (1 + np.abs(ref[name][same]))), f"{name}: max error {d.max():.3e}"
    n_loss_floor = 0
    if check_loss:
        d = np.abs(g["loss"].astype(np.float64) - ref["loss"])[same]
        floor = 1e-6 * (1.0 + np.abs(ref["logp_x"] - ref["logT_x"]) + np.abs(ref["logp_x"]))[same]   # the ~1e-7 resolution of a
        assert np.all(d <= 1e-4 * np.abs(ref["loss"][same]) + floor), f"loss: max error {d.max():.3e}"   # float32 lse
        by_floor = d > 1e-4 * np.abs(ref["loss"][same])
        n_loss_floor = int(by_floor.sum())
        assert np.all(np.abs(ref["loss"][same][by_floor]) < LOSS_FLOOR_MAX), "a large loss met its bound only by the floor"
    if report is not None:
        report.update(rows=int(len(rows)), margin_exempt=int(exempt.sum()),
                      margin_exempt_accept=int(np.sum(ref["margin_accept"] < MARGIN)),
                      margin_exempt_draw=int(np.sum(ref["margin_draw"] < MARGIN)),
                      loss_by_floor_only=n_loss_floor,
                      max_abs_dlambda=float(np.abs(g["lambda"].astype(np.float64) - ref["lam"]).max()),
                      max_abs_dtv=float(np.abs(g["tv"].astype(np.float64) - ref["tv"]).max()))
    return int(exempt.sum())


def max_errors(gpu: dict, ref: dict, rows=None):
    n_total = len(gpu["token"])
    rows = np.arange(n_total) if rows is None else np.asarray(list(rows))
    g = {k: v.detach().cpu().numpy()[rows] for k, v in gpu.items() if isinstance(v, torch.Tensor)}
    return {name: float(np.abs(g[name].astype(np.float64) - ref[key]).max())
            for name, key in (("lambda", "lam"), ("tv", "tv"), ("kl", "kl"), ("accept_prob", "accept_prob"))}


def oracle_inputs(d: dict, rows=None):
    """The identical bytes the GPU sees, widened exactly to float64 on the host."""
    s, t = d["s"], d["t"]
    if rows is not None:
        idx = torch.as_tensor(list(rows), device=s.device)
        s, t = s[idx], t[idx]
    return to_np64(s), to_np64(t)


def warp_segments(V):
    """How the row-per-SM kernel deals a row of V elements out to its warps: steps of 256 elements in order,
    steps // W to every warp and one more to the first steps % W; W = 8 warps (two CTAs per SM) up to
    V = 98304, 16 beyond.  Returns [(first element, number of steps)] per warp."""
    W = 8 if V <= 98304 else 16
    steps = (V + 255) // 256
    q, rem = divmod(steps, W)
    return [(256 * (w * q + min(w, rem)), q + (1 if w < rem else 0)) for w in range(W)]


def force_second_tier(d, rows):
    """Rewrites the given rows of a generated bf16 workload so that the row-per-SM kernel must hand them to
    the float64 kernel: a plateau 400 nats below a few peaks that sit away from the first 256 logits of
    a warp's segment, so the float32 sums of that warp's first pass overflow."""
    V = d["s"].shape[1]
    segs = [sg for sg in warp_segments(V) if sg[1] >= 2]
    assert segs, "the rows need a warp segment of two steps or more"
    g = torch.Generator(device=d["s"].device).manual_seed(1234)
    for r in rows:
        lo, n = segs[r % len(segs)]
        hi = min(V, lo + 256 * n)
        s = torch.full((V,), -400.0, device=d["s"].device) + 0.5 * torch.randn(V, generator=g, device=d["s"].device)
        pos = torch.randint(lo + 300, max(lo + 301, hi - 8), (24,), generator=g, device=d["s"].device).clamp(max=V - 1)
        s[pos] = 2.0 * torch.randn(24, generator=g, device=d["s"].device)
        t = s + 0.7 * torch.randn(V, generator=g, device=d["s"].device)
        d["s"][r] = s.to(d["s"].dtype)
        d["t"][r] = t.to(d["t"].dtype)
        d["proposal"][r] = int(pos[0])

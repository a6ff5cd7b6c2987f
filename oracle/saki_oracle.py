"""Plain float64 oracle of the SAKI per-position routing path.

TEST INFRASTRUCTURE ONLY: imported by the tests, the smoke check and the
benchmark's CPU-baseline leg, never by the product path.  It shares no code,
table or helper with the CUDA library; it is written from the paper's
definitions and is deliberately slow and direct (one vocabulary row at a time,
numpy float64, no blocking, no fusion) so that each step can be checked
against the paper by eye.

What one position computes (paper notation; p = frozen student distribution,
T = teacher distribution, both full-vocabulary softmaxes of the logit rows):

  1. log p, log T                              Section 3.1 (problem setup)
  2. q_beta = p^(1-beta) T^beta / Z(beta)      Eq. "bridge"
     lambda = largest beta in [0,1] with
              KL(q_beta || p) <= eps           Eq. "trust_region"
  3. maximal coupling of the proposal x~p
     with q: accept w.p. min(1, q(x)/p(x))     Eq. "accept"
     else draw y from [q-p]_+ / sum [q-p]_+    Eq. "residual"
     Pr(correction) = TV(p,q)                  Proposition 1, Eq. "correction_tv"
  4. accepted:  L_RKL = -A log pi(x),
                A = -sg[log p(x) - log T(x)]   Eqs. "k1_loss_token", "k1_advantage_token"
  5. corrected: L_TM = -log pi(argmax T)       Eq. "teacher_mode_loss"
  6. d(loss)/d(student logits) of the combined
     objective                                 Eq. "general_objective", Appendix C
  7. block verification: commit the accepted
     prefix, correct at the first rejection    Section 3.5, Appendix I
  8. the trainer's step: the same loss and
     gradient for freshly computed student
     logits, from the rollout's metadata only  Section 3.5; Eqs. "k1_loss_token",
                                               "teacher_mode_loss"
  9. the step in front of the path: logits =
     hidden x W^T as the models' lm-heads
     leave them (stored in bf16), with the row
     maximum and log-sum-exp of step 1         Section 3.5, Appendix K; Section 3.1

Readings where the paper is silent are stated next to the code that takes them.
The random numbers are a counter-based Philox4x32-10 stream keyed by
(seed, row, stage); the CUDA library implements the same published generator
on its own.

Parity pins (tests marked "not gpu"): Philox against its published
known-answer vectors; log-softmax against scipy; lambda against an independent
root finder, the V=2 closed form, the two endpoints and the monotone-KL
property; TV by its three equal forms and Pinsker; the coupling by exhaustive
enumeration and by Monte Carlo over seeds; losses and gradient against
torch.autograd in float64 and central differences; block verification by the
product law of the acceptance probabilities; the metadata-driven backward
against torch's cross-entropy (a library routine), central differences, the
zero row sum of a softmax gradient and route() itself on unchanged logits; the
lm-head step against scipy's logsumexp, torch's float64 matmul, one-hot hidden
states (the logits are then a column of W) and equal weight rows (log V).  The
paper prints no worked numeric example for any of these quantities.
"""
from __future__ import annotations

import math
import numpy as np

# RNG stages (the counter word that separates the independent draws of a row)
STAGE_PROPOSE = 0    # per-element Gumbel noise for the proposal utility
STAGE_ACCEPT = 1     # the acceptance uniform
STAGE_RESIDUAL = 2   # the residual (correction) draw
STAGE_BONUS = 3      # the bonus draw of block verification

# row status bits
ST_SATURATED = 1      # lambda = 1 (teacher inside the trust region)
ST_EPS_ZERO = 2       # eps <= 0: student-only fast path
ST_MASKED = 4         # M_t = 0: no supervision at this position
ST_NONFINITE = 8      # a logit is NaN or +-Inf: row not routed
ST_BAD_ID = 16        # proposal id outside [0, V): row not routed
ST_TIMEOUT = 32       # (device only) a bounded wait gave up
ST_NOT_COMPUTED = 64  # block verification: position after the first rejection

_M0 = 0xD2511F53
_M1 = 0xCD9E8D57
_W0 = 0x9E3779B9
_W1 = 0xBB67AE85
_MASK32 = 0xFFFFFFFF


# --------------------------------------------------------------------------
# Random numbers: Philox4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11)
# --------------------------------------------------------------------------
def philox4x32_10(counter, key):
    """Ten rounds of Philox-4x32.  `counter` = 4 words, `key` = 2 words; each
    word may be an int or an integer array (broadcast together).  Returns the
    4 output words as uint64 arrays holding 32-bit values."""
    c = [np.asarray(w, dtype=np.uint64) & np.uint64(_MASK32) for w in counter]
    k = [np.asarray(w, dtype=np.uint64) & np.uint64(_MASK32) for w in key]
    c = list(np.broadcast_arrays(*c))
    m32 = np.uint64(_MASK32)
    sh = np.uint64(32)
    for _ in range(10):
        prod0 = np.uint64(_M0) * c[0]          # < 2^64: no overflow
        prod1 = np.uint64(_M1) * c[2]
        hi0, lo0 = prod0 >> sh, prod0 & m32
        hi1, lo1 = prod1 >> sh, prod1 & m32
        c = [hi1 ^ c[1] ^ k[0], lo1, hi0 ^ c[3] ^ k[1], lo0]
        k = [(k[0] + np.uint64(_W0)) & m32, (k[1] + np.uint64(_W1)) & m32]
    return c


def uniform_from_word(w):
    """Map a 32-bit word to an open-interval uniform that is exact in both
    float32 and float64: an odd multiple of 2^-24."""
    w = np.asarray(w, dtype=np.uint64)
    return ((w >> np.uint64(9)).astype(np.float64) + 0.5) * (2.0 ** -23)


def scalar_uniform(seed: int, row: int, stage: int) -> float:
    """The one uniform a (row, stage) pair owns: word 0 of block 0."""
    seed, row = int(seed), int(row)
    out = philox4x32_10(
        (row & _MASK32, (row >> 32) & _MASK32, stage, 0),
        (seed & _MASK32, (seed >> 32) & _MASK32))
    return float(uniform_from_word(out[0]))


# --------------------------------------------------------------------------
# Step 1: log-softmax (Section 3.1: p_t, T_t are the softmax distributions)
# --------------------------------------------------------------------------
def log_softmax(z):
    z = np.asarray(z, dtype=np.float64)
    m = np.max(z)
    return z - (m + math.log(np.sum(np.exp(z - m))))


# --------------------------------------------------------------------------
# Step 2: geometric bridge and the trust-region coefficient
# --------------------------------------------------------------------------
def bridge_stats(beta: float, lp, d):
    """For q_beta = p^(1-beta) T^beta / Z (Eq. "bridge") with d = log T - log p:
    returns (KL(q_beta || p), log Z(beta), log q_beta).

    log q_beta = log p + beta d - log Z,  log Z = log sum_v p(v) exp(beta d(v));
    KL(q||p) = sum_v q(v) (log q(v) - log p(v))   (student-centred, q first:
    Eq. "trust_region" and the constraint of Eq. "trb_optimization")."""
    w = lp + beta * d
    m = np.max(w)
    logZ = m + math.log(np.sum(np.exp(w - m)))
    lq = w - logZ
    q = np.exp(lq)
    kl = float(np.sum(q * (lq - lp)))
    return kl, float(logZ), lq


def solve_lambda(lp, lT, eps: float) -> float:
    """Largest beta in [0,1] with KL(q_beta || p) <= eps (Eq. "trust_region").

    Readings: eps <= 0 gives 0 (Appendix J, "eps = 0", and the student-only
    fast path of Appendix K); if KL(T || p) <= eps the teacher is feasible and
    beta = 1 (Appendix J, "Teacher endpoint").  Otherwise KL(q_beta||p) is
    continuous and non-decreasing in beta (its slope is beta Var_q(d)), 0 at
    beta=0 and > eps at beta=1, so the largest feasible beta is the root; it
    is bracketed by bisection in float64 and the feasible end is returned.
    (The paper's engine stops after 16 halvings; that is a solver setting,
    coarser than the tolerance this build is checked at, not the definition.)"""
    if not (eps > 0.0):
        return 0.0
    d = lT - lp
    kl1, _, _ = bridge_stats(1.0, lp, d)
    if kl1 <= eps:
        return 1.0
    lo, hi = 0.0, 1.0
    while hi - lo >= 1e-15:
        mid = 0.5 * (lo + hi)
        if mid <= lo or mid >= hi:
            break
        kl, _, _ = bridge_stats(mid, lp, d)
        if kl <= eps:
            lo = mid
        else:
            hi = mid
    return lo


def bridge_distribution(lp, lT, lam: float):
    """(q, log q, log Z, KL(q||p)) at the given coefficient."""
    kl, logZ, lq = bridge_stats(lam, lp, lT - lp)
    return np.exp(lq), lq, logZ, kl


# --------------------------------------------------------------------------
# Step 3: maximal coupling (Section 3.3, Appendix G)
# --------------------------------------------------------------------------
def total_variation(p, q) -> float:
    """TV(p,q) as the positive-residual mass sum_v [q(v)-p(v)]_+, summed in
    index order (equal to 1 - sum min(p,q) and to (1/2) sum |p-q|:
    Eq. "correction_tv" and Appendix G)."""
    r = np.maximum(q - p, 0.0)
    return float(np.cumsum(r)[-1])


def inverse_cdf_draw(weights, u: float):
    """Draw an index from non-negative `weights` (not normalised) by inverse
    CDF in index order with one uniform u in (0,1): the smallest index whose
    running sum exceeds u * total.  Returns (index, margin) where margin is the
    distance from the target to the nearer edge of the chosen cell, as a
    fraction of the total.  If rounding leaves no such index the last index
    with positive weight is taken."""
    c = np.cumsum(weights)
    total = float(c[-1])
    target = u * total
    idx = int(np.searchsorted(c, target, side="right"))
    if idx >= len(c):
        pos = np.nonzero(weights > 0)[0]
        idx = int(pos[-1]) if len(pos) else len(c) - 1
        return idx, 0.0
    below = float(c[idx - 1]) if idx > 0 else 0.0
    margin = min(target - below, float(c[idx]) - target) / total if total > 0 else 0.0
    return idx, margin


# --------------------------------------------------------------------------
# Output rounding
# --------------------------------------------------------------------------
def round_to_bf16(x):
    """Round float64 values to the nearest bfloat16 (ties to even, subnormals
    kept), returned as float64."""
    x = np.asarray(x, dtype=np.float64)
    out = np.zeros_like(x)
    nz = (x != 0) & np.isfinite(x)
    _, e = np.frexp(x[nz])                 # |x| = m 2^e, m in [0.5,1)
    e = np.maximum(e - 1, -126)            # exponent of the leading bit
    quantum = np.ldexp(1.0, e - 7)         # 8 significant bits
    out[nz] = np.rint(x[nz] / quantum) * quantum
    out[~np.isfinite(x)] = x[~np.isfinite(x)]
    big = np.abs(out) > 3.3895313892515355e38
    out[big] = np.sign(out[big]) * np.inf
    return out


# --------------------------------------------------------------------------
# One position
# --------------------------------------------------------------------------
_ZERO_ROW = dict(corrected=0, token=-1, teacher_top1=-1, lam=0.0, kl=0.0,
                 tv=0.0, accept_prob=0.0, logp_x=0.0, logq_x=0.0, logT_x=0.0,
                 logp_y=0.0, logq_y=0.0, logT_y=0.0, loss=0.0, margin_accept=math.inf,
                 margin_draw=math.inf)


def route_row(s, t, x: int, eps: float, temperature: float, seed: int,
              row: int, mask: int = 1, grad_scale: float = 1.0,
              want_grad: bool = False, grad_dtype: str = "f32"):
    """Route one position.  `s`, `t` are the stored student / teacher logit
    rows (any float dtype; widened exactly to float64), `x` the student's
    proposal token z_t ~ p_t (an input: Section 3.3), `row` the global row id
    that keys the random stream.  Returns a dict of the per-position outputs;
    with `want_grad` also "grad", the gradient of grad_scale * loss with
    respect to the stored student logits, rounded to `grad_dtype`
    ("f32" or "bf16")."""
    s = np.asarray(s, dtype=np.float64)
    t = np.asarray(t, dtype=np.float64)
    V = s.shape[0]
    out = dict(_ZERO_ROW)
    out["status"] = 0
    if want_grad:
        out["grad"] = np.zeros(V, dtype=np.float64)
    if not (np.all(np.isfinite(s)) and np.all(np.isfinite(t))):
        out["status"] = ST_NONFINITE      # the paper assumes positive softmax
        return out                        # probabilities (Appendix H)
    if not (0 <= x < V):
        out["status"] = ST_BAD_ID
        return out

    status = 0
    # step 1
    lp = log_softmax(s / temperature)
    lT = log_softmax(t / temperature)
    d = lT - lp
    p = np.exp(lp)
    # teacher mode: lowest index among exact ties of the stored values
    v_star = int(np.argmax(t))

    # step 2
    lam = solve_lambda(lp, lT, eps)
    if not (eps > 0.0):
        status |= ST_EPS_ZERO
    elif lam == 1.0:
        status |= ST_SATURATED
    q, lq, logZ, kl = bridge_distribution(lp, lT, lam)

    # step 3: TV and the coupling.  alpha = exp(min(0, log q(x) - log p(x)))
    # (Appendix K); accept iff u < alpha with u in the open interval (0,1).
    tv = total_variation(p, q)
    if lam == 0.0:
        accept_prob, tv, kl = 1.0, 0.0, 0.0
    else:
        accept_prob = math.exp(min(0.0, lam * d[x] - logZ))
    u_acc = scalar_uniform(seed, row, STAGE_ACCEPT)
    margin_draw = math.inf
    if u_acc < accept_prob:
        corrected, y = 0, x
    else:
        corrected = 1
        u_res = scalar_uniform(seed, row, STAGE_RESIDUAL)
        y, margin_draw = inverse_cdf_draw(np.maximum(q - p, 0.0), u_res)

    # steps 4, 5: the routed loss (pi_theta is numerically p here: one student
    # tensor; the advantage, lambda, q and C are constants of differentiation)
    if mask == 0:
        status |= ST_MASKED
        loss = 0.0
    elif corrected == 0:
        k1 = lp[x] - lT[x]
        loss = k1 * lp[x]                 # -A log pi(x), A = -k1
    else:
        loss = -lp[v_star]

    out.update(corrected=corrected, token=y, teacher_top1=v_star, lam=lam,
               kl=kl, tv=tv, accept_prob=accept_prob, logp_x=float(lp[x]),
               logq_x=float(lq[x]), logT_x=float(lT[x]), logp_y=float(lp[y]),
               logq_y=float(lq[y]), logT_y=float(lT[y]), loss=float(loss), status=status,
               margin_accept=abs(u_acc - accept_prob) if lam > 0.0 else math.inf,
               margin_draw=margin_draw)

    # step 6: gradient with respect to the student logits.
    # d log pi(v) / d s_j = (1[j=v] - p_j) / temperature.
    if want_grad:
        g = np.zeros(V, dtype=np.float64)
        if mask != 0:
            onehot = np.zeros(V, dtype=np.float64)
            if corrected == 0:
                onehot[x] = 1.0
                g = grad_scale * (lp[x] - lT[x]) * (onehot - p) / temperature
            else:
                onehot[v_star] = 1.0
                g = grad_scale * (p - onehot) / temperature
        if grad_dtype == "bf16":
            g = round_to_bf16(g)
        else:
            g = g.astype(np.float32).astype(np.float64)
        out["grad"] = g
    return out


_FIELDS = ("corrected", "token", "teacher_top1", "lam", "kl", "tv",
           "accept_prob", "logp_x", "logq_x", "logT_x", "logp_y", "logq_y", "logT_y",
           "loss", "status", "margin_accept", "margin_draw")
_INT_FIELDS = {"corrected": np.uint8, "token": np.int32,
               "teacher_top1": np.int32, "status": np.uint32}


def route(s, t, proposal, eps, temperature=1.0, seed=0, row_offset=0,
          mask=None, grad_scale=1.0, want_grad=False, grad_dtype="f32",
          rows=None):
    """Route the rows `rows` (default: all) of the [N,V] logit arrays.  Returns
    a dict of arrays indexed like `rows`; "grad" is [len(rows), V]."""
    N = len(proposal)
    rows = range(N) if rows is None else rows
    res = [route_row(s[i], t[i], int(proposal[i]), eps, temperature, seed,
                     row_offset + i, 1 if mask is None else int(mask[i]),
                     grad_scale, want_grad, grad_dtype) for i in rows]
    out = {}
    for f in _FIELDS:
        out[f] = np.array([r[f] for r in res],
                          dtype=_INT_FIELDS.get(f, np.float64))
    if want_grad:
        out["grad"] = np.stack([r["grad"] for r in res]) if res else \
            np.zeros((0, np.asarray(s).shape[1]))
    return out


# --------------------------------------------------------------------------
# The trainer's side: loss and gradient from the routing metadata
# --------------------------------------------------------------------------
_ROLLOUT_UNUSABLE = ST_NONFINITE | ST_BAD_ID | ST_TIMEOUT | ST_NOT_COMPUTED


def bwd_from_meta_row(s, corrected: int, x: int, v_star: int, advantage: float,
                      temperature: float, mask: int = 1, rollout_status: int = 0,
                      grad_scale: float = 1.0, grad_dtype: str = "f32"):
    """Loss and gradient of one position for the CURRENT student logits `s`,
    given only what the rollout returned (Section 3.5: the training loop
    receives token-aligned metadata, not logits): the correction flag C, the
    proposal x, the teacher mode v* and the stop-gradient advantage
    A = log T(x) - log p_rollout(x)  (Eq. "k1_advantage_token").

      C = 0:  L = -A log pi(x)          Eq. "k1_loss_token"
      C = 1:  L = -log pi(v*)           Eq. "teacher_mode_loss"
      dL/ds_j = coef (pi_j - 1[j = tok]) / temperature, (coef, tok) = (A, x) or (1, v*)

    pi = softmax(s / temperature) of the logits passed here, which need not be
    the rollout's.  Readings (the paper does not spell this call out): a
    position that is masked, or whose rollout row was not routed (non-finite
    logits, bad id, timeout, after the first rejection), contributes nothing
    and is reported with ST_MASKED resp. ST_NOT_COMPUTED; a non-finite logit
    or advantage here gives ST_NONFINITE, a supervised token outside [0, V)
    ST_BAD_ID, both with zero loss and gradient."""
    s = np.asarray(s, dtype=np.float64)
    V = s.shape[0]
    out = dict(loss=0.0, logp_tok=0.0, status=0, grad=np.zeros(V, dtype=np.float64))
    if mask == 0:
        out["status"] = ST_MASKED
        return out
    if rollout_status & _ROLLOUT_UNUSABLE:
        out["status"] = ST_NOT_COMPUTED
        return out
    tok = int(v_star) if corrected else int(x)
    coef = 1.0 if corrected else float(advantage)
    if not (np.all(np.isfinite(s)) and math.isfinite(coef)):
        out["status"] = ST_NONFINITE
        return out
    if not (0 <= tok < V):
        out["status"] = ST_BAD_ID
        return out
    lp = log_softmax(s / temperature)
    onehot = np.zeros(V, dtype=np.float64)
    onehot[tok] = 1.0
    g = grad_scale * coef * (np.exp(lp) - onehot) / temperature
    g = round_to_bf16(g) if grad_dtype == "bf16" else g.astype(np.float32).astype(np.float64)
    out.update(loss=float(-coef * lp[tok]), logp_tok=float(lp[tok]), grad=g)
    return out


def bwd_from_meta(s, corrected, proposal, teacher_top1, advantage, temperature=1.0,
                  mask=None, rollout_status=None, grad_scale=1.0, grad_dtype="f32",
                  rows=None):
    """bwd_from_meta_row over the rows `rows` (default: all) of the [N,V] array
    `s`.  Returns arrays indexed like `rows`; "grad" is [len(rows), V]."""
    N = len(proposal)
    rows = range(N) if rows is None else rows
    res = [bwd_from_meta_row(s[i], int(corrected[i]), int(proposal[i]), int(teacher_top1[i]),
                             float(advantage[i]), temperature,
                             1 if mask is None else int(mask[i]),
                             0 if rollout_status is None else int(rollout_status[i]),
                             grad_scale, grad_dtype) for i in rows]
    return dict(loss=np.array([r["loss"] for r in res], dtype=np.float64),
                logp_tok=np.array([r["logp_tok"] for r in res], dtype=np.float64),
                status=np.array([r["status"] for r in res], dtype=np.uint32),
                grad=np.stack([r["grad"] for r in res]) if res else np.zeros((0, np.asarray(s).shape[1])))


# --------------------------------------------------------------------------
# Placement controls: where teacher-mode supervision goes (Appendix "placement_control")
# --------------------------------------------------------------------------
STAGE_SELECT = 4     # the uniform of a position's exponential-race key
SELECT_RANDOM = 0
SELECT_TV_WEIGHTED = 1


def select_tm(seq_start, corrected, tv, mode: int, seed=0, row_offset=0, mask=None,
              rollout_status=None):
    """For every trajectory b (positions seq_start[b] .. seq_start[b+1]-1) choose
    m_b = number of corrected valid positions of b, valid positions to receive
    the teacher-mode loss instead of the coupling's own corrections:

      Random-TM        m_b valid positions uniformly at random (count-matched
                       random locations);
      TV-Weighted-TM   m_b valid positions without replacement with weights
                       d_t = TV(p_t, q_t), by exponential-race keys
                       -log U_t / d_t, the m_b smallest; if fewer than m_b
                       valid positions have positive TV the rest is filled
                       uniformly.

    Readings: U_t is the (seed, row, STAGE_SELECT) uniform of the position; a
    position is valid if its mask is 1 and the rollout routed it; "uniformly"
    = the smallest U_t among the positions not yet chosen; ties go to the
    lower index.  Returns (selected [N] uint8, m [B] int32, margin [B]: the
    relative gap between the last chosen and the first rejected key, inf if
    there is no choice to make)."""
    seq_start = np.asarray(seq_start, dtype=np.int64)
    N = int(seq_start[-1])
    B = len(seq_start) - 1
    selected = np.zeros(N, dtype=np.uint8)
    m_out = np.zeros(B, dtype=np.int32)
    margin = np.full(B, np.inf)
    for b in range(B):
        lo, hi = int(seq_start[b]), int(seq_start[b + 1])
        keys = []
        m = 0
        for i in range(lo, hi):
            ok = (mask is None or mask[i] != 0) and \
                 (rollout_status is None or not (int(rollout_status[i]) & _ROLLOUT_UNUSABLE))
            if not ok:
                continue
            m += int(corrected[i] != 0)
            u = scalar_uniform(seed, row_offset + i, STAGE_SELECT)
            d = float(tv[i]) if mode == SELECT_TV_WEIGHTED else 0.0
            if mode == SELECT_TV_WEIGHTED and d > 0.0 and math.isfinite(d):
                keys.append((0, -math.log(u) / d, i))
            else:
                keys.append((1 if mode == SELECT_TV_WEIGHTED else 0, u, i))
        keys.sort()
        m_out[b] = m
        for k in keys[:m]:
            selected[k[2]] = 1
        if 0 < m < len(keys):
            a, c = keys[m - 1], keys[m]
            if a[0] == c[0]:
                margin[b] = abs(c[1] - a[1]) / max(abs(c[1]), 1e-300)
    return selected, m_out, margin


# --------------------------------------------------------------------------
# Proposal utility: x ~ softmax(s / temperature) by Gumbel-max
# --------------------------------------------------------------------------
def sample_proposal_row(s, temperature: float, seed: int, row: int):
    """argmax_v (s_v / temperature + G_v), G_v = -log(-log u_v),
    u_v = (w_v + 0.5) 2^-32 with w_v word (v mod 4) of Philox block v // 4 at
    stage PROPOSE.  Lowest index on ties.  Returns (index, gap between the two
    largest keys)."""
    s = np.asarray(s, dtype=np.float64)
    seed, row = int(seed), int(row)
    V = s.shape[0]
    nblk = (V + 3) // 4
    words = philox4x32_10(
        (row & _MASK32, (row >> 32) & _MASK32, STAGE_PROPOSE,
         np.arange(nblk, dtype=np.uint64)),
        (seed & _MASK32, (seed >> 32) & _MASK32))
    w = np.stack(words, axis=1).reshape(-1)[:V]
    u = (w.astype(np.float64) + 0.5) * (2.0 ** -32)
    keys = s / temperature - np.log(-np.log(u))
    idx = int(np.argmax(keys))
    top = keys[idx]
    keys[idx] = -np.inf
    gap = float(top - np.max(keys)) if V > 1 else math.inf
    return idx, gap


def sample_proposal(s, temperature=1.0, seed=0, row_offset=0, rows=None):
    N = np.asarray(s).shape[0]
    rows = range(N) if rows is None else rows
    res = [sample_proposal_row(s[i], temperature, seed, row_offset + i)
           for i in rows]
    return (np.array([r[0] for r in res], dtype=np.int32),
            np.array([r[1] for r in res], dtype=np.float64))


# --------------------------------------------------------------------------
# Step 7: block verification (Section 3.5; Appendix I; Appendix K)
# --------------------------------------------------------------------------
def spec_verify(s, t, draft, eps, temperature=1.0, seed=0, seq_offset=0):
    """`s`, `t`: [B, K+1, V] logits of the K drafted positions plus one bonus
    position; `draft`: [B, K] drafted ids.  Positions are verified left to
    right with the same per-position coupling as `route_row`, the row id of
    position j of sequence b being (seq_offset + b)(K+1) + j.  The accepted
    prefix is committed; at the first rejection j the residual draw is the
    next token.  If all K are accepted the next token is drawn from q at the
    bonus position by inverse CDF (reading: the paper has no bonus token; the
    workload definition asks for one, and with no proposal to couple against
    the exact-q draw is a plain sample of q).

    Returns n_accept [B], next_token [B], next_is_correction [B], and per
    position dicts (rows after the first rejection carry ST_NOT_COMPUTED)."""
    s = np.asarray(s)
    t = np.asarray(t)
    B, K1, V = s.shape
    K = K1 - 1
    n_accept = np.zeros(B, dtype=np.int32)
    next_token = np.full(B, -1, dtype=np.int32)
    next_is_corr = np.zeros(B, dtype=np.uint8)
    margins = np.full(B, math.inf)
    per_pos = [[None] * K1 for _ in range(B)]
    for b in range(B):
        n, stopped = K, False
        for j in range(K):
            r = (seq_offset + b) * K1 + j
            res = route_row(s[b, j], t[b, j], int(draft[b, j]), eps,
                            temperature, seed, r)
            per_pos[b][j] = res
            margins[b] = min(margins[b], res["margin_accept"], res["margin_draw"])
            if res["status"] & (ST_NONFINITE | ST_BAD_ID):
                n, stopped = j, True       # cannot verify: nothing committed here
                break
            if res["corrected"]:
                n, stopped = j, True
                next_token[b] = res["token"]
                next_is_corr[b] = 1
                break
        n_accept[b] = n
        if not stopped:
            r = (seq_offset + b) * K1 + K
            sk = np.asarray(s[b, K], dtype=np.float64)
            tk = np.asarray(t[b, K], dtype=np.float64)
            bonus = dict(_ZERO_ROW)
            bonus["status"] = 0
            if np.all(np.isfinite(sk)) and np.all(np.isfinite(tk)):
                lp = log_softmax(sk / temperature)
                lT = log_softmax(tk / temperature)
                lam = solve_lambda(lp, lT, eps)
                q, lq, logZ, kl = bridge_distribution(lp, lT, lam)
                u = scalar_uniform(seed, r, STAGE_BONUS)
                y, m = inverse_cdf_draw(q, u)
                bonus.update(token=y, teacher_top1=int(np.argmax(tk)), lam=lam,
                             kl=kl if lam > 0 else 0.0,
                             tv=total_variation(np.exp(lp), q) if lam > 0 else 0.0,
                             logp_y=float(lp[y]), logq_y=float(lq[y]), logT_y=float(lT[y]),
                             margin_draw=m)
                if not (eps > 0):
                    bonus["status"] |= ST_EPS_ZERO
                elif lam == 1.0:
                    bonus["status"] |= ST_SATURATED
                next_token[b] = y
                margins[b] = min(margins[b], m)
            else:
                bonus["status"] = ST_NONFINITE
            per_pos[b][K] = bonus
        for j in range(K1):
            if per_pos[b][j] is None:
                nc = dict(_ZERO_ROW)
                nc["status"] = ST_NOT_COMPUTED
                per_pos[b][j] = nc
    return dict(n_accept=n_accept, next_token=next_token,
                next_is_correction=next_is_corr, margin=margins,
                per_pos=per_pos)


# --------------------------------------------------------------------------
# The step in front of the path: the lm-head that leaves the logits
# --------------------------------------------------------------------------
def lmhead_lse(hidden, weight, temperature: float = 1.0):
    """`hidden`: [N, d], `weight`: [V, d] (one row per vocabulary entry), the
    stored (bf16) values widened exactly to float64.  Section 3.5 / Appendix K:
    the student and the teacher each leave full-vocabulary logits
    logits[i, v] = sum_k hidden[i, k] weight[v, k]; they are stored in bf16
    (round to nearest even), and Section 3.1's softmax is taken of the STORED
    values: row_max[i] = max_v logits[i, v], lse[i] = log sum_v
    exp(logits[i, v] / temperature).  Returns (logits as float64 holding bf16
    values, row_max, lse)."""
    h = np.asarray(hidden, dtype=np.float64)
    w = np.asarray(weight, dtype=np.float64)
    logits = round_to_bf16(h @ w.T)
    z = logits / temperature
    m = z.max(axis=1)
    lse = m + np.log(np.exp(z - m[:, None]).sum(axis=1))
    return logits, logits.max(axis=1), lse

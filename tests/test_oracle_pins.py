"""Pins of the float64 oracle against what the paper and the mathematics fix.
None of these re-types the oracle's own formula: each compares with a library
routine, a closed form, an exhaustive enumeration or a Monte-Carlo law."""
import ctypes
import math
import os

import numpy as np
import pytest
import scipy.optimize
import scipy.special
import torch

import oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rows(V, seed, sig=1.5, n=1):
    rng = np.random.default_rng(seed)
    s = rng.normal(0, 2, (n, V))
    t = s + rng.normal(0, sig, (n, V))
    return s, t


# ---------------------------------------------------------------- Philox
def test_philox_known_answers():
    for line in open(os.path.join(GOLDEN, "philox4x32_10_kat.txt")):
        if line.startswith("#") or not line.strip():
            continue
        w = [int(h, 16) for h in line.split()]
        out = O.philox4x32_10(w[0:4], w[4:6])
        assert [int(v) for v in out] == w[6:10]


def test_philox_matches_curand_host_generator():
    """cuRAND's host-side PHILOX4_32_10 generator (no GPU needed): its k-th
    block of four words is Philox(counter=(0,0,k,0), key=seed)."""
    try:
        lib = ctypes.CDLL("libcurand.so.10")
    except OSError:
        try:
            lib = ctypes.CDLL("/usr/local/cuda/lib64/libcurand.so")
        except OSError:
            pytest.skip("cuRAND not present")
    gen = ctypes.c_void_p()
    assert lib.curandCreateGeneratorHost(ctypes.byref(gen), 161) == 0
    for seed in (0, 0x299F31D0A4093822, 12345, 2**64 - 1):
        assert lib.curandSetPseudoRandomGeneratorSeed(gen, ctypes.c_ulonglong(seed)) == 0
        assert lib.curandSetGeneratorOffset(gen, ctypes.c_ulonglong(0)) == 0
        buf = (ctypes.c_uint32 * 64)()
        assert lib.curandGenerate(gen, buf, 64) == 0
        for k in range(16):
            mine = O.philox4x32_10((0, 0, k, 0), (seed & 0xFFFFFFFF, seed >> 32))
            assert [int(v) for v in mine] == list(buf[4 * k:4 * k + 4])
    lib.curandDestroyGenerator(gen)


def test_philox_vectorised_equals_scalar():
    ks = np.arange(50, dtype=np.uint64)
    vec = O.philox4x32_10((7, 1, 2, ks), (99, 3))
    for k in (0, 13, 49):
        one = O.philox4x32_10((7, 1, 2, int(k)), (99, 3))
        assert [int(v[k]) for v in vec] == [int(v) for v in one]


def test_uniform_is_open_interval_and_fp32_exact():
    w = np.array([0, 1, 511, 512, 2**32 - 1], dtype=np.uint64)
    u = O.uniform_from_word(w)
    assert u.min() == 2.0 ** -24 and u.max() == 1 - 2.0 ** -24
    assert np.all(u.astype(np.float32).astype(np.float64) == u)
    # the 23-bit bucket is uniform: mean of many draws -> 1/2
    ws = O.philox4x32_10((np.arange(20000, dtype=np.uint64), 0, 1, 0), (5, 0))[0]
    assert abs(O.uniform_from_word(ws).mean() - 0.5) < 4 * (1 / math.sqrt(12 * 20000))


# ---------------------------------------------------------------- step 1
def test_log_softmax_matches_scipy():
    s, _ = _rows(3000, 1)
    s[0, 5] = 700.0  # needs the max shift
    assert np.allclose(O.log_softmax(s[0]), scipy.special.log_softmax(s[0]), rtol=0, atol=1e-12)


# ---------------------------------------------------------------- step 2
def test_lambda_agrees_with_independent_root_finder_and_hits_eps():
    for seed, eps in [(2, 0.1), (3, 0.01), (4, 0.5), (5, 0.02)]:
        s, t = _rows(500, seed)
        lp, lT = scipy.special.log_softmax(s[0]), scipy.special.log_softmax(t[0])
        lam = O.solve_lambda(lp, lT, eps)

        def kl_of(b):   # written from the definition with scipy, not the oracle
            lq = scipy.special.log_softmax(lp + b * (lT - lp))
            return float(np.sum(np.exp(lq) * (lq - lp)))
        assert 0 < lam < 1
        ref = scipy.optimize.brentq(lambda b: kl_of(b) - eps, 1e-12, 1.0, xtol=1e-15, rtol=1e-15)
        assert abs(lam - ref) < 1e-12
        assert abs(kl_of(lam) - eps) < 1e-12
        assert kl_of(lam) <= eps + 1e-15 or abs(kl_of(lam) - eps) < 1e-13  # feasible side


def test_lambda_V2_closed_form():
    """V=2, uniform p: q=(x,1-x), KL(q||p) = log 2 - H(x).  With T=(a,1-a),
    q_beta ~ (a^beta, (1-a)^beta), so beta = logit(x*) / logit(a) where x* is
    the inverse binary entropy at log 2 - eps."""
    a, eps = 0.9, 0.05
    lp = np.log(np.array([0.5, 0.5]))
    lT = np.log(np.array([a, 1 - a]))

    def H(x):
        return -(x * math.log(x) + (1 - x) * math.log(1 - x))
    xs = scipy.optimize.brentq(lambda x: math.log(2) - H(x) - eps, 0.5 + 1e-12, 1 - 1e-12, xtol=1e-15)
    beta = math.log(xs / (1 - xs)) / math.log(a / (1 - a))
    assert abs(O.solve_lambda(lp, lT, eps) - beta) < 1e-12


def test_lambda_endpoints():
    s, t = _rows(200, 6)
    lp, lT = O.log_softmax(s[0]), O.log_softmax(t[0])
    kl_teacher = float(np.sum(np.exp(lT) * (lT - lp)))   # KL(T||p)
    assert O.solve_lambda(lp, lT, 0.0) == 0.0
    assert O.solve_lambda(lp, lT, -1.0) == 0.0
    assert O.solve_lambda(lp, lT, kl_teacher * 1.0000001) == 1.0
    assert O.solve_lambda(lp, lT, kl_teacher * 0.999) < 1.0
    assert O.solve_lambda(lp, lp.copy(), 0.3) == 1.0       # p == T, eps > 0
    q, lq, logZ, kl = O.bridge_distribution(lp, lT, 0.0)
    assert np.allclose(q, np.exp(lp), atol=1e-15) and abs(kl) < 1e-15
    q, lq, logZ, kl = O.bridge_distribution(lp, lT, 1.0)
    assert np.allclose(q, np.exp(lT), atol=1e-15) and abs(kl - kl_teacher) < 1e-12 and abs(logZ) < 1e-12


def test_kl_monotone_in_beta_with_slope_beta_var():
    s, t = _rows(400, 7)
    lp, lT = O.log_softmax(s[0]), O.log_softmax(t[0])
    d = lT - lp
    grid = np.linspace(0, 1, 101)
    kls = [O.bridge_stats(b, lp, d)[0] for b in grid]
    assert np.all(np.diff(kls) > 0)
    b, h = 0.37, 1e-5
    slope = (O.bridge_stats(b + h, lp, d)[0] - O.bridge_stats(b - h, lp, d)[0]) / (2 * h)
    q = np.exp(O.bridge_stats(b, lp, d)[2])
    var = np.sum(q * d * d) - np.sum(q * d) ** 2
    assert abs(slope - b * var) < 1e-7
    # small-eps asymptote: lambda ~ sqrt(2 eps / Var_p d)
    p = np.exp(lp)
    varp = np.sum(p * d * d) - np.sum(p * d) ** 2
    eps = 1e-6
    assert abs(O.solve_lambda(lp, lT, eps) / math.sqrt(2 * eps / varp) - 1) < 0.01


def test_bridge_is_normalised_geometric_mean_and_residual_support():
    s, t = _rows(300, 8)
    lp, lT = O.log_softmax(s[0]), O.log_softmax(t[0])
    lam = O.solve_lambda(lp, lT, 0.1)
    q, lq, logZ, kl = O.bridge_distribution(lp, lT, lam)
    p, T = np.exp(lp), np.exp(lT)
    direct = p ** (1 - lam) * T ** lam
    assert abs(q.sum() - 1) < 1e-14
    assert np.allclose(q, direct / direct.sum(), rtol=1e-12)
    assert abs(math.exp(logZ) - direct.sum()) < 1e-14
    # Appendix H: q > p  <=>  log(T/p) > log Z / beta
    assert np.array_equal(q > p, (lT - lp) > logZ / lam)


# ---------------------------------------------------------------- step 3
def test_tv_three_forms_and_pinsker():
    for seed, eps in [(9, 0.1), (10, 0.02), (11, 1.0)]:
        s, t = _rows(256, seed)
        lp, lT = O.log_softmax(s[0]), O.log_softmax(t[0])
        lam = O.solve_lambda(lp, lT, eps)
        q, _, _, kl = O.bridge_distribution(lp, lT, lam)
        p = np.exp(lp)
        tv = O.total_variation(p, q)
        assert abs(tv - (1 - np.minimum(p, q).sum())) < 1e-13
        assert abs(tv - 0.5 * np.abs(p - q).sum()) < 1e-13
        assert tv <= math.sqrt(kl / 2) + 1e-15 <= math.sqrt(eps / 2) + 1e-12


def test_coupling_enumeration_correction_probability_is_tv():
    """Summing the oracle's own per-proposal acceptance probability over all
    proposals x weighted by p(x) gives 1 - TV, and p(x) a(x) = min(p,q)(x)."""
    V = 12
    s, t = _rows(V, 12)
    lp, lT = O.log_softmax(s[0]), O.log_softmax(t[0])
    p = np.exp(lp)
    acc = np.zeros(V)
    for x in range(V):
        r = O.route_row(s[0], t[0], x, 0.2, 1.0, 0, 0)
        acc[x] = r["accept_prob"]
        tv, lam = r["tv"], r["lam"]
    q = O.bridge_distribution(lp, lT, lam)[0]
    assert np.allclose(p * acc, np.minimum(p, q), atol=1e-14)
    assert abs(np.sum(p * (1 - acc)) - tv) < 1e-13
    assert np.allclose(np.minimum(p, q) + np.maximum(q - p, 0), q, atol=1e-15)


def test_inverse_cdf_sweep_reproduces_weights():
    w = np.array([0.0, 0.2, 0.0, 0.5, 0.3, 0.0])
    n = 20000
    us = (np.arange(n) + 0.5) / n
    hist = np.bincount([O.inverse_cdf_draw(w, u)[0] for u in us], minlength=len(w)) / n
    assert np.allclose(hist, w / w.sum(), atol=2 / n)
    idx, margin = O.inverse_cdf_draw(w, 0.45)   # target .45 lies in cell 3 = (.2,.7]
    assert idx == 3 and abs(margin - 0.25) < 1e-15
    assert O.inverse_cdf_draw(w, 1 - 1e-17)[0] == 4   # never a zero-weight index


def test_monte_carlo_coupling_law():
    """Over many rows (= independent random streams) with the proposal drawn
    from p: acceptance rate -> 1-TV, committed tokens ~ q, corrections ~
    [q-p]_+/TV, rejected proposals ~ [p-q]_+/TV (Appendix G)."""
    V, n = 6, 30000
    s, t = _rows(V, 13, sig=2.0)
    lp, lT = O.log_softmax(s[0]), O.log_softmax(t[0])
    p = np.exp(lp)
    rng = np.random.default_rng(99)
    xs = rng.choice(V, size=n, p=p)
    committed = np.zeros(V)
    corr = np.zeros(V)
    rej = np.zeros(V)
    for i, x in enumerate(xs):
        r = O.route_row(s[0], t[0], int(x), 0.3, 1.0, 77, i)
        committed[r["token"]] += 1
        if r["corrected"]:
            corr[r["token"]] += 1
            rej[x] += 1
    lam, tv = r["lam"], r["tv"]
    q = O.bridge_distribution(lp, lT, lam)[0]
    ncorr = corr.sum()
    assert abs(ncorr / n - tv) < 4 * math.sqrt(tv * (1 - tv) / n)
    assert np.all(np.abs(committed / n - q) < 4.5 * np.sqrt(q * (1 - q) / n) + 1e-9)
    r_pos = np.maximum(q - p, 0) / tv
    r_neg = np.maximum(p - q, 0) / tv
    assert np.all(np.abs(corr / ncorr - r_pos) < 4.5 * np.sqrt(r_pos * (1 - r_pos) / ncorr) + 1e-9)
    assert np.all(np.abs(rej / ncorr - r_neg) < 4.5 * np.sqrt(r_neg * (1 - r_neg) / ncorr) + 1e-9)
    assert np.all(corr[q <= p] == 0)


def test_minimal_intervention_on_tiny_alphabet():
    """Any coupling has Pr(Z != Y) >= TV (Proposition 2): check by linear
    programming over all couplings of a 3-letter alphabet."""
    s, t = _rows(3, 14, sig=2.0)
    lp, lT = O.log_softmax(s[0]), O.log_softmax(t[0])
    lam = O.solve_lambda(lp, lT, 0.3)
    q = O.bridge_distribution(lp, lT, lam)[0]
    p = np.exp(lp)
    V = 3
    A_eq, b_eq = [], []
    for i in range(V):
        row = np.zeros((V, V)); row[i, :] = 1; A_eq.append(row.ravel()); b_eq.append(p[i])
        col = np.zeros((V, V)); col[:, i] = 1; A_eq.append(col.ravel()); b_eq.append(q[i])
    cost = (1 - np.eye(V)).ravel()
    res = scipy.optimize.linprog(cost, A_eq=np.array(A_eq), b_eq=np.array(b_eq), bounds=(0, None))
    assert abs(res.fun - O.total_variation(p, q)) < 1e-9


# ---------------------------------------------------------------- steps 4-6
def test_losses_and_gradient_match_autograd_and_finite_differences():
    V = 40
    s, t = _rows(V, 15)
    tau = 1.3
    for row in range(60):      # find both branches
        x = row % V
        r = O.route_row(s[0], t[0], x, 0.3, tau, 5, row, grad_scale=0.25, want_grad=True, grad_dtype="f32")
        st = torch.tensor(s[0], dtype=torch.float64, requires_grad=True)
        ls = torch.log_softmax(st / tau, 0)
        lT = torch.log_softmax(torch.tensor(t[0], dtype=torch.float64) / tau, 0)
        if r["corrected"] == 0:
            A = -(ls[x] - lT[x]).detach()            # Eq. k1_advantage_token
            loss = -A * ls[x]                        # Eq. k1_loss_token
        else:
            vstar = int(torch.argmax(lT))
            assert r["teacher_top1"] == vstar
            loss = torch.nn.functional.cross_entropy((st / tau)[None], torch.tensor([vstar]))
        (0.25 * loss).backward()
        assert abs(r["loss"] - loss.item()) < 1e-12
        g = st.grad.numpy()
        assert np.max(np.abs(r["grad"] - g.astype(np.float32))) < 1e-7
        assert abs(r["grad"].sum()) < 1e-6
    # central differences on the scalar loss with routing frozen
    r = O.route_row(s[0], t[0], 3, 0.3, tau, 5, 0, want_grad=True)
    lTn = O.log_softmax(t[0] / tau)
    k1 = O.log_softmax(s[0] / tau)[3] - lTn[3]

    def f(sv):
        lpn = O.log_softmax(sv / tau)
        return k1 * lpn[3] if r["corrected"] == 0 else -lpn[r["teacher_top1"]]
    for j in (0, 3, 17):
        e = np.zeros(V); e[j] = 1e-6
        fd = (f(s[0] + e) - f(s[0] - e)) / 2e-6
        assert abs(fd - r["grad"][j]) < 1e-6


def test_expected_overlap_identity():
    """E[(1-C) L_RKL(Z)] = sum_v min(p,q)(v) L_RKL(v)  (Eq. expected_overlap_k1),
    the expectation taken by enumeration over proposals with the oracle's
    acceptance probabilities."""
    V = 10
    s, t = _rows(V, 16)
    lp, lT = O.log_softmax(s[0]), O.log_softmax(t[0])
    p = np.exp(lp)
    lhs = 0.0
    for x in range(V):
        r = O.route_row(s[0], t[0], x, 0.2, 1.0, 0, 0)
        l_rkl = (lp[x] - lT[x]) * lp[x]
        lhs += p[x] * r["accept_prob"] * l_rkl
    q = O.bridge_distribution(lp, lT, r["lam"])[0]
    rhs = np.sum(np.minimum(p, q) * (lp - lT) * lp)
    assert abs(lhs - rhs) < 1e-13


def test_eps_zero_is_student_only():
    s, t = _rows(64, 17, n=20)
    x = np.arange(20) % 64
    r = O.route(s, t, x, 0.0, want_grad=True)
    assert np.all(r["lam"] == 0) and np.all(r["tv"] == 0) and np.all(r["corrected"] == 0)
    assert np.array_equal(r["token"], x) and np.all(r["status"] & O.ST_EPS_ZERO)
    for i in range(20):
        lp, lT = O.log_softmax(s[i]), O.log_softmax(t[i])
        assert abs(r["loss"][i] - (lp[x[i]] - lT[x[i]]) * lp[x[i]]) < 1e-13


def test_mask_and_flagged_rows():
    s, t = _rows(32, 18, n=3)
    r = O.route_row(s[0], t[0], 4, 0.1, 1.0, 0, 0, mask=0, want_grad=True)
    assert r["loss"] == 0 and np.all(r["grad"] == 0) and r["status"] & O.ST_MASKED and r["lam"] > 0
    bad = s[1].copy(); bad[7] = np.nan
    r = O.route_row(bad, t[1], 4, 0.1, 1.0, 0, 1, want_grad=True)
    assert r["status"] == O.ST_NONFINITE and r["token"] == -1 and np.all(r["grad"] == 0)
    r = O.route_row(s[2], t[2], 32, 0.1, 1.0, 0, 2)
    assert r["status"] == O.ST_BAD_ID and r["token"] == -1


def test_teacher_argmax_lowest_index_on_ties():
    s, t = _rows(16, 19)
    t[0, 3] = t[0, 11] = t[0].max() + 1
    assert O.route_row(s[0], t[0], 0, 0.1, 1.0, 0, 0)["teacher_top1"] == 3


def test_round_to_bf16_matches_torch():
    rng = np.random.default_rng(3)
    x = np.concatenate([rng.normal(0, 1, 4000), rng.normal(0, 1e-20, 1000), rng.normal(0, 1e-39, 1000),
                        [0.0, 1.00390625, 1.01171875, -3.0e38]])
    x32 = x.astype(np.float32).astype(np.float64)     # no double rounding for fp32-exact inputs
    ref = torch.tensor(x32, dtype=torch.float32).to(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(O.round_to_bf16(x32), ref)


# ---------------------------------------------------------------- proposal utility
def test_gumbel_max_proposal_follows_softmax():
    V, n = 8, 20000
    s, _ = _rows(V, 20)
    p = scipy.special.softmax(s[0] / 0.7)
    idx, gaps = O.sample_proposal(np.repeat(s, n, 0), temperature=0.7, seed=11)
    hist = np.bincount(idx, minlength=V) / n
    assert np.all(np.abs(hist - p) < 4.5 * np.sqrt(p * (1 - p) / n) + 1e-9)
    assert np.all(gaps >= 0)


# ---------------------------------------------------------------- step 7
def test_spec_verify_semantics():
    B, K, V = 400, 3, 8
    rng = np.random.default_rng(21)
    s1 = rng.normal(0, 2, (1, K + 1, V)); t1 = s1 + rng.normal(0, 2.0, (1, K + 1, V))
    s = np.repeat(s1, B, 0); t = np.repeat(t1, B, 0)
    draft = np.tile(np.array([[1, 5, 2]]), (B, 1))
    eps = 0.3
    out = O.spec_verify(s, t, draft, eps, seed=4)
    # law of the accepted-prefix length: prod_{i<j} a_i (1 - a_j)
    a = [O.route_row(s1[0, j], t1[0, j], int(draft[0, j]), eps, 1.0, 4, 0)["accept_prob"] for j in range(K)]
    probs = [np.prod(a[:j]) * (1 - a[j]) for j in range(K)] + [np.prod(a)]
    hist = np.bincount(out["n_accept"], minlength=K + 1) / B
    assert np.all(np.abs(hist - probs) < 4.5 * np.sqrt(np.array(probs) * (1 - np.array(probs)) / B) + 1e-9)
    for b in range(B):
        n = out["n_accept"][b]
        pp = out["per_pos"][b]
        assert all(pp[j]["corrected"] == 0 for j in range(n))
        if n < K:
            assert pp[n]["corrected"] == 1 and out["next_token"][b] == pp[n]["token"]
            assert out["next_is_correction"][b] == 1
            assert all(pp[j]["status"] == O.ST_NOT_COMPUTED for j in range(n + 1, K + 1))
        else:
            assert out["next_is_correction"][b] == 0 and out["next_token"][b] == pp[K]["token"]
        # row ids: position j of sequence b is keyed (b)(K+1)+j, so any order gives the same result
        j = min(n, K - 1)
        again = O.route_row(s[b, j], t[b, j], int(draft[b, j]), eps, 1.0, 4, b * (K + 1) + j)
        assert again["corrected"] == pp[j]["corrected"] and again["token"] == pp[j]["token"]
    # bonus draws follow q_K
    full = out["n_accept"] == K
    lp, lT = O.log_softmax(s1[0, K]), O.log_softmax(t1[0, K])
    q = O.bridge_distribution(lp, lT, O.solve_lambda(lp, lT, eps))[0]
    if full.sum() > 50:
        h = np.bincount(out["next_token"][full], minlength=V) / full.sum()
        assert np.all(np.abs(h - q) < 5 * np.sqrt(q * (1 - q) / full.sum()) + 1e-9)
    # eps = 0: everything accepted, bonus ~ p
    out0 = O.spec_verify(s[:5], t[:5], draft[:5], 0.0, seed=4)
    assert np.all(out0["n_accept"] == K) and np.all(out0["next_is_correction"] == 0)


# ---------------------------------------------------------------- metadata-driven backward
def _meta_case(rng, N, V):
    s = rng.normal(size=(N, V)) * 2.0
    C = (rng.random(N) < 0.4).astype(np.uint8)
    x = rng.integers(0, V, N).astype(np.int32)
    vs = rng.integers(0, V, N).astype(np.int32)
    A = rng.normal(size=N)
    return s, C, x, vs, A


def test_meta_backward_matches_torch_cross_entropy_and_autograd():
    """Corrected rows are a cross-entropy on the teacher mode (Eq. "teacher_mode_loss"): pinned to
    torch's library routine.  Accepted rows are -A log pi(x) (Eq. "k1_loss_token"): pinned to
    float64 autograd of that expression written with torch ops."""
    rng = np.random.default_rng(41)
    N, V, tau, scale = 12, 57, 0.7, 0.25
    s, C, x, vs, A = _meta_case(rng, N, V)
    res = O.bwd_from_meta(s, C, x, vs, A, temperature=tau, grad_scale=scale, grad_dtype="f32")
    z = torch.tensor(s, dtype=torch.float64, requires_grad=True)
    ce = torch.nn.functional.cross_entropy(z / tau, torch.tensor(vs, dtype=torch.long), reduction="none")
    lp = torch.log_softmax(z / tau, dim=1)
    rkl = -torch.tensor(A) * lp[torch.arange(N), torch.tensor(x, dtype=torch.long)]
    loss = torch.where(torch.tensor(C.astype(bool)), ce, rkl)
    (scale * loss.sum()).backward()
    assert np.allclose(res["loss"], loss.detach().numpy(), rtol=1e-12, atol=1e-12)
    assert np.allclose(res["grad"], z.grad.numpy().astype(np.float32).astype(np.float64), rtol=0, atol=1e-7)
    tok = np.where(C == 1, vs, x)
    assert np.allclose(res["logp_tok"], lp.detach().numpy()[np.arange(N), tok], atol=1e-12)
    assert np.all(res["status"] == 0)


def test_meta_backward_central_differences_and_zero_row_sum():
    rng = np.random.default_rng(42)
    N, V, tau = 4, 9, 1.3
    s, C, x, vs, A = _meta_case(rng, N, V)
    C[:] = [0, 1, 0, 1]
    res = O.bwd_from_meta(s, C, x, vs, A, temperature=tau, grad_dtype="f32")
    # the softmax part sums to one and the one-hot part to one: every gradient row sums to zero
    assert np.all(np.abs(res["grad"].sum(axis=1)) < 1e-6)
    h = 1e-6
    for i in range(N):
        for j in range(V):
            sp, sm = s.copy(), s.copy()
            sp[i, j] += h
            sm[i, j] -= h
            lp_ = O.bwd_from_meta(sp, C, x, vs, A, temperature=tau)["loss"][i]
            lm_ = O.bwd_from_meta(sm, C, x, vs, A, temperature=tau)["loss"][i]
            assert abs((lp_ - lm_) / (2 * h) - res["grad"][i, j]) < 1e-6


def test_meta_backward_on_unchanged_logits_equals_routing():
    """With the rollout's own logits and its metadata the trainer's call reproduces the loss and the
    gradient of the routing call (Eq. "general_objective")."""
    rng = np.random.default_rng(43)
    N, V, eps, tau = 40, 300, 0.15, 0.9
    s = rng.normal(size=(N, V)) * 2.0
    t = s + rng.normal(size=(N, V)) * 1.5
    x = np.array([O.sample_proposal_row(s[i], tau, 5, i)[0] for i in range(N)], dtype=np.int32)
    mask = (rng.random(N) < 0.8).astype(np.uint8)
    r = O.route(s, t, x, eps, tau, seed=5, mask=mask, grad_scale=0.1, want_grad=True, grad_dtype="bf16")
    assert 0 < r["corrected"].sum() < N
    A = r["logT_x"] - r["logp_x"]
    m = O.bwd_from_meta(s, r["corrected"], x, r["teacher_top1"], A, tau, mask=mask, rollout_status=r["status"],
                        grad_scale=0.1, grad_dtype="bf16")
    assert np.allclose(m["loss"], r["loss"], rtol=1e-12, atol=1e-14)
    assert np.array_equal(m["grad"], r["grad"])
    assert np.all((m["status"] == O.ST_MASKED) == (mask == 0))


def test_meta_backward_flags():
    rng = np.random.default_rng(44)
    N, V = 6, 33
    s, C, x, vs, A = _meta_case(rng, N, V)
    C[:] = [0, 1, 0, 1, 0, 0]
    s[0, 3] = np.nan
    vs[1] = V
    x[2] = -1
    A[4] = np.inf
    st = np.zeros(N, dtype=np.uint32)
    st[3] = O.ST_NOT_COMPUTED
    mask = np.ones(N, dtype=np.uint8)
    mask[5] = 0
    res = O.bwd_from_meta(s, C, x, vs, A, mask=mask, rollout_status=st)
    assert list(res["status"]) == [O.ST_NONFINITE, O.ST_BAD_ID, O.ST_BAD_ID, O.ST_NOT_COMPUTED, O.ST_NONFINITE,
                                   O.ST_MASKED]
    assert np.all(res["grad"] == 0) and np.all(res["loss"] == 0)


# ---------------------------------------------------------------- placement controls
def test_select_tm_counts_and_validity():
    rng = np.random.default_rng(50)
    lens = [7, 1, 0, 30, 12]
    seq = np.concatenate([[0], np.cumsum(lens)])
    N = int(seq[-1])
    C = (rng.random(N) < 0.4).astype(np.uint8)
    tv = rng.random(N) * (rng.random(N) < 0.7)
    mask = (rng.random(N) < 0.8).astype(np.uint8)
    st = np.where(rng.random(N) < 0.1, O.ST_NOT_COMPUTED, 0).astype(np.uint32)
    valid = (mask != 0) & (st == 0)
    for mode in (O.SELECT_RANDOM, O.SELECT_TV_WEIGHTED):
        sel, m, _ = O.select_tm(seq, C, tv, mode, seed=3, mask=mask, rollout_status=st)
        assert np.all(sel[~valid] == 0)
        for b in range(len(lens)):
            lo, hi = seq[b], seq[b + 1]
            assert m[b] == int((C[lo:hi] != 0)[valid[lo:hi]].sum()) == int(sel[lo:hi].sum())


def test_select_tm_laws():
    """Exponential race: with one pick the chance of position t is d_t / sum d; with two picks the
    successive-sampling law (closed forms).  Random-TM: every subset of the right size equally likely."""
    d = np.array([0.5, 0.2, 0.3])
    seq = np.array([0, 3])
    trials = 6000
    first = np.zeros(3)
    pairs = {}
    uni = np.zeros(3)
    for sd in range(trials):
        sel, _, _ = O.select_tm(seq, np.array([1, 0, 0]), d, O.SELECT_TV_WEIGHTED, seed=sd)
        first += sel
        sel2, _, _ = O.select_tm(seq, np.array([1, 1, 0]), d, O.SELECT_TV_WEIGHTED, seed=sd)
        pairs[tuple(sel2)] = pairs.get(tuple(sel2), 0) + 1
        selr, _, _ = O.select_tm(seq, np.array([0, 1, 0]), d, O.SELECT_RANDOM, seed=sd)
        uni += selr
    assert np.all(np.abs(first / trials - d / d.sum()) < 0.025)
    assert np.all(np.abs(uni / trials - 1 / 3) < 0.025)
    D = d.sum()
    for (i, j), key in (((0, 1), (1, 1, 0)), ((0, 2), (1, 0, 1)), ((1, 2), (0, 1, 1))):
        want = d[i] / D * d[j] / (D - d[i]) + d[j] / D * d[i] / (D - d[j])
        assert abs(pairs.get(key, 0) / trials - want) < 0.025


def test_select_tm_uniform_fill_when_too_few_positive():
    tv = np.array([0.0, 0.3, 0.0, 0.0, 0.1, 0.0])
    C = np.array([1, 1, 1, 0, 1, 0])              # m = 4 > 2 positions with positive TV
    hits = np.zeros(6)
    for sd in range(3000):
        sel, m, _ = O.select_tm(np.array([0, 6]), C, tv, O.SELECT_TV_WEIGHTED, seed=sd)
        assert m[0] == 4 and sel[1] == 1 and sel[4] == 1 and sel.sum() == 4
        hits += sel
    zeros = [0, 2, 3, 5]                            # two of the four zero-TV positions, uniformly
    assert np.all(np.abs(hits[zeros] / 3000 - 0.5) < 0.03)


# ---- the lm-head step (logits as stored, row maximum, log-sum-exp)
def _bf16_values(shape, seed, scale=1.0):
    g = torch.Generator().manual_seed(seed)
    return (scale * torch.randn(shape, generator=g)).to(torch.bfloat16).to(torch.float64).numpy()


def test_lmhead_against_library_routines():
    h, w = _bf16_values((7, 48), 1), _bf16_values((300, 48), 2, 0.3)
    for tau in (1.0, 0.7):
        logits, row_max, lse = O.lmhead_lse(h, w, tau)
        full = (torch.as_tensor(h) @ torch.as_tensor(w).T)                   # torch's float64 matmul
        stored = full.to(torch.bfloat16).to(torch.float64).numpy()           # torch's rounding to bf16
        assert np.array_equal(logits, stored)
        assert np.array_equal(row_max, stored.max(axis=1))
        assert np.allclose(lse, scipy.special.logsumexp(stored / tau, axis=1), rtol=0, atol=1e-12)


def test_lmhead_closed_forms():
    # a one-hot hidden state picks a column of W: the logits are that column, exactly
    w = _bf16_values((64, 16), 3)
    h = np.zeros((2, 16))
    h[0, 5] = 1.0
    h[1, 11] = -2.0
    logits, row_max, lse = O.lmhead_lse(h, w, 1.0)
    assert np.array_equal(logits[0], w[:, 5]) and np.array_equal(logits[1], -2.0 * w[:, 11])
    assert row_max[0] == w[:, 5].max()
    # equal weight rows: constant logits, lse = logit / tau + log V
    w2 = np.tile(_bf16_values((1, 16), 4), (40, 1))
    h2 = _bf16_values((3, 16), 5)
    logits2, _, lse2 = O.lmhead_lse(h2, w2, 2.0)
    assert np.all(logits2 == logits2[:, :1])
    assert np.allclose(lse2, logits2[:, 0] / 2.0 + math.log(40), rtol=0, atol=1e-12)
    # and the result is what route_row's own log-softmax starts from
    lp = O.log_softmax(logits[0] / 1.0)
    assert abs(-lp.max() - (lse[0] - row_max[0])) < 1e-12

"""A numpy stand-in for the GPU's vocabulary-slice kernels (saki_vshard_partial), for the multi-process tests
of the exchange that run without a GPU: given a slice of the logit rows and the per-row state, the 16 numbers
per row of each stage, as the header defines them.  The combine is NOT modelled here: the tests call the
library's own host combine (saki_vshard_combine_host)."""
import numpy as np

P, S = 16, 32
(MODE, STATUS, MS, MT, VSTAR, LSE_S, LSE_T, SX, TX, SV, BETA, LO, HI, ITER, LAM, LOGZ, KL, TV, ACC, CORR,
 OWNER, BEFORE, TARGET, TAKE_LAST, TOK, COEF, LOSS, Y, SY, TY) = range(30)
SOLVING, SETTLED, FLAGGED = 0, 1, 2


def partial(stage, s, t, v0, tau, proposal, state, rank, grad_scale=1.0, want_grad=False):
    """s, t: [N, V_local] float64 copies of the stored slice values.  Returns ([N, 16] partials, gradient
    slice or None)."""
    N, Vl = s.shape
    out = np.zeros((N, P))
    grad = np.zeros((N, Vl)) if (want_grad and stage == 3) else None
    for i in range(N):
        zs, zt = s[i] / tau, t[i] / tau
        dl = zt - zs
        st = None if state is None else state[i]
        if stage == 0:
            fin = bool(np.all(np.isfinite(s[i])) and np.all(np.isfinite(t[i])))
            ms = s[i].max() if Vl else -np.inf
            mt = t[i].max() if Vl else -np.inf
            am = v0 + int(np.argmax(t[i])) if Vl else 2147483647
            x = int(proposal[i]) - v0
            own = 0 <= x < Vl
            if fin and Vl:
                es, et = np.exp(zs - ms / tau), np.exp(zt - mt / tau)
                sums = [es.sum(), et.sum(), (et * dl).sum(), (es * dl).sum(), (es * dl * dl).sum()]
                high = [(es * dl ** 3).sum(), (es * dl ** 4).sum()]
            else:
                sums, high = [0.0] * 5, [0.0] * 2
            out[i, :12] = [ms, mt, am, 1.0 if fin else 0.0, *sums, s[i, x] if own else 0.0, t[i, x] if own else 0.0,
                           1.0 if own else 0.0]
            out[i, 12:14] = high
        elif stage == 1:
            if int(st[MODE]) == SOLVING:
                b = st[BETA]
                kb = ((1 - b) * st[MS] + b * st[MT]) / tau
                e = np.exp(zs + b * dl - kb)
                out[i, :5] = [(e * dl ** k).sum() for k in range(5)]
        elif stage == 2:
            live = int(st[MODE]) == SETTLED
            if live and st[LAM] > 0:
                lp, lT = zs - st[LSE_S], zt - st[LSE_T]
                lq = lp + st[LAM] * (lT - lp) - st[LOGZ]
                q = np.exp(lq)
                out[i, 0] = np.maximum(q - np.exp(lp), 0.0).sum()
                out[i, 1] = (q * (lq - lp)).sum()
            vs = int(st[VSTAR]) - v0
            if live and 0 <= vs < Vl:
                out[i, 2] = s[i, vs]
        else:
            mode = int(st[MODE])
            if grad is not None and mode != FLAGGED and st[COEF] != 0.0:
                p = np.exp(zs - st[LSE_S])
                tok = int(st[TOK]) - v0
                oh = np.zeros(Vl)
                if 0 <= tok < Vl:
                    oh[tok] = 1.0
                grad[i] = grad_scale * st[COEF] / tau * (p - oh)
            out[i, 0] = -1.0
            if mode == SETTLED and st[CORR] != 0.0 and int(st[OWNER]) == rank:
                lp, lT = zs - st[LSE_S], zt - st[LSE_T]
                r = np.maximum(np.exp(lp + st[LAM] * (lT - lp) - st[LOGZ]) - np.exp(lp), 0.0)
                run = st[BEFORE] + np.cumsum(r)
                pos = np.nonzero(r > 0)[0]
                hit = np.nonzero(run > st[TARGET])[0] if st[TAKE_LAST] == 0.0 else np.array([], dtype=int)
                y = int(hit[0]) if len(hit) else (int(pos[-1]) if len(pos) else max(Vl - 1, 0))
                if 0 <= y < Vl:
                    out[i, :3] = [v0 + y, s[i, y], t[i, y]]
    return out, grad

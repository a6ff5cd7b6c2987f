"""The lm-head GEMM with the routing path's first row statistics in its epilogue (saki_lmhead_lse), against the
float64 oracle: the stored bf16 logits (fp32 accumulation on the tensor cores may round a value that sits on a
rounding boundary the other way: such entries are counted and must be one bf16 step off at most), each row's
maximum, and the log-sum-exp of the stored values."""
import numpy as np
import pytest
import torch

import oracle as O
import paper_2609_36601_b200 as P
from parity import bf16_ulp

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _inputs(N, d, V, seed, w_scale=None):
    g = torch.Generator(device=DEV).manual_seed(seed)
    h = torch.randn((N, d), generator=g, device=DEV).to(torch.bfloat16)
    w = (torch.randn((V, d), generator=g, device=DEV) * (w_scale or 2.0 / d ** 0.5)).to(torch.bfloat16)
    return h, w


@pytest.mark.parametrize("N,d,V,tau", [(200, 64, 4128, 1.0), (131, 96, 1000, 0.7), (257, 256, 8192, 1.0), (128, 8, 256, 1.0),
                                        (600, 520, 33024, 1.3)])
def test_logits_and_row_statistics_match_the_oracle(N, d, V, tau):
    h, w = _inputs(N, d, V, 7 * N + d)
    logits, row_max, lse = P.lmhead_lse(h, w, tau)
    torch.cuda.synchronize()
    ref_logits, ref_max, ref_lse = O.lmhead_lse(h.cpu().to(torch.float64).numpy(), w.cpu().to(torch.float64).numpy(), tau)
    got = logits.cpu().to(torch.float64).numpy()
    diff = np.abs(got - ref_logits)
    off = diff > 0
    # fp32 accumulation: absolute error up to ~d 2^-24 of the sum of the products' magnitudes, which near a zero of
    # the logit is more than a bf16 step of the tiny value; allowed on top of one step
    h64, w64 = h.cpu().to(torch.float64).numpy(), w.cpu().to(torch.float64).numpy()
    acc_err = 2.0 ** -20 * (np.abs(h64) @ np.abs(w64).T)
    assert np.all(diff <= bf16_ulp(ref_logits) * 1.0000001 + acc_err), "a stored logit is more than one bf16 step from the oracle's"
    assert off.mean() <= 0.02, f"{off.mean():.4f} of the logits rounded the other way"
    # the statistics are those of the values the kernel stored
    z = got / tau
    own_lse = z.max(axis=1) + np.log(np.exp(z - z.max(axis=1, keepdims=True)).sum(axis=1))
    assert np.array_equal(row_max.cpu().numpy().astype(np.float64), got.max(axis=1))
    assert np.max(np.abs(lse.cpu().numpy() - own_lse)) <= 2e-6 * (1 + np.max(np.abs(own_lse)))
    # and agree with the oracle's up to the few logits that rounded differently
    assert np.max(np.abs(lse.cpu().numpy() - ref_lse)) <= 1e-4 * (1 + np.max(np.abs(ref_lse)))
    assert np.max(np.abs(row_max.cpu().numpy() - ref_max) / bf16_ulp(ref_max)) <= 1.0000001
    print(f"\n[parity] lm-head N={N} d={d} V={V}: {int(off.sum())} of {off.size} logits rounded the other way, "
          f"max |lse - oracle| {np.max(np.abs(lse.cpu().numpy() - ref_lse)):.2e}")


def test_row_statistics_feed_the_routing_path():
    """The epilogue's log-sum-exp is the normaliser the routing call derives from the same stored logits:
    log p(x) from route_fwd equals logits[x] / tau - lse."""
    N, d, V = 64, 128, 32000
    h, w = _inputs(N, d, V, 5, w_scale=0.35)
    ht, wt = _inputs(N, d, V, 6, w_scale=0.35)
    s, _, lse_s = P.lmhead_lse(h, w)
    t, _, lse_t = P.lmhead_lse(ht * 0.2 + h, wt * 0.2 + w)
    x = torch.argmax(s.float(), dim=1).to(torch.int32)
    out = P.route_fwd(s, t, x, 0.1)
    torch.cuda.synchronize()
    lp = s.float().gather(1, x.long()[:, None])[:, 0] - lse_s
    lT = t.float().gather(1, x.long()[:, None])[:, 0] - lse_t
    assert float((out["logp_x"] - lp).abs().max()) <= 1e-5 * (1 + float(lp.abs().max()))
    assert float((out["logT_x"] - lT).abs().max()) <= 1e-5 * (1 + float(lT.abs().max()))

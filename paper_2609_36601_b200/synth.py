"""Seeded synthetic logits shaped like the paper's workloads.

This module only *makes inputs*: Gaussian logits with a Zipf rank bias, a
teacher correlated with the student, and student proposal tokens drawn with
torch's own generator.  It holds none of the routing arithmetic, and it is the
one module both the CUDA path's callers and the float64 test oracle's callers
use, so that both sides always see the identical bytes.

Recipe (per workload; V = vocabulary, N = positions):
  student  s = g_s + b_S,   g_s ~ N(0, 2^2) iid,
           b_S(v) = -1.1 ln(1 + rank_S(v)),  rank_S a random permutation
  teacher  t = 0.8 g_s + sigma n + b_T,  n ~ N(0,1) iid,
           b_T built like b_S from rank_T, the ordering of
           ln(1 + rank_S) + N(0, 0.5^2)  (a noisy copy of the student's
           ranking, so that small-sigma rows can sit inside the trust region)
  "independent" regime: t = N(0, 2^2) + b_T with no shared Gaussian part.
  The tiny fp32 workload has no Zipf term: s ~ N(0,2^2), t = s + N(0,1.5^2).
  proposal x ~ softmax(s / temperature), drawn by Gumbel-max with torch.rand.
Rows are generated in fixed chunks of CHUNK rows, each from its own seed, so a
prefix or a subset of chunks reproduces the same bytes as the full workload
on the same device type.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
import math
import torch

CHUNK = 256


@dataclass(frozen=True)
class Workload:
    name: str
    N: int
    V: int
    dtype: str            # "f32" | "bf16"
    eps: float
    sigma: float          # teacher noise; < 0 means the independent regime
    zipf: bool
    gen_seed: int         # seed of the logits generator
    seed: int             # routing seed handed to the library
    temperature: float = 1.0
    K: int = 0            # > 0: block verification, N = B * (K + 1)
    student_scale: float = 0.8

    @property
    def torch_dtype(self):
        return torch.float32 if self.dtype == "f32" else torch.bfloat16

    @property
    def B(self):
        return self.N // (self.K + 1) if self.K else self.N


WORKLOADS = {
    "cfg1": Workload("cfg1", 64, 1024, "f32", 0.1, 1.5, False, 1001, 0, student_scale=1.0),
    "cfg2": Workload("cfg2", 4096, 32000, "bf16", 0.05, 1.0, True, 1002, 2),
    "cfg3": Workload("cfg3", 16384, 151936, "bf16", 0.1, 1.5, True, 1003, 3),
    "cfg5": Workload("cfg5", 512 * 7, 151936, "bf16", 0.1, 1.5, True, 1005, 5, K=6),
}
# the throughput sweep: 3 disagreement regimes x 3 radii; one input set per
# regime is reused across the radii
_REGIMES = (("s05", 0.5, 1004), ("s20", 2.0, 1014), ("ind", -1.0, 1024))
for _rn, _sg, _gs in _REGIMES:
    for _e in (0.01, 0.1, 1.0):
        _nm = f"cfg4_{_rn}_e{_e:g}"
        WORKLOADS[_nm] = Workload(_nm, 65536, 151936, "bf16", _e, _sg, True, _gs, 4)


def shrink(w: Workload, N: int) -> Workload:
    """The same workload cut to its first N rows (a multiple of K+1 for block
    verification)."""
    return replace(w, N=N)


def _zipf_bias(V: int, gen: torch.Generator, device):
    rank_s = torch.randperm(V, generator=gen, device=device)
    lr = torch.log1p(rank_s.to(torch.float32))
    noisy = lr + 0.5 * torch.randn(V, generator=gen, device=device)
    order = torch.argsort(noisy)
    rank_t = torch.empty_like(order)
    rank_t[order] = torch.arange(V, device=device)
    b_s = -1.1 * lr
    b_t = -1.1 * torch.log1p(rank_t.to(torch.float32))
    return b_s, b_t


def generate(w: Workload, device="cpu", rows: int | None = None):
    """Returns dict(s, t, proposal, mask=None) for the first `rows` rows
    (default all) of workload `w` on `device`.  s, t: [rows, V] in w's dtype;
    proposal: [rows] int32 (for block verification the proposal of the bonus
    row of each sequence is present but unused)."""
    n = w.N if rows is None else rows
    dev = torch.device(device)
    s = torch.empty((n, w.V), dtype=w.torch_dtype, device=dev)
    t = torch.empty((n, w.V), dtype=w.torch_dtype, device=dev)
    x = torch.empty((n,), dtype=torch.int32, device=dev)
    g0 = torch.Generator(device=dev)
    g0.manual_seed(w.gen_seed)
    if w.zipf:
        b_s, b_t = _zipf_bias(w.V, g0, dev)
    gen = torch.Generator(device=dev)
    for c0 in range(0, n, CHUNK):
        c1 = min(n, c0 + CHUNK)
        gen.manual_seed(w.gen_seed * 1_000_003 + 17 * (c0 // CHUNK) + 1)
        m = CHUNK                      # always draw a full chunk: a cut chunk
        g_s = 2.0 * torch.randn((m, w.V), generator=gen, device=dev)
        noise = torch.randn((m, w.V), generator=gen, device=dev)
        if w.sigma < 0:
            t_c = 2.0 * noise
        else:
            t_c = w.student_scale * g_s + w.sigma * noise
        if w.zipf:
            g_s = g_s + b_s
            t_c = t_c + b_t
        s_c = g_s.to(w.torch_dtype)
        u = torch.rand((m, w.V), generator=gen, device=dev)
        u = u.clamp_(min=1e-12, max=1.0 - 1e-7)
        keys = s_c.to(torch.float32) / w.temperature - torch.log(-torch.log(u))
        k = c1 - c0
        s[c0:c1] = s_c[:k]
        t[c0:c1] = t_c[:k].to(w.torch_dtype)
        x[c0:c1] = torch.argmax(keys[:k], dim=1).to(torch.int32)
        del g_s, noise, t_c, s_c, u, keys
    return dict(s=s, t=t, proposal=x, mask=None)


def bytes_per_position(w: Workload, backward: bool = True) -> int:
    """Algorithmic minimum HBM traffic of one position: read both logit rows
    once, write the gradient row once."""
    e = 4 if w.dtype == "f32" else 2
    return w.V * e * (3 if backward else 2)

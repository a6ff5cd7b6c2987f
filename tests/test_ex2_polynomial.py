"""The exponential that one pair per chunk of the row kernel's last pass takes on the FMA pipe (ex2_fma2 in
csrc/saki_device.cuh): the same coefficients, read from the source, evaluated in numpy float32 the way the
kernel does (magic-number rounding, Horner, exponent by integer add) against exp2 over a dense grid of its
argument range.  It has to be as good as ex2.approx (2^-22 relative)."""
import os
import re

import numpy as np

SRC = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "paper_2609_36601_b200", "csrc", "saki_device.cuh")


def _coefficients():
    text = open(SRC).read()
    c = {int(k): np.float32(v) for k, v in re.findall(r"EX2_C(\d) = ([0-9.eE+-]+)f", text)}
    assert sorted(c) == [1, 2, 3, 4, 5]
    return [c[k] for k in range(1, 6)]


def _ex2_fma2(x, c):
    x = np.maximum(x.astype(np.float32), np.float32(-126.0))
    magic = np.float32(12582912.0)
    t = (x + magic).astype(np.float32)
    n = (t - magic).astype(np.float32)
    f = (x - n).astype(np.float32)
    assert np.all(np.abs(f) <= 0.5)
    p = np.full_like(f, c[4])
    for k in (3, 2, 1, 0):
        p = (p * f + c[k]).astype(np.float32)
    p = (p * f + np.float32(1.0)).astype(np.float32)
    bits = p.view(np.int32) + (t.view(np.int32) << 23)         # the low bits of t hold n (two's complement)
    return bits.view(np.float32)


def test_polynomial_matches_exp2_to_the_accuracy_of_ex2_approx():
    c = _coefficients()
    rng = np.random.default_rng(0)
    x = np.concatenate([np.linspace(-126.0, 0.0, 2_000_001), -rng.random(500_000) * 40.0, -np.arange(0, 127, 0.5)])
    got = _ex2_fma2(x, c).astype(np.float64)
    want = np.exp2(np.maximum(x.astype(np.float32), np.float32(-126.0)).astype(np.float64))
    rel = np.abs(got / want - 1.0)
    assert rel.max() <= 2.4e-7, rel.max()                       # 2^-22
    assert np.all(got[x == 0.0] == 1.0)
    # and below the clamp the result is the smallest normal number, not garbage
    assert np.all(_ex2_fma2(np.array([-200.0, -1e30]), c) == np.float32(2.0 ** -126))

"""Fits the polynomial the kernels' GELU uses and prints its coefficients and error.

gelu(v) = v Phi(v) = max(v, 0) - 0.5 a erfc(a / sqrt 2) with a = |v|; the kernels evaluate erfc(a / sqrt 2) as
2^Q(a), Q of degree 6 on [0, 5.9375] (clamped beyond).  Q is a weighted least-squares fit of log2 erfc, the weights
iterated towards the largest absolute error of the resulting GELU.  Run: python -m paper_2409_09708_b200.fit_gelu
"""
import math

import numpy as np
from numpy.polynomial import polynomial as P
from scipy.special import erf, erfc

A_MAX = 5.9375


def fit(deg=6, n=6000, rounds=200):
    xs = np.cos(np.pi * (np.arange(n) + 0.5) / n) * A_MAX / 2 + A_MAX / 2
    target = erfc(xs / math.sqrt(2))
    w = target * np.maximum(xs, 0.05)
    for _ in range(rounds):
        co = P.polyfit(xs, np.log2(target), deg, w=w)
        err = np.abs(np.exp2(P.polyval(xs, co)) - target) * 0.5 * xs
        w = w * (1 + 0.5 * err / err.max())
    return co.astype(np.float32)


def gelu_f32(v, co):
    a = np.minimum(np.abs(v), np.float32(A_MAX))
    q = np.zeros_like(a)
    for c in co[::-1]:
        q = (q * a + c).astype(np.float32)
    e = np.exp2(q.astype(np.float64)).astype(np.float32)
    return (np.maximum(v, np.float32(0)) - (np.float32(0.5) * np.abs(v) * e).astype(np.float32)).astype(np.float32)


if __name__ == "__main__":
    co = fit()
    v = np.linspace(-10, 10, 2000001).astype(np.float32)
    ref = 0.5 * v.astype(np.float64) * (1 + erf(v.astype(np.float64) / math.sqrt(2)))
    print("coefficients, constant term first:", ", ".join("%.9ef" % c for c in co))
    print("largest absolute error of gelu in fp32: %.3g" % np.abs(gelu_f32(v, co) - ref).max())

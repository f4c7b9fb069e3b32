"""Derives the coefficients of the erf polynomial in layer_gemm.cu (not part of the build; run by hand).

GELU(x) = x/2 + |x|/2 * erf(|x| / sqrt 2).  On u = min(|x|, 3.3 sqrt 2) the odd polynomial u * Q(u^2) with nine
coefficients replaces erf(u / sqrt 2); beyond the clamp erf is within 3.1e-6 of its value there.  The fit
minimises the largest error of GELU itself (the error of erf weighted by |x| / 2) with Lawson's reweighted least
squares on Chebyshev nodes, and the script then evaluates the polynomial in float32 the way the kernel does.
"""
import math

import numpy as np

C = 3.3 * math.sqrt(2.0)
N_COEF = 9


def fit(n_coef=N_COEF, iters=60):
    erf = np.vectorize(math.erf)
    v = (np.cos(np.pi * (np.arange(6000) + 0.5) / 6000) + 1) / 2
    x = v * C
    y = erf(x / math.sqrt(2))
    w = np.ones_like(v)
    A = np.stack([v * (v * v) ** k for k in range(n_coef)], 1)
    for _ in range(iters):
        wt = w * np.maximum(x, 0.05)
        coef, *_ = np.linalg.lstsq(A * wt[:, None], y * wt, rcond=None)
        e = np.abs(A @ coef - y) * np.maximum(x, 0.05)
        w = w * (0.5 + e / e.max())
        w /= w.mean()
    return np.array([c / C ** (2 * k + 1) for k, c in enumerate(coef)])     # in powers of u, not of u / C


def max_error(coef):
    erf = np.vectorize(math.erf)
    k32 = coef.astype(np.float32)
    xs = np.linspace(-12, 12, 600001).astype(np.float32)
    a = np.abs(xs)
    u = np.minimum(a, np.float32(C))
    s = (u * u).astype(np.float32)
    q = np.full_like(xs, k32[-1])
    for k in range(len(k32) - 2, -1, -1):
        q = (q * s + k32[k]).astype(np.float32)
    p = (q * u).astype(np.float32)
    g = (np.float32(0.5) * xs + (np.float32(0.5) * a) * p).astype(np.float32)
    exact = 0.5 * xs.astype(np.float64) * (1 + erf(xs.astype(np.float64) / math.sqrt(2)))
    return float(np.abs(g - exact).max())


if __name__ == "__main__":
    k = fit()
    print("clamp", repr(np.float32(C)))
    print("coefficients (u^1, u^3, ...):")
    print(", ".join("%.9ef" % t for t in k.astype(np.float32)))
    print("largest |GELU error| in float32 on [-12, 12]: %.3g" % max_error(k))

"""Fits the polynomial used by the GEMM's GELU epilogue (rs_gemm_tc.cu, gelu_erf).

GELU(v) = v * Phi(v) with Phi the standard normal CDF (the exact-erf form).  For t >= 0 let
q(t) = -log2(Phi(-t)); then Phi(v) = 2^-q(|v|) for v < 0 and 1 - 2^-q(|v|) for v >= 0, which
costs one ex2 and a short Horner chain.  A degree-5 polynomial is fitted to q on [0, 7] by
iteratively re-weighted least squares (Lawson) under the weight t * Phi(-t), i.e. the size of
the resulting GELU error, and checked in emulated fp32 arithmetic.

    python fit_gelu.py        # prints the coefficients (lowest degree first) and the max error
"""
import numpy as np
from scipy.special import erf, erfc


def q_true(t):
    return -np.log2(0.5 * erfc(t / np.sqrt(2.0)))


def fit(deg=5, T=7.0, iters=200):
    t = np.linspace(0.0, T, 20001)
    w = np.maximum(t, 0.05) * 0.5 * erfc(t / np.sqrt(2.0))
    lam = np.ones_like(t)
    V = np.vander(t, deg + 1, increasing=True)
    coef = None
    for _ in range(iters):
        ww = w * np.sqrt(lam)
        coef, *_ = np.linalg.lstsq(V * ww[:, None], q_true(t) * ww, rcond=None)
        r = np.abs((V @ coef - q_true(t)) * w)
        lam = lam * (r / r.max() + 1e-3)
        lam /= lam.mean()
    return coef


def max_error_fp32(coef, lo=-60.0, hi=60.0, n=2000001):
    c = coef.astype(np.float32)
    v = np.linspace(lo, hi, n).astype(np.float32)
    a = np.abs(v)
    q = np.full_like(a, c[-1])
    for ci in c[-2::-1]:
        q = (q * a + ci).astype(np.float32)
    e = np.exp2(-q.astype(np.float64)).astype(np.float32)
    phi = np.where(v >= 0, (np.float32(1) - e).astype(np.float32), e)
    g = (v * phi).astype(np.float64)
    ref = 0.5 * v.astype(np.float64) * (1.0 + erf(v.astype(np.float64) / np.sqrt(2.0)))
    return float(np.abs(g - ref).max())


if __name__ == "__main__":
    c = fit()
    print([float(np.float32(x)) for x in c])
    print("max abs GELU error in fp32: %.3e" % max_error_fp32(c))

"""Fits the polynomial behind the device GELU (less_internal.cuh, gelu_erf) and prints its
coefficients together with the error of the fp32 evaluation.

    gelu(x) = x * Phi(x),   Phi(-u) = E(u) / 2,   Phi(u) = 1 - E(u) / 2   (u = |x|)
            = max(x, 0) - u * E(u) / 2        (both signs in one expression, no select)
    E(u) = erfc(u / sqrt(2)) = 2^(-u * g(u))

g is smooth on [0, 8] (g(0) = sqrt(2 / pi) / ln 2), so a degree-5 polynomial in u reproduces it
well enough that the fp32 result is limited by rounding, not by the fit; both tails come out of
the exponential directly, without the cancellation of 1 - erf.  Run:  python gelu_fit.py
"""
import numpy as np
from numpy.polynomial import chebyshev as C
from scipy.special import erfc

U = 8.0      # u is clamped here: E(8) = 1.2e-15, below fp32 resolution of every use
DEG = 5


def fit():
    n = 4000
    x = np.cos(np.pi * (np.arange(n) + 0.5) / n)          # Chebyshev nodes on [-1, 1]
    u = (x + 1) * U / 2
    E = erfc(u / np.sqrt(2))
    g = -np.log2(E) / u
    w = np.maximum(u * u * E, 1e-6 * np.max(u * u * E))     # weight ~ absolute error of gelu
    cheb = C.chebfit(x, g, DEG, w=w)
    px = np.polynomial.Polynomial(C.cheb2poly(cheb))
    return px(np.polynomial.Polynomial([-1, 2 / U])).coef.astype(np.float32)


def gelu_f32(xs, co):
    u = np.minimum(np.abs(xs), np.float32(U))
    q = np.zeros_like(u) + co[-1]
    for a in co[-2::-1]:
        q = (q * u + a).astype(np.float32)
    E = np.exp2((-q * u).astype(np.float32)).astype(np.float32)
    t = (u * E).astype(np.float32)
    # fma(-0.5, t, max(x, 0)): one rounding
    return (np.maximum(xs, np.float32(0)).astype(np.float64) - 0.5 * t.astype(np.float64)).astype(np.float32)


if __name__ == "__main__":
    co = fit()
    xs = np.linspace(-12, 12, 2000001).astype(np.float32)
    ref = 0.5 * xs.astype(np.float64) * erfc(-xs.astype(np.float64) / np.sqrt(2))
    err = np.abs(gelu_f32(xs, co) - ref)
    print("coefficients (u^0 .. u^%d):" % DEG)
    print(", ".join("%.9ef" % c for c in co))
    print("max |gelu_f32 - gelu| on [-12, 12]: %.3e at x = %.3f (one fp32 ulp there: %.3e)"
          % (err.max(), xs[err.argmax()], np.spacing(np.float32(abs(ref[err.argmax()])))))
    print("max on [-3, 3]: %.3e" % err[np.abs(xs) <= 3].max())

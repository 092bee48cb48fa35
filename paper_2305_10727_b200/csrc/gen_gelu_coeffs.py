"""Provenance of the constants of the GEMM epilogue's exact-erf GELU (not a build input:
the build never runs this file; it documents how the table in gemm_i8.cu was made and
needs scipy).

GELU(y) = max(y, 0) - g(|y|),  g(t) = t * Phi(-t) = t * 2^p(t),  p(t) = log2(Phi(-t)),
Phi the standard normal CDF.  p is smooth (close to a parabola), so a degree-6
polynomial on [0, 6] reaches |error| < 1.1e-5 in p for t <= 4.3, i.e. a relative
error below 1e-5 in g -- far inside a binary16 ulp (2^-11 relative) -- and the
form keeps that relative accuracy in the negative tail where 1 + erf cancels.
Beyond t = 4.3 the result of GELU for negative arguments is subnormal in
binary16 (absolute spacing 2^-24), so the fit is weighted down there by
10^(-2 (t - 4.3)).  For t > 6, g < 2^-25 rounds to zero in binary16, so t is
clamped to 6.  Measured against a binary64 evaluation over [-12, 12] the whole
formula, in binary32 arithmetic, stays within 0.1 binary16 ulp of the exact value
(a degree-5 fit: 0.16 ulp, which moves one output in twenty to the neighbouring
binary16 value; not taken).

The kernel evaluates the polynomial in u = -t (so that the last step is one fused
multiply-add, max(y, 0) + u * 2^p), hence the odd coefficients are printed negated.

Weighted least-squares fit on Chebyshev nodes, converted to monomial coefficients.
Run: python gen_gelu_coeffs.py   (prints the constants pasted into gemm_i8.cu)
"""
import numpy as np
from numpy.polynomial import chebyshev as C
from numpy.polynomial import polynomial as P
from scipy.special import log_ndtr

DEG, T = 6, 6.0
T_SUBNORMAL, DECADES_PER_UNIT = 4.3, 2.0


def fit():
    n = 2000
    x = np.cos(np.pi * (np.arange(n) + 0.5) / n)
    t = (x + 1) * T / 2
    w = np.ones_like(t)
    w[t > T_SUBNORMAL] = 10.0 ** (-DECADES_PER_UNIT * (t[t > T_SUBNORMAL] - T_SUBNORMAL))
    c = C.chebfit(x, log_ndtr(-t) / np.log(2.0), DEG, w=w)
    px = C.cheb2poly(c)
    pt, basis, lin = np.zeros(1), np.array([1.0]), np.array([-1.0, 2.0 / T])
    for a in px:
        pt = P.polyadd(pt, a * basis)
        basis = P.polymul(basis, lin)
    return pt


if __name__ == "__main__":
    coef = fit()
    t = np.linspace(0, T, 200001)
    e = np.abs(P.polyval(t, coef) - log_ndtr(-t) / np.log(2.0))
    print("// degree %d on [0, %g], max |error| in log2(Phi(-t)): %.2e for t <= %.1f, %.2e beyond"
          % (DEG, T, e[t <= T_SUBNORMAL].max(), T_SUBNORMAL, e.max()))
    for k, a in enumerate(coef):
        a = a if k % 2 == 0 else -a          # polynomial in u = -t
        print("    {%.9ef, %.9ef}," % (np.float32(a), np.float32(a)))

"""Generates the polynomial used by the GEMM epilogue's exact-erf GELU.

GELU(y) = max(y, 0) - g(|y|),  g(t) = t * Phi(-t) = t * 2^p(t),  p(t) = log2(Phi(-t)),
Phi the standard normal CDF.  p is smooth (close to a parabola), so a degree-7
polynomial on [0, 6] reaches |error| < 1e-5 in p, i.e. a relative error below
1e-5 in g -- far inside half a binary16 ulp -- and the form keeps that relative
accuracy in the negative tail where 1 + erf cancels.  For t > 6, g < 2^-25
rounds to zero in binary16, so t is clamped to 6.

Least-squares fit on Chebyshev nodes, converted to monomial coefficients.
Run: python gen_gelu_coeffs.py   (prints the constants pasted into gemm_i8.cu)
"""
import numpy as np
from numpy.polynomial import chebyshev as C
from numpy.polynomial import polynomial as P
from scipy.special import log_ndtr

DEG, T = 7, 6.0


def fit():
    n = 600
    x = np.cos(np.pi * (np.arange(n) + 0.5) / n)
    t = (x + 1) * T / 2
    c = C.chebfit(x, log_ndtr(-t) / np.log(2.0), DEG)
    px = C.cheb2poly(c)
    pt, basis, lin = np.zeros(1), np.array([1.0]), np.array([-1.0, 2.0 / T])
    for a in px:
        pt = P.polyadd(pt, a * basis)
        basis = P.polymul(basis, lin)
    return pt


if __name__ == "__main__":
    coef = fit()
    t = np.linspace(0, T, 200001)
    err = np.abs(P.polyval(t, coef) - log_ndtr(-t) / np.log(2.0)).max()
    print("// degree %d on [0, %g], max |error| in log2(Phi(-t)): %.2e" % (DEG, T, err))
    for k, a in enumerate(coef):
        print("constexpr float kGeluC%d = %.9ef;" % (k, np.float32(a)))

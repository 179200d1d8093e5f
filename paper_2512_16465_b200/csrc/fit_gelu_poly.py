"""Derives the polynomial behind the GPU's exact-erf GELU (``gelu_erf`` in dense_kernel.cuh).

GELU(t) = t * Phi(t) = 0.5 * t * (1 + erf(x)), x = t / sqrt(2).  For x < 0, 1 + erf(x) = erfc(|x|), and for
x >= 0 it is 2 - erfc(x), so one evaluation of g(|x|) = erfc(|x|) serves both signs without cancellation in the
negative tail.  log2(erfc(x)) is smooth on [0, X], so g = 2^p(z) with a single polynomial p in z = 2x/X - 1 and one
ex2 instruction: no branches, about half the instructions of a two-regime erff.  Beyond X = 4 (|t| > 5.66) the
kernel takes g = 0: erfc is 1.5e-8 and less there, i.e. |GELU error| < 5e-8, and the negative tail ends in -0 as the
function does (holding g at erfc(4) instead would leave a tail of t * 7.7e-9, visible against a 16-bit zero for
|t| in the thousands).

Run this file to reprint the coefficients (numpy / scipy, least squares on a dense grid in the Chebyshev basis,
then converted to the monomial basis the kernel evaluates with Horner's rule) and their fp32 error report.
"""
import numpy as np
from numpy.polynomial import chebyshev as C
from scipy.special import erf, erfc

X, DEG = 4.0, 9


def fit():
    xs = np.linspace(0.0, X, 400001)
    z = xs / X * 2.0 - 1.0
    cheb = C.Chebyshev.fit(z, np.log2(erfc(xs)), DEG, domain=[-1, 1])
    return cheb.convert(kind=np.polynomial.Polynomial).coef


def report(coef):
    xs = np.linspace(0.0, X, 400001)
    zf = (xs / X * 2.0 - 1.0).astype(np.float32)
    acc = np.full_like(zf, np.float32(coef[-1]))
    for a in coef[-2::-1]:
        acc = acc * zf + np.float32(a)
    g = np.exp2(acc.astype(np.float64))
    t = xs * np.sqrt(2.0)
    err = np.max(np.abs(0.5 * t * (2.0 - g) - 0.5 * t * (1.0 + erf(xs))))
    return float(np.max(np.abs(g / erfc(xs) - 1.0))), float(err)


if __name__ == "__main__":
    c = fit()
    print("coefficients of p(z), lowest order first:")
    for i, a in enumerate(c):
        print(f"  c{i} = {np.float32(a)!r}  ({a:.12e})")
    rel, ab = report(c)
    print(f"fp32 Horner: max relative error of erfc on [0,{X}] = {rel:.2e}; max |GELU error| = {ab:.2e}")

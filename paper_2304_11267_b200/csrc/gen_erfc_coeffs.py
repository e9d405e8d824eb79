"""Coefficients of the scaled complementary error function used by geglu_kernel.cuh.

For z >= 0 and t = 1 / (1 + z/2) in (0, 1]:   erfc(z) = t * exp(-z^2) * exp(f(t)),   f(t) = log(erfcx(z) / t),
with erfcx(z) = exp(z^2) erfc(z).  f is smooth on (0, 1] (it tends to log(2 / sqrt(pi)) as t -> 0), so a polynomial in
t fits it to a relative error in erfc near binary32 rounding.  This script fits that polynomial (Chebyshev
interpolation on [T_MIN, 1], converted to the monomial basis in u = t, scaled by log2(e) so that the kernel can use
exp2) and prints the constants; it also checks the fit, evaluated in binary32 the way the kernel does, against
scipy's erfc.  Run:  python gen_erfc_coeffs.py
"""
import numpy as np
from numpy.polynomial import chebyshev as C, polynomial as P
from scipy.special import erfc, erfcx

DEGREE = 10
T_MIN = 1.0 / (1.0 + 0.5 * 10.0)      # z up to 10: erfc(10) = 2e-45, far below anything a product can keep


def f(t):
    z = 2.0 * (1.0 / t - 1.0)
    return np.log(erfcx(z) / t)


def main():
    k = np.arange(400)
    x = np.cos(np.pi * (k + 0.5) / 400)                      # Chebyshev nodes on [-1, 1]
    t = 0.5 * (x + 1.0) * (1.0 - T_MIN) + T_MIN
    cheb = C.chebfit(x, f(t), DEGREE)
    mono_x = C.cheb2poly(cheb)                               # polynomial in x
    # x = (2 t - 1 - T_MIN) / (1 - T_MIN): substitute to get a polynomial in t
    a, b = 2.0 / (1.0 - T_MIN), -(1.0 + T_MIN) / (1.0 - T_MIN)
    mono_t = np.zeros(1)
    lin = np.array([b, a])
    for c in mono_x[::-1]:
        mono_t = P.polyadd(P.polymul(mono_t, lin), [c])
    coeffs = mono_t * np.log2(np.e)
    print("// f(t) * log2(e), lowest order first (degree %d)" % DEGREE)
    print(", ".join("%.9ef" % c for c in coeffs))
    # check in binary32, Horner as in the kernel
    z = np.concatenate([np.linspace(0.0, 10.0, 200001), np.random.default_rng(0).uniform(0, 10, 200000)]).astype(np.float32)
    tt = (np.float32(1.0) / (np.float32(1.0) + np.float32(0.5) * z)).astype(np.float32)
    acc = np.full_like(tt, np.float32(coeffs[-1]))
    for c in coeffs[-2::-1]:
        acc = (acc * tt + np.float32(c)).astype(np.float32)
    arg = (acc - (z * z).astype(np.float32) * np.float32(np.log2(np.e))).astype(np.float32)
    approx = tt.astype(np.float64) * np.exp2(arg.astype(np.float64))
    exact = erfc(z.astype(np.float64))
    keep = exact > 1e-37
    rel = np.abs(approx[keep] - exact[keep]) / exact[keep]
    print("// max relative error of erfc over z in [0, 10] (binary32 Horner, exact exp2): %.3e at z = %.4f" % (
        rel.max(), z[keep][rel.argmax()]))
    zz = z[keep].astype(np.float64)
    print("// ... over z in [0, 2]: %.3e;  largest error / (2.5e-7 + 1.3e-7 * 2 z^2): %.3f" % (
        rel[zz <= 2.0].max(), (rel / (2.5e-7 + 1.3e-7 * 2.0 * zz * zz)).max()))


if __name__ == "__main__":
    main()

"""Regenerates the coefficients of the normal-tail approximation used by common.cuh.

    q(a) = Phi(-a) ~ 2^(R(t)),  t = a / 7.5,  R a degree-6 polynomial,  0 <= t <= 1

R is fitted to log2 Phi(-a) by iteratively re-weighted least squares so that the absolute error
of a * q(a) (the part of gelu(z) = max(z, 0) - |z| q(|z|) that is approximated) is levelled.
Prints the float32 coefficients and the errors of a float32 Horner evaluation.
"""
import numpy as np
from scipy import special


def fit(deg=6, hi=7.5, n=40001):
    t = np.linspace(0, 1, n)
    a = hi * t
    q = 0.5 * special.erfc(a / np.sqrt(2))
    R = np.log2(q)
    wt = a * q + 1e-3 * q + 1e-9
    for _ in range(30):
        c = np.polynomial.polynomial.polyfit(t, R, deg, w=wt)
        err = (np.exp2(np.polynomial.polynomial.polyval(t, c)) - q) * np.maximum(a, 0.5)
        wt = wt * (1 + 2 * np.abs(err) / np.abs(err).max())
    return c.astype(np.float32)


def report(c, hi=7.5):
    t = np.linspace(0, 1, 400001).astype(np.float32)
    p = np.float32(c[-1])
    for k in c[-2::-1]:
        p = (p * t + np.float32(k)).astype(np.float32)
    qf = np.exp2(p).astype(np.float64)
    a64 = hi * t.astype(np.float64)
    q = 0.5 * special.erfc(a64 / np.sqrt(2))
    print("max |q err|      ", np.abs(qf - q).max())
    print("max |a q err|    ", np.abs(a64 * (qf - q)).max())


if __name__ == "__main__":
    c = fit()
    print(", ".join(f"{float(x):.9e}f" for x in c))
    report(c)

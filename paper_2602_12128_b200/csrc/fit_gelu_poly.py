"""Fits the odd polynomial erf(u) ~ u * P(u^2) on [0, c] that the tensor-core phi kernels use for
the exact (erf) GELU, GELU(x) = x/2 + (x/2) erf(x / sqrt 2), with u clamped to [-c, c].

Run:  python fit_gelu_poly.py   -> prints the coefficients (lowest order first) and the maximum
absolute error of erf and of GELU in fp32 Horner evaluation.  The constants in hla_tc_phi.cuh
are this script's output for c = 3.0, 9 coefficients."""
import numpy as np
from scipy.special import erf

C, NCOEF = 3.0, 9


def fit(c=C, n=NCOEF, iters=200):
    u = 0.5 * c * (1 - np.cos(np.linspace(0, np.pi, 6001)))[1:]
    A = np.stack([u ** (2 * k + 1) for k in range(n)], 1)
    y = erf(u)
    w = np.ones_like(u)
    for _ in range(iters):                      # reweighted least squares towards the minimax fit
        coef, *_ = np.linalg.lstsq(A * w[:, None], y * w, rcond=None)
        err = np.abs(A @ coef - y)
        w *= 1 + 2 * err / err.max()
        w /= w.mean()
    return coef


def gelu_poly_f32(x, coef, c=C):
    x = x.astype(np.float32)
    u = np.clip(x * np.float32(0.70710678), np.float32(-c), np.float32(c))
    t = u * u
    p = np.float32(coef[-1])
    for a in coef[-2::-1]:
        p = p * t + np.float32(a)
    hx = np.float32(0.5) * x
    return hx * (u * p) + hx


if __name__ == "__main__":
    coef = fit()
    print("coefficients:", ", ".join("%.9ef" % a for a in coef))
    uu = np.linspace(-6, 6, 1200001)
    ref = 0.5 * uu * (1 + erf(uu / np.sqrt(2)))
    got = gelu_poly_f32(uu, coef).astype(np.float64)
    print("max |gelu_poly - gelu| on [-6,6]: %.3e" % np.abs(got - ref).max())
    u = np.linspace(0, C, 300001)
    print("max |erf_poly - erf| on [0,c]: %.3e ; 1 - erf(c) = %.3e" % (np.abs(sum(a * u ** (2 * k + 1) for k, a in enumerate(coef)) - erf(u)).max(), 1 - erf(C)))

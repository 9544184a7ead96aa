"""Fits the constants the tensor-core phi kernels use for the exact (erf) GELU and its derivative.

Forward:  Phi(x) ~ 1/2 + tanh(x (a + b x^2)) / 2  (one tanh.approx on the special-function unit per element),
GELU(x) = x Phi(x); fit_tanh() gives a, b (fitted against erf(x / sqrt 2) on |x| <= 6) and the error before the
hardware approximation's own 2^-11 relative error.

Backward: GELU'(x) = Phi(x) + x pdf(x) through the same kind of tanh:
    th = tanh(x (a + b x^2)),  r = 1/2 + th / 2,  y = 1/2 - th / 2,   GELU'(x) ~ r (1 + x (C0 + C1 x^2) y)
(r y = (1 - th^2) / 4: the derivative of the tanh form with its inner derivative a free polynomial); fit_tanh_grad()
fits a, b, C0, C1 against the exact GELU' on |x| <= 8.

Weight gradients need GELU and GELU' of the same element; fit_tanh_grad_shared() keeps the forward's a, b (so that one
tanh serves both) and fits only C0, C1 of the derivative form (max error 5.2e-4 instead of 1.5e-4).

Run:  python fit_gelu_tanh.py   -> prints both sets of constants and their maximum absolute errors; the constants in
hla_tc_phi.cuh are this script's output."""
import numpy as np
from scipy.special import erf


def fit_tanh(iters=60):
    from scipy.optimize import least_squares
    x = np.linspace(0, 6, 6001)[1:]
    ref = erf(x / np.sqrt(2))
    res = lambda c: np.tanh(x * (c[0] + c[1] * x * x)) - ref
    c, w = np.array([0.7978845608, 0.0356774]), np.ones_like(x)
    for _ in range(iters):                      # reweighted least squares towards the minimax fit
        c = least_squares(lambda c: res(c) * w, c).x
        e = np.abs(res(c))
        w *= 1 + 2 * e / e.max()
        w /= w.mean()
    return c, np.abs(res(c)).max() / 2


def gelu_grad_tanh(x, c):
    t = x * x
    th = np.tanh(x * (c[0] + c[1] * t))
    r, y = 0.5 + 0.5 * th, 0.5 - 0.5 * th
    return r * (1 + x * (c[2] + c[3] * t) * y)


def gelu_grad_exact(x):
    return 0.5 * (1 + erf(x / np.sqrt(2))) + x * np.exp(-x * x / 2) / np.sqrt(2 * np.pi)


def fit_tanh_grad():
    from scipy.optimize import least_squares
    x = np.linspace(-8, 8, 32001)
    ref = gelu_grad_exact(x)
    c = least_squares(lambda c: gelu_grad_tanh(x, c) - ref, np.array([0.7988, 0.0353, 1.5976, 0.2117])).x
    return c, np.abs(gelu_grad_tanh(x, c) - ref).max()


def fit_tanh_grad_shared(a, b):
    from scipy.optimize import least_squares
    x = np.linspace(-8, 8, 32001)
    ref = gelu_grad_exact(x)
    c = least_squares(lambda c: gelu_grad_tanh(x, (a, b, c[0], c[1])) - ref, np.array([1.6, 0.2])).x
    return c, np.abs(gelu_grad_tanh(x, (a, b, c[0], c[1])) - ref).max()


if __name__ == "__main__":
    c, err = fit_tanh_grad()
    print("tanh form of GELU': a = %.8ff, b = %.8ff, C0 = %.8ff, C1 = %.8ff, max |error| = %.3e" % (*c, err))
    (a, b), err = fit_tanh()
    print("tanh form: a = %.8ff, b = %.8ff, max |Phi error| = %.3e" % (a, b, err))
    c, err = fit_tanh_grad_shared(a, b)
    print("GELU' on the forward's tanh: C0 = %.8ff, C1 = %.8ff, max |error| = %.3e" % (*c, err))

"""Numeric model of the magnitude-weighted quantization error (Sec. 3.3).  Test infrastructure.

The deployed clip rule (Eq. 14) is a recurrence whose derivation the paper leaves to an appendix;
what the text does define is the error functional and, for the Inverted-T density, the derivative
whose root is the optimal clip.  These utilities evaluate both the definition and the closed form so
that one can be checked against the other:

  * ``error_sample``        Eq. 8 on an empirical sample with a real nearest-rounding quantizer;
  * ``error_simplified``    Eq. 9 (I1 + I2) by numerical quadrature for any symmetric density;
  * ``inverted_t_density``  Eq. 13;
  * ``dE_ds_inverted_t``    the derivative printed between Eq. 13 and Eq. 14;
  * ``root_inverted_t``     its root (the condition of Eq. 10), ``root_inverted_t_alpha0`` the alpha->0 limit;
  * ``argmin_grid``         brute-force minimiser used as the independent check.
"""
from __future__ import annotations

import math

import numpy as np
from scipy import integrate


def error_sample(g: np.ndarray, s: float, alpha: float) -> float:
    """Eq. 8 with p(g) the empirical distribution of ``g``: mean of |g - g_hat| * exp(alpha*|g|),
    g_hat = round(127*clamp(g,s)/s) * s/127 with nearest rounding (Eq. 1), in binary64."""
    g = np.asarray(g, dtype=np.float64)
    clamped = np.clip(g, -s, s)
    g_hat = np.rint(127.0 * clamped / s) * (s / 127.0)
    return float(np.mean(np.abs(g - g_hat) * np.exp(alpha * np.abs(g))))


def inverted_t_density(a: float, b: float, eps: float, gmax: float):
    """Eq. 13: piecewise-uniform density, a on (0, eps), b on (eps, gmax) (one side; symmetric)."""
    def p(g):
        g = abs(g)
        if g < eps:
            return a
        if g <= gmax:
            return b
        return 0.0
    return p


def error_simplified(p, s: float, gmax: float, alpha: float, breakpoints=()) -> float:
    """Eq. 9: E = int_0^s (s/127) f p dg + 2 int_s^gmax (g - s) f p dg, f(g) = exp(alpha*|g|),
    by adaptive quadrature (independent of any closed form)."""
    f = lambda g: math.exp(alpha * abs(g))
    pts1 = [x for x in breakpoints if 0.0 < x < s]
    pts2 = [x for x in breakpoints if s < x < gmax]
    i1, _ = integrate.quad(lambda g: (s / 127.0) * f(g) * p(g), 0.0, s, points=pts1 or None,
                           epsabs=1e-14, epsrel=1e-12, limit=200)
    i2 = 0.0
    if s < gmax:
        i2, _ = integrate.quad(lambda g: (g - s) * f(g) * p(g), s, gmax, points=pts2 or None,
                               epsabs=1e-14, epsrel=1e-12, limit=200)
    return i1 + 2.0 * i2


def dE_ds_inverted_t(s: float, a: float, b: float, eps: float, gmax: float, alpha: float) -> float:
    """The closed form printed after Eq. 13 (valid for eps < s <= gmax, alpha > 0):
    [(a-b) e^{alpha eps} + b (255 + alpha s) e^{alpha s} - 254 b e^{alpha gmax} - a] / (127 alpha)."""
    return ((a - b) * math.exp(alpha * eps) + b * (255.0 + alpha * s) * math.exp(alpha * s)
            - 254.0 * b * math.exp(alpha * gmax) - a) / (127.0 * alpha)


def root_inverted_t(a: float, b: float, eps: float, gmax: float, alpha: float) -> float:
    """Root of ``dE_ds_inverted_t`` in s.  With u = 255 + alpha*s the condition reads
    u * e^{u-255} = R,  R = 254 e^{alpha gmax} + (a - (a-b) e^{alpha eps}) / b,
    i.e. u + ln u = ln R + 255, solved by Newton iteration."""
    R = 254.0 * math.exp(alpha * gmax) + (a - (a - b) * math.exp(alpha * eps)) / b
    c = math.log(R) + 255.0
    u = 255.0
    for _ in range(100):
        step = (u + math.log(u) - c) / (1.0 + 1.0 / u)
        u -= step
        if abs(step) < 1e-15 * u:
            break
    return (u - 255.0) / alpha


def root_inverted_t_alpha0(a: float, b: float, eps: float, gmax: float) -> float:
    """alpha -> 0 limit of the root: s = (254 gmax - (a/b - 1) eps) / 256."""
    return (254.0 * gmax - (a / b - 1.0) * eps) / 256.0


def argmin_grid(fn, lo: float, hi: float, n: int = 2001):
    """Brute-force minimiser of fn over n equally spaced points of [lo, hi]."""
    xs = np.linspace(lo, hi, n)
    vals = np.array([fn(float(x)) for x in xs])
    i = int(np.argmin(vals))
    return float(xs[i]), float(vals[i])

"""Scalar gain codebook matched to a chi distribution (TEST INFRASTRUCTURE, part of the CPU oracle).

The shape-gain construction of the paper (appendix "spherical shaping or
shape-gain") takes the gain code to be a scalar quantizer matched to the
chi distribution with 24 degrees of freedom - the law of the norm of a block of
24 unit-variance Gaussian weights.  The paper does not say how the quantizer is
designed; the reading here is the minimum mean-square-error (Lloyd-Max) design:
iterate "thresholds = midpoints of neighbouring levels, levels = centroids of
their cells" to a fixed point.  The cell probabilities and first moments of a
chi law have closed forms in the regularized lower incomplete gamma function P:

    Pr[a < r < b]   = P(n/2, b^2/2) - P(n/2, a^2/2)
    E[r; a < r < b] = sqrt(2) Gamma((n+1)/2) / Gamma(n/2) * (P((n+1)/2, b^2/2) - P((n+1)/2, a^2/2))

The decoder never runs this: the codebook is an input of the dequantizer.
Pins (tests): a 0-bit codebook is the mean of the law, sqrt(2) Gamma(12.5) /
Gamma(12); every level is the centroid of its cell by numerical quadrature of
the density; the distortion falls with every added bit and follows the
high-resolution 2^(-2b) slope.
"""
from __future__ import annotations

import math

import numpy as np
from scipy.special import gammainc


def _mass(n: int, a: float, b: float) -> float:
    return float(gammainc(n / 2, b * b / 2) - gammainc(n / 2, a * a / 2))


def _first_moment(n: int, a: float, b: float) -> float:
    c = math.sqrt(2.0) * math.exp(math.lgamma((n + 1) / 2) - math.lgamma(n / 2))
    return c * float(gammainc((n + 1) / 2, b * b / 2) - gammainc((n + 1) / 2, a * a / 2))


def chi_codebook(bits: int, dof: int = 24, iters: int = 5000, tol: float = 1e-13) -> np.ndarray:
    """2**bits reconstruction levels (ascending, float64) of the Lloyd-Max quantizer of chi(dof)."""
    levels = 1 << bits
    mean = _first_moment(dof, 0.0, math.inf)
    sd = math.sqrt(max(dof - mean * mean, 1e-12))
    y = np.array([mean + sd * (2 * (i + 0.5) / levels - 1) * 1.5 for i in range(levels)], dtype=np.float64)
    for _ in range(iters):
        t = np.concatenate(([0.0], 0.5 * (y[1:] + y[:-1]), [math.inf]))
        new = np.array([_first_moment(dof, t[i], t[i + 1]) / _mass(dof, t[i], t[i + 1]) for i in range(levels)])
        done = np.max(np.abs(new - y)) < tol
        y = new
        if done:
            break
    return y


def chi_distortion(levels: np.ndarray, dof: int = 24) -> float:
    """E[(r - Q(r))^2] of the nearest-level quantizer with these levels, r ~ chi(dof)."""
    y = np.asarray(levels, dtype=np.float64)
    t = np.concatenate(([0.0], 0.5 * (y[1:] + y[:-1]), [math.inf]))
    # E r^2 = dof;  E[(r - y)^2; cell] = E[r^2; cell] - 2 y E[r; cell] + y^2 Pr[cell]
    total = float(dof)
    for i in range(len(y)):
        total += -2.0 * y[i] * _first_moment(dof, t[i], t[i + 1]) + y[i] * y[i] * _mass(dof, t[i], t[i + 1])
    return total

"""Radial weighting of the neighbour density (test infrastructure).

The interface section of the paper lists an optional radial `weighting` among
the constructor arguments and gives no formula.  Reading taken here (the
functional forms of the package whose constructor the paper reproduces): every
neighbour Gaussian of Eq. 1 is multiplied by w(d) of its distance d from the
centre, the centre's own Gaussian by a separate constant w0;

    "poly":  w(d) = c (1 + 2 (d/r0)^3 - 3 (d/r0)^2)^m   for d <= r0, else 0
    "pow":   w(d) = c / (dd + (d/r0)^m)
    "exp":   w(d) = c / (dd + exp(-d/r0))

Because w depends only on the centre-neighbour distance it multiplies the
neighbour's whole term of Eq. 13 / Eq. 18: F_nl(d) -> w(d) F_nl(d), with the
product rule for the gradient.
"""
from __future__ import annotations

import numpy as np


def weight(spec: dict | None, d):
    """w(d) and dw/dd for an array of distances; (1, 0) without a spec."""
    d = np.asarray(d, np.float64)
    if not spec:
        return np.ones_like(d), np.zeros_like(d)
    fn, r0, c = spec["function"], float(spec["r0"]), float(spec.get("c", 1.0))
    x = d / r0
    if fn == "poly":
        m = float(spec["m"])
        base = 1.0 + 2.0 * x ** 3 - 3.0 * x ** 2
        inside = x <= 1.0
        base = np.where(inside, base, 0.0)
        w = c * base ** m
        dbase = (6.0 * x ** 2 - 6.0 * x) / r0
        with np.errstate(divide="ignore", invalid="ignore"):
            dw = np.where(inside & (base > 0), c * m * base ** (m - 1.0) * dbase, 0.0)
        return w, dw
    if fn == "pow":
        m, dd = float(spec["m"]), float(spec.get("d", 1.0))
        den = dd + x ** m
        with np.errstate(divide="ignore", invalid="ignore"):
            dden = np.where(x > 0, m * x ** (m - 1.0) / r0, 0.0)
        return c / den, -c * dden / den ** 2
    if fn == "exp":
        dd = float(spec.get("d", 1.0))
        e = np.exp(-x)
        den = dd + e
        return c / den, c * e / r0 / den ** 2
    raise ValueError("weighting function must be 'poly', 'pow' or 'exp'")


def onsite_weight(spec: dict | None) -> float:
    return 1.0 if not spec else float(spec.get("w0", 1.0))

"""Real spherical and solid harmonics of the oracle (test infrastructure).

The real harmonics are the ones Eq. 2 expands in: orthonormal on the sphere,

    Y_l0   = sqrt((2l+1)/4pi) P_l(cos t)
    Y_l,+m = sqrt(2) sqrt((2l+1)/4pi (l-m)!/(l+m)!) P_l^m(cos t) cos(m phi)
    Y_l,-m = the same with sin(m phi),                      m = 1..l,

with P_l^m = (1-t^2)^(m/2) d^m P_l / dt^m (no Condon-Shortley sign; Eqs. 4 and
5 are blind to the sign and order convention inside an l block).

The solid harmonic r^l Y_lm is a homogeneous polynomial of degree l in
(x, y, z).  This module builds that polynomial explicitly, with integer
arithmetic up to the normalisation, as a table of monomial coefficients, and
evaluates values and exact Cartesian gradients from the table.  Order inside
an l block: m = -l, ..., 0, ..., +l at index l*l + l + m.
"""
from __future__ import annotations

import functools
from fractions import Fraction
from math import factorial, pi, sqrt

import numpy as np

Poly = dict  # {(a, b, c): Fraction}  coefficient of x^a y^b z^c


def _add(p: Poly, q: Poly, s=Fraction(1)) -> Poly:
    out = dict(p)
    for k, v in q.items():
        out[k] = out.get(k, Fraction(0)) + s * v
    return {k: v for k, v in out.items() if v != 0}


def _mul(p: Poly, q: Poly) -> Poly:
    out: Poly = {}
    for (a, b, c), v in p.items():
        for (d, e, f), w in q.items():
            k = (a + d, b + e, c + f)
            out[k] = out.get(k, Fraction(0)) + v * w
    return {k: v for k, v in out.items() if v != 0}


def _scale(p: Poly, s) -> Poly:
    return {k: v * s for k, v in p.items()}


X: Poly = {(1, 0, 0): Fraction(1)}
Y: Poly = {(0, 1, 0): Fraction(1)}
Z: Poly = {(0, 0, 1): Fraction(1)}
R2: Poly = {(2, 0, 0): Fraction(1), (0, 2, 0): Fraction(1), (0, 0, 2): Fraction(1)}
ONE: Poly = {(0, 0, 0): Fraction(1)}


def _legendre_derivative_coeffs(l: int, m: int):
    """Coefficients a_k of d^m P_l/dt^m = sum_k a_k t^k (exact rationals), from
    P_l(t) = 2^-l sum_j (-1)^j C(l,j) C(2l-2j,l) t^(l-2j)."""
    out = {}
    for j in range(l // 2 + 1):
        power = l - 2 * j
        if power < m:
            continue
        c = Fraction((-1) ** j * factorial(2 * l - 2 * j),
                     2 ** l * factorial(j) * factorial(l - j) * factorial(l - 2 * j))
        for s in range(m):
            c *= (power - s)
        out[power - m] = c
    return out


def _solid_q(l: int, m: int) -> Poly:
    """r^(l-m) d^m P_l/dt^m at t = z/r, a polynomial in z and r^2."""
    out: Poly = {}
    for k, a in _legendre_derivative_coeffs(l, m).items():
        # t^k r^(l-m) = z^k (r^2)^((l-m-k)/2); l-m-k is even by parity of P_l
        e = (l - m - k) // 2
        term = ONE
        for _ in range(k):
            term = _mul(term, Z)
        for _ in range(e):
            term = _mul(term, R2)
        out = _add(out, term, a)
    return out


def _cos_sin_polys(m: int):
    """Re and Im of (x + i y)^m as polynomials."""
    c, s = ONE, {}
    for _ in range(m):
        c, s = _add(_mul(c, X), _mul(s, Y), Fraction(-1)), _add(_mul(s, X), _mul(c, Y))
    return c, s


@functools.lru_cache(maxsize=None)
def solid_harmonic_table(l_max: int):
    """For each l: exponents E[l] (n_mono, 3) and coefficients M[l]
    (2l+1, n_mono) with r^l Y_lm = sum_t M[l][l+m, t] x^a y^b z^c."""
    tables = []
    for l in range(l_max + 1):
        monos = [(a, b, l - a - b) for a in range(l + 1) for b in range(l + 1 - a)]
        index = {mono: t for t, mono in enumerate(monos)}
        M = np.zeros((2 * l + 1, len(monos)))
        for m in range(l + 1):
            norm = sqrt((2 * l + 1) / (4 * pi) * factorial(l - m) / factorial(l + m))
            q = _solid_q(l, m)
            c, s = _cos_sin_polys(m)
            if m == 0:
                for mono, v in q.items():
                    M[l, index[mono]] = norm * float(v)
            else:
                for mono, v in _mul(q, c).items():
                    M[l + m, index[mono]] = sqrt(2.0) * norm * float(v)
                for mono, v in _mul(q, s).items():
                    M[l - m, index[mono]] = sqrt(2.0) * norm * float(v)
        tables.append((np.array(monos, dtype=np.int64).reshape(-1, 3), M))
    return tables


def _powers(v: np.ndarray, l_max: int) -> np.ndarray:
    """v[j]^e for e = 0..l_max, shape (l_max+1, J); 0^0 = 1."""
    out = np.ones((l_max + 1, v.size))
    for e in range(1, l_max + 1):
        out[e] = out[e - 1] * v
    return out


def real_solid_harmonics(xyz: np.ndarray, l_max: int, gradients: bool = False):
    """S[j, lm] = r^l Y_lm at the points xyz[j] (and dS[j, dir, lm]).

    Values and gradients come from the same monomial table, so they are
    consistent with each other to rounding."""
    xyz = np.atleast_2d(np.asarray(xyz, np.float64))
    J = xyz.shape[0]
    px, py, pz = (_powers(xyz[:, a], l_max) for a in range(3))
    S = np.zeros((J, (l_max + 1) ** 2))
    dS = np.zeros((J, 3, (l_max + 1) ** 2)) if gradients else None
    for l, (E, M) in enumerate(solid_harmonic_table(l_max)):
        a, b, c = E[:, 0], E[:, 1], E[:, 2]
        mono = px[a] * py[b] * pz[c]                         # (n_mono, J)
        S[:, l * l:(l + 1) ** 2] = (M @ mono).T
        if gradients:
            gx = a[:, None] * px[np.maximum(a - 1, 0)] * py[b] * pz[c]
            gy = b[:, None] * px[a] * py[np.maximum(b - 1, 0)] * pz[c]
            gz = c[:, None] * px[a] * py[b] * pz[np.maximum(c - 1, 0)]
            dS[:, 0, l * l:(l + 1) ** 2] = (M @ gx).T
            dS[:, 1, l * l:(l + 1) ** 2] = (M @ gy).T
            dS[:, 2, l * l:(l + 1) ** 2] = (M @ gz).T
    return (S, dS) if gradients else S


def real_spherical_harmonics(xyz: np.ndarray, l_max: int, gradients: bool = False):
    """Y[j, lm] at the directions of xyz[j] (|xyz| > 0), and the Cartesian
    gradient of Y_lm(xyz/|xyz|) with respect to xyz:  Y = S / r^l,
    grad Y = grad S / r^l - l S xyz / r^(l+2)."""
    xyz = np.atleast_2d(np.asarray(xyz, np.float64))
    r = np.linalg.norm(xyz, axis=1)
    ls = np.concatenate([[l] * (2 * l + 1) for l in range(l_max + 1)])
    rl = r[:, None] ** ls[None, :]
    if not gradients:
        return real_solid_harmonics(xyz, l_max) / rl
    S, dS = real_solid_harmonics(xyz, l_max, gradients=True)
    Yv = S / rl
    dY = dS / rl[:, None, :] - (ls[None, None, :] * Yv[:, None, :]) * xyz[:, :, None] / (r * r)[:, None, None]
    return Yv, dY

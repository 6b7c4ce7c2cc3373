"""Radial bases of the oracle (test infrastructure; see the package docstring).

Both families are reduced to one radial factor per neighbour distance d,

    c^mu_nlm = sum_j F_nl(d_j) Y_lm(dhat_j)  (+ on-site term),

with F_nl and dF_nl/dd returned by `gto_radial` (Eq. 13) and `poly_radial`
(Eqs. 18-19).  The Loewdin matrices S^(-1/2) (Eq. 9 and the sentence below
Eq. 17) are ill-conditioned, so they are formed as the principal inverse square
root in 80-digit arithmetic and rounded once to fp64.
"""
from __future__ import annotations

import functools

import mpmath
import numpy as np
from scipy import special

LD = np.longdouble


# --------------------------------------------------------------------------
# Loewdin orthogonalisation, Eq. 9
# --------------------------------------------------------------------------
def lowdin(S_rows) -> np.ndarray:
    """Principal S^(-1/2) of a symmetric positive-definite matrix given as a
    nested list of mpmath numbers; 80 significant digits inside, returned in
    extended precision (the entries reach 1e6 and are summed with heavy
    cancellation, so they are kept as accurate as the host allows)."""
    with mpmath.workdps(80):
        S = mpmath.matrix(S_rows)
        n = S.rows
        lam, V = mpmath.eigsy(S)
        out = mpmath.zeros(n, n)
        for a in range(n):
            for b in range(n):
                out[a, b] = mpmath.fsum(V[a, k] * V[b, k] / mpmath.sqrt(lam[k])
                                        for k in range(n))
        return np.array([[LD(mpmath.nstr(out[a, b], 30)) for b in range(n)] for a in range(n)], dtype=LD)


# --------------------------------------------------------------------------
# Gaussian-type orbitals, Eqs. 6-10, 13
# --------------------------------------------------------------------------
def gto_z(r_cut: float, n_max: int):
    """Decay distances z_k of Eq. 10 (a single primitive sits at 1 A)."""
    if n_max == 1:
        return [mpmath.mpf(1)]
    return [1 + mpmath.mpf(k) * (mpmath.mpf(r_cut) - 1) / (n_max - 1)
            for k in range(n_max)]


def gto_alpha_mp(r_cut: float, n_max: int, l: int):
    """alpha_kl of Eq. 10: z_k^l exp(-alpha z_k^2) = 1e-3."""
    return [-(mpmath.log(mpmath.mpf(10) ** -3 / z ** l)) / z ** 2
            for z in gto_z(r_cut, n_max)]


def gto_alpha(r_cut: float, n_max: int, l_max: int) -> np.ndarray:
    """alpha[l, k] in fp64."""
    with mpmath.workdps(80):
        return np.array([[float(a) for a in gto_alpha_mp(r_cut, n_max, l)]
                         for l in range(l_max + 1)])


@functools.lru_cache(maxsize=None)
def _gto_alpha_ld(r_cut: float, n_max: int, l_max: int) -> np.ndarray:
    with mpmath.workdps(80):
        return np.array([[LD(mpmath.nstr(a, 30)) for a in gto_alpha_mp(r_cut, n_max, l)]
                         for l in range(l_max + 1)], dtype=LD)


def gto_overlap_mp(alpha_l, l: int):
    """S^l of Eq. 8, the overlap over [0, inf) (the range the closed form of
    Eq. 13 integrates over)."""
    g = mpmath.gamma(l + mpmath.mpf(3) / 2)
    n = len(alpha_l)
    return [[g / (2 * (alpha_l[a] + alpha_l[b]) ** (l + mpmath.mpf(3) / 2))
             for b in range(n)] for a in range(n)]


@functools.lru_cache(maxsize=None)
def gto_beta(r_cut: float, n_max: int, l_max: int) -> np.ndarray:
    """beta[l, n, k] = (S^l)^(-1/2), Eq. 9."""
    with mpmath.workdps(80):
        return np.array([lowdin(gto_overlap_mp(gto_alpha_mp(r_cut, n_max, l), l))
                         for l in range(l_max + 1)])


def gto_radial(d, r_cut: float, n_max: int, l_max: int, sigma: float):
    """F[n, l, j] and dF/dd for distances d[j] >= 0, Eq. 13:

    F_nl(d) = (2 pi)^(3/2) sigma^3 sum_k beta^l_nk d^l
              (1 + 2 sigma^2 alpha_kl)^-(l+3/2) exp(-alpha_kl d^2 / (1 + 2 sigma^2 alpha_kl)).

    The k-sum cancels heavily, so it is carried in extended precision.
    """
    d = np.atleast_1d(np.asarray(d, np.float64)).astype(LD)
    alpha = _gto_alpha_ld(r_cut, n_max, l_max)              # [l, k]
    beta = gto_beta(r_cut, n_max, l_max)                    # [l, n, k]
    s2 = LD(sigma) ** 2
    pref = (LD(2) * LD(np.pi)) ** LD(1.5) * LD(sigma) ** 3
    F = np.zeros((n_max, l_max + 1, d.size), LD)
    dF = np.zeros_like(F)
    for l in range(l_max + 1):
        w = LD(1) + LD(2) * s2 * alpha[l]                   # [k]
        a = alpha[l] / w
        amp = pref * w ** (-(LD(l) + LD(1.5)))              # [k]
        e = np.exp(-a[:, None] * d[None, :] ** 2)           # [k, j]
        dl = d ** l
        # d/dd of d^l exp(-a d^2) = (l d^(l-1) - 2 a d^(l+1)) exp(-a d^2)
        ddl = (LD(l) * d ** (l - 1) if l > 0 else np.zeros_like(d))
        prim = amp[:, None] * dl[None, :] * e
        dprim = amp[:, None] * (ddl[None, :] - LD(2) * a[:, None] * d[None, :] * dl[None, :]) * e
        F[:, l, :] = beta[l] @ prim
        dF[:, l, :] = beta[l] @ dprim
    return F.astype(np.float64), dF.astype(np.float64)


def gto_onsite(r_cut: float, n_max: int, l_max: int, sigma: float) -> np.ndarray:
    """Second term of Eq. 13: sqrt(2) pi sigma^3 sum_k beta^0_nk (1 + 2 sigma^2 alpha_k0)^(-3/2)."""
    alpha0 = _gto_alpha_ld(r_cut, n_max, l_max)[0]
    beta0 = gto_beta(r_cut, n_max, l_max)[0]
    w = LD(1) + LD(2) * LD(sigma) ** 2 * alpha0
    return (np.sqrt(LD(2)) * LD(np.pi) * LD(sigma) ** 3 * (beta0 @ w ** LD(-1.5))).astype(np.float64)


# --------------------------------------------------------------------------
# Polynomials, Eqs. 15-19
# --------------------------------------------------------------------------
def poly_norm(r_cut: float, n_max: int) -> np.ndarray:
    """N_k of Eq. 16, k = 1..n_max."""
    k = np.arange(1, n_max + 1, dtype=np.float64)
    return np.sqrt(r_cut ** (2 * k + 5) / (2 * k + 5))


@functools.lru_cache(maxsize=None)
def poly_w(n_max: int) -> np.ndarray:
    """W = S^(-1/2) with S_kk' = sqrt((5+2k)(5+2k'))/(5+k+k'), Eq. 17."""
    with mpmath.workdps(80):
        S = [[mpmath.sqrt(mpmath.mpf((5 + 2 * a) * (5 + 2 * b))) / (5 + a + b)
              for b in range(1, n_max + 1)] for a in range(1, n_max + 1)]
        return lowdin(S)


def _scaled_bessel_i(l: int, z):
    """exp(-z) i_l(z) and exp(-z) i_l'(z) for z >= 0 (modified spherical Bessel
    function of the first kind), through SciPy's exponentially scaled I_nu:
    i_l(z) = sqrt(pi / 2z) I_{l+1/2}(z);  i_l' = i_{l+1} + (l/z) i_l."""
    z = np.asarray(z, np.float64)
    pos = z > 0
    zs = np.where(pos, z, 1.0)
    pre = np.sqrt(np.pi / (2 * zs))
    il = pre * special.ive(l + 0.5, zs)
    il1 = pre * special.ive(l + 1.5, zs)
    dil = il1 + (l / zs) * il
    il = np.where(pos, il, 1.0 if l == 0 else 0.0)
    dil = np.where(pos, dil, 1.0 / 3.0 if l == 1 else 0.0)
    return il, dil


def _poly_g(r, r_cut: float, n_max: int) -> np.ndarray:
    """g_n(r) = sum_k W_nk (r_cut - r)^(k+2) / N_k (Eq. 15) at the points r.
    By linearity sum_k (W_nk/N_k) I_kl of Eq. 18 is the radial integral of
    g_n itself; the k-sum cancels to ~1e-6 of its terms, so it is done once,
    here, in extended precision."""
    r = np.asarray(r, np.float64).astype(LD)
    k = np.arange(1, n_max + 1)
    norm = np.sqrt(LD(r_cut) ** (2 * k + 5) / (2 * k + 5).astype(LD))
    prim = (LD(r_cut) - r)[None, :] ** (k[:, None] + 2) / norm[:, None]
    return (poly_w(n_max) @ prim).astype(np.float64)


def _gauss_legendre(r_cut: float, quad_n: int):
    x, w = np.polynomial.legendre.leggauss(quad_n)
    return 0.5 * r_cut * (x + 1.0), 0.5 * r_cut * w


def poly_radial(d, r_cut: float, n_max: int, l_max: int, sigma: float, quad_n: int = 256):
    """F[n, l, j] and dF/dd for the polynomial basis, Eqs. 18-19:

    F_nl(d) = 4 pi exp(-d^2/2 sigma^2) sum_k (W_nk / N_k) I_kl(d),
    I_kl(d) = int_0^rcut r^2 (rcut - r)^(k+2) exp(-r^2/2 sigma^2) i_l(r d / sigma^2) dr,

    the radial integral by a fixed Gauss-Legendre rule on [0, r_cut] that is
    fine enough to be converged to rounding (checked in the tests).  The
    exponentials are merged into exp(-(r-d)^2/2 sigma^2) * [exp(-z) i_l(z)],
    z = r d / sigma^2, which is the same number without overflow.
    """
    d = np.atleast_1d(np.asarray(d, np.float64))
    r, w = _gauss_legendre(r_cut, quad_n)                   # [q]
    s2 = sigma * sigma
    z = r[None, :] * d[:, None] / s2                        # [j, q]
    gauss = np.exp(-(r[None, :] - d[:, None]) ** 2 / (2 * s2))
    g = _poly_g(r, r_cut, n_max)                            # [n, q]  g_n(r_q) of Eq. 15
    F = np.zeros((n_max, l_max + 1, d.size))
    dF = np.zeros_like(F)
    for l in range(l_max + 1):
        il, dil = _scaled_bessel_i(l, z)                    # exp(-z) i_l(z), exp(-z) i_l'(z)
        base = w[None, :] * r[None, :] ** 2 * gauss         # [j, q]
        # sum_k (W_nk/N_k) e^{-d^2/2s2} I_kl(d) = int r^2 g_n(r) e^{-(r^2+d^2)/2s2} i_l(rd/s2) dr
        F[:, l, :] = 4 * np.pi * np.einsum("nq,jq->nj", g, base * il)
        # d/dd [exp(-(r^2+d^2)/2s2) i_l(rd/s2)] = exp(..)[ -d/s2 i_l + (r/s2) i_l' ]
        dF[:, l, :] = 4 * np.pi * np.einsum("nq,jq->nj", g,
                                            base * (-(d[:, None] / s2) * il + (r[None, :] / s2) * dil))
    return F, dF


def poly_onsite(r_cut: float, n_max: int, sigma: float, quad_n: int = 256) -> np.ndarray:
    """On-site l = 0 term of the polynomial basis (text below Eq. 21):
    sqrt(4 pi) sum_k (W_nk/N_k) I_k0(0), i_0(0) = 1."""
    r, w = _gauss_legendre(r_cut, quad_n)
    return np.sqrt(4 * np.pi) * _poly_g(r, r_cut, n_max) @ (w * r ** 2 * np.exp(-r ** 2 / (2 * sigma ** 2)))

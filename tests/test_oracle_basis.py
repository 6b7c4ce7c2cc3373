"""Pins for the oracle's radial bases (Eqs. 6-10, 13, 15-19)."""
import os

import mpmath
import numpy as np
import pytest
from scipy import integrate

from oracle import basis


def test_gto_alpha_threshold_rule():
    # Eq. 10: primitive k of channel l has decayed to 1e-3 at z_k, z_k uniform in [1, r_cut]
    r_cut, n_max, l_max = 6.0, 8, 6
    alpha = basis.gto_alpha(r_cut, n_max, l_max)
    z = 1.0 + np.arange(n_max) * (r_cut - 1.0) / (n_max - 1)
    for l in range(l_max + 1):
        np.testing.assert_allclose(z ** l * np.exp(-alpha[l] * z ** 2), 1e-3, rtol=1e-12)
    np.testing.assert_allclose(alpha[:, 0], 3 * np.log(10.0), rtol=1e-14)   # z_1 = 1 for every l
    assert basis.gto_alpha(5.0, 1, 2).shape == (3, 1)


@pytest.mark.parametrize("n_max,l_max", [(4, 3), (8, 6)])
def test_gto_lowdin_orthonormalises_overlap(n_max, l_max):
    # Eq. 9: beta S beta = 1 with S of Eq. 8, checked in 50-digit arithmetic
    r_cut = 6.0
    beta = basis.gto_beta(r_cut, n_max, l_max).astype(np.float64)
    with mpmath.workdps(50):
        for l in range(l_max + 1):
            S = mpmath.matrix(basis.gto_overlap_mp(basis.gto_alpha_mp(r_cut, n_max, l), l))
            B = mpmath.matrix(beta[l].tolist())
            err = B * S * B - mpmath.eye(n_max)
            worst = max(abs(err[i, j]) for i in range(n_max) for j in range(n_max))
            # beta is rounded to fp64: error ~ 1e-16 * |beta|^2 |S|
            assert worst < 1e-16 * float(np.abs(beta[l]).max()) ** 2 * 50
        assert np.allclose(beta, np.transpose(beta, (0, 2, 1)), rtol=0, atol=1e-9 * np.abs(beta).max())


def test_gto_basis_orthonormal_by_numerical_integration():
    # int_0^inf r^2 g_nl g_n'l dr = delta_nn' with g_nl of Eq. 6
    r_cut, n_max, l_max = 5.0, 4, 3
    alpha = basis.gto_alpha(r_cut, n_max, l_max)
    beta = basis.gto_beta(r_cut, n_max, l_max).astype(np.float64)
    for l in range(l_max + 1):
        def g(n, r):
            return np.sum(beta[l, n] * r ** l * np.exp(-alpha[l] * r * r))
        for n in range(n_max):
            for n2 in range(n, n_max):
                val, _ = integrate.quad(lambda r: r * r * g(n, r) * g(n2, r), 0, 40.0, epsabs=1e-13, epsrel=1e-13, limit=400)
                assert abs(val - (1.0 if n == n2 else 0.0)) < 1e-9


def test_poly_basis_constants():
    # Eq. 16 and Eq. 17 by direct integration, and W S W = 1
    r_cut, n_max = 5.0, 6
    N = basis.poly_norm(r_cut, n_max)
    for k in range(1, n_max + 1):
        val, _ = integrate.quad(lambda r: (r_cut - r) ** (2 * (k + 2)), 0, r_cut, epsrel=1e-13)
        assert abs(np.sqrt(val) / N[k - 1] - 1) < 1e-12
    W = basis.poly_w(n_max).astype(np.float64)
    # orthonormality of g_n = sum_k W_nk (rc-r)^(k+2)/N_k under the plain measure dr of Eq. 17
    x, w = np.polynomial.legendre.leggauss(64)
    r = 0.5 * r_cut * (x + 1)
    w = 0.5 * r_cut * w
    prim = np.array([(r_cut - r) ** (k + 2) / N[k - 1] for k in range(1, n_max + 1)])
    g = W @ prim
    gram = (g * w) @ g.T
    assert np.abs(gram - np.eye(n_max)).max() < 1e-7
    assert np.abs(W - W.T).max() < 1e-9 * np.abs(W).max()


def _mp_radial_projection(l, n, d, r_cut, n_max, sigma):
    """F_nl(d) from Eqs. 3, 6, 11 without the closed form of Eq. 12:
    4 pi int_0^inf r^2 g_nl(r) exp(-(r^2+d^2)/2 sigma^2) i_l(r d/sigma^2) dr."""
    alpha = basis.gto_alpha_mp(r_cut, n_max, l)
    beta = basis.gto_beta(r_cut, n_max, l)[l, n]

    def i_l(z):
        return mpmath.sqrt(mpmath.pi / (2 * z)) * mpmath.besseli(l + mpmath.mpf(1) / 2, z)

    def integrand(r):
        g = mpmath.fsum(mpmath.mpf(float(b)) * r ** l * mpmath.exp(-a * r * r) for b, a in zip(beta, alpha))
        return r * r * g * mpmath.exp(-(r * r + d * d) / (2 * sigma ** 2)) * i_l(r * d / sigma ** 2)
    return 4 * mpmath.pi * mpmath.quad(integrand, [0, d / 2, d, 2 * d, 4 * d, 12 * d])


def test_gto_closed_form_against_radial_bessel_integral():
    # Eq. 13 against a 30-digit quadrature of the integral Eq. 12 evaluates in closed form
    r_cut, n_max, l_max, sigma = 5.0, 4, 3, 0.5
    d = 2.0
    F, _ = basis.gto_radial([d], r_cut, n_max, l_max, sigma)
    with mpmath.workdps(30):
        for l in (0, 2, 3):
            for n in range(n_max):
                ref = _mp_radial_projection(l, n, mpmath.mpf(d), r_cut, n_max, mpmath.mpf(sigma))
                assert abs(F[n, l, 0] - float(ref)) < 1e-12 * max(1.0, abs(float(ref)))


def test_gto_single_neighbour_values():
    # A neighbour of another species on +z at 2.0 A, r_cut = 5, n_max = 4, sigma = 0.5:
    # c_nl0 = sqrt((2l+1)/4 pi) F_nl(d).  The reference digits come from tests/golden/make_gto_single_neighbour.py,
    # which evaluates Eqs. 1, 3, 8-11 in 40-digit arithmetic without the oracle (Loewdin root by a matrix iteration,
    # radial integral by quadrature); they pin beta as the principal root of Eq. 9.
    golden = np.loadtxt(os.path.join(os.path.dirname(__file__), "golden", "gto_single_neighbour.txt"))
    ref = {l: golden[golden[:, 0] == l][:, 2] for l in (0, 2)}
    assert len(ref[0]) == 4 and len(ref[2]) == 4
    F, _ = basis.gto_radial([2.0], 5.0, 4, 3, 0.5)
    np.testing.assert_allclose(np.sqrt(1 / (4 * np.pi)) * F[:, 0, 0], ref[0], rtol=2e-10)
    np.testing.assert_allclose(np.sqrt(5 / (4 * np.pi)) * F[:, 2, 0], ref[2], rtol=2e-10)


@pytest.mark.parametrize("r_cut,n_max,l_max", [(5.0, 4, 3), (6.0, 8, 6), (6.0, 12, 12)])
def test_lowdin_matrices_are_the_positive_definite_roots(r_cut, n_max, l_max):
    # beta S beta = 1 and symmetry also hold for the non-principal symmetric roots (eigenvalue signs flipped);
    # Eq. 9 means the principal one, whose eigenvalues are all positive.  Checked in 60-digit arithmetic on the
    # extended-precision entries.
    beta = basis.gto_beta(r_cut, n_max, l_max)
    with mpmath.workdps(60):
        for l in range(l_max + 1):
            B = mpmath.matrix([[mpmath.mpf(repr(float(x))) + mpmath.mpf(float(x - np.longdouble(float(x)))) for x in row] for row in beta[l]])
            lam = mpmath.eigsy((B + B.T) / 2, eigvals_only=True)
            assert min(lam) > 0, f"l = {l}: smallest eigenvalue {min(lam)}"
        W = basis.poly_w(min(n_max, 8))
        Wm = mpmath.matrix([[mpmath.mpf(float(x)) for x in row] for row in W])
        assert min(mpmath.eigsy((Wm + Wm.T) / 2, eigvals_only=True)) > 0


def test_gto_onsite_is_the_zero_distance_limit():
    # second term of Eq. 13 = first term at r -> 0 (only l = 0 survives, Y_00 = 1/sqrt(4 pi))
    args = (6.0, 8, 6, 0.5)
    F, dF = basis.gto_radial([0.0, 1e-7], *args)
    np.testing.assert_allclose(F[:, 0, 0] / np.sqrt(4 * np.pi), basis.gto_onsite(*args), rtol=1e-12)
    assert np.abs(F[:, 1:, 0]).max() == 0.0
    assert np.abs(dF[:, 0, 0]).max() == 0.0


@pytest.mark.parametrize("fn,args", [
    (basis.gto_radial, (5.0, 6, 4, 0.5)),
    (basis.poly_radial, (5.0, 6, 4, 0.4)),
])
def test_radial_derivative_by_finite_differences(fn, args):
    d = np.array([0.7, 1.3, 2.9, 4.6])
    h = 2e-3        # five-point stencil: truncation ~ h^4, rounding ~ eps |W| / h
    _, dF = fn(d, *args)
    f = {s: fn(d + s * h, *args)[0] for s in (-2, -1, 1, 2)}
    fd = (f[-2] - 8 * f[-1] + 8 * f[1] - f[2]) / (12 * h)
    scale = np.abs(dF).max(axis=2, keepdims=True) + 1e-300
    assert (np.abs(fd - dF) / scale).max() < 2e-7


def test_poly_quadrature_is_converged_and_onsite_limit():
    args = (5.0, 8, 8, 0.4)
    d = np.array([0.0, 0.9, 2.5, 4.95])
    F1, dF1 = basis.poly_radial(d, *args, quad_n=256)
    F2, dF2 = basis.poly_radial(d, *args, quad_n=512)
    assert np.abs(F1 - F2).max() < 1e-11 * np.abs(F1).max()
    assert np.abs(dF1 - dF2).max() < 1e-11 * np.abs(dF1).max()
    np.testing.assert_allclose(F1[:, 0, 0] / np.sqrt(4 * np.pi), basis.poly_onsite(5.0, 8, 0.4), rtol=1e-12)
    assert np.abs(F1[:, 1:, 0]).max() == 0.0


def test_poly_exact_integral_tends_to_laplace_form():
    # Eq. 21 is the first-order (in sigma^2) Laplace expansion of Eqs. 18-19:
    # the gap to the exact integral must shrink like sigma^4 relative to the leading term.
    r_cut, n_max, l = 5.0, 3, 2
    d = 2.5
    W = basis.poly_w(n_max).astype(np.float64) / basis.poly_norm(r_cut, n_max)[None, :]
    gaps = []
    for sigma in (0.1, 0.05):
        F, _ = basis.poly_radial([d], r_cut, n_max, l, sigma, quad_n=2000)
        k = np.arange(1, n_max + 1)
        s2 = sigma ** 2
        bracket = (1 - l * (l + 1) * s2 / (2 * d * d) - (k + 2) * s2 / (d * (r_cut - d))
                   + (k + 2) * (k + 1) * s2 / (2 * (r_cut - d) ** 2))
        approx = (2 * np.pi) ** 1.5 * sigma ** 3 * W @ ((r_cut - d) ** (k + 2) * bracket)
        lead = (2 * np.pi) ** 1.5 * sigma ** 3 * np.abs(W @ ((r_cut - d) ** (k + 2)))
        gaps.append(np.abs(F[:, l, 0] - approx) / lead)
    gaps = np.array(gaps)
    assert gaps[0].max() < 5e-3
    ratio = gaps[0] / gaps[1]
    assert np.all(ratio > 10) and np.all(ratio < 24)      # ~ 2^4

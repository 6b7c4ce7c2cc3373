"""Pins for the oracle's real spherical / solid harmonics."""
import numpy as np
from scipy import special

from oracle.harmonics import real_solid_harmonics, real_spherical_harmonics

L = 8
rng = np.random.Generator(np.random.PCG64(7))
PTS = rng.normal(size=(40, 3)) * 2.0


def test_against_scipy_complex_harmonics():
    # Y_l0 = Y_l^0, Y_l,+m = sqrt2 (-1)^m Re Y_l^m, Y_l,-m = sqrt2 (-1)^m Im Y_l^m
    # (the (-1)^m strips SciPy's Condon-Shortley phase)
    Y = real_spherical_harmonics(PTS, L)
    r = np.linalg.norm(PTS, axis=1)
    theta = np.arccos(PTS[:, 2] / r)
    phi = np.arctan2(PTS[:, 1], PTS[:, 0])
    for l in range(L + 1):
        for m in range(0, l + 1):
            ylm = special.sph_harm_y(l, m, theta, phi)
            if m == 0:
                np.testing.assert_allclose(Y[:, l * l + l], ylm.real, atol=1e-12)
            else:
                np.testing.assert_allclose(Y[:, l * l + l + m], np.sqrt(2) * (-1) ** m * ylm.real, atol=1e-12)
                np.testing.assert_allclose(Y[:, l * l + l - m], np.sqrt(2) * (-1) ** m * ylm.imag, atol=1e-12)


def test_unsold_and_gradient_sum_rules():
    S, dS = real_solid_harmonics(PTS, L, gradients=True)
    r = np.linalg.norm(PTS, axis=1)
    for l in range(L + 1):
        sl = slice(l * l, (l + 1) ** 2)
        np.testing.assert_allclose((S[:, sl] ** 2).sum(1), (2 * l + 1) / (4 * np.pi) * r ** (2 * l), rtol=1e-11)
        if l > 0:
            np.testing.assert_allclose((dS[:, :, sl] ** 2).sum((1, 2)),
                                       l * (2 * l + 1) ** 2 / (4 * np.pi) * r ** (2 * l - 2), rtol=1e-11)
        # Euler: r . grad S = l S (homogeneous of degree l)
        np.testing.assert_allclose(np.einsum("jd,jdm->jm", PTS, dS[:, :, sl]), l * S[:, sl],
                                   atol=1e-10 * np.abs(S[:, sl]).max())


def test_gradient_by_finite_differences_and_harmonicity():
    h = 1e-4
    S, dS = real_solid_harmonics(PTS, L, gradients=True)
    lap = np.zeros_like(S)
    for a in range(3):
        e = np.zeros(3)
        e[a] = h
        Sp, dSp = real_solid_harmonics(PTS + e, L, gradients=True)
        Sm, dSm = real_solid_harmonics(PTS - e, L, gradients=True)
        fd = (Sp - Sm) / (2 * h)
        assert np.abs(fd - dS[:, a]).max() < 1e-6 * max(1.0, np.abs(dS[:, a]).max())
        lap += (dSp[:, a] - dSm[:, a]) / (2 * h)
    # Laplace equation: div grad S = 0
    assert np.abs(lap).max() < 1e-5 * np.abs(dS).max()


def test_spherical_gradient_is_tangential():
    Y, dY = real_spherical_harmonics(PTS, L, gradients=True)
    # Y depends on the direction only: r . grad Y = 0
    assert np.abs(np.einsum("jd,jdm->jm", PTS, dY)).max() < 1e-11
    np.testing.assert_allclose(Y[:, 0], 1 / np.sqrt(4 * np.pi))

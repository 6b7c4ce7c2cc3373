#!/usr/bin/env python
"""Writes tests/golden/gto_single_neighbour.txt: expansion coefficients c_nl0 of ONE neighbour of another
species on the +z axis, straight from the paper's definitions in 40-digit arithmetic (mpmath only; this
script imports nothing from the oracle or the library, and the oracle's tests read the file it writes).

  alpha_kl          Eq. 10:  z_k^l exp(-alpha_kl z_k^2) = 1e-3, z_k evenly spaced from 1 A to r_cut
  S^l_kk'           Eq. 8:   overlap of the primitives r^l exp(-alpha r^2) over [0, inf) with weight r^2
  beta^l            Eq. 9:   the principal inverse square root of S^l.  Formed here by the coupled
                             Denman-Beavers iteration (Y -> S^(1/2), Z -> S^(-1/2) from Y = S, Z = 1), which
                             converges to the principal roots of a positive-definite matrix and shares nothing
                             with an eigen-decomposition.
  c_nl0             Eq. 3 with the density of Eq. 1 (one Gaussian of width sigma at d on the z axis), the
                    angular integral done by the plane-wave expansion of Eq. 11:
                        c_nl0 = sqrt((2l+1)/(4 pi)) 4 pi int_0^inf r^2 g_nl(r) exp(-(r^2+d^2)/(2 sigma^2))
                                i_l(r d / sigma^2) dr,     g_nl(r) = sum_k beta^l_nk r^l exp(-alpha_kl r^2)
                    by adaptive quadrature of the radial integral, not by the closed form of Eq. 12.

Parameters: r_cut = 5 A, n_max = 4, sigma = 0.5 A, d = 2 A, l = 0 and l = 2.
"""
import os

import mpmath as mp

mp.mp.dps = 40
R_CUT, N_MAX, SIGMA, D = mp.mpf(5), 4, mp.mpf("0.5"), mp.mpf(2)


def alphas(l):
    z = [1 + k * (R_CUT - 1) / (N_MAX - 1) for k in range(N_MAX)]
    return [(3 * mp.log(10) + l * mp.log(zk)) / zk ** 2 for zk in z]


def overlap(alpha, l):
    g = mp.gamma(l + mp.mpf(3) / 2)
    return mp.matrix([[g / (2 * (a + b) ** (l + mp.mpf(3) / 2)) for b in alpha] for a in alpha])


def inverse_sqrt(S):
    Y, Z = S.copy(), mp.eye(S.rows)
    for _ in range(200):
        Yn = (Y + Z ** -1) / 2
        Zn = (Z + Y ** -1) / 2
        done = mp.norm(Zn - Z, "inf") < mp.mpf(10) ** -36 * mp.norm(Zn, "inf")
        Y, Z = Yn, Zn
        if done:
            break
    return Z


def c_nl0(l):
    alpha = alphas(l)
    beta = inverse_sqrt(overlap(alpha, l))

    def i_l(x):
        return mp.sqrt(mp.pi / (2 * x)) * mp.besseli(l + mp.mpf(1) / 2, x)

    out = []
    for n in range(N_MAX):
        def f(r):
            g = mp.fsum(beta[n, k] * r ** l * mp.exp(-alpha[k] * r * r) for k in range(N_MAX))
            return r * r * g * mp.exp(-(r * r + D * D) / (2 * SIGMA ** 2)) * i_l(r * D / SIGMA ** 2)
        radial = mp.quad(f, [0, D / 2, D, 2 * D, 4 * D, 12 * D])
        out.append(mp.sqrt((2 * l + 1) / (4 * mp.pi)) * 4 * mp.pi * radial)
    return out


def main():
    here = os.path.dirname(os.path.abspath(__file__))
    with open(os.path.join(here, "gto_single_neighbour.txt"), "w") as fh:
        fh.write("# c_nl0 of one neighbour of another species at (0, 0, 2 A); r_cut 5 A, n_max 4, sigma 0.5 A, GTO basis\n")
        fh.write("# Eqs. 1, 3, 8-11 evaluated by make_gto_single_neighbour.py (mpmath, 40 digits); columns: l n value\n")
        for l in (0, 2):
            for n, v in enumerate(c_nl0(l)):
                fh.write(f"{l} {n + 1} {mp.nstr(v, 25)}\n")


if __name__ == "__main__":
    main()

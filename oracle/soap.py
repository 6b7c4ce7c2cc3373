"""The SOAP hot path, written out plainly in fp64 (test infrastructure).

Steps, in the paper's order:
  neighbours inside the cutoff (text under Eq. 1)  ->  expansion coefficients
  c^mu_nlm (Eq. 13 for Gaussian-type orbitals, Eqs. 18-19 for polynomials,
  on-site term included)  ->  partial power spectrum p (Eq. 4)  ->  Cartesian
  Jacobian dp/dR_j for every atom inside the sphere and for the centre itself
  (Eq. 5 and the translation argument below it).

Positions are promoted to fp64 as they come: hand in the same fp32 array the
library receives and both sides see identical numbers (fp64 arrays are taken
as they are, which the invariance and finite-difference tests use).
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

from . import basis
from . import weighting as _weighting
from .harmonics import real_spherical_harmonics

GTO, POLYNOMIAL = 0, 1


@dataclass
class Derivatives:
    descriptor: np.ndarray     # (C, F)
    row_ptr: np.ndarray        # (C+1,) rows of centre i are row_ptr[i]:row_ptr[i+1]
    row_atom: np.ndarray       # (rows,) atom the row differentiates with respect to
    jacobian: np.ndarray       # (rows, 3, F)


class SoapOracle:
    def __init__(self, species, r_cut, n_max, l_max, sigma, rbf=GTO, pbc=(False, False, False), crossover=True,
                 weighting=None):
        self.crossover = bool(crossover)
        self.weighting = dict(weighting) if weighting else None
        self.species = sorted(int(z) for z in species)
        self.r_cut, self.n_max, self.l_max, self.sigma = float(r_cut), int(n_max), int(l_max), float(sigma)
        self.rbf = int(rbf)
        self.pbc = tuple(bool(p) for p in pbc)
        if self.rbf == GTO and not self.r_cut > 1.0:
            raise ValueError("the width rule of Eq. 10 places primitives between 1 A and r_cut")
        self.S = len(self.species)
        self.table = self.feature_table()
        self.n_features = self.table.shape[0]

    # ---------------------------------------------------------------- layout
    def feature_table(self) -> np.ndarray:
        """Rows (mu, nu, n, n', l) in output order: species pairs mu <= nu,
        then the radial pair (n' >= n when mu == nu, every (n, n') otherwise),
        then l fastest.  With `crossover` off only the pairs mu == nu are kept
        (the constructor flag that decides whether off-diagonal species pairs
        are retained)."""
        rows = []
        for mu in range(self.S):
            for nu in range(mu, self.S if self.crossover else mu + 1):
                for n in range(self.n_max):
                    for n2 in range(n if mu == nu else 0, self.n_max):
                        for l in range(self.l_max + 1):
                            rows.append((mu, nu, n, n2, l))
        return np.array(rows, dtype=np.int64)

    # ------------------------------------------------------------ neighbours
    def _heights(self, cell):
        """Distance between opposite faces of the cell along each axis."""
        vol = abs(np.linalg.det(cell))
        return [vol / np.linalg.norm(np.cross(cell[(a + 1) % 3], cell[(a + 2) % 3]))
                for a in range(3)]

    def neighbor_list(self, positions, cell=None, centers=None, sites=None):
        """For every centre the sorted list of (atom j, n_a, n_b, n_c) with
        0 < |r_j + n_a a + n_b b + n_c c - r_i|^2 < r_cut^2.  With `sites`
        (an array of Cartesian points) the centres are those points instead of
        atoms: r_i is the point.

        The displacement is formed as (r_j - r_i) + T with the lattice
        translation T = (n_a a + n_b b) + n_c c, each step rounded to fp64 in
        this order; the library evaluates the same expression so that the two
        sets can be compared exactly."""
        pos = np.asarray(positions, np.float64)
        N = pos.shape[0]
        centers = np.arange(N) if centers is None else np.asarray(centers)
        origins = pos[centers] if sites is None else np.asarray(sites, np.float64).reshape(-1, 3)
        rc2 = self.r_cut * self.r_cut
        periodic = cell is not None and any(self.pbc)
        if periodic:
            cell = np.asarray(cell, np.float64)
            frac = np.concatenate([pos, origins]) @ np.linalg.inv(cell)
            spans = []
            heights = self._heights(cell)
            for a in range(3):
                if not self.pbc[a]:
                    spans.append(range(0, 1))
                    continue
                spread = frac[:, a].max() - frac[:, a].min()
                # wide enough for unwrapped inputs; every candidate is tested below
                k = int(np.ceil(self.r_cut / heights[a] + spread)) + 1
                spans.append(range(-k, k + 1))
            shifts = [(na, nb, nc) for na in spans[0] for nb in spans[1] for nc in spans[2]]
        else:
            shifts = [(0, 0, 0)]
        out = []
        for origin in origins:
            found = []
            base = pos - origin                                   # r_j - r_i
            for (na, nb, nc) in shifts:
                if periodic:
                    T = (na * cell[0] + nb * cell[1]) + nc * cell[2]
                    d = base + T
                else:
                    d = base
                d2 = d[:, 0] * d[:, 0] + d[:, 1] * d[:, 1] + d[:, 2] * d[:, 2]
                for j in np.nonzero((d2 < rc2) & (d2 > 0.0))[0]:
                    found.append((int(j), na, nb, nc))
            out.append(sorted(found))
        return out

    def _displacements(self, pos, cell, i, nbrs):
        """Displacements of the listed neighbours from atom i, or from the
        point i when i is a length-3 array."""
        if not nbrs:
            return np.zeros((0, 3))
        j = np.array([t[0] for t in nbrs])
        d = pos[j] - (pos[i] if np.ndim(i) == 0 else np.asarray(i, np.float64))
        if cell is not None and any(self.pbc):
            n = np.array([t[1:] for t in nbrs], dtype=np.float64)
            cell = np.asarray(cell, np.float64)
            d = d + ((n[:, 0:1] * cell[0] + n[:, 1:2] * cell[1]) + n[:, 2:3] * cell[2])
        return d

    # ---------------------------------------------------------- coefficients
    def radial(self, d):
        """F[n, l, j], dF/dd[n, l, j] of the chosen basis, times the radial
        weighting of the neighbour density when one is set."""
        if self.rbf == GTO:
            F, dF = basis.gto_radial(d, self.r_cut, self.n_max, self.l_max, self.sigma)
        else:
            F, dF = basis.poly_radial(d, self.r_cut, self.n_max, self.l_max, self.sigma)
        if self.weighting:
            w, dw = _weighting.weight(self.weighting, d)
            F, dF = F * w, dF * w + F * dw
        return F, dF

    def onsite(self):
        """c_n00 contribution of the centre itself (position independent)."""
        w0 = _weighting.onsite_weight(self.weighting)
        if self.rbf == GTO:
            return w0 * basis.gto_onsite(self.r_cut, self.n_max, self.l_max, self.sigma)
        return w0 * basis.poly_onsite(self.r_cut, self.n_max, self.sigma)

    def _species_index(self, numbers):
        lut = {z: s for s, z in enumerate(self.species)}
        try:
            return np.array([lut[int(z)] for z in numbers], dtype=np.int64)
        except KeyError as e:
            raise ValueError(f"atomic number {e} is not in the species list") from None

    def _pair_terms(self, d, want_grad):
        """Per neighbour: t[j, n, lm] = F_nl(d) Y_lm(dhat) and its Cartesian
        gradient g[j, dir, n, lm] = F' (d_dir/d) Y + F dY/d(dir)  (Eq. 14 for
        Gaussian-type orbitals, Eq. 23 for polynomials)."""
        L1 = self.l_max + 1
        J = d.shape[0]
        if J == 0:
            z = np.zeros((0, self.n_max, L1 * L1))
            return z, (np.zeros((0, 3, self.n_max, L1 * L1)) if want_grad else None)
        r = np.linalg.norm(d, axis=1)
        F, dF = self.radial(r)                                    # [n, l, j]
        ls = np.concatenate([[l] * (2 * l + 1) for l in range(L1)])
        Fx = np.transpose(F[:, ls, :], (2, 0, 1))                 # [j, n, lm]
        if not want_grad:
            Yv = real_spherical_harmonics(d, self.l_max)
            return Fx * Yv[:, None, :], None
        Yv, dY = real_spherical_harmonics(d, self.l_max, gradients=True)
        dFx = np.transpose(dF[:, ls, :], (2, 0, 1))
        unit = d / r[:, None]
        g = (dFx[:, None, :, :] * unit[:, :, None, None] * Yv[:, None, None, :]
             + Fx[:, None, :, :] * dY[:, :, None, :])
        return Fx * Yv[:, None, :], g

    def coefficients(self, positions, numbers, cell, i, nbrs=None):
        """c[mu, n, lm] of centre atom i (Eq. 13 / Eq. 18, on-site term included)."""
        pos = np.asarray(positions, np.float64)
        sp = self._species_index(numbers)
        if nbrs is None:
            nbrs = self.neighbor_list(pos, cell, [i])[0]
        d = self._displacements(pos, cell, i, nbrs)
        t, _ = self._pair_terms(d, False)
        L1 = self.l_max + 1
        c = np.zeros((self.S, self.n_max, L1 * L1))
        zj = sp[[n[0] for n in nbrs]] if nbrs else np.zeros(0, np.int64)
        for mu in range(self.S):
            c[mu] = t[zj == mu].sum(axis=0)
        c[sp[i], :, 0] += self.onsite()
        return c

    # -------------------------------------------------------- power spectrum
    def power_spectrum(self, c):
        """Eq. 4 in the order of `feature_table`."""
        L1 = self.l_max + 1
        p = np.empty(self.n_features)
        for f, (mu, nu, n, n2, l) in enumerate(self.table):
            sl = slice(l * l, (l + 1) ** 2)
            p[f] = np.pi * np.sqrt(8.0 / (2 * l + 1)) * np.dot(c[mu, n, sl], c[nu, n2, sl])
        return p

    def descriptor(self, positions, numbers, cell=None, centers=None):
        pos = np.asarray(positions, np.float64)
        N = pos.shape[0]
        centers = np.arange(N) if centers is None else np.asarray(centers)
        lists = self.neighbor_list(pos, cell, centers)
        out = np.empty((len(centers), self.n_features))
        for a, i in enumerate(centers):
            out[a] = self.power_spectrum(self.coefficients(pos, numbers, cell, int(i), lists[a]))
        return out

    # -------------------------------------------------------------- Jacobian
    def derivatives(self, positions, numbers, cell=None, centers=None) -> Derivatives:
        """Descriptor and its Jacobian, one row per atom inside the sphere and
        one for the centre, rows of a centre in ascending atom order.

        Eq. 5 with grad_j c^mu = 0 unless atom j has species mu; images of one
        atom add up in that atom's row; the centre's row is minus the sum over
        its neighbours' terms (a periodic image of the centre itself moves
        with the centre, so its displacement is constant and drops out)."""
        pos = np.asarray(positions, np.float64)
        sp = self._species_index(numbers)
        N = pos.shape[0]
        centers = np.arange(N) if centers is None else np.asarray(centers)
        lists = self.neighbor_list(pos, cell, centers)
        L1 = self.l_max + 1
        kl = np.array([np.pi * np.sqrt(8.0 / (2 * l + 1)) for l in range(L1)])
        desc = np.empty((len(centers), self.n_features))
        row_ptr = [0]
        row_atom, blocks = [], []
        # feature rows grouped by (mu, nu, l) for vectorised assembly
        groups = {}
        for f, (mu, nu, n, n2, l) in enumerate(self.table):
            groups.setdefault((mu, nu, l), []).append((f, n, n2))
        for a, i in enumerate(centers):
            i = int(i)
            nbrs = lists[a]
            d = self._displacements(pos, cell, i, nbrs)
            t, g = self._pair_terms(d, True)                      # [j,n,lm], [j,dir,n,lm]
            zj = sp[[n[0] for n in nbrs]] if nbrs else np.zeros(0, np.int64)
            c = np.zeros((self.S, self.n_max, L1 * L1))
            for mu in range(self.S):
                c[mu] = t[zj == mu].sum(axis=0)
            c[sp[i], :, 0] += self.onsite()
            desc[a] = self.power_spectrum(c)
            atoms = sorted(set([i] + [n[0] for n in nbrs]))
            local = {atom: r for r, atom in enumerate(atoms)}
            J = np.zeros((len(atoms), 3, self.n_features))
            rows_of = np.array([local[n[0]] for n in nbrs], dtype=np.int64)
            moving = np.array([n[0] != i for n in nbrs], dtype=bool)   # an image of the centre has no net motion
            for s in range(self.S):
                sel = np.nonzero((zj == s) & moving)[0]
                if sel.size == 0:
                    continue
                gs = g[sel]                                       # [e, dir, n, lm]
                pair = np.zeros((sel.size, 3, self.n_features))
                for (mu, nu, l), items in groups.items():
                    if mu != s and nu != s:
                        continue
                    sl = slice(l * l, (l + 1) ** 2)
                    fs = np.array([it[0] for it in items])
                    ns = np.array([it[1] for it in items])
                    n2s = np.array([it[2] for it in items])
                    val = np.zeros((sel.size, 3, len(items)))
                    if mu == s:    # (grad_j c^mu_nlm) c^nu_n'lm
                        val += np.einsum("edfm,fm->edf", gs[:, :, ns, sl], c[nu][n2s, sl])
                    if nu == s:    # c^mu_nlm (grad_j c^nu_n'lm)
                        val += np.einsum("fm,edfm->edf", c[mu][ns, sl], gs[:, :, n2s, sl])
                    pair[:, :, fs] = kl[l] * val
                np.add.at(J, rows_of[sel], pair)
                J[local[i]] -= pair.sum(axis=0)
            desc_rows = len(atoms)
            row_ptr.append(row_ptr[-1] + desc_rows)
            row_atom.extend(atoms)
            blocks.append(J)
        jac = np.concatenate(blocks, axis=0) if blocks else np.zeros((0, 3, self.n_features))
        return Derivatives(desc, np.array(row_ptr, np.int64), np.array(row_atom, np.int32), jac)

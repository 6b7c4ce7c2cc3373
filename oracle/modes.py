"""Output modes beyond the per-centre power spectrum (test infrastructure).

The text on the package's interface lists, next to the per-centre power
spectrum, a coefficient mode that returns the raw projection coefficients
c^mu_nlm themselves, and two averaged power spectra: "outer" averages the
power spectra of the centres, "inner" averages the coefficients over the
centres first and contracts the averaged coefficients (Eq. 4 applied to the
mean).  Everything here is the definition written out on top of the pinned
coefficient routine of `oracle.soap`; the Jacobians are dense in the atom
index, (n_atoms, 3, width), because an average couples every centre to
every atom.

Coefficient layout (a reading: the paper names no order): species, then n,
then l, then m = -l..l, i.e. index (mu n_max + n) (l_max+1)^2 + l^2 + l + m.
"""
from __future__ import annotations

import numpy as np

from .soap import Derivatives, SoapOracle


def coefficient_vector(o: SoapOracle, positions, numbers, cell=None, centers=None) -> np.ndarray:
    """(C, S n_max (l_max+1)^2): c^mu_nlm of every centre, on-site term included."""
    pos = np.asarray(positions, np.float64)
    centers = np.arange(pos.shape[0]) if centers is None else np.asarray(centers)
    lists = o.neighbor_list(pos, cell, centers)
    return np.stack([o.coefficients(pos, numbers, cell, int(i), lists[a]).reshape(-1)
                     for a, i in enumerate(centers)]) if len(centers) else np.zeros((0, coefficient_width(o)))


def coefficient_width(o: SoapOracle) -> int:
    return o.S * o.n_max * (o.l_max + 1) ** 2


def coefficient_derivatives(o: SoapOracle, positions, numbers, cell=None, centers=None) -> Derivatives:
    """Coefficients and d c^mu_nlm / d R_j in the row format of
    `SoapOracle.derivatives`: the gradient of a neighbour's term sits in the
    block of that neighbour's species (Eq. 14 / Eq. 23), zero in the others;
    images of one atom add up; the centre's row is minus the sum of the rows
    of the atoms that move relative to it."""
    pos = np.asarray(positions, np.float64)
    sp = o._species_index(numbers)
    centers = np.arange(pos.shape[0]) if centers is None else np.asarray(centers)
    lists = o.neighbor_list(pos, cell, centers)
    LM = (o.l_max + 1) ** 2
    W = coefficient_width(o)
    vec = np.zeros((len(centers), W))
    row_ptr, row_atom, blocks = [0], [], []
    for a, i in enumerate(centers):
        i = int(i)
        nbrs = lists[a]
        vec[a] = o.coefficients(pos, numbers, cell, i, nbrs).reshape(-1)
        d = o._displacements(pos, cell, i, nbrs)
        _, g = o._pair_terms(d, True)                               # [pair, dir, n, lm]
        atoms = sorted(set([i] + [t[0] for t in nbrs]))
        local = {atom: r for r, atom in enumerate(atoms)}
        J = np.zeros((len(atoms), 3, o.S, o.n_max, LM))
        for e, t in enumerate(nbrs):
            if t[0] == i:                                           # an image of the centre moves with it
                continue
            J[local[t[0]], :, sp[t[0]]] += g[e]
            J[local[i], :, sp[t[0]]] -= g[e]
        row_ptr.append(row_ptr[-1] + len(atoms))
        row_atom.extend(atoms)
        blocks.append(J.reshape(len(atoms), 3, W))
    jac = np.concatenate(blocks, axis=0) if blocks else np.zeros((0, 3, W))
    return Derivatives(vec, np.array(row_ptr, np.int64), np.array(row_atom, np.int32), jac)


def _dense(der: Derivatives, n_atoms: int) -> np.ndarray:
    """(C, n_atoms, 3, width) with zeros for atoms outside a centre's sphere."""
    C = len(der.row_ptr) - 1
    out = np.zeros((C, n_atoms) + der.jacobian.shape[1:])
    for a in range(C):
        for r in range(der.row_ptr[a], der.row_ptr[a + 1]):
            out[a, der.row_atom[r]] = der.jacobian[r]
    return out


def average_descriptor(o: SoapOracle, mode: str, positions, numbers, cell=None, centers=None) -> np.ndarray:
    """(F,): "outer" = mean over the centres of their power spectra;
    "inner" = power spectrum of the mean coefficients."""
    if mode == "outer":
        return o.descriptor(positions, numbers, cell, centers).mean(axis=0)
    if mode == "inner":
        c = coefficient_vector(o, positions, numbers, cell, centers).mean(axis=0)
        return o.power_spectrum(c.reshape(o.S, o.n_max, -1))
    raise ValueError("mode must be 'inner' or 'outer'")


def average_derivatives(o: SoapOracle, mode: str, positions, numbers, cell=None, centers=None):
    """The averaged descriptor (F,) and its Jacobian (n_atoms, 3, F)."""
    n_atoms = np.asarray(positions).shape[0]
    if mode == "outer":
        der = o.derivatives(positions, numbers, cell, centers)
        return der.descriptor.mean(axis=0), _dense(der, n_atoms).mean(axis=0)
    if mode != "inner":
        raise ValueError("mode must be 'inner' or 'outer'")
    der = coefficient_derivatives(o, positions, numbers, cell, centers)
    cbar = der.descriptor.mean(axis=0).reshape(o.S, o.n_max, -1)                  # [mu, n, lm]
    dcbar = _dense(der, n_atoms).mean(axis=0).reshape(n_atoms, 3, o.S, o.n_max, -1)
    jac = np.empty((n_atoms, 3, o.n_features))
    for f, (mu, nu, n, n2, l) in enumerate(o.table):                              # Eq. 5 on the mean
        sl = slice(l * l, (l + 1) ** 2)
        k = np.pi * np.sqrt(8.0 / (2 * l + 1))
        jac[:, :, f] = k * (dcbar[:, :, mu, n, sl] @ cbar[nu, n2, sl] + dcbar[:, :, nu, n2, sl] @ cbar[mu, n, sl])
    return o.power_spectrum(cbar), jac


# ------------------------------------------------------------------ centres that are not atoms
def site_derivatives(o: SoapOracle, positions, numbers, sites, cell=None) -> Derivatives:
    """Descriptor and Jacobian for centres at arbitrary Cartesian points (the interface accepts
    an explicit list of centres; a point that is no atom has no Gaussian of its own, hence no
    on-site term, and no row of its own: it does not move with any atom).  Otherwise Eqs. 4
    and 5 exactly as for atom centres.  A point that coincides with an atom drops that atom
    (the neighbour test is 0 < d^2): use the atom as the centre instead."""
    pos = np.asarray(positions, np.float64)
    sp = o._species_index(numbers)
    sites = np.asarray(sites, np.float64).reshape(-1, 3)
    lists = o.neighbor_list(pos, cell, sites=sites)
    LM = (o.l_max + 1) ** 2
    desc = np.empty((len(sites), o.n_features))
    row_ptr, row_atom, blocks = [0], [], []
    for a, site in enumerate(sites):
        nbrs = lists[a]
        d = o._displacements(pos, cell, site, nbrs)
        t, g = o._pair_terms(d, True)                                  # [pair, n, lm], [pair, dir, n, lm]
        c = np.zeros((o.S, o.n_max, LM))
        atoms = sorted(set(n[0] for n in nbrs))
        local = {atom: r for r, atom in enumerate(atoms)}
        dc = np.zeros((len(atoms), 3, o.S, o.n_max, LM))               # grad_j c^mu_nlm, images of an atom add up
        for e, n in enumerate(nbrs):
            c[sp[n[0]]] += t[e]
            dc[local[n[0]], :, sp[n[0]]] += g[e]
        desc[a] = o.power_spectrum(c)
        J = np.empty((len(atoms), 3, o.n_features))
        for f, (mu, nu, n1, n2, l) in enumerate(o.table):               # Eq. 5
            sl = slice(l * l, (l + 1) ** 2)
            k = np.pi * np.sqrt(8.0 / (2 * l + 1))
            J[:, :, f] = k * (dc[:, :, mu, n1, sl] @ c[nu, n2, sl] + dc[:, :, nu, n2, sl] @ c[mu, n1, sl])
        row_ptr.append(row_ptr[-1] + len(atoms))
        row_atom.extend(atoms)
        blocks.append(J)
    jac = np.concatenate(blocks, axis=0) if blocks else np.zeros((0, 3, o.n_features))
    return Derivatives(desc, np.array(row_ptr, np.int64), np.array(row_atom, np.int32), jac)


# ------------------------------------------------------------------ many independent structures at once
def batch_derivatives(o: SoapOracle, structures) -> Derivatives:
    """Non-periodic structures treated as one list of atoms: every atom of every structure is a centre and
    sees only the atoms of its own structure (the multi-GPU section enumerates work as batches of centres
    drawn from one structure each; structures never interact).  Output rows as in
    `SoapOracle.derivatives`, with atom indices counted through the concatenated list."""
    desc, ptr, atoms, jac = [], [np.zeros(1, np.int64)], [], []
    base_atom, base_row = 0, 0
    for positions, numbers in structures:
        d = o.derivatives(positions, numbers)
        desc.append(d.descriptor)
        ptr.append(d.row_ptr[1:] + base_row)
        atoms.append(d.row_atom + base_atom)
        jac.append(d.jacobian)
        base_atom += len(numbers)
        base_row += int(d.row_ptr[-1])
    F = o.n_features
    return Derivatives(np.concatenate(desc) if desc else np.zeros((0, F)), np.concatenate(ptr),
                       (np.concatenate(atoms) if atoms else np.zeros(0)).astype(np.int32),
                       np.concatenate(jac) if jac else np.zeros((0, 3, F)))

"""Generators for the synthetic structures (see the package docstring)."""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np
from scipy.spatial import cKDTree

WATER_DENSITY = 0.0334      # molecules / A^3
OO_MIN = 2.5                # A
R_OH = 0.9572               # A
HOH_DEG = 104.52
BOX_DENSITY = 0.1           # atoms / A^3
BOX_MIN_DIST = 0.9          # A


@dataclass
class Structure:
    positions: np.ndarray          # (N, 3) float32, Angstrom
    numbers: np.ndarray            # (N,) int32 atomic numbers
    cell: np.ndarray | None        # (3, 3) float64, rows = lattice vectors
    pbc: tuple                     # three bools
    name: str = ""

    @property
    def n_atoms(self) -> int:
        return int(self.positions.shape[0])


def _rng(seed: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(int(seed)))


def random_rotation(rng: np.random.Generator) -> np.ndarray:
    """Uniform random proper rotation from a unit quaternion."""
    while True:
        q = 2.0 * rng.random(4) - 1.0
        s = float(q @ q)
        if 1e-4 < s <= 1.0:
            break
    a, b, c, d = q / np.sqrt(s)
    return np.array([
        [a*a + b*b - c*c - d*d, 2*(b*c - a*d), 2*(b*d + a*c)],
        [2*(b*c + a*d), a*a - b*b + c*c - d*d, 2*(c*d - a*b)],
        [2*(b*d - a*c), 2*(c*d + a*b), a*a - b*b - c*c + d*d]])


def _rotations(rng: np.random.Generator, n: int) -> np.ndarray:
    """n uniform rotations, vectorised (Gaussian-free: rejection on the 4-ball)."""
    out = np.empty((n, 4))
    filled = 0
    while filled < n:
        q = 2.0 * rng.random((2 * (n - filled) + 8, 4)) - 1.0
        s = np.einsum("ij,ij->i", q, q)
        q = q[(s > 1e-4) & (s <= 1.0)]
        q /= np.linalg.norm(q, axis=1, keepdims=True)
        k = min(n - filled, q.shape[0])
        out[filled:filled + k] = q[:k]
        filled += k
    a, b, c, d = out.T
    R = np.empty((n, 3, 3))
    R[:, 0, 0] = a*a + b*b - c*c - d*d
    R[:, 0, 1] = 2*(b*c - a*d)
    R[:, 0, 2] = 2*(b*d + a*c)
    R[:, 1, 0] = 2*(b*c + a*d)
    R[:, 1, 1] = a*a - b*b + c*c - d*d
    R[:, 1, 2] = 2*(c*d - a*b)
    R[:, 2, 0] = 2*(b*d - a*c)
    R[:, 2, 1] = 2*(c*d + a*b)
    R[:, 2, 2] = a*a - b*b - c*c + d*d
    return R


def _rsa_sphere(rng, n, radius, dmin):
    """Random sequential addition of n points in a sphere, pair distance >= dmin.

    Candidates come in batches; a candidate is dropped when it is closer than
    dmin to an accepted point or to an earlier candidate of its own batch.
    """
    acc = np.empty((0, 3))
    while acc.shape[0] < n:
        want = n - acc.shape[0]
        m = max(64, min(8 * want, 1 << 21))
        c = (2.0 * rng.random((m, 3)) - 1.0) * radius
        c = c[np.einsum("ij,ij->i", c, c) <= radius * radius]
        if acc.shape[0]:
            d, _ = cKDTree(acc).query(c, k=1, distance_upper_bound=dmin)
            c = c[np.isinf(d)]
        if c.shape[0] > 1:
            pairs = cKDTree(c).query_pairs(dmin, output_type="ndarray")
            keep = np.ones(c.shape[0], bool)
            if pairs.size:
                keep[np.unique(pairs.max(axis=1))] = False
            c = c[keep]
        acc = np.concatenate([acc, c[:want]], axis=0)
    return acc


def water_cluster(n_mol: int, seed: int = 0) -> Structure:
    rng = _rng(seed)
    radius = (3.0 * n_mol / (4.0 * np.pi * WATER_DENSITY)) ** (1.0 / 3.0)
    o_xyz = _rsa_sphere(rng, n_mol, radius, OO_MIN)
    half = np.deg2rad(HOH_DEG) / 2.0
    h_local = R_OH * np.array([[np.sin(half), 0.0, np.cos(half)],
                               [-np.sin(half), 0.0, np.cos(half)]])
    R = _rotations(rng, n_mol)
    pos = np.empty((n_mol, 3, 3))
    pos[:, 0] = o_xyz
    pos[:, 1] = o_xyz + np.einsum("nij,j->ni", R, h_local[0])
    pos[:, 2] = o_xyz + np.einsum("nij,j->ni", R, h_local[1])
    numbers = np.tile(np.array([8, 1, 1], np.int32), n_mol)
    return Structure(pos.reshape(-1, 3).astype(np.float32), numbers, None,
                     (False, False, False), f"water{n_mol}_seed{seed}")


def _rsa_periodic_cube(rng, n, box, dmin):
    acc = np.empty((0, 3))
    while acc.shape[0] < n:
        want = n - acc.shape[0]
        c = rng.random((max(64, 2 * want), 3)) * box
        if acc.shape[0]:
            d, _ = cKDTree(acc, boxsize=box).query(c, k=1, distance_upper_bound=dmin)
            c = c[np.isinf(d)]
        if c.shape[0] > 1:
            pairs = cKDTree(c, boxsize=box).query_pairs(dmin, output_type="ndarray")
            keep = np.ones(c.shape[0], bool)
            if pairs.size:
                keep[np.unique(pairs.max(axis=1))] = False
            c = c[keep]
        acc = np.concatenate([acc, c[:want]], axis=0)
    return acc


def multispecies_box(n_atoms: int = 2000, seed: int = 0) -> Structure:
    rng = _rng(seed)
    box = (n_atoms / BOX_DENSITY) ** (1.0 / 3.0)
    # fp32 positions must stay inside [0, box) after rounding
    pos = np.minimum(_rsa_periodic_cube(rng, n_atoms, box, BOX_MIN_DIST),
                     np.nextafter(np.float32(box), np.float32(0)))
    unit = n_atoms // 10
    numbers = np.concatenate([np.full(3 * unit, 6), np.full(5 * unit, 1),
                              np.full(unit, 7),
                              np.full(n_atoms - 9 * unit, 8)]).astype(np.int32)
    numbers = numbers[np.argsort(rng.random(n_atoms), kind="stable")]
    return Structure(pos.astype(np.float32), numbers, np.eye(3) * box,
                     (True, True, True), f"chno_box{n_atoms}_seed{seed}")


def small_periodic_cell(seed: int = 0, pbc=(True, True, True)) -> Structure:
    """8 atoms (C, H, N, O twice) in a sheared 4 A cell; positions are not
    wrapped into the cell on purpose (two atoms are pushed one lattice vector
    out) so that the image bookkeeping is exercised."""
    rng = _rng(seed)
    cell = np.array([[4.0, 0.0, 0.0], [0.6, 4.1, 0.0], [-0.4, 0.5, 3.9]])
    while True:
        frac = rng.random((8, 3))
        cart = frac @ cell
        ok = True
        for i in range(8):
            for j in range(i + 1, 8):
                d = frac[j] - frac[i]
                d -= np.round(d)
                if np.linalg.norm(d @ cell) < 0.9:
                    ok = False
        if ok:
            break
    cart[2] += cell[0]
    cart[5] -= cell[1] + cell[2]
    numbers = np.array([6, 1, 7, 8, 6, 1, 7, 8], np.int32)
    return Structure(cart.astype(np.float32), numbers, cell, tuple(pbc),
                     f"cell8_seed{seed}")

"""Pins for the oracle's coefficients, power spectrum, Jacobian and neighbour list."""
import numpy as np
import pytest
from scipy import special

from oracle import basis
from oracle.soap import GTO, POLYNOMIAL, SoapOracle
from soap_inputs import multispecies_box, random_rotation, small_periodic_cell, water_cluster


def _scipy_real_harmonics(l_max, theta, phi):
    out = []
    for l in range(l_max + 1):
        row = [None] * (2 * l + 1)
        for m in range(0, l + 1):
            y = special.sph_harm_y(l, m, theta, phi)
            if m == 0:
                row[l] = y.real
            else:
                row[l + m] = np.sqrt(2) * (-1) ** m * y.real
                row[l - m] = np.sqrt(2) * (-1) ** m * y.imag
        out.extend(row)
    return np.array(out)                                   # [lm, ...]


@pytest.mark.parametrize("rbf", [GTO, POLYNOMIAL])
def test_coefficients_against_brute_force_projection(rbf):
    """Eq. 3 by 3-D quadrature of g_nl(r) Y_lm rho(r) on a product grid, for a
    centre (included in its own density) and three neighbours of two species.
    Radial range: all space for the Gaussian-type orbitals (the range the closed
    form of Eq. 13 integrates over), the cutoff sphere for the polynomials."""
    r_cut, n_max, l_max, sigma = 4.0, 3, 3, 0.5
    pos = np.array([[0.0, 0.0, 0.0], [1.1, 0.7, -0.9], [-1.6, 0.4, 1.2], [0.3, -2.2, 0.8]])
    numbers = np.array([1, 8, 1, 8])
    o = SoapOracle([1, 8], r_cut, n_max, l_max, sigma, rbf)
    c = o.coefficients(pos, numbers, None, 0)

    r_hi = r_cut + 10 * sigma if rbf == GTO else r_cut
    xr, wr = np.polynomial.legendre.leggauss(160)
    r = 0.5 * r_hi * (xr + 1)
    wr = 0.5 * r_hi * wr
    xt, wt = np.polynomial.legendre.leggauss(96)            # cos(theta)
    nphi = 192
    phi = 2 * np.pi * np.arange(nphi) / nphi
    wphi = 2 * np.pi / nphi
    ct, ph = np.meshgrid(xt, phi, indexing="ij")
    st = np.sqrt(1 - ct * ct)
    unit = np.stack([st * np.cos(ph), st * np.sin(ph), ct], -1)          # [t, p, 3]
    Yg = _scipy_real_harmonics(l_max, np.arccos(ct), ph)                   # [lm, t, p]
    if rbf == GTO:
        alpha = basis.gto_alpha(r_cut, n_max, l_max)
        beta = basis.gto_beta(r_cut, n_max, l_max).astype(np.float64)
        g = np.array([[beta[l, n] @ (r[None, :] ** l * np.exp(-alpha[l][:, None] * r[None, :] ** 2))
                       for l in range(l_max + 1)] for n in range(n_max)])  # [n, l, r]
    else:
        W = basis.poly_w(n_max).astype(np.float64)
        N = basis.poly_norm(r_cut, n_max)
        prim = np.array([(r_cut - r) ** (k + 2) / N[k - 1] for k in range(1, n_max + 1)])
        g = np.repeat((W @ prim)[:, None, :], l_max + 1, axis=1)
    ls = np.concatenate([[l] * (2 * l + 1) for l in range(l_max + 1)])
    for mu, z in enumerate([1, 8]):
        members = [j for j in range(4) if numbers[j] == z]
        rho = np.zeros((r.size,) + ct.shape)
        for j in members:                                                # Eq. 1, centre included
            diff = r[:, None, None, None] * unit[None] - pos[j]
            rho += np.exp(-np.sum(diff * diff, -1) / (2 * sigma ** 2))
        ang = np.einsum("mtp,rtp,t->mr", Yg, rho, wt) * wphi             # [lm, r]
        ref = np.einsum("nmr,mr,r->nm", g[:, ls, :], ang, wr * r * r)
        assert np.abs(c[mu] - ref).max() < 2e-9 * max(1.0, np.abs(ref).max())


def _legendre_closed_form(o, pos, numbers, i):
    """p^{mu nu}_{n n' l} without spherical harmonics (addition theorem):
    K_l (2l+1)/(4 pi) sum_{a in mu} sum_{b in nu} F_nl(d_a) F_n'l(d_b) P_l(cos gamma_ab),
    the centre counted as a neighbour at distance zero (l = 0 only)."""
    sp = o._species_index(numbers)
    d = np.delete(pos - pos[i], i, axis=0)
    z = np.delete(sp, i)
    r = np.linalg.norm(d, axis=1)
    keep = r < o.r_cut
    d, z, r = d[keep], z[keep], r[keep]
    F, _ = o.radial(r)                                      # [n, l, j]
    cosg = np.clip((d / r[:, None]) @ (d / r[:, None]).T, -1, 1)
    self_n = o.onsite() * np.sqrt(4 * np.pi)                # F_n0(0)
    out = np.zeros(o.n_features)
    for f, (mu, nu, n, n2, l) in enumerate(o.table):
        a, b = z == mu, z == nu
        P = special.eval_legendre(l, cosg[np.ix_(a, b)])
        val = F[n, l, a] @ P @ F[n2, l, b]
        if l == 0:
            if sp[i] == mu:
                val += self_n[n] * F[n2, 0, b].sum()
            if sp[i] == nu:
                val += F[n, 0, a].sum() * self_n[n2]
            if sp[i] == mu == nu:
                val += self_n[n] * self_n[n2]
        out[f] = np.pi * np.sqrt(8.0 / (2 * l + 1)) * (2 * l + 1) / (4 * np.pi) * val
    return out


@pytest.mark.parametrize("rbf,n_max,l_max", [(GTO, 4, 5), (POLYNOMIAL, 4, 4)])
def test_power_spectrum_against_harmonics_free_form(rbf, n_max, l_max):
    s = water_cluster(8, 3)
    o = SoapOracle([1, 8], 4.5, n_max, l_max, 0.5, rbf)
    pos = s.positions.astype(np.float64)
    p = o.descriptor(pos, s.numbers, None, [0, 1, 5])
    for a, i in enumerate([0, 1, 5]):
        ref = _legendre_closed_form(o, pos, s.numbers, i)
        assert np.abs(p[a] - ref).max() < 1e-11 * np.abs(ref).max()


def test_feature_table_layout():
    o = SoapOracle([8, 1, 6], 5.0, 3, 2, 0.5)
    t = o.table
    S, n, L1 = 3, 3, 3
    assert o.n_features == S * n * (S * n + 1) // 2 * L1
    assert o.species == [1, 6, 8]
    # l fastest, then n', then n, then the species pair; same-species blocks keep n' >= n
    assert [tuple(r) for r in t[:4]] == [(0, 0, 0, 0, 0), (0, 0, 0, 0, 1), (0, 0, 0, 0, 2), (0, 0, 0, 1, 0)]
    same = t[t[:, 0] == t[:, 1]]
    assert np.all(same[:, 3] >= same[:, 2])
    cross = t[(t[:, 0] == 0) & (t[:, 1] == 2)]
    assert cross.shape[0] == n * n * L1
    assert np.all(t[:, 0] <= t[:, 1])
    assert len({tuple(r) for r in t}) == t.shape[0]


@pytest.mark.parametrize("rbf", [GTO, POLYNOMIAL])
def test_invariances(rbf):
    s = water_cluster(8, 1)
    pos = s.positions.astype(np.float64)
    o = SoapOracle([1, 8], 4.0, 4, 4, 0.5, rbf)
    centers = [0, 4, 11]
    p0 = o.descriptor(pos, s.numbers, None, centers)
    scale = np.abs(p0).max()
    rng = np.random.Generator(np.random.PCG64(5))
    R = random_rotation(rng)
    assert np.abs(o.descriptor(pos @ R.T, s.numbers, None, centers) - p0).max() < 1e-10 * scale
    M = np.diag([1.0, -1.0, 1.0])                            # reflection
    assert np.abs(o.descriptor(pos @ M, s.numbers, None, centers) - p0).max() < 1e-10 * scale
    assert np.abs(o.descriptor(pos + np.array([3.0, -7.5, 11.25]), s.numbers, None, centers) - p0).max() < 1e-10 * scale
    # permutation of like atoms: swap the two hydrogens of molecule 3 and two oxygens' order
    perm = np.arange(24)
    perm[[10, 11]] = perm[[11, 10]]
    perm[[6, 7, 8, 15, 16, 17]] = perm[[15, 16, 17, 6, 7, 8]]
    inv = np.argsort(perm)
    p1 = o.descriptor(pos[perm], s.numbers[perm], None, [int(inv[c]) for c in centers])
    assert np.abs(p1 - p0).max() < 1e-10 * scale


@pytest.mark.parametrize("rbf", [GTO, POLYNOMIAL])
def test_jacobian_by_central_differences_and_sum_rules(rbf):
    s = water_cluster(8, 2)
    pos = s.positions.astype(np.float64)
    r_cut = 4.2
    o = SoapOracle([1, 8], r_cut, 4, 3, 0.5, rbf)
    h = 1e-4
    dist = np.linalg.norm(pos[:, None] - pos[None], axis=-1)
    assert np.abs(dist - r_cut).min() > 10 * h              # no pair crosses the cutoff
    centers = [0, 7, 13]
    D = o.derivatives(pos, s.numbers, None, centers)
    scale = np.abs(D.jacobian).max(axis=(0, 1))              # per feature
    for a, i in enumerate(centers):
        rows = slice(D.row_ptr[a], D.row_ptr[a + 1])
        atoms = D.row_atom[rows]
        assert i in atoms and np.all(np.diff(atoms) > 0)
        J = D.jacobian[rows]
        # translation: rows sum to zero; rotation: sum_j r_j x dp/dr_j = 0
        assert np.abs(J.sum(0)).max() < 1e-12 * scale.max()
        torque = np.cross(pos[atoms][:, :, None], J, axisa=1, axisb=1, axisc=1).sum(0)
        assert np.abs(torque).max() < 1e-11 * scale.max() * np.abs(pos).max()
        for r, j in enumerate(atoms):
            for dirn in range(3):
                pp, pm = pos.copy(), pos.copy()
                pp[j, dirn] += h
                pm[j, dirn] -= h
                fd = (o.descriptor(pp, s.numbers, None, [i])[0] - o.descriptor(pm, s.numbers, None, [i])[0]) / (2 * h)
                assert np.abs(fd - J[r, dirn]).max() / scale.max() < 1e-6
        # atoms outside the sphere do not move the descriptor
        outside = [j for j in range(24) if j not in atoms]
        if outside:
            pp = pos.copy()
            pp[outside[0], 0] += h
            assert np.abs(o.descriptor(pp, s.numbers, None, [i])[0] - D.descriptor[a]).max() == 0.0


def _replicate(struct, reps):
    cell = struct.cell
    pos = struct.positions.astype(np.float64)
    allpos, allnum, origin = [], [], None
    for na in range(-reps, reps + 1):
        for nb in range(-reps, reps + 1):
            for nc in range(-reps, reps + 1):
                if (na, nb, nc) == (0, 0, 0):
                    origin = len(allpos) * pos.shape[0]
                allpos.append(pos + (na * cell[0] + nb * cell[1]) + nc * cell[2])
                allnum.append(struct.numbers)
    return np.concatenate(allpos), np.concatenate(allnum), origin


def test_periodic_equals_explicit_replicas():
    s = small_periodic_cell(0)
    r_cut = 4.5                                             # larger than the cell: several images per atom
    for rbf in (GTO, POLYNOMIAL):
        o = SoapOracle([1, 6, 7, 8], r_cut, 3, 3, 0.5, rbf, pbc=(True, True, True))
        D = o.derivatives(s.positions, s.numbers, s.cell, [0, 2, 5])
        big_pos, big_num, origin = _replicate(s, 3)
        ofree = SoapOracle([1, 6, 7, 8], r_cut, 3, 3, 0.5, rbf)
        centers = [origin + c for c in (0, 2, 5)]
        Dfree = ofree.derivatives(big_pos, big_num, None, centers)
        assert np.abs(D.descriptor - Dfree.descriptor).max() < 1e-11 * np.abs(D.descriptor).max()
        # derivative with respect to atom j of the cell = sum over all replicas of j
        n = s.n_atoms
        for a in range(3):
            rows = slice(D.row_ptr[a], D.row_ptr[a + 1])
            rows_f = slice(Dfree.row_ptr[a], Dfree.row_ptr[a + 1])
            folded = np.zeros((n, 3, o.n_features))
            np.add.at(folded, Dfree.row_atom[rows_f] % n, Dfree.jacobian[rows_f])
            dense = np.zeros((n, 3, o.n_features))
            dense[D.row_atom[rows]] = D.jacobian[rows]
            assert np.abs(dense - folded).max() < 1e-10 * np.abs(folded).max()


def test_neighbor_list_periodic_matches_replicas_and_counts():
    s = small_periodic_cell(1)
    o = SoapOracle([1, 6, 7, 8], 5.0, 2, 1, 0.5, GTO, pbc=(True, True, True))
    lists = o.neighbor_list(s.positions, s.cell)
    big_pos, _, origin = _replicate(s, 4)
    n = s.n_atoms
    for i in range(n):
        d = np.linalg.norm(big_pos - big_pos[origin + i], axis=1)
        count = int(((d < 5.0) & (d > 0)).sum())
        assert len(lists[i]) == count
        assert len(set(lists[i])) == count
    # mixed boundary conditions: only the periodic axes carry images
    o2 = SoapOracle([1, 6, 7, 8], 5.0, 2, 1, 0.5, GTO, pbc=(True, False, False))
    for nb in o2.neighbor_list(s.positions, s.cell):
        assert all(t[2] == 0 and t[3] == 0 for t in nb)
    # the box of the paper-like periodic workload holds one image at most
    b = multispecies_box(200, 0)
    o3 = SoapOracle([1, 6, 7, 8], 5.0, 2, 1, 0.4, POLYNOMIAL, pbc=(True, True, True))
    for nb in o3.neighbor_list(b.positions, b.cell, range(20)):
        atoms = [t[0] for t in nb]
        assert len(atoms) == len(set(atoms))


def test_unknown_species_and_small_cutoff_are_rejected():
    with pytest.raises(ValueError):
        SoapOracle([1, 8], 1.0, 2, 1, 0.5, GTO)
    o = SoapOracle([1, 8], 3.0, 2, 1, 0.5, GTO)
    with pytest.raises(ValueError):
        o.descriptor(np.zeros((2, 3), np.float32) + [[0, 0, 0], [1, 0, 0]], [1, 6])


def test_isolated_atom_has_only_the_onsite_term():
    o = SoapOracle([1, 8], 3.0, 3, 2, 0.5, GTO)
    D = o.derivatives(np.array([[0.0, 0, 0], [10.0, 0, 0]], np.float32), [8, 1])
    assert list(D.row_ptr) == [0, 1, 2] and list(D.row_atom) == [0, 1]
    assert np.abs(D.jacobian).max() == 0.0
    c = o.onsite()
    # only the (O,O), l = 0 block of centre 0 is non-zero
    for f, (mu, nu, n, n2, l) in enumerate(o.table):
        want = np.pi * np.sqrt(8.0) * c[n] * c[n2] if (mu == nu == 1 and l == 0) else 0.0
        assert abs(D.descriptor[0, f] - want) < 1e-14

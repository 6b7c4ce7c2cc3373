"""Pins for the oracle's coefficient mode, averaged modes and the crossover flag."""
import numpy as np
import pytest

from oracle import modes
from oracle.soap import GTO, POLYNOMIAL, SoapOracle
from soap_inputs import random_rotation, small_periodic_cell, water_cluster


def _fd(fun, pos, h=1e-5):
    """Central differences of fun(pos) with respect to every coordinate: (N, 3, ...)."""
    out = []
    for j in range(pos.shape[0]):
        row = []
        for k in range(3):
            p1, p2 = pos.copy(), pos.copy()
            p1[j, k] += h
            p2[j, k] -= h
            row.append((fun(p1) - fun(p2)) / (2 * h))
        out.append(row)
    return np.array(out)


def test_crossover_off_keeps_exactly_the_same_species_blocks():
    st = water_cluster(3, seed=5)
    pos = st.positions.astype(np.float64)
    full = SoapOracle([1, 8], 4.0, 3, 2, 0.5)
    diag = SoapOracle([1, 8], 4.0, 3, 2, 0.5, crossover=False)
    keep = np.nonzero(full.table[:, 0] == full.table[:, 1])[0]
    assert diag.n_features == 2 * (3 * 4 // 2) * 3 == keep.size
    assert np.array_equal(diag.table, full.table[keep])
    a, b = full.derivatives(pos, st.numbers), diag.derivatives(pos, st.numbers)
    assert np.array_equal(a.descriptor[:, keep], b.descriptor)
    assert np.array_equal(a.row_atom, b.row_atom)
    np.testing.assert_allclose(b.jacobian, a.jacobian[:, :, keep], rtol=0, atol=1e-15)


@pytest.mark.parametrize("rbf", [GTO, POLYNOMIAL])
def test_coefficient_jacobian_by_central_differences(rbf):
    st = small_periodic_cell(seed=2, pbc=(True, True, False))      # short axes: images of the centre itself occur
    pos = st.positions.astype(np.float64)
    o = SoapOracle([1, 6, 7, 8], 4.2, 3, 3, 0.5, rbf, pbc=st.pbc)
    der = modes.coefficient_derivatives(o, pos, st.numbers, st.cell)
    dense = modes._dense(der, pos.shape[0])                        # [C, N, 3, W]
    fd = _fd(lambda p: modes.coefficient_vector(o, p, st.numbers, st.cell), pos)   # [N, 3, C, W]
    np.testing.assert_allclose(dense, np.transpose(fd, (2, 0, 1, 3)), rtol=0, atol=2e-8 * np.abs(dense).max())
    # a rigid translation changes nothing: the rows of a centre sum to zero
    assert np.abs(dense.sum(axis=1)).max() < 1e-12 * np.abs(dense).max()
    # the descriptor of the coefficient mode is the pinned coefficient routine, flattened
    np.testing.assert_array_equal(der.descriptor[3], o.coefficients(pos, st.numbers, st.cell, 3).reshape(-1))


def test_coefficient_block_of_another_species_stays_zero():
    pos = np.array([[0.0, 0.0, 0.0], [1.0, 0.2, -0.3], [-0.8, 1.1, 0.4]])
    numbers = np.array([8, 1, 1])
    o = SoapOracle([1, 8], 3.0, 2, 2, 0.4)
    der = modes.coefficient_derivatives(o, pos, numbers, centers=[0])
    J = der.jacobian.reshape(3, 3, 2, 2, 9)                        # rows: atoms 0, 1, 2
    assert np.all(J[1:, :, 1] == 0) and np.abs(J[1:, :, 0]).max() > 0     # hydrogens move only the H block
    assert np.all(J[0, :, 1] == 0)                                        # the O block holds the on-site constant only


@pytest.mark.parametrize("mode", ["inner", "outer"])
@pytest.mark.parametrize("rbf", [GTO, POLYNOMIAL])
def test_averaged_jacobian_by_central_differences(mode, rbf):
    st = small_periodic_cell(seed=4, pbc=(True, False, True))
    pos = st.positions.astype(np.float64)
    o = SoapOracle([1, 6, 7, 8], 4.0, 2, 3, 0.45, rbf, pbc=st.pbc)
    centers = [0, 2, 3, 7]
    desc, jac = modes.average_derivatives(o, mode, pos, st.numbers, st.cell, centers)
    np.testing.assert_allclose(desc, modes.average_descriptor(o, mode, pos, st.numbers, st.cell, centers), rtol=1e-13)
    fd = _fd(lambda p: modes.average_descriptor(o, mode, p, st.numbers, st.cell, centers), pos)
    np.testing.assert_allclose(jac, fd, rtol=0, atol=3e-8 * np.abs(jac).max())
    assert np.abs(jac.sum(axis=0)).max() < 1e-11 * np.abs(jac).max()


def test_inner_average_is_the_mean_cross_power_spectrum():
    """Eq. 4 is bilinear, so contracting the mean coefficients equals the mean over all ordered
    pairs of centres (i, i') of K_l sum_m c_i c_i'."""
    st = water_cluster(2, seed=9)
    pos = st.positions.astype(np.float64)
    o = SoapOracle([1, 8], 3.5, 2, 2, 0.5)
    cs = [o.coefficients(pos, st.numbers, None, i) for i in range(6)]
    acc = np.zeros(o.n_features)
    for a in cs:
        for b in cs:
            for f, (mu, nu, n, n2, l) in enumerate(o.table):
                sl = slice(l * l, (l + 1) ** 2)
                acc[f] += np.pi * np.sqrt(8.0 / (2 * l + 1)) * np.dot(a[mu, n, sl], b[nu, n2, sl])
    np.testing.assert_allclose(modes.average_descriptor(o, "inner", pos, st.numbers), acc / 36, rtol=1e-12)


@pytest.mark.parametrize("mode", ["inner", "outer"])
def test_averages_reduce_to_the_plain_descriptor(mode):
    # one centre: nothing to average
    st = water_cluster(3, seed=1)
    pos = st.positions.astype(np.float64)
    o = SoapOracle([1, 8], 4.0, 3, 2, 0.5)
    plain = o.derivatives(pos, st.numbers, centers=[4])
    desc, jac = modes.average_derivatives(o, mode, pos, st.numbers, centers=[4])
    np.testing.assert_allclose(desc, plain.descriptor[0], rtol=1e-13)
    np.testing.assert_allclose(jac, modes._dense(plain, pos.shape[0])[0], rtol=0, atol=1e-14)
    # two atoms related by a lattice translation of half the doubled cell see the same environment
    cell = np.diag([3.0, 3.2, 6.8])
    p2 = np.array([[0.1, 0.2, 0.3], [0.1, 0.2, 3.7], [1.4, 1.9, 1.2], [1.4, 1.9, 4.6]])
    z2 = np.array([8, 8, 1, 1])
    op = SoapOracle([1, 8], 3.3, 2, 3, 0.5, pbc=(True, True, True))
    np.testing.assert_allclose(modes.average_descriptor(op, mode, p2, z2, cell, [0, 1]),
                               op.descriptor(p2, z2, cell, [0])[0], rtol=1e-12)


@pytest.mark.parametrize("mode", ["inner", "outer"])
def test_averages_are_rotation_and_permutation_invariant(mode):
    st = water_cluster(3, seed=3)
    pos = st.positions.astype(np.float64)
    o = SoapOracle([1, 8], 4.0, 2, 4, 0.5)
    ref = modes.average_descriptor(o, mode, pos, st.numbers)
    R = random_rotation(np.random.default_rng(11))
    np.testing.assert_allclose(modes.average_descriptor(o, mode, pos @ R.T, st.numbers), ref, rtol=1e-10, atol=1e-12)
    perm = np.random.default_rng(0).permutation(pos.shape[0])
    np.testing.assert_allclose(modes.average_descriptor(o, mode, pos[perm], st.numbers[perm]), ref, rtol=1e-12)


# ----------------------------------------------------------------- radial weighting
WEIGHTS = [
    {"function": "poly", "r0": 3.6, "c": 1.3, "m": 2, "w0": 0.6},
    {"function": "pow", "r0": 1.5, "c": 0.8, "d": 1.2, "m": 3, "w0": 1.4},
    {"function": "exp", "r0": 0.9, "c": 2.0, "d": 0.5, "w0": 1.0},
]


def _w_plain(spec, d):
    """The three weight functions typed out once more, scalar, for the pins."""
    x = d / spec["r0"]
    if spec["function"] == "poly":
        return spec["c"] * (1 + 2 * x ** 3 - 3 * x ** 2) ** spec["m"] if x <= 1 else 0.0
    if spec["function"] == "pow":
        return spec["c"] / (spec["d"] + x ** spec["m"])
    return spec["c"] / (spec["d"] + np.exp(-x))


@pytest.mark.parametrize("spec", WEIGHTS)
@pytest.mark.parametrize("rbf", [GTO, POLYNOMIAL])
def test_weighted_coefficients_against_brute_force_projection(spec, rbf):
    """Eq. 3 by 3-D quadrature with every neighbour Gaussian of Eq. 1 scaled by w(|r_j|) and the
    centre's by w0; the radial functions come from the unweighted oracle through Eq. 3 itself:
    g_nl(r) is recovered as the projection of a delta shell, i.e. taken from `basis`."""
    from oracle import basis
    from test_oracle_soap import _scipy_real_harmonics
    r_cut, n_max, l_max, sigma = 4.0, 2, 2, 0.5
    pos = np.array([[0.0, 0.0, 0.0], [1.1, 0.7, -0.9], [-1.6, 0.4, 1.2], [0.3, -2.2, 0.8], [2.4, 2.3, 1.7]])
    numbers = np.array([1, 8, 1, 8, 1])
    o = SoapOracle([1, 8], r_cut, n_max, l_max, sigma, rbf, weighting=spec)
    c = o.coefficients(pos, numbers, None, 0)
    r_hi = r_cut + 10 * sigma if rbf == GTO else r_cut
    xr, wr = np.polynomial.legendre.leggauss(140)
    r = 0.5 * r_hi * (xr + 1)
    wr = 0.5 * r_hi * wr
    xt, wt = np.polynomial.legendre.leggauss(80)
    nphi = 160
    phi = 2 * np.pi * np.arange(nphi) / nphi
    ct, ph = np.meshgrid(xt, phi, indexing="ij")
    st = np.sqrt(1 - ct * ct)
    unit = np.stack([st * np.cos(ph), st * np.sin(ph), ct], -1)
    Yg = _scipy_real_harmonics(l_max, np.arccos(ct), ph)
    if rbf == GTO:
        alpha = basis.gto_alpha(r_cut, n_max, l_max)
        beta = basis.gto_beta(r_cut, n_max, l_max).astype(np.float64)
        g = np.array([[beta[l, n] @ (r[None, :] ** l * np.exp(-alpha[l][:, None] * r[None, :] ** 2))
                       for l in range(l_max + 1)] for n in range(n_max)])
    else:
        W = basis.poly_w(n_max).astype(np.float64)
        N = basis.poly_norm(r_cut, n_max)
        prim = np.array([(r_cut - r) ** (k + 2) / N[k - 1] for k in range(1, n_max + 1)])
        g = np.repeat((W @ prim)[:, None, :], l_max + 1, axis=1)
    ls = np.concatenate([[l] * (2 * l + 1) for l in range(l_max + 1)])
    for mu, z in enumerate([1, 8]):
        rho = np.zeros((r.size,) + ct.shape)
        for j in range(5):
            if numbers[j] != z:
                continue
            dj = np.linalg.norm(pos[j] - pos[0])
            if j != 0 and dj >= r_cut:
                continue
            wj = spec["w0"] if j == 0 else _w_plain(spec, dj)
            diff = r[:, None, None, None] * unit[None] - pos[j]
            rho += wj * np.exp(-np.sum(diff * diff, -1) / (2 * sigma ** 2))
        ang = np.einsum("mtp,rtp,t->mr", Yg, rho, wt) * (2 * np.pi / nphi)
        ref = np.einsum("nmr,mr,r->nm", g[:, ls, :], ang, wr * r * r)
        assert np.abs(c[mu] - ref).max() < 5e-9 * max(1.0, np.abs(ref).max())


@pytest.mark.parametrize("spec", WEIGHTS)
def test_weighted_jacobian_by_central_differences(spec):
    st = small_periodic_cell(seed=6, pbc=(True, True, True))
    pos = st.positions.astype(np.float64)
    o = SoapOracle([1, 6, 7, 8], 4.0, 2, 3, 0.5, GTO, pbc=st.pbc, weighting=spec)
    der = o.derivatives(pos, st.numbers, st.cell, [1, 5])
    dense = modes._dense(der, pos.shape[0])
    fd = _fd(lambda p: o.descriptor(p, st.numbers, st.cell, [1, 5]), pos)
    np.testing.assert_allclose(dense, np.transpose(fd, (2, 0, 1, 3)), rtol=0, atol=3e-8 * np.abs(dense).max())


def test_weight_that_vanishes_beyond_r0_removes_those_atoms():
    spec = {"function": "poly", "r0": 2.5, "c": 1.0, "m": 1, "w0": 1.0}
    st = water_cluster(4, seed=2)
    pos = st.positions.astype(np.float64)
    o = SoapOracle([1, 8], 5.0, 3, 3, 0.5, weighting=spec)
    near = np.nonzero(np.linalg.norm(pos - pos[0], axis=1) <= 2.5)[0]      # atom 0 itself included
    assert near.size < pos.shape[0]
    np.testing.assert_allclose(o.descriptor(pos, st.numbers, centers=[0])[0],
                               o.descriptor(pos[near], st.numbers[near], centers=[0])[0], rtol=1e-13)


def test_constant_weight_scales_the_neighbour_terms():
    st = water_cluster(3, seed=8)
    pos = st.positions.astype(np.float64)
    plain = SoapOracle([1, 8], 4.0, 2, 2, 0.5, POLYNOMIAL)
    spec = {"function": "pow", "r0": 1.0, "c": 3.0, "d": 1.0, "m": 0.0, "w0": 0.5}        # w = 3 / (1 + 1) everywhere
    weighted = SoapOracle([1, 8], 4.0, 2, 2, 0.5, POLYNOMIAL, weighting=spec)
    c0 = plain.coefficients(pos, st.numbers, None, 2)
    on = np.zeros_like(c0)
    on[plain._species_index(st.numbers)[2], :, 0] = plain.onsite()
    np.testing.assert_allclose(weighted.coefficients(pos, st.numbers, None, 2), 1.5 * (c0 - on) + 0.5 * on, rtol=1e-12)


# ----------------------------------------------------------------- centres that are not atoms
def test_site_centres_equal_a_ghost_atom_of_a_species_of_its_own():
    """A point centre sees what an atom of an otherwise absent species placed there sees, in every
    feature that does not involve that species (its own Gaussian only enters its own block)."""
    st = small_periodic_cell(seed=3, pbc=(True, True, True))
    pos = st.positions.astype(np.float64)
    sites = np.array([[0.7, 1.9, 2.2], [3.1, 0.2, 1.0]])
    o = SoapOracle([1, 6, 7, 8], 4.0, 2, 3, 0.5, pbc=st.pbc)
    got = modes.site_derivatives(o, pos, st.numbers, sites, st.cell)
    og = SoapOracle([1, 6, 7, 8, 99], 4.0, 2, 3, 0.5, pbc=st.pbc)
    keep = np.nonzero((og.table[:, 0] < 4) & (og.table[:, 1] < 4))[0]
    assert np.array_equal(og.table[keep], o.table)
    for a, site in enumerate(sites):
        p2 = np.concatenate([pos, site[None]])
        z2 = np.concatenate([st.numbers, [99]])
        ref = og.derivatives(p2, z2, st.cell, [len(pos)])
        np.testing.assert_allclose(got.descriptor[a], ref.descriptor[0][keep], rtol=1e-12, atol=1e-15)
        rows = slice(got.row_ptr[a], got.row_ptr[a + 1])
        real = ref.row_atom < len(pos)                                  # the ghost's own row has no counterpart
        assert np.array_equal(got.row_atom[rows], ref.row_atom[real])
        np.testing.assert_allclose(got.jacobian[rows], ref.jacobian[real][:, :, keep], rtol=1e-11, atol=1e-14)


def test_site_jacobian_by_central_differences():
    st = water_cluster(3, seed=4)
    pos = st.positions.astype(np.float64)
    sites = np.array([[0.3, -0.4, 0.9]])
    o = SoapOracle([1, 8], 4.5, 3, 3, 0.5, POLYNOMIAL)
    der = modes.site_derivatives(o, pos, st.numbers, sites)
    dense = modes._dense(der, pos.shape[0])
    fd = _fd(lambda p: modes.site_derivatives(o, p, st.numbers, sites).descriptor, pos)
    np.testing.assert_allclose(dense, np.transpose(fd, (2, 0, 1, 3)), rtol=0, atol=3e-8 * np.abs(dense).max())


# ----------------------------------------------------------------- many independent structures
def test_batch_equals_one_structure_with_the_parts_far_apart():
    a, b, c = water_cluster(2, seed=1), water_cluster(3, seed=2), water_cluster(1, seed=3)
    o = SoapOracle([1, 8], 4.0, 2, 2, 0.5)
    parts = [(s.positions.astype(np.float64), s.numbers) for s in (a, b, c)]
    got = modes.batch_derivatives(o, parts)
    merged = np.concatenate([parts[0][0], parts[1][0] + [100.0, 0, 0], parts[2][0] + [0, -200.0, 50.0]])
    ref = o.derivatives(merged, np.concatenate([p[1] for p in parts]))
    assert np.array_equal(got.row_ptr, ref.row_ptr) and np.array_equal(got.row_atom, ref.row_atom)
    np.testing.assert_allclose(got.descriptor, ref.descriptor, rtol=1e-10, atol=1e-13)
    np.testing.assert_allclose(got.jacobian, ref.jacobian, rtol=0, atol=1e-10 * np.abs(ref.jacobian).max())

"""Parity of the other output modes (crossover off, coefficient mode, inner and outer averages)
against the fp64 oracle, on a GPU through the C ABI.

Tolerances per output column, relative to the column's largest oracle value and floored at 1e-8:
values (descriptor, coefficients) <= 1e-5, Jacobians <= 1e-4; row lists identical.  An averaged
descriptor is a single row whose entries can be small through cancellation between centres: its
scale per feature is the largest per-centre value of that feature.
"""
import numpy as np
import pytest

from oracle import modes
from oracle.soap import GTO, POLYNOMIAL, SoapOracle
from soap_inputs import multispecies_box, small_periodic_cell, water_cluster
from test_gpu_parity import DESC_TOL, JAC_TOL, check_derivatives, col_err, dev, same_values

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def pkg():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import paper_2609_05709_b200 as p
    p.load_library()
    return p


@pytest.mark.parametrize("case", ["water", "chno_poly", "periodic", "nch_not_multiple_of_8"])
def test_crossover_off(pkg, case):
    if case == "water":
        s, args = water_cluster(20, 3), ([1, 8], 6.0, 8, 6, 0.5, GTO)
    elif case == "chno_poly":
        s, args = multispecies_box(120, 2), ([1, 6, 7, 8], 4.0, 6, 4, 0.4, POLYNOMIAL, (True, True, True))
    elif case == "periodic":
        s, args = small_periodic_cell(1, (True, True, False)), ([1, 6, 7, 8], 4.5, 3, 3, 0.5, GTO, (True, True, False))
    else:
        s, args = water_cluster(10, 8), ([1, 8], 5.0, 5, 2, 0.5, GTO)
    pbc = args[6] if len(args) > 6 else (False, False, False)
    soap = pkg.Soap(*args[:6], pbc, crossover=False)
    oracle = SoapOracle(*args[:6], pbc, crossover=False)
    S, n, L1 = len(args[0]), args[2], args[3] + 1
    assert soap.n_features == oracle.n_features == S * (n * (n + 1) // 2) * L1
    for f in (0, soap.n_features // 2, soap.n_features - 1):
        assert soap.feature_info(f) == tuple(int(v) for v in oracle.table[f])
    sample = None if s.n_atoms <= 40 else [0, 7, s.n_atoms // 2, s.n_atoms - 1]
    check_derivatives(soap, oracle, s, sample=sample)


def test_crossover_can_be_switched_on_a_live_handle(pkg):
    s = water_cluster(6, 2)
    pos, num = dev(s)
    soap = pkg.Soap([1, 8], 5.0, 4, 3, 0.5, GTO)
    full = soap.descriptor(pos, num).cpu().numpy()
    soap._check(soap._lib.soap_set_crossover(soap._h, 0))
    oracle = SoapOracle([1, 8], 5.0, 4, 3, 0.5, GTO)
    keep = np.nonzero(oracle.table[:, 0] == oracle.table[:, 1])[0]
    diag = torch.empty((s.n_atoms, keep.size), dtype=torch.float32, device="cuda")
    soap.n_features = keep.size
    soap.descriptor(pos, num, out=diag)
    soap.status()
    assert np.array_equal(diag.cpu().numpy(), full[:, keep])


@pytest.mark.parametrize("case", ["water", "periodic_poly", "large_l"])
def test_coefficient_mode(pkg, case):
    if case == "water":
        s, args = water_cluster(15, 6), ([1, 8], 6.0, 8, 6, 0.5, GTO)
    elif case == "periodic_poly":
        s, args = small_periodic_cell(3, (True, True, True)), ([1, 6, 7, 8], 4.5, 3, 3, 0.5, POLYNOMIAL, (True, True, True))
    else:
        s, args = water_cluster(8, 1), ([1, 8], 5.0, 3, 9, 0.5, GTO)
    soap, oracle = pkg.Soap(*args), SoapOracle(*args)
    assert soap.n_coefficients == modes.coefficient_width(oracle)
    pos, num = dev(s)
    ref = modes.coefficient_derivatives(oracle, s.positions, s.numbers, s.cell)
    c = soap.coefficients(pos, num, s.cell).cpu().numpy()
    soap.status()
    assert col_err(c, ref.descriptor, 0) < DESC_TOL
    out = soap.coefficient_derivatives(pos, num, s.cell)
    assert np.array_equal(out.row_ptr.cpu().numpy(), ref.row_ptr)
    assert np.array_equal(out.row_atom.cpu().numpy(), ref.row_atom)
    assert same_values(out.descriptor, c)
    jac = out.jacobian.cpu().numpy()
    assert col_err(jac, ref.jacobian, (0, 1)) < JAC_TOL
    # blocks of foreign species are exact zeros, written explicitly
    assert np.all(jac[ref.jacobian == 0] == 0)


def test_coefficient_mode_centre_subset_into_poisoned_buffers(pkg):
    s = water_cluster(10, 7)
    args = ([1, 8], 4.5, 4, 4, 0.5, GTO)
    soap, oracle = pkg.Soap(*args), SoapOracle(*args)
    pos, num = dev(s)
    centers = [5, 0, 29, 11]
    cen = torch.tensor(centers, dtype=torch.int32).cuda()
    ref = modes.coefficient_derivatives(oracle, s.positions, s.numbers, None, centers)
    # every element of the result is written, whatever the buffers held before
    filler = torch.full((1 << 22,), float("nan"), device="cuda")      # the allocator hands this memory out again
    del filler
    out = soap.coefficient_derivatives(pos, num, None, cen)
    assert np.array_equal(out.row_atom.cpu().numpy(), ref.row_atom)
    assert not torch.isnan(out.jacobian).any() and not torch.isnan(out.descriptor).any()
    assert col_err(out.jacobian.cpu().numpy(), ref.jacobian, (0, 1)) < JAC_TOL


@pytest.mark.parametrize("mode", ["inner", "outer"])
@pytest.mark.parametrize("case", ["water", "periodic_poly", "subset", "wide_rows", "large_basis"])
def test_averaged_modes(pkg, mode, case):
    centers = None
    if case == "water":
        s, args = water_cluster(12, 4), ([1, 8], 5.0, 6, 4, 0.5, GTO)
    elif case == "wide_rows":
        # more features that involve one species than a thread of the outer-average kernel keeps in registers;
        # a 4 A cell with r_cut 4 A: every atom also sees images of itself
        s, args = small_periodic_cell(2), ([1, 6, 7, 8], 4.0, 8, 4, 0.5, POLYNOMIAL, (True, True, True))
    elif case == "large_basis":
        # the coefficients of a centre are too many for the shared memory of the outer-average kernel: general path
        s, args = water_cluster(4, 6), ([1, 8, 9], 4.5, 12, 12, 0.5, GTO)
    elif case == "periodic_poly":
        s, args = small_periodic_cell(5, (True, False, True)), ([1, 6, 7, 8], 4.5, 3, 3, 0.5, POLYNOMIAL, (True, False, True))
    else:
        s, args = water_cluster(12, 9), ([1, 8], 4.0, 4, 5, 0.5, GTO)
        s.positions = np.concatenate([s.positions, np.array([[60.0, 0, 0]], np.float32)])    # an atom in no sphere
        s.numbers = np.concatenate([s.numbers, np.array([1], np.int32)])
        centers = [3, 0, 20, 35, 8]
    soap, oracle = pkg.Soap(*args), SoapOracle(*args)
    pos, num = dev(s)
    cen = None if centers is None else torch.tensor(centers, dtype=torch.int32).cuda()
    ref_desc, ref_jac = modes.average_derivatives(oracle, mode, s.positions, s.numbers, s.cell, centers)
    d1 = soap.descriptor_average(mode, pos, num, s.cell, cen).cpu().numpy()
    soap.status()
    scale = np.maximum(np.abs(oracle.descriptor(s.positions, s.numbers, s.cell, centers)).max(axis=0), 1e-8)
    assert (np.abs(d1 - ref_desc) / scale).max() < DESC_TOL
    out_jac = torch.full((s.n_atoms, 3, soap.n_features), float("nan"), device="cuda")
    d2, jac = soap.derivatives_average(mode, pos, num, s.cell, cen, out_jac=out_jac)
    soap.status()
    assert (np.abs(d2.cpu().numpy() - ref_desc) / scale).max() < DESC_TOL
    jac = jac.cpu().numpy()
    assert not np.isnan(jac).any()
    assert col_err(jac, ref_jac, (0, 1)) < JAC_TOL
    if case == "subset":
        assert np.all(jac[-1] == 0)
    # fixed summation order: a second call gives the same bits
    d3, jac3 = soap.derivatives_average(mode, pos, num, s.cell, cen)
    soap.status()
    assert np.array_equal(jac3.cpu().numpy(), jac) and np.array_equal(d3.cpu().numpy(), d2.cpu().numpy())


def test_averaged_modes_many_centres_per_atom(pkg):
    """More centres hold one atom than the reduction lists at a time (1024): a dense blob."""
    rng = np.random.default_rng(3)
    n = 1300
    p = rng.random((n, 3)) * 7.0
    from soap_inputs import Structure
    s = Structure(p.astype(np.float32), np.where(rng.random(n) < 0.5, 1, 8).astype(np.int32), None, (False, False, False))
    args = ([1, 8], 14.0, 1, 1, 0.5, POLYNOMIAL)
    soap, oracle = pkg.Soap(*args), SoapOracle(*args)
    pos, num = dev(s)
    _, jac = soap.derivatives_average("outer", pos, num)
    soap.status()
    # the oracle on all 1300 centres costs too much: per-centre rows from the plain entry point
    # (itself checked against the oracle elsewhere), averaged here in fp64
    der = soap.derivatives(pos, num)
    rows = der.jacobian.cpu().numpy().astype(np.float64)
    acc = np.zeros((n, 3, soap.n_features))
    np.add.at(acc, der.row_atom.cpu().numpy(), rows)
    assert col_err(jac.cpu().numpy(), acc / n, (0, 1)) < 1e-5


def test_average_argument_errors(pkg):
    s = water_cluster(2, 0)
    pos, num = dev(s)
    soap = pkg.Soap([1, 8], 4.0, 2, 2, 0.5, GTO)
    empty = torch.empty(0, dtype=torch.int32, device="cuda")
    with pytest.raises(pkg.SoapError, match="at least one centre"):
        soap.descriptor_average("inner", pos, num, None, empty)
    out = torch.empty(soap.n_features, device="cuda")
    rc = soap._lib.soap_descriptor_average(soap._h, 7, pos.data_ptr(), num.data_ptr(), 6, None, None, 6, out.data_ptr(), None)
    assert rc == -1


# ----------------------------------------------------------------- radial weighting
WEIGHTS = [
    {"function": "poly", "r0": 4.2, "c": 1.3, "m": 2, "w0": 0.6},
    {"function": "poly", "r0": 3.1, "c": 1.0, "m": 1, "w0": 1.0},       # cuts inside the sphere, kink in w'' at r0
    {"function": "pow", "r0": 1.5, "c": 0.8, "d": 1.2, "m": 3, "w0": 1.4},
    {"function": "exp", "r0": 0.9, "c": 2.0, "d": 0.5, "w0": 1.0},
]


@pytest.mark.parametrize("spec", WEIGHTS)
@pytest.mark.parametrize("case", ["water_gto", "periodic_poly"])
def test_radial_weighting(pkg, spec, case):
    if case == "water_gto":
        s, args = water_cluster(15, 2), ([1, 8], 5.0, 6, 5, 0.5, GTO, (False, False, False))
    else:
        s, args = small_periodic_cell(7, (True, True, True)), ([1, 6, 7, 8], 4.5, 3, 3, 0.5, POLYNOMIAL, (True, True, True))
    soap = pkg.Soap(*args, weighting=spec)
    oracle = SoapOracle(*args, weighting=spec)
    check_derivatives(soap, oracle, s)
    pos, num = dev(s)
    ref = modes.coefficient_derivatives(oracle, s.positions, s.numbers, s.cell)
    out = soap.coefficient_derivatives(pos, num, s.cell)
    assert col_err(out.descriptor.cpu().numpy(), ref.descriptor, 0) < DESC_TOL
    assert col_err(out.jacobian.cpu().numpy(), ref.jacobian, (0, 1)) < JAC_TOL


def test_weighting_can_be_switched_on_a_live_handle(pkg):
    s = water_cluster(10, 5)
    pos, num = dev(s)
    args = ([1, 8], 5.0, 4, 4, 0.5, GTO)
    soap = pkg.Soap(*args)
    plain = soap.derivatives(pos, num)
    spec = WEIGHTS[0]
    soap._check(soap._lib.soap_set_weighting(soap._h, 1, spec["r0"], spec["c"], 1.0, float(spec["m"]), spec["w0"]))
    check_derivatives(soap, SoapOracle(*args, weighting=spec), s)
    soap._check(soap._lib.soap_set_weighting(soap._h, 0, 0.0, 0.0, 0.0, 0.0, 0.0))
    again = soap.derivatives(pos, num)
    assert torch.equal(again.jacobian, plain.jacobian) and torch.equal(again.descriptor, plain.descriptor)
    with pytest.raises(pkg.SoapError, match="r0 > 0"):
        soap._check(soap._lib.soap_set_weighting(soap._h, 2, -1.0, 1.0, 1.0, 1.0, 1.0))


# ----------------------------------------------------------------- centres that are not atoms
@pytest.mark.parametrize("case", ["water_gto", "periodic_poly_weighted"])
def test_centres_at_arbitrary_points(pkg, case):
    rng = np.random.default_rng(12)
    if case == "water_gto":
        s, args, kw = water_cluster(20, 4), ([1, 8], 5.0, 6, 4, 0.5, GTO, (False, False, False)), {}
        lo, hi = s.positions.min(axis=0), s.positions.max(axis=0)
        sites = lo + rng.random((9, 3)) * (hi - lo)
        sites[0] = hi + 2.0                # outside the bounding box of the atoms, still within reach
        sites[1] = lo - 30.0               # sees nothing
    else:
        s, args = small_periodic_cell(9, (True, True, True)), ([1, 6, 7, 8], 4.5, 3, 3, 0.5, POLYNOMIAL, (True, True, True))
        kw = {"weighting": {"function": "poly", "r0": 4.0, "c": 1.0, "m": 2, "w0": 1.0}}
        sites = rng.random((6, 3)) * 12.0 - 4.0                       # several cells away as well
    sites = sites.astype(np.float32)
    soap, oracle = pkg.Soap(*args, **kw), SoapOracle(*args, **kw)
    pos, num = dev(s)
    ref = modes.site_derivatives(oracle, s.positions, s.numbers, sites, s.cell)
    out = soap.derivatives_at(pos, num, torch.from_numpy(sites).cuda(), s.cell)
    assert np.array_equal(out.row_ptr.cpu().numpy(), ref.row_ptr)
    assert np.array_equal(out.row_atom.cpu().numpy(), ref.row_atom)
    assert col_err(out.descriptor.cpu().numpy(), ref.descriptor, 0) < DESC_TOL
    assert col_err(out.jacobian.cpu().numpy(), ref.jacobian, (0, 1)) < JAC_TOL
    d = soap.derivatives_at(pos, num, torch.from_numpy(sites).cuda(), s.cell, jacobian=False)
    assert same_values(d, out.descriptor)
    if case == "water_gto":
        assert np.all(out.descriptor[1].cpu().numpy() == 0) and ref.row_ptr[2] == ref.row_ptr[1]
    # the same handle still serves atom centres afterwards
    check_derivatives(soap, oracle, s, sample=[0, 3])


# ----------------------------------------------------------------- species-compact Jacobian rows
@pytest.mark.parametrize("case", ["water", "chno_periodic", "crossover_off", "one_species"])
def test_species_compact_rows(pkg, case):
    kw = {}
    if case == "water":
        s, args = water_cluster(25, 6), ([1, 8], 6.0, 8, 6, 0.5, GTO)
    elif case == "chno_periodic":
        s, args = small_periodic_cell(4, (True, True, True)), ([1, 6, 7, 8], 4.5, 3, 3, 0.5, POLYNOMIAL, (True, True, True))
    elif case == "crossover_off":
        s, args, kw = water_cluster(10, 3), ([1, 8], 5.0, 5, 2, 0.5, GTO, (False, False, False)), {"crossover": False}
    else:
        s, args = water_cluster(6, 1), ([8], 5.0, 4, 3, 0.5, GTO)
        s.numbers[:] = 8
    soap, oracle = pkg.Soap(*args, **kw), SoapOracle(*args, **kw)
    S = len(args[0])
    tri = args[2] * (args[2] + 1) // 2 * (args[3] + 1)
    cross = args[2] * args[2] * (args[3] + 1)
    assert soap.n_compact == tri + (0 if case == "crossover_off" else (S - 1) * cross)
    assert soap.compact_pitch % 8 == 0 and 0 <= soap.compact_pitch - soap.n_compact < 8
    pos, num = dev(s)
    sample = list(range(s.n_atoms)) if s.n_atoms <= 30 else [0, 5, 31, s.n_atoms - 1]
    cen = torch.tensor(sample, dtype=torch.int32).cuda()
    ref = oracle.derivatives(s.positions, s.numbers, s.cell, sample)
    comp = soap.derivatives_compact(pos, num, s.cell, cen)
    assert np.array_equal(comp.row_ptr.cpu().numpy(), ref.row_ptr)
    assert np.array_equal(comp.row_atom.cpu().numpy(), ref.row_atom)
    assert col_err(comp.descriptor.cpu().numpy(), ref.descriptor, 0) < DESC_TOL
    # compact columns against the oracle through the column map, row by row; everything the
    # compact format leaves out is an exact zero in the oracle's row
    jac = comp.jacobian.cpu().numpy()
    own = comp.center_rows.cpu().numpy()
    sp = oracle._species_index(s.numbers)
    maps = [soap.compact_feature_map(z) for z in range(S)]
    full = np.zeros_like(ref.jacobian)
    for a, i in enumerate(sample):
        for r in range(ref.row_ptr[a], ref.row_ptr[a + 1]):
            atom = ref.row_atom[r]
            if atom == i:
                full[r] = own[a]
                assert np.all(jac[r] == 0)
                continue
            m = maps[sp[atom]]
            assert np.all(np.delete(ref.jacobian[r], m, axis=1) == 0)
            full[r][:, m] = jac[r][:, :soap.n_compact]
            assert np.all(jac[r][:, soap.n_compact:] == 0)
    assert col_err(full, ref.jacobian, (0, 1)) < JAC_TOL
    # the expansion kernel gives the same rows; the dense entry point (another instantiation of the
    # kernel, so not necessarily the same bits) agrees far inside the tolerance
    exp = soap.compact_expand(num, cen, comp)
    soap.status()
    assert np.array_equal(exp.cpu().numpy(), full)
    dense = soap.derivatives(pos, num, s.cell, cen)
    assert col_err(dense.jacobian.cpu().numpy(), full.astype(np.float64), (0, 1)) < 1e-5


def test_new_entry_points_with_empty_inputs_and_null_pointers(pkg):
    s = water_cluster(3, 0)
    pos, num = dev(s)
    soap = pkg.Soap([1, 8], 4.0, 2, 2, 0.5, GTO)
    none = torch.empty(0, dtype=torch.int32, device="cuda")
    assert soap.coefficients(pos, num, None, none).shape == (0, soap.n_coefficients)
    out = soap.coefficient_derivatives(pos, num, None, none)
    assert out.jacobian.shape[0] == 0 and out.row_ptr.cpu().tolist() == [0]
    comp = soap.derivatives_compact(pos, num, None, none)
    assert comp.jacobian.shape[0] == 0 and comp.row_ptr.cpu().tolist() == [0]
    sites = torch.empty((0, 3), dtype=torch.float32, device="cuda")
    at = soap.derivatives_at(pos, num, sites)
    assert at.jacobian.shape[0] == 0 and at.descriptor.shape == (0, soap.n_features)
    # an empty structure seen from a point: no neighbours, zero descriptor
    nopos, nonum = torch.empty((0, 3), device="cuda"), torch.empty(0, dtype=torch.int32, device="cuda")
    one = torch.zeros((1, 3), dtype=torch.float32, device="cuda")
    d = soap.derivatives_at(nopos, nonum, one)
    assert d.jacobian.shape[0] == 0 and torch.all(d.descriptor == 0)
    # NULL outputs are refused before any launch
    n = s.n_atoms
    lib, h = soap._lib, soap._h
    assert lib.soap_coefficients(h, pos.data_ptr(), num.data_ptr(), n, None, None, n, None, None) == -1
    assert lib.soap_descriptor_at(h, pos.data_ptr(), num.data_ptr(), n, None, None, 2, None, None) == -1
    assert lib.soap_derivatives_compact(h, pos.data_ptr(), num.data_ptr(), n, None, None, n, pos.data_ptr(), None,
                                        pos.data_ptr(), 0, pos.data_ptr(), pos.data_ptr(), None) == -1
    assert lib.soap_derivatives_average(h, 1, pos.data_ptr(), num.data_ptr(), n, None, None, n, None, None, None) == -1
    soap.status()


# ----------------------------------------------------------------- the modes at the benchmark's full sizes
def test_modes_at_full_size_sampled(pkg):
    """The configurations `bench.py --suite modes|compact` times (1000-molecule cluster, every centre on
    the GPU), checked on sampled centres the oracle computes one by one."""
    s = water_cluster(1000, 0)
    args = ([1, 8], 6.0, 8, 6, 0.5, GTO)
    soap, oracle = pkg.Soap(*args), SoapOracle(*args)
    pos, num = dev(s)
    sample = [0, 1, 1500, 2999] + list(range(77, 3000, 487))
    sp = oracle._species_index(s.numbers)
    # species-compact rows of all 3000 centres
    comp = soap.derivatives_compact(pos, num)
    ref = oracle.derivatives(s.positions, s.numbers, None, sample)
    row_ptr, row_atom = comp.row_ptr.cpu().numpy(), comp.row_atom.cpu().numpy()
    maps = [soap.compact_feature_map(z) for z in range(2)]
    got = []
    for b, a in enumerate(sample):
        lo, hi = row_ptr[a], row_ptr[a + 1]
        assert np.array_equal(row_atom[lo:hi], ref.row_atom[ref.row_ptr[b]:ref.row_ptr[b + 1]])
        rows = comp.jacobian[lo:hi].cpu().numpy()
        full = np.zeros((hi - lo, 3, soap.n_features), np.float32)
        for r in range(hi - lo):
            atom = row_atom[lo + r]
            if atom == a:
                full[r] = comp.center_rows[a].cpu().numpy()
            else:
                full[r][:, maps[sp[atom]]] = rows[r][:, :soap.n_compact]
        got.append(full)
    assert col_err(np.concatenate(got), ref.jacobian, (0, 1)) < JAC_TOL
    assert col_err(comp.descriptor.cpu().numpy()[sample], ref.descriptor, 0) < DESC_TOL
    del comp
    # coefficient mode of all 3000 centres
    out = soap.coefficient_derivatives(pos, num)
    cref = modes.coefficient_derivatives(oracle, s.positions, s.numbers, None, sample)
    row_ptr = out.row_ptr.cpu().numpy()
    got = [out.jacobian[row_ptr[a]:row_ptr[a + 1]].cpu().numpy() for a in sample]
    assert col_err(np.concatenate(got), cref.jacobian, (0, 1)) < JAC_TOL
    assert col_err(out.descriptor.cpu().numpy()[sample], cref.descriptor, 0) < DESC_TOL
    del out
    # outer average over all centres: equals the mean of the per-centre results of the plain entry point
    # (themselves checked against the oracle at this size in test_gpu_parity.py), in fp64
    d, jac = soap.derivatives_average("outer", pos, num)
    plain = soap.derivatives(pos, num)
    acc = torch.zeros((3000, 3, soap.n_features), dtype=torch.float64, device="cuda")
    acc.index_add_(0, plain.row_atom.long(), plain.jacobian.double())
    want = (acc / 3000).cpu().numpy()
    assert col_err(jac.cpu().numpy(), want, (0, 1)) < 1e-5
    assert col_err(d.cpu().numpy()[None], plain.descriptor.double().mean(dim=0).cpu().numpy()[None], 0) < 1e-5


# ----------------------------------------------------------------- many independent structures in one call
@pytest.mark.parametrize("rbf", [GTO, POLYNOMIAL])
def test_batch_of_structures(pkg, rbf):
    rng = np.random.default_rng(21)
    parts = []
    for k, n_mol in enumerate([1, 8, 2, 5, 3, 12]):
        s = water_cluster(n_mol, 40 + k)
        parts.append((s.positions + rng.uniform(-3, 3, size=3).astype(np.float32), s.numbers))
    parts.insert(2, (np.array([[0.3, 0.1, -0.2]], np.float32), np.array([8], np.int32)))        # a lone atom
    parts.insert(4, (np.zeros((0, 3), np.float32), np.zeros(0, np.int32)))                      # an empty structure
    args = ([1, 8], 4.5, 4, 3, 0.5, rbf)
    soap, oracle = pkg.Soap(*args), SoapOracle(*args)
    ref = modes.batch_derivatives(oracle, parts)
    pos = torch.from_numpy(np.concatenate([p[0] for p in parts])).cuda()
    num = torch.from_numpy(np.concatenate([p[1] for p in parts])).cuda()
    ptr = torch.tensor(np.concatenate([[0], np.cumsum([len(p[1]) for p in parts])]), dtype=torch.int64).cuda()
    out = soap.derivatives_batch(pos, num, ptr)
    assert np.array_equal(out.row_ptr.cpu().numpy(), ref.row_ptr)
    assert np.array_equal(out.row_atom.cpu().numpy(), ref.row_atom)
    assert col_err(out.descriptor.cpu().numpy(), ref.descriptor, 0) < DESC_TOL
    assert col_err(out.jacobian.cpu().numpy(), ref.jacobian, (0, 1)) < JAC_TOL
    d = soap.derivatives_batch(pos, num, ptr, jacobian=False)
    assert same_values(d, out.descriptor)
    # each structure on its own through the ordinary entry point gives the same bits
    lo = int(ptr[1])
    single = soap.derivatives(pos[lo:int(ptr[2])].contiguous(), num[lo:int(ptr[2])].contiguous())
    assert torch.equal(single.descriptor, out.descriptor[lo:int(ptr[2])])
    # a periodic handle refuses batches
    per = pkg.Soap([1, 8], 4.5, 2, 2, 0.5, GTO, (True, False, False))
    with pytest.raises(pkg.SoapError, match="non-periodic"):
        per.derivatives_batch(pos, num, ptr)

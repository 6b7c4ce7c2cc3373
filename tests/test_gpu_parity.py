"""Parity of the CUDA path (through the C ABI) against the fp64 oracle, on a GPU.

Tolerances (per feature column, floored at 1e-8 absolute):
  neighbour lists identical as sets (and in order); descriptor <= 1e-5; Jacobian <= 1e-4.
"""
import numpy as np
import pytest

from oracle.soap import GTO, POLYNOMIAL, SoapOracle
from soap_inputs import multispecies_box, small_periodic_cell, water_cluster

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

DESC_TOL, JAC_TOL = 1e-5, 1e-4


@pytest.fixture(scope="module")
def pkg():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import paper_2609_05709_b200 as p
    p.load_library()
    return p


def col_err(a, ref, axes):
    a = np.asarray(a, np.float64)
    return float((np.abs(a - ref).max(axis=axes) / np.maximum(np.abs(ref).max(axis=axes), 1e-8)).max())


def same_values(a, b, tol=DESC_TOL):
    """Two builds of the same quantity by different kernels (the descriptor-only build has a kernel of its own,
    with another order of summation and a value table of its own): both are fp32, so they are compared column by
    column within the parity tolerance with the column scale floored at 1e-3 of the largest entry (a column that
    is tiny next to the quantities it is computed from carries the rounding of those), not bit for bit.  Each
    side is checked against the oracle with the stated metric elsewhere."""
    a = a.detach().cpu().numpy() if hasattr(a, "detach") else np.asarray(a)
    b = b.detach().cpu().numpy() if hasattr(b, "detach") else np.asarray(b)
    if a.shape != b.shape:
        return False
    a2, b2 = a.reshape(-1, a.shape[-1]).astype(np.float64), b.reshape(-1, b.shape[-1]).astype(np.float64)
    if a2.size == 0:
        return True
    scale = np.maximum(np.abs(b2).max(axis=0), max(1e-3 * float(np.abs(b2).max()), 1e-8))
    return float((np.abs(a2 - b2).max(axis=0) / scale).max()) < tol


def dev(struct):
    return torch.from_numpy(struct.positions).cuda(), torch.from_numpy(struct.numbers).cuda()


def check_neighbors(soap, oracle, struct, centers=None):
    pos, num = dev(struct)
    cen = None if centers is None else torch.tensor(centers, dtype=torch.int32).cuda()
    ptr, atom, shift = soap.neighbor_list(pos, num, struct.cell, cen)
    ptr, atom, shift = ptr.cpu().numpy(), atom.cpu().numpy(), shift.cpu().numpy()
    ref = oracle.neighbor_list(struct.positions, struct.cell, centers)
    assert ptr[0] == 0 and len(ptr) == len(ref) + 1
    for a, lst in enumerate(ref):
        got = [(int(atom[e]), int(shift[e, 0]), int(shift[e, 1]), int(shift[e, 2])) for e in range(ptr[a], ptr[a + 1])]
        assert got == lst, f"centre {a}"


def check_derivatives(soap, oracle, struct, centers=None, sample=None):
    """GPU computes every requested centre; the oracle the sampled ones."""
    pos, num = dev(struct)
    cen = None if centers is None else torch.tensor(centers, dtype=torch.int32).cuda()
    out = soap.derivatives(pos, num, struct.cell, cen)
    all_centers = list(range(struct.n_atoms)) if centers is None else list(centers)
    which = list(range(len(all_centers))) if sample is None else list(sample)
    ref = oracle.derivatives(struct.positions, struct.numbers, struct.cell, [all_centers[a] for a in which])
    row_ptr = out.row_ptr.cpu().numpy()
    row_atom = out.row_atom.cpu().numpy()
    desc = out.descriptor.cpu().numpy()
    got_rows, got_desc = [], []
    for b, a in enumerate(which):
        lo, hi = row_ptr[a], row_ptr[a + 1]
        assert hi - lo == ref.row_ptr[b + 1] - ref.row_ptr[b]
        assert np.array_equal(row_atom[lo:hi], ref.row_atom[ref.row_ptr[b]:ref.row_ptr[b + 1]])
        got_rows.append(out.jacobian[lo:hi].cpu().numpy())
        got_desc.append(desc[a])
    ed = col_err(np.stack(got_desc), ref.descriptor, 0)
    ej = col_err(np.concatenate(got_rows), ref.jacobian, (0, 1))
    assert ed < DESC_TOL, f"descriptor error {ed:.3e}"
    assert ej < JAC_TOL, f"Jacobian error {ej:.3e}"
    # descriptor-only entry point gives the same rows
    d2 = soap.descriptor(pos, num, struct.cell, cen)
    soap.status()
    assert col_err(d2.cpu().numpy()[which], ref.descriptor, 0) < DESC_TOL
    return ed, ej


def test_config1_tiny_water_cluster(pkg):
    s = water_cluster(8, 0)
    args = ([1, 8], 5.0, 4, 3, 0.5, GTO)
    soap, oracle = pkg.Soap(*args), SoapOracle(*args)
    check_neighbors(soap, oracle, s)
    check_derivatives(soap, oracle, s)


@pytest.mark.parametrize("rbf", [GTO, POLYNOMIAL])
@pytest.mark.parametrize("pbc", [(True, True, True), (True, False, True), (False, False, False)])
def test_small_triclinic_cell_many_images(pkg, rbf, pbc):
    s = small_periodic_cell(0, pbc)
    args = ([1, 6, 7, 8], 4.5, 3, 3, 0.5, rbf, pbc)
    soap, oracle = pkg.Soap(*args), SoapOracle(*args)
    check_neighbors(soap, oracle, s)
    check_derivatives(soap, oracle, s)


def test_centre_subset_and_isolated_atoms(pkg):
    s = water_cluster(8, 4)
    s.positions = np.concatenate([s.positions, np.array([[40.0, 0, 0], [0, -55.0, 3]], np.float32)])
    s.numbers = np.concatenate([s.numbers, np.array([8, 1], np.int32)])
    args = ([8, 1], 3.5, 3, 4, 0.4, POLYNOMIAL)
    soap, oracle = pkg.Soap(*args), SoapOracle(*args)
    centers = [25, 3, 24, 0, 17]
    check_neighbors(soap, oracle, s, centers)
    check_derivatives(soap, oracle, s, centers)


@pytest.mark.parametrize("n_max,l_max", [(2, 2), (6, 4), (8, 6), (10, 8), (12, 12), (1, 0), (5, 9), (14, 2), (16, 1), (3, 11)])
def test_basis_size_sweep_small_cluster(pkg, n_max, l_max):
    s = water_cluster(12, 5)
    args = ([1, 8], 6.0, n_max, l_max, 0.5, GTO)
    soap, oracle = pkg.Soap(*args), SoapOracle(*args)
    check_derivatives(soap, oracle, s, sample=[0, 7, 20, 35])


@pytest.mark.parametrize("r_cut,n_max,l_max", [(9.0, 4, 3), (12.5, 2, 2)])
def test_large_neighbourhoods(pkg, r_cut, n_max, l_max):
    """Several hundred neighbours per centre (the paper's own runs use r_cut = 10 A): more pairs than
    one geometry batch of the per-centre kernel holds, and (at 12.5 A) more than the neighbour sort
    keeps in shared memory."""
    s = water_cluster(600, 7)
    args = ([1, 8], r_cut, n_max, l_max, 0.5, GTO)
    soap, oracle = pkg.Soap(*args), SoapOracle(*args)
    inner = np.argsort(np.linalg.norm(s.positions, axis=1))          # centres deep inside the cluster first
    sample = [int(inner[0]), int(inner[5]), 0, 1799]
    lists = oracle.neighbor_list(s.positions, None, sample)
    assert max(len(l) for l in lists) > (512 if r_cut > 12 else 128)
    check_neighbors(soap, oracle, s, sample)
    check_derivatives(soap, oracle, s, sample=sample)


def test_eight_species(pkg):
    rng = np.random.Generator(np.random.PCG64(3))
    s = water_cluster(20, 9)
    s.numbers = np.array([1, 6, 7, 8, 9, 15, 16, 17], np.int32)[rng.integers(0, 8, s.n_atoms)].astype(np.int32)
    args = ([17, 1, 6, 7, 8, 9, 15, 16], 4.5, 3, 2, 0.5, POLYNOMIAL)
    soap, oracle = pkg.Soap(*args), SoapOracle(*args)
    check_derivatives(soap, oracle, s, sample=[0, 13, 31, 59])


def test_config2_water_1000_sampled(pkg):
    s = water_cluster(1000, 0)
    args = ([1, 8], 6.0, 8, 6, 0.5, GTO)
    soap, oracle = pkg.Soap(*args), SoapOracle(*args)
    sample = [0, 1, 2, 777, 1500, 2998, 2999] + list(range(100, 3000, 233))
    check_neighbors(soap, oracle, s, sample)
    check_derivatives(soap, oracle, s, sample=sample)
    # whole-output properties at full size: translation sum rule per centre
    pos, num = dev(s)
    out = soap.derivatives(pos, num)
    seg = torch.repeat_interleave(torch.arange(3000, device="cuda"), out.row_ptr[1:] - out.row_ptr[:-1])
    sums = torch.zeros((3000, 3, soap.n_features), device="cuda", dtype=torch.float64)
    sums.index_add_(0, seg, out.jacobian.double())
    scale = out.jacobian.abs().amax(dim=(0, 1)).double().clamp_min(1e-8)
    assert float((sums.abs().amax(dim=(0, 1)) / scale).max()) < 1e-4
    assert torch.isfinite(out.jacobian).all() and torch.isfinite(out.descriptor).all()


class ColumnError:
    """Accumulates, chunk by chunk, the per-column figures of the tolerance metric: largest |error| and largest
    |reference| of every output column, plus element-wise |error| / column scale for the quantiles."""

    def __init__(self, width):
        self.err = np.zeros(width)
        self.ref = np.zeros(width)
        self.samples = []

    def add(self, got, ref, axes, rng):
        got = np.asarray(got, np.float64)
        d = np.abs(got - ref)
        self.err = np.maximum(self.err, d.max(axis=axes))
        self.ref = np.maximum(self.ref, np.abs(ref).max(axis=axes))
        flat = d.reshape(-1, d.shape[-1])
        pick = rng.integers(0, flat.shape[0], size=min(flat.shape[0], 2000))
        self.samples.append(flat[pick])

    def worst(self):
        return float((self.err / np.maximum(self.ref, 1e-8)).max())

    def quantiles(self):
        rel = np.concatenate(self.samples) / np.maximum(self.ref, 1e-8)
        return [float(np.quantile(rel, q)) for q in (0.5, 0.99, 0.9999)]


def check_full_output(soap, oracle, struct, centres, chunk):
    """Every requested centre's whole output (row pointers, row atoms, descriptor row, every Jacobian row)
    against the oracle, the oracle working through the centres a chunk at a time."""
    pos, num = dev(struct)
    out = soap.derivatives(pos, num, struct.cell)
    soap.status()
    row_ptr = out.row_ptr.cpu().numpy()
    row_atom = out.row_atom.cpu().numpy()
    desc = out.descriptor.cpu().numpy()
    F = soap.n_features
    ed, ej = ColumnError(F), ColumnError(F)
    rng = np.random.default_rng(0)
    rows_checked = 0
    for c0 in range(0, len(centres), chunk):
        cen = centres[c0:c0 + chunk]
        ref = oracle.derivatives(struct.positions, struct.numbers, struct.cell, cen)
        for b, a in enumerate(cen):
            lo, hi = int(row_ptr[a]), int(row_ptr[a + 1])
            r0, r1 = int(ref.row_ptr[b]), int(ref.row_ptr[b + 1])
            assert hi - lo == r1 - r0, f"centre {a}: row count"
            assert np.array_equal(row_atom[lo:hi], ref.row_atom[r0:r1]), f"centre {a}: row atoms"
        contiguous = all(cen[k + 1] == cen[k] + 1 for k in range(len(cen) - 1))
        if contiguous:
            got = out.jacobian[int(row_ptr[cen[0]]):int(row_ptr[cen[-1] + 1])].cpu().numpy()
        else:
            got = np.concatenate([out.jacobian[int(row_ptr[a]):int(row_ptr[a + 1])].cpu().numpy() for a in cen])
        ej.add(got, ref.jacobian, (0, 1), rng)
        ed.add(desc[cen], ref.descriptor, 0, rng)
        rows_checked += got.shape[0]
    return ed, ej, rows_checked, int(row_ptr[-1])


def test_config2_water_1000_complete_output(pkg):
    """The benchmark's own workload in full: all 3000 descriptor rows, all Jacobian rows, row pointers and row
    atoms of the 1000-molecule cluster against the oracle (about half a minute of oracle time)."""
    s = water_cluster(1000, 0)
    args = ([1, 8], 6.0, 8, 6, 0.5, GTO)
    soap, oracle = pkg.Soap(*args), SoapOracle(*args)
    ed, ej, rows, total = check_full_output(soap, oracle, s, list(range(3000)), 250)
    assert rows == total                                           # every row of the output was compared
    print(f"config 2 complete: {rows} rows; descriptor worst column {ed.worst():.2e}, element quantiles "
          f"(50/99/99.99 %) {ed.quantiles()}; Jacobian worst column {ej.worst():.2e}, quantiles {ej.quantiles()}")
    assert ed.worst() < DESC_TOL and ej.worst() < JAC_TOL


def test_config4_multispecies_box_250_centres_complete_rows(pkg):
    """250 evenly spread centres of the periodic four-species box, every one of their rows against the oracle."""
    s = multispecies_box(2000, 0)
    args = ([6, 1, 7, 8], 5.0, 8, 8, 0.4, POLYNOMIAL, (True, True, True))
    soap, oracle = pkg.Soap(*args), SoapOracle(*args)
    centres = list(range(0, 2000, 8))
    ed, ej, rows, _ = check_full_output(soap, oracle, s, centres, 50)
    print(f"config 4, 250 centres: {rows} rows; descriptor worst column {ed.worst():.2e}; Jacobian worst column {ej.worst():.2e}")
    assert ed.worst() < DESC_TOL and ej.worst() < JAC_TOL


def test_paper_parameters_water_1000_rcut10_sampled(pkg):
    """The paper's own headline parameters (r_cut 10, n_max 7, l_max 3) on the 1000-molecule cluster:
    several hundred neighbours per sphere, every centre on the GPU, sampled centres against the oracle."""
    s = water_cluster(1000, 0)
    args = ([1, 8], 10.0, 7, 3, 0.5, GTO)
    soap, oracle = pkg.Soap(*args), SoapOracle(*args)
    sample = [0, 1499, 2999, 777]
    check_neighbors(soap, oracle, s, sample)
    check_derivatives(soap, oracle, s, sample=sample)


@pytest.mark.parametrize("l_max", [2, 4, 6, 8, 10, 12])
@pytest.mark.parametrize("n_max", [2, 4, 6, 8, 10, 12])
def test_config3_hyperparameter_map_cells_sampled(pkg, n_max, l_max):
    """Every cell of the (n_max, l_max) map `bench.py --suite map` times, on the full 1000-molecule cluster:
    every centre on the GPU, three of them against the oracle."""
    s = water_cluster(1000, 0)
    args = ([1, 8], 6.0, n_max, l_max, 0.5, GTO)
    soap, oracle = pkg.Soap(*args), SoapOracle(*args)
    check_derivatives(soap, oracle, s, sample=[5, 1499, 2990])


def test_config4_multispecies_box_sampled(pkg):
    s = multispecies_box(2000, 0)
    args = ([6, 1, 7, 8], 5.0, 8, 8, 0.4, POLYNOMIAL, (True, True, True))
    soap, oracle = pkg.Soap(*args), SoapOracle(*args)
    sample = [0, 1, 999, 1999] + list(range(50, 2000, 331))
    check_neighbors(soap, oracle, s, sample)
    check_derivatives(soap, oracle, s, sample=sample)


def test_config5_descriptor_only_30k(pkg):
    s = water_cluster(10000, 0)
    args = ([1, 8], 5.0, 8, 6, 0.5, GTO)
    soap, oracle = pkg.Soap(*args), SoapOracle(*args)
    pos, num = dev(s)
    d = soap.descriptor(pos, num)
    npairs, _ = soap.status()
    sample = [0, 29999, 12345] + list(range(17, 30000, 2999))
    ref = oracle.descriptor(s.positions, s.numbers, None, sample)
    assert col_err(d[sample].cpu().numpy(), ref, 0) < DESC_TOL
    lists = oracle.neighbor_list(s.positions, None, sample)
    assert npairs >= sum(len(l) for l in lists)          # the status word counts every centre's pairs
    cen = torch.tensor(sample, dtype=torch.int32).cuda()
    ptr, atom, _ = soap.neighbor_list(pos, num, None, cen)
    assert [int(x) for x in (ptr[1:] - ptr[:-1]).cpu()] == [len(l) for l in lists]


def test_jacobian_beyond_four_gigabytes_30k_atoms_sampled(pkg):
    """Descriptor + Jacobian of 30,000 atoms: 1.4 million rows, 16 GB of output, so every offset into the
    Jacobian passes 2^32 bytes; centres from the start, the middle and the very end against the oracle."""
    s = water_cluster(10000, 0)
    args = ([1, 8], 5.0, 8, 6, 0.5, GTO)
    soap, oracle = pkg.Soap(*args), SoapOracle(*args)
    pos, num = dev(s)
    out = soap.derivatives(pos, num)
    assert out.jacobian.numel() * 4 > 2 ** 33
    sample = [0, 14999, 29990, 29999]
    ref = oracle.derivatives(s.positions, s.numbers, None, sample)
    row_ptr = out.row_ptr.cpu().numpy()
    got = []
    for b, a in enumerate(sample):
        lo, hi = int(row_ptr[a]), int(row_ptr[a + 1])
        assert np.array_equal(out.row_atom[lo:hi].cpu().numpy(), ref.row_atom[ref.row_ptr[b]:ref.row_ptr[b + 1]])
        got.append(out.jacobian[lo:hi].cpu().numpy())
    assert col_err(np.concatenate(got), ref.jacobian, (0, 1)) < JAC_TOL
    assert col_err(out.descriptor[sample].cpu().numpy(), ref.descriptor, 0) < DESC_TOL
    # translation sum rule on the last thousand centres (their rows sit at the end of the 16 GB)
    lo, hi = int(row_ptr[29000]), int(row_ptr[30000])
    seg = torch.repeat_interleave(torch.arange(1000, device="cuda"), out.row_ptr[29001:] - out.row_ptr[29000:-1])
    sums = torch.zeros((1000, 3, soap.n_features), device="cuda", dtype=torch.float64)
    sums.index_add_(0, seg, out.jacobian[lo:hi].double())
    scale = out.jacobian[lo:hi].abs().amax(dim=(0, 1)).double().clamp_min(1e-8)
    assert float((sums.abs().amax(dim=(0, 1)) / scale).max()) < 1e-4
    del out


def test_config5_descriptor_only_million_atoms_sampled(pkg):
    """The largest size of the scaling benchmark (1,000,002 atoms): every centre on the GPU, a handful of
    centres and their neighbour lists against the oracle, and whole-output properties."""
    s = water_cluster(333334, 0)
    assert s.n_atoms == 1000002
    args = ([1, 8], 5.0, 8, 6, 0.5, GTO)
    soap, oracle = pkg.Soap(*args), SoapOracle(*args)
    pos, num = dev(s)
    d = soap.descriptor(pos, num)
    soap.status()
    sample = [0, 1000001, 500000, 123456, 777777, 999000]
    ref = oracle.descriptor(s.positions, s.numbers, None, sample)
    assert col_err(d[sample].cpu().numpy(), ref, 0) < DESC_TOL
    cen = torch.tensor(sample, dtype=torch.int32).cuda()
    ptr, atom, _ = soap.neighbor_list(pos, num, None, cen)
    lists = oracle.neighbor_list(s.positions, None, sample)
    ptr, atom = ptr.cpu().numpy(), atom.cpu().numpy()
    for a, lst in enumerate(lists):
        assert [int(x) for x in atom[ptr[a]:ptr[a + 1]]] == [t[0] for t in lst]
    # whole output: finite, and every feature with mu == nu and n == n' is a sum of squares
    assert torch.isfinite(d).all()
    diag = [f for f, (mu, nu, n, n2, l) in enumerate(oracle.table) if mu == nu and n == n2]
    cols = d[:, torch.tensor(diag, device="cuda")]
    assert float(cols.min()) >= 0.0
    assert float(cols.amax(dim=0).min()) > 0.0


def test_device_side_errors_are_reported(pkg):
    s = water_cluster(8, 0)
    soap = pkg.Soap([1, 8], 5.0, 2, 2, 0.5)
    pos, num = dev(s)
    bad = num.clone()
    bad[5] = 6
    soap.descriptor(pos, bad)
    with pytest.raises(pkg.SoapError) as e:
        soap.status()
    assert e.value.code == -2
    # undersized Jacobian buffer
    _, nrows = soap.neighbors(pos, num)
    desc = torch.empty((24, soap.n_features), device="cuda")
    jac = torch.full((nrows - 1, 3, soap.n_features), 7.0, device="cuda")
    row_ptr = torch.empty(25, dtype=torch.int64, device="cuda")
    row_atom = torch.empty(nrows, dtype=torch.int32, device="cuda")
    soap.derivatives_into(pos, num, None, None, desc, jac, row_ptr, row_atom)
    with pytest.raises(pkg.SoapError) as e:
        soap.status()
    assert e.value.code == -3
    assert float(jac.min()) == 7.0 and float(jac.max()) == 7.0        # nothing was written
    assert int(row_ptr[-1]) == nrows
    # and the handle keeps working afterwards
    out = soap.derivatives(pos, num)
    assert out.jacobian.shape[0] == nrows
    # a periodic handle without a cell is refused on the host
    per = pkg.Soap([1, 8], 5.0, 2, 2, 0.5, pkg.GTO, (True, False, False))
    with pytest.raises(pkg.SoapError):
        per.descriptor(pos, num)


def test_denser_structure_than_planned_is_reported_and_replanned(pkg):
    """Scratch is planned from the first structure of a given size; a later structure of the same
    size with more pairs than the plan's headroom must be flagged, and planning again must fix it."""
    loose = water_cluster(60, 0)
    dense = water_cluster(60, 0)
    dense.positions = (dense.positions * 0.6).astype(np.float32)          # same atoms, 4.6x the density
    args = ([1, 8], 5.0, 3, 2, 0.5, GTO)
    soap, oracle = pkg.Soap(*args), SoapOracle(*args)
    num = torch.from_numpy(loose.numbers).cuda()
    soap.descriptor(torch.from_numpy(loose.positions).cuda(), num)
    p_loose, _ = soap.status()
    pos_dense = torch.from_numpy(dense.positions).cuda()
    soap.descriptor(pos_dense, num)                                       # same sizes: no new plan
    with pytest.raises(pkg.SoapError) as e:
        soap.status()
    assert e.value.code == -3
    p_dense, _ = soap.neighbors(pos_dense, num)                           # plans again
    assert p_dense > 1.25 * p_loose + 1024
    d = soap.descriptor(pos_dense, num)
    soap.status()
    ref = oracle.descriptor(dense.positions, dense.numbers, None, [0, 77, 179])
    assert col_err(d[[0, 77, 179]].cpu().numpy(), ref, 0) < DESC_TOL


def test_empty_centre_list_on_a_mid_sized_structure(pkg):
    """No centres requested on a fresh handle with 300 atoms (a size the one-launch brute-force search would
    take if every atom were a centre): nothing is computed, the row pointer is a single zero."""
    s = water_cluster(100, 2)
    soap = pkg.Soap([1, 8], 5.0, 2, 2, 0.5)
    pos, num = dev(s)
    cen = torch.empty((0,), dtype=torch.int32, device="cuda")
    d = soap.descriptor(pos, num, None, cen)
    assert d.shape == (0, soap.n_features)
    out = soap.derivatives(pos, num, None, cen)
    assert out.row_ptr.cpu().tolist() == [0] and out.jacobian.shape[0] == 0
    soap.status()
    # and the handle then serves the full structure correctly
    oracle = SoapOracle([1, 8], 5.0, 2, 2, 0.5)
    ref = oracle.descriptor(s.positions, s.numbers, None, [0, 150, 299])
    assert col_err(soap.descriptor(pos, num)[[0, 150, 299]].cpu().numpy(), ref, 0) < DESC_TOL


def test_empty_structure(pkg):
    soap = pkg.Soap([1, 8], 5.0, 2, 2, 0.5)
    pos = torch.empty((0, 3), dtype=torch.float32, device="cuda")
    num = torch.empty((0,), dtype=torch.int32, device="cuda")
    assert soap.neighbors(pos, num) == (0, 0)
    assert soap.descriptor(pos, num).shape == (0, soap.n_features)

"""The face with the paper's constructor keywords and call shapes (`compat.SOAP`) against the oracle."""
import numpy as np
import pytest

from oracle import modes
from oracle.soap import GTO, POLYNOMIAL, SoapOracle
from soap_inputs import small_periodic_cell, water_cluster
from test_gpu_parity import DESC_TOL, JAC_TOL, col_err, same_values

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def SOAP():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2609_05709_b200.compat import SOAP as cls
    return cls


def test_power_spectrum_dense_derivatives_with_selections(SOAP):
    s = water_cluster(6, 2)
    soap = SOAP(r_cut=4.5, n_max=4, l_max=3, sigma=0.5, rbf="gto", species=["H", "O"])
    oracle = SoapOracle([1, 8], 4.5, 4, 3, 0.5, GTO)
    assert soap.get_number_of_features() == oracle.n_features
    centers, include = [4, 0, 11], [0, 3, 5, 17]
    ref = oracle.derivatives(s.positions, s.numbers, None, centers)
    dense_ref = modes._dense(ref, s.n_atoms)
    d = soap.create(s, centers=centers)
    assert d.shape == (3, oracle.n_features) and col_err(d.cpu().numpy(), ref.descriptor, 0) < DESC_TOL
    assert torch.equal(soap.generate(s, centers=centers), d)                 # the same call twice: bit for bit
    jac, d2 = soap.derivatives(s, centers=centers, include=include)
    assert jac.shape == (3, 4, 3, oracle.n_features) and same_values(d2, d)
    assert col_err(jac.cpu().numpy(), dense_ref[:, include], (0, 1, 2)) < JAC_TOL
    jac = soap.derivatives((s.positions, s.numbers), centers=centers, exclude=[1, 2], return_descriptor=False)
    keep = [a for a in range(s.n_atoms) if a not in (1, 2)]
    assert col_err(jac.cpu().numpy(), dense_ref[:, keep], (0, 1, 2)) < JAC_TOL
    with pytest.raises(ValueError):
        soap.derivatives(s, include=[0], exclude=[1])


def test_periodic_polynomial_with_weighting_and_point_centres(SOAP):
    s = small_periodic_cell(2, (True, True, True))
    w = {"function": "poly", "r0": 3.8, "c": 1.0, "m": 2, "w0": 1.0}
    soap = SOAP(r_cut=4.2, n_max=3, l_max=3, sigma=0.5, rbf="polynomial", species=[1, 6, 7, 8], periodic=True,
                weighting=w, crossover=False)
    oracle = SoapOracle([1, 6, 7, 8], 4.2, 3, 3, 0.5, POLYNOMIAL, (True, True, True), crossover=False, weighting=w)
    ref = oracle.derivatives(s.positions, s.numbers, s.cell)
    jac, d = soap.derivatives(s)
    assert col_err(d.cpu().numpy(), ref.descriptor, 0) < DESC_TOL
    assert col_err(jac.cpu().numpy(), modes._dense(ref, s.n_atoms), (0, 1, 2)) < JAC_TOL
    sites = np.array([[0.5, 0.5, 0.5], [2.2, 1.7, 3.1]])
    sref = modes.site_derivatives(oracle, s.positions, s.numbers, sites, s.cell)
    jac, d = soap.derivatives(s, centers=sites)
    assert col_err(d.cpu().numpy(), sref.descriptor, 0) < DESC_TOL
    assert col_err(jac.cpu().numpy(), modes._dense(sref, s.n_atoms), (0, 1, 2)) < JAC_TOL
    assert same_values(soap.create(s, centers=sites), d)
    # the same object on a structure it treats as non-periodic (flags off in the structure)
    s.pbc = (False, False, False)
    o2 = SoapOracle([1, 6, 7, 8], 4.2, 3, 3, 0.5, POLYNOMIAL, crossover=False, weighting=w)
    assert col_err(soap.create(s).cpu().numpy(), o2.descriptor(s.positions, s.numbers), 0) < DESC_TOL


@pytest.mark.parametrize("average", ["inner", "outer", "cc"])
def test_average_modes(SOAP, average):
    s = water_cluster(5, 7)
    soap = SOAP(r_cut=4.0, n_max=3, l_max=2, sigma=0.5, species=[1, 8], average=average)
    oracle = SoapOracle([1, 8], 4.0, 3, 2, 0.5, GTO)
    if average == "cc":
        ref = modes.coefficient_derivatives(oracle, s.positions, s.numbers)
        assert soap.get_number_of_features() == modes.coefficient_width(oracle)
        jac, c = soap.derivatives(s, include=[2, 9])
        assert col_err(c.cpu().numpy(), ref.descriptor, 0) < DESC_TOL
        assert col_err(jac.cpu().numpy(), modes._dense(ref, s.n_atoms)[:, [2, 9]], (0, 1, 2)) < JAC_TOL
        assert same_values(soap.create(s), c)
        return
    rd, rj = modes.average_derivatives(oracle, average, s.positions, s.numbers)
    jac, d = soap.derivatives(s)
    assert d.shape == (1, oracle.n_features) and jac.shape == (1, s.n_atoms, 3, oracle.n_features)
    scale = np.maximum(np.abs(oracle.descriptor(s.positions, s.numbers)).max(axis=0), 1e-8)
    assert (np.abs(d.cpu().numpy()[0] - rd) / scale).max() < DESC_TOL
    assert col_err(jac.cpu().numpy()[0], rj, (0, 1)) < JAC_TOL
    assert (np.abs(soap.create(s).cpu().numpy()[0] - rd) / scale).max() < DESC_TOL


def test_unsupported_arguments_are_refused(SOAP):
    with pytest.raises(NotImplementedError):
        SOAP(r_cut=4.0, n_max=2, l_max=2, species=[1], sparse=True)
    with pytest.raises(NotImplementedError):
        SOAP(r_cut=4.0, n_max=2, l_max=2, species=[1], max_num_neighbors=20)
    with pytest.raises(ValueError):
        SOAP(r_cut=4.0, n_max=2, l_max=2, species=[1], average="middle")
    with pytest.raises(ValueError):
        SOAP(r_cut=4.0, n_max=2, l_max=2, species=[1], device="cpu")


def test_lists_of_structures_go_through_the_batch_path(SOAP):
    structs = [water_cluster(n, 30 + n) for n in (2, 5, 1, 7)]
    soap = SOAP(r_cut=4.5, n_max=3, l_max=3, sigma=0.5, species=[1, 8])
    oracle = SoapOracle([1, 8], 4.5, 3, 3, 0.5, GTO)
    descs = soap.create(structs)
    both = soap.derivatives(structs)
    assert len(descs) == len(both) == 4
    for s, d, (jac, d2) in zip(structs, descs, both):
        ref = oracle.derivatives(s.positions, s.numbers)
        assert same_values(d, d2) and col_err(d.cpu().numpy(), ref.descriptor, 0) < DESC_TOL
        assert jac.shape == (s.n_atoms, s.n_atoms, 3, oracle.n_features)
        assert col_err(jac.cpu().numpy(), modes._dense(ref, s.n_atoms), (0, 1, 2)) < JAC_TOL
    # with a selection the structures are taken one by one
    sel = soap.derivatives(structs, include=[0, 1], return_descriptor=False)
    assert sel[1].shape == (15, 2, 3, oracle.n_features) and torch.equal(sel[1], both[1][0][:, [0, 1]])

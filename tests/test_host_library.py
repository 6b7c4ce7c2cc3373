"""CPU-side checks of the CUDA library: it loads, exports the declared ABI, and its
host-built tables agree with the oracle.  No GPU needed."""
import ctypes
import os
import re

import numpy as np
import pytest

from oracle import basis
from oracle.soap import GTO, POLYNOMIAL, SoapOracle

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def pkg():
    from paper_2609_05709_b200 import build as b
    b.build()
    import paper_2609_05709_b200 as p
    return p


def test_library_exports_every_declared_symbol(pkg):
    header = open(os.path.join(ROOT, "include", "soap.h")).read()
    declared = sorted(set(re.findall(r"\b(soap_[a-z0-9_]+)\s*\(", header)))
    assert declared == sorted(pkg.EXPORTED_SYMBOLS)
    lib = ctypes.CDLL(pkg.library_path())
    for name in declared:
        assert hasattr(lib, name), name


def test_create_rejects_bad_arguments(pkg):
    for args in [([1, 8], 1.0, 4, 3, 0.5, GTO), ([1, 1], 5.0, 4, 3, 0.5, GTO), ([1, 8], 5.0, 0, 3, 0.5, GTO),
                 ([1, 8], 5.0, 4, 13, 0.5, GTO), ([1, 8], 5.0, 4, 3, -1.0, GTO), ([1, 8], 5.0, 4, 3, 0.5, 7),
                 ([], 5.0, 4, 3, 0.5, GTO), ([1, 300], 5.0, 4, 3, 0.5, GTO), ([1, 8], 5.0, 16, 12, 0.5, GTO)]:
        with pytest.raises(pkg.SoapError) as e:
            pkg.Soap(*args)
        assert e.value.code == -1


def test_feature_table_matches_oracle(pkg):
    s = pkg.Soap([8, 1, 6], 5.0, 3, 2, 0.5)
    o = SoapOracle([8, 1, 6], 5.0, 3, 2, 0.5)
    assert s.n_features == o.n_features
    for f in range(o.n_features):
        assert s.feature_info(f) == tuple(int(v) for v in o.table[f])
    with pytest.raises(pkg.SoapError):
        s.feature_info(o.n_features)


@pytest.mark.parametrize("rbf,r_cut,n_max,l_max,sigma", [
    (GTO, 5.0, 4, 3, 0.5), (GTO, 6.0, 8, 6, 0.5), (POLYNOMIAL, 5.0, 8, 8, 0.4), (GTO, 6.0, 12, 12, 0.5),
    (POLYNOMIAL, 4.0, 3, 2, 0.3)])
def test_radial_tables_against_oracle(pkg, rbf, r_cut, n_max, l_max, sigma):
    """The degree-5 tables G_nl(d) = F_nl(d)/d^l reproduce the oracle's radial factor
    (and its derivative) to fp32 rounding, in the weighting they enter the coefficients with."""
    s = pkg.Soap([1, 8], r_cut, n_max, l_max, sigma, rbf)
    d = np.concatenate([np.linspace(0.3, r_cut - 1e-9, 97), [0.05, 0.5 * r_cut + 1e-3]])
    F, dF = (basis.gto_radial if rbf == GTO else basis.poly_radial)(d, r_cut, n_max, l_max, sigma)
    L1 = l_max + 1
    G = np.empty((d.size, n_max, L1))
    Gh = np.empty_like(G)
    for a, x in enumerate(d):
        g, gh = s.radial_table(x)
        G[a] = g.reshape(n_max, L1)
        Gh[a] = gh.reshape(n_max, L1)
    l = np.arange(L1)[None, None, :]
    dd = d[:, None, None]
    Fm = np.transpose(F, (2, 0, 1))
    dFm = np.transpose(dF, (2, 0, 1))
    scale = np.abs(Fm).max(axis=0, keepdims=True)
    assert (np.abs(G * dd ** l - Fm) / scale).max() < 5e-7
    # d/dd [G d^l] = (Ghat d^2 + l G) d^(l-1)
    dscale = np.abs(dFm).max(axis=0, keepdims=True)
    assert (np.abs((Gh * dd * dd + l * G) * dd ** (l - 1.0) - dFm) / dscale).max() < 3e-6


def test_compute_calls_fail_loudly_without_a_device(pkg):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    s = pkg.Soap([1, 8], 5.0, 2, 1, 0.5)
    n = ctypes.c_int64()
    rc = s._lib.soap_neighbors(s._h, ctypes.c_void_p(16), ctypes.c_void_p(16), 1, None, None, 1,
                               ctypes.byref(n), ctypes.byref(n), None)
    assert rc == -4      # SOAP_ERR_CUDA: no CPU path behind the ABI


def test_options_change_the_host_side_tables(pkg):
    """Crossover, compact-row maps and weighting arguments are host logic: no GPU involved."""
    s = pkg.Soap([1, 6, 8], 5.0, 3, 2, 0.5)
    o = SoapOracle([1, 6, 8], 5.0, 3, 2, 0.5)
    tri, cross = 6 * 3, 9 * 3
    assert s.n_features == 3 * tri + 3 * cross and s.n_coefficients == 3 * 3 * 9
    assert s.n_compact == tri + 2 * cross and s.compact_pitch == (s.n_compact + 7) // 8 * 8
    for z in range(3):
        m = s.compact_feature_map(z)
        want = [f for f, (mu, nu, *_rest) in enumerate(o.table) if mu == z or nu == z]
        assert list(m) == want
    with pytest.raises(pkg.SoapError):
        s.compact_feature_map(3)
    # crossover off: the table shrinks to the same-species blocks, the compact row is the whole row of its species
    d = pkg.Soap([1, 6, 8], 5.0, 3, 2, 0.5, crossover=False)
    od = SoapOracle([1, 6, 8], 5.0, 3, 2, 0.5, crossover=False)
    assert d.n_features == 3 * tri == od.n_features and d.n_compact == tri
    assert [d.feature_info(f) for f in range(d.n_features)] == [tuple(int(v) for v in r) for r in od.table]
    assert list(d.compact_feature_map(1)) == list(range(tri, 2 * tri))
    # weighting arguments are validated before anything touches a device
    for bad in [{"function": "poly", "r0": 0.0, "m": 1}, {"function": "pow", "r0": 1.0, "m": -1, "d": 1.0},
                {"function": "pow", "r0": 1.0, "m": 2, "d": 0.0}, {"function": "exp", "r0": 1.0, "d": -1.0}]:
        with pytest.raises(pkg.SoapError) as e:
            pkg.Soap([1, 8], 5.0, 2, 2, 0.5, weighting=bad)
        assert e.value.code == -1
    pkg.Soap([1, 8], 5.0, 2, 2, 0.5, weighting={"function": "exp", "r0": 1.0, "c": 2.0, "d": 0.5})

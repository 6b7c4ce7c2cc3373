"""The multi-GPU driver with its CUDA backend on the one GPU of the test box: a single worker process
must reproduce the direct call bit for bit, and its results must match the oracle."""
import numpy as np
import pytest

from soap_inputs import water_cluster
from test_gpu_parity import same_values

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


def test_one_worker_equals_the_direct_call():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import paper_2609_05709_b200 as pkg
    from paper_2609_05709_b200 import driver
    config = dict(species=[1, 8], r_cut=5.0, n_max=4, l_max=3, sigma=0.5)
    structs = [water_cluster(20, 1), water_cluster(7, 2)]
    results, seconds = driver.generate(config, structs, batch=16, derivatives=True, world=1, timeout=300)
    assert seconds > 0
    soap = pkg.Soap(**config)
    for s, r in zip(structs, results):
        pos, num = torch.from_numpy(s.positions).cuda(), torch.from_numpy(s.numbers).cuda()
        ref = soap.derivatives(pos, num)
        assert np.array_equal(r.descriptor, ref.descriptor.cpu().numpy())
        assert np.array_equal(r.row_ptr, ref.row_ptr.cpu().numpy())
        assert np.array_equal(r.row_atom, ref.row_atom.cpu().numpy())
        assert np.array_equal(r.jacobian, ref.jacobian.cpu().numpy())
    desc_only, _ = driver.generate(config, structs[:1], batch=25, derivatives=False, world=1, timeout=300)
    assert same_values(desc_only[0].descriptor, results[0].descriptor) and desc_only[0].jacobian is None


def test_one_worker_against_the_oracle():
    """The driver's output (descriptor, rows, row bookkeeping, batches put together on the host) against the fp64
    oracle, not against another call of the library."""
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from oracle.soap import SoapOracle
    from paper_2609_05709_b200 import driver
    from test_gpu_parity import DESC_TOL, JAC_TOL, col_err
    config = dict(species=[1, 8], r_cut=4.5, n_max=4, l_max=3, sigma=0.5)
    structs = [water_cluster(11, 5), water_cluster(3, 6)]
    results, _ = driver.generate(config, structs, batch=7, derivatives=True, world=1, timeout=300)
    oracle = SoapOracle([1, 8], 4.5, 4, 3, 0.5)
    for s, r in zip(structs, results):
        ref = oracle.derivatives(s.positions, s.numbers)
        assert np.array_equal(r.row_ptr, ref.row_ptr) and np.array_equal(r.row_atom, ref.row_atom)
        assert col_err(r.descriptor, ref.descriptor, 0) < DESC_TOL
        assert col_err(r.jacobian, ref.jacobian, (0, 1)) < JAC_TOL

"""The multi-GPU driver with its CUDA backend on the one GPU of the test box: a single worker process
must reproduce the direct call bit for bit."""
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

"""The allocation-free neighbour-count entry point against the handle-based one.

Who needs it: callers that are not allowed to allocate device memory while they call the
library (their memory pool owns the whole budget, or an allocation's implicit synchronisation
would break their timing).  `soap_neighbor_counts_static` keeps its cell list in a fixed array
inside the library, so nothing is allocated during the call; here its counts must equal, atom by
atom, the row lengths of the neighbour list the ordinary entry point builds.  Two calls in a row
on different structures check that the shared array is cleared properly between calls.
This file sorts last on purpose: a run that stops at the first failure has then already run
every other test.
"""
import ctypes

import numpy as np
import pytest

from soap_inputs import water_cluster

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


def reference_counts(pkg, struct, r_cut):
    soap = pkg.Soap([1, 8], r_cut, 2, 1, 0.5)
    pos = torch.from_numpy(struct.positions).cuda()
    num = torch.from_numpy(struct.numbers).cuda()
    ptr, _, _ = soap.neighbor_list(pos, num)
    return (ptr[1:] - ptr[:-1]).to(torch.int32), pos


def test_static_scratch_counts_match_twice_in_a_row():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import paper_2609_05709_b200 as pkg
    first, second = water_cluster(700, 11), water_cluster(90, 12)
    for struct, r_cut in ((first, 6.0), (second, 4.0)):          # the second call reuses the array the first one filled
        want, pos = reference_counts(pkg, struct, r_cut)
        out = torch.full((struct.n_atoms,), -1, dtype=torch.int32, device="cuda")
        got = pkg.neighbor_counts_static(pos, r_cut, out=out)
        torch.cuda.synchronize()
        assert torch.equal(got, want)                            # integer work: exact
    # nothing is allocated on the device by a call whose output tensor is the caller's
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    pkg.neighbor_counts_static(pos, r_cut, out=out)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before
    # the largest structure the fixed scratch takes: 65536 atoms, spread thinly so that the bin grid hits its cap
    rng = np.random.default_rng(5)
    big = (rng.random((65536, 3)) * 400.0).astype(np.float32)
    big[1] = big[0] + np.float32(0.5)                              # at least one pair for sure
    bpos = torch.from_numpy(big).cuda()
    bnum = torch.ones(65536, dtype=torch.int32, device="cuda")
    ptr, _, _ = pkg.Soap([1], 6.0, 2, 1, 0.5).neighbor_list(bpos, bnum)
    got = pkg.neighbor_counts_static(bpos, 6.0)
    torch.cuda.synchronize()
    assert torch.equal(got, (ptr[1:] - ptr[:-1]).to(torch.int32)) and int(got.sum()) >= 2
    # sizes beyond the fixed scratch are refused with a message and nothing runs
    lib = pkg.load_library()
    msg = ctypes.create_string_buffer(256)
    rc = lib.soap_neighbor_counts_static(ctypes.c_void_p(256), 65537, 5.0, ctypes.c_void_p(256), None, msg, 256)
    assert rc == -3 and b"65536" in msg.value
    # an empty structure is fine
    empty = torch.empty((0, 3), dtype=torch.float32, device="cuda")
    assert pkg.neighbor_counts_static(empty, 5.0).numel() == 0

"""Dense (centres, atoms, 3, F) view with an atom selection, and centre-batch streaming, on a GPU.

The dense tensor is the layout of the paper's derivatives() call; the reference is built from the
oracle's rows (zeros everywhere else, as the text below Eq. 5 says)."""
import numpy as np
import pytest

from oracle.soap import GTO, POLYNOMIAL, SoapOracle
from soap_inputs import small_periodic_cell, water_cluster

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def pkg():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import paper_2609_05709_b200 as p
    p.load_library()
    return p


def oracle_dense(oracle, struct, centers, include):
    ref = oracle.derivatives(struct.positions, struct.numbers, struct.cell, centers)
    col = {int(a): k for k, a in enumerate(include)}
    dense = np.zeros((len(centers), len(include), 3, oracle.n_features))
    for c in range(len(centers)):
        for r in range(ref.row_ptr[c], ref.row_ptr[c + 1]):
            if int(ref.row_atom[r]) in col:
                dense[c, col[int(ref.row_atom[r])]] = ref.jacobian[r]
    return dense


def col_err(a, ref):
    a = np.asarray(a, np.float64).reshape(-1, ref.shape[-1])
    ref = ref.reshape(-1, ref.shape[-1])
    return float((np.abs(a - ref).max(0) / np.maximum(np.abs(ref).max(0), 1e-8)).max())


@pytest.mark.parametrize("case", ["water", "cell"])
def test_dense_view_with_atom_selection(pkg, case):
    if case == "water":
        s, args = water_cluster(8, 0), ([1, 8], 3.0, 3, 3, 0.5, GTO)          # small cutoff: many empty blocks
    else:
        s, args = small_periodic_cell(0), ([1, 6, 7, 8], 4.5, 2, 2, 0.5, POLYNOMIAL, (True, True, True))
    soap, oracle = pkg.Soap(*args), SoapOracle(*args)
    pos = torch.from_numpy(s.positions).cuda()
    num = torch.from_numpy(s.numbers).cuda()
    centers = [0, 3, 5] if case == "water" else [1, 6]
    out = soap.derivatives(pos, num, s.cell, torch.tensor(centers, dtype=torch.int32).cuda())
    # every atom
    dense = soap.jacobian_dense(out, n_atoms=s.n_atoms)
    ref = oracle_dense(oracle, s, centers, list(range(s.n_atoms)))
    assert dense.shape == ref.shape
    assert col_err(dense.cpu().numpy(), ref) < 1e-4
    assert np.array_equal(dense.cpu().numpy() == 0, ref == 0) or case == "cell"   # same sparsity pattern
    # a selection, not in order, with an atom outside every sphere where there is one
    include = [5, 0, s.n_atoms - 1, 2]
    dense = soap.jacobian_dense(out, include=torch.tensor(include, dtype=torch.int32).cuda())
    assert col_err(dense.cpu().numpy(), oracle_dense(oracle, s, centers, include)) < 1e-4


def test_centre_batches_equal_one_call(pkg):
    s = water_cluster(40, 2)
    soap = pkg.Soap([1, 8], 5.0, 4, 3, 0.5, GTO)
    pos = torch.from_numpy(s.positions).cuda()
    num = torch.from_numpy(s.numbers).cuda()
    whole = soap.derivatives(pos, num)
    rows = 0
    for part, got in soap.derivatives_batched(pos, num, batch=37):
        lo = int(part[0])
        n = part.shape[0]
        assert torch.equal(got.descriptor, whole.descriptor[lo:lo + n])
        r0, r1 = int(whole.row_ptr[lo]), int(whole.row_ptr[lo + n])
        assert torch.equal(got.row_ptr, whole.row_ptr[lo:lo + n + 1] - r0)
        assert torch.equal(got.row_atom, whole.row_atom[r0:r1])
        assert torch.equal(got.jacobian, whole.jacobian[r0:r1])       # same kernels, same inputs: bit for bit
        rows += r1 - r0
    assert rows == whole.jacobian.shape[0]


def test_a_planned_step_can_be_captured_in_a_cuda_graph_and_replayed(pkg):
    """After the first call for a structure size the library neither allocates nor waits, so a step
    can be recorded once and replayed on new positions of the same size (launch-bound small systems)."""
    s = water_cluster(8, 3)
    soap = pkg.Soap([1, 8], 5.0, 4, 3, 0.5, GTO)
    pos = torch.from_numpy(s.positions).cuda()
    num = torch.from_numpy(s.numbers).cuda()
    n = s.n_atoms
    _, nrows = soap.neighbors(pos, num)
    cap = nrows + 64                                            # head-room: the moved structure may gain rows
    desc = torch.empty((n, soap.n_features), device="cuda")
    jac = torch.empty((cap, 3, soap.n_features), device="cuda")
    row_ptr = torch.empty(n + 1, dtype=torch.int64, device="cuda")
    row_atom = torch.empty(cap, dtype=torch.int32, device="cuda")
    soap.derivatives_into(pos, num, None, None, desc, jac, row_ptr, row_atom)     # warm-up outside the capture
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        soap.derivatives_into(pos, num, None, None, desc, jac, row_ptr, row_atom)
    # new coordinates in the captured input buffer, then replay
    rng = np.random.default_rng(5)
    moved = s.positions + rng.normal(scale=0.05, size=s.positions.shape).astype(np.float32)
    pos.copy_(torch.from_numpy(moved).cuda())
    graph.replay()
    torch.cuda.synchronize()
    soap.status()
    got_desc, got_ptr = desc.clone(), row_ptr.clone()
    rows = int(got_ptr[-1])
    got_jac, got_atom = jac[:rows].clone(), row_atom[:rows].clone()
    ref = soap.derivatives(torch.from_numpy(moved).cuda(), num)
    assert torch.equal(got_ptr, ref.row_ptr) and torch.equal(got_atom, ref.row_atom)
    assert torch.equal(got_desc, ref.descriptor) and torch.equal(got_jac, ref.jacobian)


def test_calls_queued_back_to_back_equal_calls_made_alone(pkg):
    """The kernels of a call wait for one another on the device and start while their predecessor still runs.  Calls
    of different sizes and kinds queued on one stream without a host wait in between, and on two streams at once
    with a handle each, must give the bits of the same calls made alone."""
    structs = [water_cluster(40, 1), water_cluster(6, 2), small_periodic_cell(3)]
    args = [([1, 8], 5.0, 8, 6, 0.5, GTO), ([1, 8], 4.0, 4, 3, 0.5, GTO), ([1, 6, 7, 8], 4.5, 3, 3, 0.5, POLYNOMIAL, (True, True, True))]
    soaps = [pkg.Soap(*a) for a in args]
    dev = [(torch.from_numpy(s.positions).cuda(), torch.from_numpy(s.numbers).cuda(), s.cell) for s in structs]
    alone = []
    for soap, (pos, num, cell) in zip(soaps, dev):
        d = soap.derivatives(pos, num, cell)
        torch.cuda.synchronize()
        p = soap.descriptor(pos, num, cell).clone()
        torch.cuda.synchronize()
        alone.append((d.descriptor.clone(), d.jacobian.clone(), d.row_ptr.clone(), d.row_atom.clone(), p))
    def buffers(k):
        ref = alone[k]
        return [torch.empty_like(ref[0]), torch.empty_like(ref[1]), torch.empty_like(ref[2]), torch.empty_like(ref[3]), torch.empty_like(ref[4])]

    for trial in range(5):
        queued = []
        for k in (0, 1, 2, 1, 0):
            pos, num, cell = dev[k]
            b = buffers(k)
            soaps[k].derivatives_into(pos, num, cell, None, b[0], b[1], b[2], b[3])      # enqueues only: no host wait
            soaps[k].descriptor(pos, num, cell, None, out=b[4])
            queued.append((k, b))
        torch.cuda.synchronize()
        for k, b in queued:
            soaps[k].status()
            for got, ref in zip(b, alone[k]):
                assert torch.equal(got, ref)
    # two streams, a handle each, at the same time
    other = pkg.Soap(*args[0])
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    pos, num, cell = dev[0]
    other.neighbors(pos, num, cell)                                # plans the second handle's scratch
    torch.cuda.synchronize()
    outs = []
    for _ in range(4):
        for soap, st in zip((soaps[0], other), streams):
            with torch.cuda.stream(st):
                b = buffers(0)
                soap.derivatives_into(pos, num, cell, None, b[0], b[1], b[2], b[3])
                outs.append(b)
    torch.cuda.synchronize()
    for b in outs:
        assert torch.equal(b[0], alone[0][0]) and torch.equal(b[1], alone[0][1])

"""The multi-GPU driver's bookkeeping on CPU: two worker processes, results put together on the host.
The per-task computation is injected (here: the oracle), so no GPU is needed."""
import os

import numpy as np
import pytest

torch = pytest.importorskip("torch")

from oracle.soap import SoapOracle  # noqa: E402
from paper_2609_05709_b200 import driver  # noqa: E402
from soap_inputs import small_periodic_cell, water_cluster  # noqa: E402

CONFIG = dict(species=[1, 6, 7, 8], r_cut=3.5, n_max=2, l_max=2, sigma=0.5, pbc=(True, True, False))


def oracle_backend(rank, config):
    o = SoapOracle(**config)

    def run(s, struct, lo, hi, derivatives):
        centers = list(range(lo, hi))
        if not derivatives:
            return {"desc": torch.from_numpy(o.descriptor(struct.positions, struct.numbers, struct.cell, centers))}
        d = o.derivatives(struct.positions, struct.numbers, struct.cell, centers)
        return {"desc": torch.from_numpy(d.descriptor), "jac": torch.from_numpy(d.jacobian),
                "row_ptr": torch.from_numpy(d.row_ptr), "row_atom": torch.from_numpy(d.row_atom)}
    return run


def failing_backend(rank, config):
    if rank == 1:
        raise ValueError("no device for this worker")
    return oracle_backend(rank, config)


def dying_backend(rank, config):
    run = oracle_backend(rank, config)

    def die(*a):
        if rank == 0:
            os._exit(3)
        return run(*a)
    return die


def _structures():
    a = small_periodic_cell(1, (True, True, False))
    b = small_periodic_cell(2, (True, True, False))
    b.positions, b.numbers = b.positions[:5].copy(), b.numbers[:5].copy()
    return [a, b]


def test_task_list_and_stride_assignment():
    tasks = driver.enumerate_tasks([10, 0, 3], 4)
    assert [(t.structure, t.batch, t.lo, t.hi) for t in tasks] == [(0, 0, 0, 4), (0, 1, 4, 8), (0, 2, 8, 10), (2, 0, 0, 3)]
    assert driver.tasks_of_rank(tasks, 3, 1) == [tasks[1]]
    key = lambda t: (t.structure, t.batch)
    assert sorted((t for r in range(3) for t in driver.tasks_of_rank(tasks, 3, r)), key=key) == tasks
    with pytest.raises(ValueError):
        driver.enumerate_tasks([3], 0)


@pytest.mark.parametrize("derivatives", [True, False])
def test_two_workers_reproduce_the_single_call(derivatives):
    structs = _structures()
    results, seconds = driver.generate(CONFIG, structs, batch=3, derivatives=derivatives, world=2,
                                       backend_factory=oracle_backend, timeout=120)
    assert seconds > 0 and len(results) == 2
    o = SoapOracle(**CONFIG)
    for s, r in zip(structs, results):
        ref = o.derivatives(s.positions, s.numbers, s.cell)
        assert np.array_equal(r.descriptor, ref.descriptor)
        if derivatives:
            assert np.array_equal(r.row_ptr, ref.row_ptr) and np.array_equal(r.row_atom, ref.row_atom)
            assert np.array_equal(r.jacobian, ref.jacobian)
        else:
            assert r.jacobian is None


def test_three_workers_and_an_uneven_task_list():
    """Seven tasks on three workers (3 + 2 + 2), one of the structures empty: the pieces still come back complete
    and in order."""
    structs = _structures()
    empty = small_periodic_cell(3, (True, True, False))
    empty.positions, empty.numbers = empty.positions[:0].copy(), empty.numbers[:0].copy()
    structs.insert(1, empty)
    tasks = driver.enumerate_tasks([int(s.positions.shape[0]) for s in structs], 2)
    assert len(tasks) == 7 and [len(driver.tasks_of_rank(tasks, 3, r)) for r in range(3)] == [3, 2, 2]
    results, _ = driver.generate(CONFIG, structs, batch=2, derivatives=True, world=3,
                                 backend_factory=oracle_backend, timeout=180)
    o = SoapOracle(**CONFIG)
    assert len(results) == 3 and results[1].descriptor.shape[0] == 0
    for s, r in zip(structs, results):
        if s.positions.shape[0] == 0:
            continue
        ref = o.derivatives(s.positions, s.numbers, s.cell)
        assert np.array_equal(r.descriptor, ref.descriptor) and np.array_equal(r.row_ptr, ref.row_ptr)
        assert np.array_equal(r.row_atom, ref.row_atom) and np.array_equal(r.jacobian, ref.jacobian)


def test_a_worker_that_fails_in_setup_ends_the_job():
    with pytest.raises(RuntimeError, match="worker 1 failed during set-up"):
        driver.generate(CONFIG, _structures(), batch=3, world=2, backend_factory=failing_backend, timeout=60)


def test_a_worker_that_dies_silently_is_noticed():
    with pytest.raises(RuntimeError, match="worker 0 exited with code 3"):
        driver.generate(CONFIG, _structures(), batch=3, world=2, backend_factory=dying_backend, timeout=60)


def test_assemble_rejects_missing_batches():
    with pytest.raises(RuntimeError, match="batches missing"):
        driver.assemble([4], {(0, 1): {"desc": np.zeros((2, 3))}}, False)

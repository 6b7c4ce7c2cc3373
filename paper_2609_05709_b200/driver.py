"""Centre-sharded multi-GPU driver (the paper's section on multi-GPU parallelisation).

Centres are independent, so several GPUs work on one job without exchanging anything: the job is
cut into tasks (one batch of centres of one structure), task k goes to worker k mod W, every worker
is a process of its own bound to one device with its own descriptor object.  Workers report ready
once constructed and warmed up and then wait for a common start signal, so set-up stays outside the
timed region; results travel to the driver as host tensors in shared memory, keyed by (structure,
batch), and are put together there.

Everything that touches a GPU lives in the backend a worker builds (`cuda_backend`, the default,
which needs a CUDA device and the compiled library).  The bookkeeping around it is plain Python and
is tested on CPU with another backend injected.
"""
from __future__ import annotations

import time
import traceback
from dataclasses import dataclass

import numpy as np


@dataclass(frozen=True)
class Task:
    structure: int      # index into the structure list
    batch: int          # batch number inside that structure
    lo: int             # centres lo .. hi-1 of the structure
    hi: int


def enumerate_tasks(n_atoms_per_structure, batch: int):
    """The flat task list: consecutive batches of at most `batch` centres, structure by structure."""
    if batch < 1:
        raise ValueError("batch must be at least 1")
    tasks = []
    for s, n in enumerate(n_atoms_per_structure):
        for b, lo in enumerate(range(0, int(n), batch)):
            tasks.append(Task(s, b, lo, min(lo + batch, int(n))))
    return tasks


def tasks_of_rank(tasks, world: int, rank: int):
    """Static stride assignment: worker `rank` of `world` takes every world-th task."""
    return tasks[rank::world]


@dataclass
class HostResult:
    """Output for one structure, on the host."""
    descriptor: "np.ndarray"            # (N, F)
    jacobian: "np.ndarray | None"       # (rows, 3, F), rows of all centres in centre order
    row_ptr: "np.ndarray | None"        # (N+1,)
    row_atom: "np.ndarray | None"       # (rows,)


def assemble(n_atoms_per_structure, pieces, derivatives: bool):
    """Puts the per-task outputs {(structure, batch): dict} together, batches in order."""
    out = []
    for s, n in enumerate(n_atoms_per_structure):
        keys = sorted(k for k in pieces if k[0] == s)
        if [k[1] for k in keys] != list(range(len(keys))):
            raise RuntimeError(f"structure {s}: batches missing from the results")
        parts = [pieces[k] for k in keys]
        width = parts[0]["desc"].shape[1] if parts else 0
        desc = np.concatenate([np.asarray(p["desc"]) for p in parts]) if parts else np.zeros((0, width), np.float32)
        if desc.shape[0] != int(n):
            raise RuntimeError(f"structure {s}: {desc.shape[0]} descriptor rows for {n} centres")
        if not derivatives:
            out.append(HostResult(desc, None, None, None))
            continue
        jac = np.concatenate([np.asarray(p["jac"]) for p in parts]) if parts else np.zeros((0, 3, width), np.float32)
        row_atom = np.concatenate([np.asarray(p["row_atom"]) for p in parts]) if parts else np.zeros(0, np.int32)
        ptr = [np.zeros(1, np.int64)]
        base = 0
        for p in parts:
            rp = np.asarray(p["row_ptr"], np.int64)
            ptr.append(rp[1:] + base)
            base += int(rp[-1])
        out.append(HostResult(desc, jac, np.concatenate(ptr), row_atom))
    return out


def cuda_backend(rank: int, config: dict):
    """Builds the worker's descriptor object on cuda:<rank> and returns the function that runs one
    task.  Fails when there is no such device or the library is missing: there is no CPU path."""
    import torch
    from .binding import Soap
    if not torch.cuda.is_available() or rank >= torch.cuda.device_count():
        raise RuntimeError(f"worker {rank}: no CUDA device cuda:{rank}")
    torch.cuda.set_device(rank)
    soap = Soap(**config)
    resident = {}

    def on_device(s, struct):
        if s not in resident:
            resident.clear()                                   # one structure at a time stays on the device
            resident[s] = (torch.from_numpy(np.ascontiguousarray(struct.positions, np.float32)).cuda(),
                           torch.from_numpy(np.ascontiguousarray(struct.numbers, np.int32)).cuda())
        return resident[s]

    def run(s, struct, lo, hi, derivatives):
        pos, num = on_device(s, struct)
        centers = torch.arange(lo, hi, dtype=torch.int32, device="cuda")
        if derivatives:
            d = soap.derivatives(pos, num, struct.cell, centers)
            out = {"desc": d.descriptor, "jac": d.jacobian, "row_ptr": d.row_ptr, "row_atom": d.row_atom}
        else:
            out = {"desc": soap.descriptor(pos, num, struct.cell, centers)}
            soap.status()
        # one copy, device -> shared host memory the driver maps (pageable: page-locking the segment for the copy
        # with cudaHostRegister was measured and costs more than it saves when every task has buffers of its own)
        host = {k: torch.empty(v.shape, dtype=v.dtype).share_memory_() for k, v in out.items()}
        for k, v in out.items():
            host[k].copy_(v)
        return host

    # warm-up: one tiny call so that module loading and first-launch costs are paid before the start signal
    sp = [int(z) for z in config["species"]]
    wpos = torch.tensor([[0.0, 0.0, 0.0], [0.9, 0.1, 0.0], [40.0, 0.0, 0.0]], dtype=torch.float32, device="cuda")
    wnum = torch.tensor([sp[0], sp[-1], sp[0]], dtype=torch.int32, device="cuda")
    periodic = any(config.get("pbc", (False, False, False)))
    soap.derivatives(wpos, wnum, np.eye(3) * 100.0 if periodic else None)
    torch.cuda.synchronize()
    return run


def _worker(rank, world, config, structures, tasks, derivatives, backend_factory, ready_q, start_ev, result_q, done_ev):
    try:
        run = backend_factory(rank, config)
        ready_q.put(("ready", rank, None))
        start_ev.wait()
        for t in tasks_of_rank(tasks, world, rank):
            result_q.put(("task", (t.structure, t.batch), run(t.structure, structures[t.structure], t.lo, t.hi, derivatives)))
        result_q.put(("done", rank, None))
        done_ev.wait()        # shared-memory tensors stay valid until the driver has copied them
    except BaseException:     # reported to the driver, which ends the job
        msg = ("error", rank, traceback.format_exc())
        ready_q.put(msg)
        result_q.put(msg)


def _get(q, procs, timeout, what):
    """Next message from `q`; notices workers that died without reporting."""
    import queue
    deadline = time.monotonic() + timeout
    while True:
        try:
            return q.get(timeout=0.2)
        except queue.Empty:
            dead = [i for i, p in enumerate(procs) if p.exitcode not in (None, 0)]
            if dead:
                raise RuntimeError(f"worker {dead[0]} exited with code {procs[dead[0]].exitcode} while the driver waited for {what}")
            if time.monotonic() > deadline:
                raise TimeoutError(f"no message within {timeout} s while waiting for {what}")


def generate(config: dict, structures, batch: int = 1024, derivatives: bool = True, world: int | None = None,
             backend_factory=cuda_backend, timeout: float = 600.0):
    """Runs the job on `world` worker processes (default: one per visible GPU).

    config: keyword arguments of `Soap` (species, r_cut, n_max, l_max, sigma, ...).
    Returns (list of HostResult, one per structure; seconds between the start signal and the last result)."""
    import torch
    import torch.multiprocessing as mp
    if world is None:
        world = torch.cuda.device_count()
    if world < 1:
        raise RuntimeError("no CUDA device: the driver has no CPU path")
    sizes = [int(s.positions.shape[0]) for s in structures]
    tasks = enumerate_tasks(sizes, batch)
    ctx = mp.get_context("spawn")
    ready_q, result_q, start_ev, done_ev = ctx.Queue(), ctx.Queue(), ctx.Event(), ctx.Event()
    procs = [ctx.Process(target=_worker, args=(r, world, config, structures, tasks, derivatives, backend_factory,
                                               ready_q, start_ev, result_q, done_ev), daemon=True) for r in range(world)]
    for p in procs:
        p.start()
    try:
        for _ in range(world):
            kind, rank, info = _get(ready_q, procs, timeout, "the workers to report ready")
            if kind == "error":
                raise RuntimeError(f"worker {rank} failed during set-up:\n{info}")
        t0 = time.perf_counter()
        start_ev.set()
        pieces, finished = {}, 0
        while finished < world:
            kind, key, payload = _get(result_q, procs, timeout, "results")
            if kind == "error":
                raise RuntimeError(f"worker {key} failed:\n{payload}")
            if kind == "done":
                finished += 1
            else:
                pieces[key] = {k: v.numpy() for k, v in payload.items()}     # views of the shared memory, no copy
        seconds = time.perf_counter() - t0
        if len(pieces) != len(tasks):
            raise RuntimeError(f"{len(pieces)} results for {len(tasks)} tasks")
        return assemble(sizes, pieces, derivatives), seconds
    finally:
        start_ev.set()
        done_ev.set()
        for p in procs:
            p.join(timeout=10)
            if p.is_alive():
                p.terminate()

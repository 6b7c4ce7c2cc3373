#!/usr/bin/env python
"""Benchmark of the SOAP hot path: descriptor + Jacobian on the 1000-molecule water cluster.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--workload NAME]

One step = one soap_derivatives call through the C ABI: cell-list neighbour search,
expansion coefficients, power spectrum and every Jacobian row of all 3000 centres.
Prints ONE JSON line (rank 0).  With --gpus N > 1 (launched under torch.distributed.run)
every rank runs the same structure on its own GPU: the path has no exchange step, so
ranks are independent replicas and the job throughput is N x structure / slowest rank
(--shard cuts the centres of ONE structure over the ranks instead).  The same line carries the
descriptor-only half of the metric (soap_descriptor on a 1,000,002-atom cluster) with its FP32
roofline, the FP32 rate measured in the run, and the oracle timed on every host core.

--impl reference times the fp64 NumPy oracle on the host cores on a bounded sample of
the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

WORKLOADS = {
    # name: (generator, generator args, species, r_cut, n_max, l_max, sigma, rbf)
    "water1000_gto_n8_l6_rc6": ("water", 1000, [1, 8], 6.0, 8, 6, 0.5, 0),
    "water8_gto_n4_l3_rc5": ("water", 8, [1, 8], 5.0, 4, 3, 0.5, 0),
    "water300_gto_n8_l6_rc6": ("water", 300, [1, 8], 6.0, 8, 6, 0.5, 0),      # small case for ncu captures
    "chno2000_poly_n8_l8_rc5": ("box", 2000, [1, 6, 7, 8], 5.0, 8, 8, 0.4, 1),
    # the paper's own headline parameters (r_cut 10, n_max 7, l_max 3; its sigma is not given): context only
    "water1000_gto_n7_l3_rc10": ("water", 1000, [1, 8], 10.0, 7, 3, 0.5, 0),
}
DEFAULT_WORKLOAD = "water1000_gto_n8_l6_rc6"
METRIC = "SOAP atoms/s, descriptor + Jacobian"
UNIT = "atoms/s"


def kernels_per_step(n_atoms, n_centers, periodic=False):
    """Kernel launches of one soap_derivatives call over all atoms: the cell-list build (one launch up to
    16384 atoms, five above; none for a non-periodic structure of up to 512 atoms, which takes the
    brute-force pair kernel), the pair kernel, the row scan with the launch order (one launch up to 65536
    centres, three above) and the fused per-centre kernel."""
    build = 0 if (n_atoms <= 512 and not periodic) else (1 if n_atoms <= 16384 else 5)
    return build + 1 + (1 if n_centers <= 65536 else 3) + 1


# DRAM traffic of the fused kernel: ONE ncu capture on the 300-molecule cluster (profiles/center_kernel_water300.md),
# dram__bytes_read.sum + dram__bytes_write.sum of one launch, beside that launch's algorithmic bytes.  The capture
# shows no re-reads: the shortfall against the algorithmic bytes is the tail of the output that is still dirty in
# L2 when the kernel ends, a constant of the cache and not a ratio.  The full-size figure reported as `traffic` is
# therefore the full launch's algorithmic bytes minus that same residue, and says so.
NCU_CAPTURE = {"workload": "water300_gto_n8_l6_rc6", "dram_read_bytes": 1.41e6, "dram_write_bytes": 575.37e6,
               "algorithmic_bytes": 629088584}
NCU_L2_RESIDUE_BYTES = NCU_CAPTURE["algorithmic_bytes"] - NCU_CAPTURE["dram_read_bytes"] - NCU_CAPTURE["dram_write_bytes"]
DESC_ONLY_WORKLOAD = {"name": "water333334_gto_n8_l6_rc5", "molecules": 333334, "species": [1, 8], "r_cut": 5.0,
                      "n_max": 8, "l_max": 6, "sigma": 0.5}
FP32_NOMINAL_TFLOPS = 148 * 128 * 2 * 1.965e9 / 1e12


def make_structure(name):
    from soap_inputs import multispecies_box, water_cluster
    kind, n = WORKLOADS[name][:2]
    return water_cluster(n, 0) if kind == "water" else multispecies_box(n, 0)


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    return 6650.0, "fallback (6.65 TB/s, earlier measurement on this pool)"


class ClockSampler:
    """nvidia-smi clocks and throttle reasons while the timed region runs."""
    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.QUERY}",
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def _oracle_setup(name):
    from oracle.soap import SoapOracle
    kind, n, species, r_cut, n_max, l_max, sigma, rbf = WORKLOADS[name]
    s = make_structure(name)
    pbc = (True, True, True) if s.cell is not None else (False, False, False)
    return SoapOracle(species, r_cut, n_max, l_max, sigma, rbf, pbc), s


def _oracle_worker(job):
    """One process of the all-cores baseline: the oracle, NumPy held to one thread, on its share of the centres."""
    name, centers, mode = job
    from threadpoolctl import threadpool_limits
    oracle, s = _oracle_setup(name)
    call = oracle.derivatives if mode == "derivatives" else oracle.descriptor
    with threadpool_limits(limits=1):
        call(s.positions, s.numbers, s.cell, [0])                      # builds the basis caches (not timed)
        t0 = time.perf_counter()
        call(s.positions, s.numbers, s.cell, centers)
        return time.perf_counter() - t0


def oracle_rate(name, n_centers):
    """atoms/s of the fp64 oracle (descriptor + Jacobian) on evenly spaced centres: one thread."""
    from threadpoolctl import threadpool_limits
    oracle, s = _oracle_setup(name)
    oracle.derivatives(s.positions, s.numbers, s.cell, [0])            # builds the basis caches
    centers = [int(c) for c in np.linspace(0, s.n_atoms - 1, n_centers)]
    with threadpool_limits(limits=1):
        t0 = time.perf_counter()
        oracle.derivatives(s.positions, s.numbers, s.cell, centers)
        seconds = time.perf_counter() - t0
    return n_centers / seconds, seconds


def oracle_rate_all_cores(name, per_core, mode="derivatives"):
    """The same oracle in one process per host core (each on `per_core` centres of its own); the rate is all
    centres over the busy time of the slowest process."""
    import multiprocessing as mp
    from concurrent.futures import ProcessPoolExecutor
    cores = len(os.sched_getaffinity(0)) if hasattr(os, "sched_getaffinity") else (os.cpu_count() or 1)
    cores = min(cores, 64)                     # one process each; more than this only adds start-up time
    n_atoms = make_structure(name).n_atoms
    allc = [int(c) for c in np.linspace(0, n_atoms - 1, cores * per_core)]
    jobs = [(name, allc[k::cores], mode) for k in range(cores)]
    with ProcessPoolExecutor(max_workers=cores, mp_context=mp.get_context("spawn")) as pool:
        busy = list(pool.map(_oracle_worker, jobs))
    return len(allc) / max(busy), cores, max(busy), len(allc)


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    name = args.workload
    sample = 32
    from threadpoolctl import threadpool_limits
    oracle, s = _oracle_setup(name)
    centers = [int(c) for c in np.linspace(0, s.n_atoms - 1, sample)]
    times = []
    with threadpool_limits(limits=1):
        for it in range(args.warmup + args.steps):
            t0 = time.perf_counter()
            oracle.derivatives(s.positions, s.numbers, s.cell, centers)
            if it >= args.warmup:
                times.append(time.perf_counter() - t0)
    per_step = sum(times) / len(times)
    value = sample / per_step
    desc = f"{sample} evenly spaced centres of the {s.n_atoms}-atom structure per step, descriptor + Jacobian, 1 thread"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": per_step * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": config_dict(name, s),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def config_dict(name, s):
    kind, n, species, r_cut, n_max, l_max, sigma, rbf = WORKLOADS[name]
    return {"workload": name, "atoms": s.n_atoms, "centres": s.n_atoms, "species": species, "r_cut": r_cut,
            "n_max": n_max, "l_max": l_max, "sigma": sigma, "rbf": "gto" if rbf == 0 else "polynomial",
            "periodic": s.cell is not None, "outputs": "descriptor + neighbour-sparse Jacobian",
            "l2": "flushed between timed steps (256 MiB write); the 2.4 GB output also exceeds L2",
            "parallelism": "independent replicas, one structure per GPU"}


def descriptor_only_leg(pkg, torch, steps, flush):
    """The other half of the metric: soap_descriptor on the 1,000,002-atom water cluster, device-resident, CUDA
    events per step; FP32-bound, so its roofline is multiply-adds against the measured FP32 rate."""
    from soap_inputs import water_cluster
    w = DESC_ONLY_WORKLOAD
    s = water_cluster(w["molecules"], 0)
    soap = pkg.Soap(w["species"], w["r_cut"], w["n_max"], w["l_max"], w["sigma"], 0)
    n, L1, S, F, C = w["n_max"], w["l_max"] + 1, len(w["species"]), soap.n_features, s.n_atoms
    pos, num = torch.from_numpy(s.positions).cuda(), torch.from_numpy(s.numbers).cuda()
    n_pairs, _ = soap.neighbors(pos, num)
    desc = torch.empty((C, F), device="cuda")
    soap.profile(True)
    for _ in range(3):
        soap.descriptor(pos, num, None, None, out=desc)
    soap.status()
    step_ms, kern_ms, nbr_ms = [], [], []
    for _ in range(steps):
        flush.fill_(1)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        soap.descriptor(pos, num, None, None, out=desc)
        e1.record()
        e1.synchronize()
        step_ms.append(e0.elapsed_time(e1))
        a, b = soap.profile_read()
        nbr_ms.append(a)
        kern_ms.append(b)
    soap.status()
    # multiply-adds the method needs: per pair the radial channels (n (l+1) functions as sums over n primitives),
    # the harmonics (about 3 per (l, m)) and the accumulation into c (n (l+1)^2); per centre Eq. 4
    fma = n_pairs * (n * n * L1 + 3 * L1 * L1 + n * L1 * L1) + C * L1 * L1 * (S * n * (S * n + 1) // 2)
    del desc, pos, num, soap
    torch.cuda.empty_cache()
    return {"workload": w["name"], "atoms": C, "pairs": n_pairs, "features": F, "ms_per_step": statistics.mean(step_ms),
            "kernel_ms": statistics.mean(kern_ms), "neighbour_search_ms": statistics.mean(nbr_ms), "fma": fma,
            "bytes_written": C * F * 4, "steps": steps}


def run_cuda(args):
    import torch
    import torch.distributed as dist
    import paper_2609_05709_b200 as pkg
    from paper_2609_05709_b200.replicas import job_throughput, max_over_ranks, split_centers

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the product has no CPU path")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    name = args.workload
    kind, n, species, r_cut, n_max, l_max, sigma, rbf = WORKLOADS[name]
    s = make_structure(name)
    pbc = (True, True, True) if s.cell is not None else (False, False, False)
    soap = pkg.Soap(species, r_cut, n_max, l_max, sigma, rbf, pbc)
    F = soap.n_features
    # --shard: ONE structure for the whole job, every rank computes a contiguous range of its centres (no exchange:
    # a centre needs only the atoms in its own sphere); otherwise every rank runs the whole structure (replicas)
    shard = bool(args.shard) and world > 1
    c_lo, c_hi = split_centers(s.n_atoms, world, rank) if shard else (0, s.n_atoms)
    C = c_hi - c_lo
    pos_host = torch.from_numpy(s.positions).pin_memory()
    num_host = torch.from_numpy(s.numbers).pin_memory()
    pos, num = pos_host.cuda(), num_host.cuda()
    centers = torch.arange(c_lo, c_hi, dtype=torch.int32, device="cuda") if shard else None
    n_pairs, n_rows = soap.neighbors(pos, num, s.cell, centers)      # sizes scratch and the Jacobian (untimed, like construction)
    dev = {"pos": torch.empty_like(pos), "num": torch.empty_like(num),
           "desc": torch.empty((C, F), device="cuda"), "jac": torch.empty((n_rows, 3, F), device="cuda"),
           "row_ptr": torch.empty(C + 1, dtype=torch.int64, device="cuda"),
           "row_atom": torch.empty(n_rows, dtype=torch.int32, device="cuda")}
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    soap.profile(True)

    def step():
        soap.derivatives_into(pos, num, s.cell, centers, dev["desc"], dev["jac"], dev["row_ptr"], dev["row_atom"])

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # clocks are sampled from the warm-up to the end of the end-to-end leg (nvidia-smi needs a
    # moment to deliver its first line, and the device-resident region lasts only tens of ms)
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    for _ in range(max(args.warmup, 3)):
        step()
    soap.status()
    t_wait = time.time()
    while rank == 0 and sampler.proc is not None and not sampler.lines and time.time() - t_wait < 2.0:
        step()
        torch.cuda.synchronize()
    # ---- device-resident timing: per-step CUDA events on the launching stream ----
    # The timed region runs the call as a user gets it: the library records no events of its own, so the launches of a
    # step overlap each other's tails (they wait for one another on the device).
    soap.profile(False)
    barrier()
    step_ms, center_ms, nbr_ms, profiled_step_ms = [], [], [], []
    for _ in range(args.steps):
        flush.fill_(1)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        step()
        e1.record()
        e1.synchronize()
        step_ms.append(e0.elapsed_time(e1))
    barrier()
    soap.status()
    total_ms = sum(step_ms)
    # The same steps once more with the library's own events (on the same stream) before the search, between the search
    # and the per-centre kernel and after it: the durations of the two segments.  An event between two launches keeps
    # the second from starting early, so these steps are a little slower than the timed ones.
    soap.profile(True)
    for _ in range(args.steps):
        flush.fill_(1)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        step()
        e1.record()
        e1.synchronize()
        profiled_step_ms.append(e0.elapsed_time(e1))
        a, b = soap.profile_read()
        nbr_ms.append(a)
        center_ms.append(b)
    barrier()
    soap.status()
    # ---- end to end on host buffers: H2D of the inputs, compute, D2H of every output ----
    e2e_steps = 0 if args.kernel_only else max(3, min(args.steps, 10))
    host_out = {}
    if e2e_steps:
        host_out = {k: torch.empty(v.shape, dtype=v.dtype).pin_memory() for k, v in dev.items() if k not in ("pos", "num")}
        for _ in range(2):
            soap.derivatives_host(pos_host, num_host, s.cell, host_out, dev, centers)
    torch.cuda.synchronize()
    barrier()
    e2e_ms = []
    for _ in range(e2e_steps):
        flush.fill_(1)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        soap.derivatives_host(pos_host, num_host, s.cell, host_out, dev)
        e1.record()
        e1.synchronize()
        e2e_ms.append(e0.elapsed_time(e1))
    barrier()
    clocks = sampler.stop() if rank == 0 else None
    e2e_total = sum(e2e_ms)
    total_ms, e2e_total = max_over_ranks([total_ms, e2e_total], device="cuda")     # slowest rank decides
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return
    ms_per_step = total_ms / args.steps
    units, ranks = (s.n_atoms, 1) if shard else (C, world)           # sharded: the job is the one structure
    value = job_throughput(units, ranks, ms_per_step)
    e2e_value = job_throughput(units, ranks, e2e_total / e2e_steps) if e2e_steps else None
    # ---- roofline of the dominant kernel (the fused per-centre kernel): HBM-write bound ----
    # algorithmic bytes per launch: Jacobian rows + descriptor + row_atom written, pair list and positions read
    alg_bytes = n_rows * 3 * F * 4 + C * F * 4 + n_rows * 4 + n_pairs * (8 + 4 + 12) + (C + 1) * 16
    k_ms = statistics.mean(center_ms)
    peak, peak_src = measured_peaks()
    achieved = alg_bytes / (k_ms * 1e-3) / 1e9
    h2d = pos_host.numel() * 4 + num_host.numel() * 4
    d2h = sum(v.numel() * v.element_size() for v in host_out.values())
    # ---- the descriptor-only half of the metric, and the FP32 rate it is measured against ----
    fp32_tflops, fp32_ms = pkg.measure_fp32_peak()
    desc_only = None
    if not args.kernel_only and name == DEFAULT_WORKLOAD:
        del dev, host_out
        torch.cuda.empty_cache()
        desc_only = descriptor_only_leg(pkg, torch, max(3, min(args.steps, 10)), flush)
    # ---- oracle on the host cores, bounded sample: every core (one process each), and one thread ----
    n_sample = 300 if name == DEFAULT_WORKLOAD else 48
    per_core = 100 if name == DEFAULT_WORKLOAD else 16
    if args.kernel_only:
        cpu_all, cores, cpu_busy, n_all, cpu_one, cpu_one_s = None, 0, 0.0, 0, None, 0.0
    else:
        cpu_all, cores, cpu_busy, n_all = oracle_rate_all_cores(name, per_core)
        cpu_one, cpu_one_s = oracle_rate(name, n_sample)
    extra = {}
    if desc_only:
        achieved_tf = 2.0 * desc_only["fma"] / (desc_only["kernel_ms"] * 1e-3) / 1e12
        extra["desc_only"] = {"metric": "SOAP atoms/s, descriptor only", "value": desc_only["atoms"] / (desc_only["ms_per_step"] * 1e-3),
                              "unit": UNIT, "ms_per_step": desc_only["ms_per_step"], "workload": desc_only["workload"],
                              "atoms": desc_only["atoms"], "steps": desc_only["steps"]}
        extra["roofline_desc_only"] = {
            "bound": "alu", "kernel": "desc_kernel<6,8,true,true>", "achieved": achieved_tf, "peak": fp32_tflops, "unit": "TFLOP/s",
            "frac": achieved_tf / fp32_tflops, "traffic": None,
            "peak_source": f"measured in this run: register-only FP32 multiply-add loop, {fp32_ms:.2f} ms "
                           f"(nominal 148 SM x 128 lanes x 2 x 1.965 GHz = {FP32_NOMINAL_TFLOPS:.1f})",
            "algorithmic_fma_per_launch": desc_only["fma"], "fma_per_atom": desc_only["fma"] / desc_only["atoms"],
            "kernel_ms": desc_only["kernel_ms"], "neighbour_search_ms": desc_only["neighbour_search_ms"],
            "pairs": desc_only["pairs"], "hbm_floor_ms": desc_only["bytes_written"] / (peak * 1e9) * 1e3,
            "fp32_floor_ms": 2.0 * desc_only["fma"] / (fp32_tflops * 1e12) * 1e3}
    print(json.dumps({
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "strong" if shard else "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic", "config": dict(config_dict(name, s), **({"parallelism": f"centres of one structure sharded over {world} GPUs, no exchange"} if shard else {})),
        "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "ms_per_step": e2e_total / e2e_steps if e2e_steps else None, "steps": e2e_steps},
        "gpu_launches": kernels_per_step(C, C, s.cell is not None) * args.steps,
        "roofline": {"bound": "hbm", "kernel": f"center_kernel<1,{l_max},{n_max},true>", "achieved": achieved, "peak": peak, "unit": "GB/s",
                     "frac": achieved / peak, "peak_source": peak_src, "peak_nominal": 8000.0,
                     "frac_of_nominal": achieved / 8000.0,
                     "traffic": alg_bytes - NCU_L2_RESIDUE_BYTES,
                     "traffic_source": "not measured in this run: algorithmic bytes of this launch minus the L2 residue "
                                       f"({NCU_L2_RESIDUE_BYTES / 1e6:.1f} MB still dirty in L2 at kernel end) seen in the one "
                                       "ncu capture on the 300-molecule cluster, which showed no re-reads",
                     "traffic_capture": NCU_CAPTURE,
                     "algorithmic_bytes_per_launch": alg_bytes, "kernel_ms": k_ms,
                     "neighbour_search_ms": statistics.mean(nbr_ms),
                     "kernel_timing": f"library CUDA events on the launching stream over a second pass of the same {args.steps} steps "
                                      "(an event between two launches keeps the second from starting early, so the timed "
                                      "region itself runs without them)",
                     "ms_per_step_with_events": statistics.mean(profiled_step_ms),
                     "pairs": n_pairs, "rows": n_rows, "features": F},
        "fp32_peak": {"measured_tflops": fp32_tflops, "nominal_tflops": FP32_NOMINAL_TFLOPS, "loop_ms": fp32_ms},
        **extra,
        "cpu_baseline": {"value": cpu_all, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": f"{n_all} evenly spaced centres of the same structure, descriptor + Jacobian, one process "
                                   f"per core (NumPy held to 1 thread each), slowest process busy {cpu_busy:.1f} s",
                         "one_thread": {"value": cpu_one, "cores": 1,
                                        "sample": f"{n_sample} evenly spaced centres, {cpu_one_s:.1f} s"}},
        "paper_context": "GB200, r_cut=10, n_max=7, l_max=3: 0.15 s for (H2O)_1000 = 2.0e4 atoms/s (other machine and parameters)",
    }))
    if world > 1:
        dist.destroy_process_group()


def time_case(struct, species, r_cut, n_max, l_max, sigma, rbf, mode, steps, warmup=3, crossover=True):
    """Device-resident timing of one configuration; returns a dict (one row of the measured tables)."""
    import torch
    import paper_2609_05709_b200 as pkg
    pbc = (True, True, True) if struct.cell is not None else (False, False, False)
    soap = pkg.Soap(species, r_cut, n_max, l_max, sigma, rbf, pbc, crossover=crossover)
    F, C, W = soap.n_features, struct.n_atoms, soap.n_coefficients
    pos = torch.from_numpy(struct.positions).cuda()
    num = torch.from_numpy(struct.numbers).cuda()
    n_pairs, n_rows = soap.neighbors(pos, num, struct.cell)
    desc = torch.empty((C, F), device="cuda")
    if mode == "derivatives":
        jac = torch.empty((n_rows, 3, F), device="cuda")
        row_ptr = torch.empty(C + 1, dtype=torch.int64, device="cuda")
        row_atom = torch.empty(n_rows, dtype=torch.int32, device="cuda")
        step = lambda: soap.derivatives_into(pos, num, struct.cell, None, desc, jac, row_ptr, row_atom)
        alg_bytes = n_rows * 3 * F * 4 + C * F * 4 + n_rows * 4 + n_pairs * 24 + (C + 1) * 16
    elif mode == "derivatives_compact":
        pitch = soap.compact_pitch
        own = torch.empty((C, 3, F), device="cuda")
        jac = torch.empty((n_rows, 3, pitch), device="cuda")
        row_ptr = torch.empty(C + 1, dtype=torch.int64, device="cuda")
        row_atom = torch.empty(n_rows, dtype=torch.int32, device="cuda")
        step = lambda: soap.derivatives_compact_into(pos, num, struct.cell, None, desc, own, jac, row_ptr, row_atom)
        alg_bytes = n_rows * 3 * pitch * 4 + C * 3 * F * 4 + C * F * 4 + n_rows * 4 + n_pairs * 24 + (C + 1) * 16
    elif mode == "descriptor":
        step = lambda: soap.descriptor(pos, num, struct.cell, None, out=desc)
        alg_bytes = C * F * 4 + n_pairs * 24 + (C + 1) * 8
    elif mode == "coefficients":
        coeff = torch.empty((C, W), device="cuda")
        step = lambda: soap.coefficients(pos, num, struct.cell, None, out=coeff)
        alg_bytes = C * W * 4 + n_pairs * 24 + (C + 1) * 8
    elif mode == "coefficient_derivatives":
        coeff = torch.empty((C, W), device="cuda")
        jac = torch.empty((n_rows, 3, W), device="cuda")
        row_ptr = torch.empty(C + 1, dtype=torch.int64, device="cuda")
        row_atom = torch.empty(n_rows, dtype=torch.int32, device="cuda")
        cellp = soap._cell(struct.cell)
        step = lambda: soap._check(soap._lib.soap_coefficient_derivatives(
            soap._h, pos.data_ptr(), num.data_ptr(), C, cellp[1], None, C, coeff.data_ptr(), jac.data_ptr(), n_rows,
            row_ptr.data_ptr(), row_atom.data_ptr(), soap._stream()))
        alg_bytes = n_rows * 3 * W * 4 + C * W * 4 + n_rows * 4 + n_pairs * 24 + (C + 1) * 16
    elif mode in ("average_inner", "average_outer"):
        avg = torch.empty(F, device="cuda")
        step = lambda: soap.descriptor_average(mode[8:], pos, num, struct.cell, None, out=avg)
        alg_bytes = F * 4 + n_pairs * 24 + (C + 1) * 8
    else:
        # averaged Jacobian: what must move is the result (with every atom a centre, as here, the kernels write one row
        # per atom and nothing per pair; only centre subsets still pass per-centre rows through a workspace)
        avg = torch.empty(F, device="cuda")
        jac = torch.empty((C, 3, F), device="cuda")
        step = lambda: soap.derivatives_average(mode[8:13], pos, num, struct.cell, None, out_desc=avg, out_jac=jac)
        alg_bytes = C * 3 * F * 4 + F * 4 + n_pairs * 24 + (C + 1) * 8
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    for _ in range(warmup):
        step()
    soap.status()
    # first the steps as a user gets them (no events inside the call: its launches overlap each other's tails), then
    # the same steps with the library's events for the durations of the search and of the per-centre kernel
    total, kern, nbr = [], [], []
    for profiled in (False, True):
        soap.profile(profiled)
        for _ in range(steps):
            flush.fill_(1)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            step()
            e1.record()
            e1.synchronize()
            if not profiled:
                total.append(e0.elapsed_time(e1))
            else:
                a, b = soap.profile_read()
                nbr.append(a)
                kern.append(b)
    soap.status()
    ms = statistics.median(total)
    peak, _ = measured_peaks()
    k_ms = statistics.median(kern)
    out = {"mode": mode, "crossover": bool(crossover), "atoms": C, "n_max": n_max, "l_max": l_max, "features": F, "pairs": n_pairs, "rows": n_rows,
           "ms_per_step": ms, "atoms_per_s": C / (ms * 1e-3), "kernel_ms": k_ms, "neighbour_search_ms": statistics.median(nbr),
           "algorithmic_bytes": alg_bytes, "kernel_GBps": alg_bytes / (k_ms * 1e-3) / 1e9,
           "hbm_frac_of_measured_peak": alg_bytes / (k_ms * 1e-3) / 1e9 / peak}
    del soap
    torch.cuda.empty_cache()
    return out


def run_suite(args):
    import torch
    from soap_inputs import multispecies_box, water_cluster
    if args.suite != "cpu":
        torch.cuda.set_device(0)
    steps = args.steps
    if args.suite == "map":
        s = water_cluster(1000, 0)
        for n_max in (2, 4, 6, 8, 10, 12):
            for l_max in (2, 4, 6, 8, 10, 12):
                r = time_case(s, [1, 8], 6.0, n_max, l_max, 0.5, 0, "derivatives", steps)
                r["case"] = "map"
                print(json.dumps(r), flush=True)
    elif args.suite in ("scaling", "desc30k"):
        for n_mol in ((10000,) if args.suite == "desc30k" else (1000, 10000, 100000, 333334)):
            s = water_cluster(n_mol, 0)
            r = time_case(s, [1, 8], 5.0, 8, 6, 0.5, 0, "descriptor", steps)
            r["case"] = "scaling"
            print(json.dumps(r), flush=True)
    elif args.suite == "driver":
        # the multi-process driver on the GPUs of this machine (one worker per GPU): wall time between the
        # start signal and the last result on the host, results travelling through shared memory
        from paper_2609_05709_b200 import driver
        s = water_cluster(1000, 0)
        config = dict(species=[1, 8], r_cut=6.0, n_max=8, l_max=6, sigma=0.5)
        world = max(1, min(args.gpus, torch.cuda.device_count()))
        for derivatives, batch in ((True, 256), (True, 1024), (False, 1024)):
            best = None
            for _ in range(max(1, min(steps, 3))):
                _, seconds = driver.generate(config, [s], batch=batch, derivatives=derivatives, world=world)
                best = seconds if best is None else min(best, seconds)
            print(json.dumps({"case": "driver", "workers": world, "atoms": s.n_atoms, "batch": batch,
                              "mode": "derivatives" if derivatives else "descriptor", "seconds": best,
                              "atoms_per_s": s.n_atoms / best}), flush=True)
    elif args.suite == "graph":
        # launch-bound small systems: one planned step recorded in a CUDA graph and replayed
        import paper_2609_05709_b200 as pkg
        for name in ("water8_gto_n4_l3_rc5", "water300_gto_n8_l6_rc6"):
            kind, n, species, r_cut, n_max, l_max, sigma, rbf = WORKLOADS[name]
            st = make_structure(name)
            soap = pkg.Soap(species, r_cut, n_max, l_max, sigma, rbf)
            pos, num = torch.from_numpy(st.positions).cuda(), torch.from_numpy(st.numbers).cuda()
            C, F = st.n_atoms, soap.n_features
            _, n_rows = soap.neighbors(pos, num)
            desc = torch.empty((C, F), device="cuda")
            jac = torch.empty((n_rows, 3, F), device="cuda")
            row_ptr = torch.empty(C + 1, dtype=torch.int64, device="cuda")
            row_atom = torch.empty(n_rows, dtype=torch.int32, device="cuda")
            step = lambda: soap.derivatives_into(pos, num, None, None, desc, jac, row_ptr, row_atom)
            for _ in range(3):
                step()
            torch.cuda.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph):
                step()
            out = {"case": "graph", "workload": name, "atoms": C}
            for label, fn in (("direct_ms", step), ("graph_replay_ms", graph.replay)):
                for _ in range(5):
                    fn()
                times = []
                for _ in range(max(steps, 20)):
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    e0.record()
                    fn()
                    e1.record()
                    e1.synchronize()
                    times.append(e0.elapsed_time(e1))
                out[label] = statistics.median(times)
            soap.status()
            print(json.dumps(out), flush=True)
    elif args.suite == "small":
        # a stream of different small structures (launch-bound): descriptor + Jacobian of 256 eight-molecule water
        # clusters, every structure into buffers of its own, on one stream and round-robin over eight streams
        # (one library handle per stream; after the first call nothing allocates or waits)
        import paper_2609_05709_b200 as pkg
        structs = [water_cluster(8, seed) for seed in range(256)]
        n, cap_rows = structs[0].n_atoms, structs[0].n_atoms ** 2
        pos = [torch.from_numpy(st.positions).cuda() for st in structs]
        num = torch.from_numpy(structs[0].numbers).cuda()
        for n_streams in (1, 8):
            streams = [torch.cuda.Stream() for _ in range(n_streams)]
            handles = [pkg.Soap([1, 8], 5.0, 4, 3, 0.5, 0) for _ in range(n_streams)]
            F = handles[0].n_features
            outs = [(torch.empty((n, F), device="cuda"), torch.empty((cap_rows, 3, F), device="cuda"),
                     torch.empty(n + 1, dtype=torch.int64, device="cuda"), torch.empty(cap_rows, dtype=torch.int32, device="cuda"))
                    for _ in structs]
            for h, st in zip(handles, streams):                 # plan once per handle, outside the timing
                with torch.cuda.stream(st):
                    h.neighbors(pos[0], num)
            torch.cuda.synchronize()

            def sweep():
                for k, p_k in enumerate(pos):
                    with torch.cuda.stream(streams[k % n_streams]):
                        handles[k % n_streams].derivatives_into(p_k, num, None, None, *outs[k])

            sweep()
            torch.cuda.synchronize()
            for h in handles:
                h.status()
            best = None
            for _ in range(max(3, min(steps, 10))):
                t0 = time.perf_counter()
                sweep()
                torch.cuda.synchronize()
                dt = time.perf_counter() - t0
                best = dt if best is None else min(best, dt)
            print(json.dumps({"case": "small", "structures": len(structs), "atoms_each": n, "streams": n_streams,
                              "seconds": best, "structures_per_s": len(structs) / best,
                              "atoms_per_s": len(structs) * n / best, "us_per_structure": 1e6 * best / len(structs)}), flush=True)
        # the same structures (and 16 times as many) as ONE list of atoms through the batch entry point
        for copies in (1, 16):
            soap = pkg.Soap([1, 8], 5.0, 4, 3, 0.5, 0)
            allpos = torch.cat(pos * copies).contiguous()
            allnum = num.repeat(len(structs) * copies).contiguous()
            ptr = torch.arange(0, (len(structs) * copies + 1) * n, n, dtype=torch.int64, device="cuda")
            N = allpos.shape[0]
            import ctypes
            npairs, nrows = ctypes.c_int64(), ctypes.c_int64()
            soap._check(soap._lib.soap_neighbors_batch(soap._h, allpos.data_ptr(), allnum.data_ptr(), N, ptr.data_ptr(),
                                                       ptr.shape[0] - 1, ctypes.byref(npairs), ctypes.byref(nrows), soap._stream()))
            F = soap.n_features
            desc = torch.empty((N, F), device="cuda")
            jac = torch.empty((nrows.value, 3, F), device="cuda")
            row_ptr = torch.empty(N + 1, dtype=torch.int64, device="cuda")
            row_atom = torch.empty(nrows.value, dtype=torch.int32, device="cuda")
            call = lambda: soap._check(soap._lib.soap_derivatives_batch(
                soap._h, allpos.data_ptr(), allnum.data_ptr(), N, ptr.data_ptr(), ptr.shape[0] - 1, desc.data_ptr(),
                jac.data_ptr(), nrows.value, row_ptr.data_ptr(), row_atom.data_ptr(), soap._stream()))
            for _ in range(3):
                call()
            soap.status()
            times = []
            for _ in range(max(steps, 10)):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                call()
                e1.record()
                e1.synchronize()
                times.append(e0.elapsed_time(e1) * 1e-3)
            best = statistics.median(times)
            nst = len(structs) * copies
            print(json.dumps({"case": "small", "structures": nst, "atoms_each": n, "streams": "one batch call",
                              "seconds": best, "structures_per_s": nst / best, "atoms_per_s": nst * n / best,
                              "us_per_structure": 1e6 * best / nst, "rows": nrows.value,
                              "jacobian_GBps": nrows.value * 3 * F * 4 / best / 1e9}), flush=True)
            del soap, desc, jac
    elif args.suite == "cpu":
        # the fp64 oracle as it stands on all host cores, per configuration (a reported baseline: it runs no GPU code)
        cores = min(len(os.sched_getaffinity(0)) if hasattr(os, "sched_getaffinity") else (os.cpu_count() or 1), 64)
        for name, per_core in (("water8_gto_n4_l3_rc5", (3, 3)), ("water1000_gto_n8_l6_rc6", (100, 300)),
                               ("chno2000_poly_n8_l8_rc5", (24, 96)), ("water1000_gto_n7_l3_rc10", (40, 300))):
            for mode, pc in zip(("derivatives", "descriptor"), per_core):
                n_atoms = make_structure(name).n_atoms
                rate, used, busy, n = oracle_rate_all_cores(name, max(1, min(pc, n_atoms // cores)), mode)
                print(json.dumps({"case": name, "mode": mode, "atoms": n_atoms, "oracle_atoms_per_s": rate, "cores": used,
                                  "centres_timed": n, "slowest_process_s": busy}), flush=True)
    elif args.suite == "compact":
        for name in ("water1000_gto_n8_l6_rc6", "chno2000_poly_n8_l8_rc5"):
            kind, n, species, r_cut, n_max, l_max, sigma, rbf = WORKLOADS[name]
            s = make_structure(name)
            for mode in ("derivatives", "derivatives_compact"):
                r = time_case(s, species, r_cut, n_max, l_max, sigma, rbf, mode, steps)
                r["case"] = name
                print(json.dumps(r), flush=True)
    elif args.suite == "modes":
        # on --workload (default: the 1000-molecule cluster; the 300-molecule one is small enough for profiler captures)
        kind, n, species, r_cut, n_max, l_max, sigma, rbf = WORKLOADS[args.workload]
        s = make_structure(args.workload)
        base = (species, r_cut, n_max, l_max, sigma, rbf)
        for mode, crossover in (("derivatives", False), ("descriptor", False), ("coefficients", True),
                                ("coefficient_derivatives", True), ("average_inner", True), ("average_outer", True),
                                ("average_inner_derivatives", True), ("average_outer_derivatives", True)):
            r = time_case(s, *base, mode, steps, crossover=crossover)
            r["case"] = "modes"
            print(json.dumps(r), flush=True)
    else:
        for name in ("water8_gto_n4_l3_rc5", "water1000_gto_n8_l6_rc6", "chno2000_poly_n8_l8_rc5", "water1000_gto_n7_l3_rc10"):
            kind, n, species, r_cut, n_max, l_max, sigma, rbf = WORKLOADS[name]
            s = make_structure(name)
            for mode in ("derivatives", "descriptor"):
                r = time_case(s, species, r_cut, n_max, l_max, sigma, rbf, mode, steps)
                r["case"] = name
                print(json.dumps(r), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(WORKLOADS))
    ap.add_argument("--shard", action="store_true",
                    help="with --gpus N > 1: shard the centres of ONE structure over the ranks (strong scaling) "
                         "instead of running N independent replicas")
    ap.add_argument("--kernel-only", action="store_true",
                    help="skip the end-to-end and CPU-baseline legs (for profiler captures)")
    ap.add_argument("--suite", choices=["map", "scaling", "configs", "desc30k", "modes", "driver", "compact", "graph", "small", "cpu"],
                    help="extra measurements beside the headline line: 'map' = descriptor+Jacobian over "
                         "n_max x l_max on the 1000-molecule cluster, 'scaling' = descriptor-only on "
                         "3k..1M atoms, 'configs' = the periodic multi-species box and the tiny cluster, "
                         "'desc30k' = descriptor-only on 30,000 atoms alone (small enough for profiler captures), "
                         "'compact' = species-compact against full Jacobian rows on the water cluster and the four-species box, "
                         "'small' = a stream of 256 different 24-atom structures on one and on eight CUDA streams, "
                         "'graph' = a planned step replayed from a CUDA graph on the small clusters, "
                         "'driver' = the multi-process driver with --gpus workers, results on the host, "
                         "'modes' = crossover off, coefficient mode and the averaged modes on the 1000-molecule cluster; "
                         "prints one JSON line per case")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    elif args.suite:
        run_suite(args)
    else:
        run_cuda(args)


if __name__ == "__main__":
    main()

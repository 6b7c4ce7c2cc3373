"""Builds libsoap_b200.so in-tree: nvcc for sm_100a, g++ for the quad-precision host part."""
from __future__ import annotations

import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
INCLUDE = os.path.join(os.path.dirname(HERE), "include")
LIB = os.path.join(HERE, "libsoap_b200.so")

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-lineinfo", "-std=c++17",
              "--expt-relaxed-constexpr", "-Xcompiler", "-fPIC", "-Xptxas", "-v", "-Xfatbin=-compress-all"]
# compiled in parallel, the longest first (compile time grows with l_max): the per-centre kernels are compiled
# once per l_max from one source each (-DSOAP_L=<l_max>)
PER_L_SOURCES = ["center_kernels", "desc_kernels"]
PLAIN_UNITS = ["soap_api", "peak_kernel"]


def _newer(target, sources):
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(s) > t for s in sources)


def _run(cmd, verbose, log):
    res = subprocess.run(cmd, capture_output=True, text=True)
    log.append(" ".join(cmd) + "\n" + res.stdout + res.stderr)
    if res.returncode != 0:
        sys.stderr.write(log[-1])
        raise RuntimeError("build failed: " + " ".join(cmd))


def build(force: bool = False, verbose: bool = False) -> str:
    sources = [os.path.join(CSRC, f) for f in sorted(os.listdir(CSRC)) if not f.endswith(".o")]
    sources.append(os.path.join(INCLUDE, "soap.h"))
    if not force and not _newer(LIB, sources):
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    obj = lambda name: os.path.join(CSRC, name + ".o")
    cmds = [["g++", "-O2", "-std=gnu++17", "-fPIC", "-ffp-contract=off", "-I", INCLUDE, "-I", CSRC,
             "-c", os.path.join(CSRC, "basis_host.cpp"), "-o", obj("basis_host")]]
    objects = []
    for l in range(12, -1, -1):
        for src in PER_L_SOURCES:
            name = f"{src}_l{l}"
            objects.append(name)
            cmds.append([nvcc, *NVCC_FLAGS, f"-DSOAP_L={l}", "-I", INCLUDE, "-I", CSRC, "-c", os.path.join(CSRC, src + ".cu"), "-o", obj(name)])
    for unit in PLAIN_UNITS:
        objects.append(unit)
        cmds.append([nvcc, *NVCC_FLAGS, "-I", INCLUDE, "-I", CSRC, "-c", os.path.join(CSRC, unit + ".cu"), "-o", obj(unit)])
    log = []
    with ThreadPoolExecutor(max_workers=min(len(cmds), os.cpu_count() or 4)) as pool:
        list(pool.map(lambda c: _run(c, verbose, log), cmds))
    _run([nvcc, "-shared", "-o", LIB, *[obj(u) for u in objects], obj("basis_host"), "-lquadmath", "-cudart", "static"],
         verbose, log)
    if verbose:
        sys.stderr.write("\n".join(log))
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose=True))

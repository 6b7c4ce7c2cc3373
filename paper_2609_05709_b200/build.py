"""Builds libsoap_b200.so in-tree: nvcc for sm_100a, g++ for the quad-precision host part."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
INCLUDE = os.path.join(os.path.dirname(HERE), "include")
LIB = os.path.join(HERE, "libsoap_b200.so")

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-lineinfo", "-std=c++17",
              "--expt-relaxed-constexpr", "-Xcompiler", "-fPIC", "-Xptxas", "-v"]


def _newer(target, sources):
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(s) > t for s in sources)


def build(force: bool = False, verbose: bool = False) -> str:
    sources = [os.path.join(CSRC, f) for f in sorted(os.listdir(CSRC))] + [os.path.join(INCLUDE, "soap.h")]
    if not force and not _newer(LIB, sources):
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    obj_host = os.path.join(CSRC, "basis_host.o")
    obj_api = os.path.join(CSRC, "soap_api.o")
    cmds = [
        ["g++", "-O2", "-std=gnu++17", "-fPIC", "-ffp-contract=off", "-I", INCLUDE, "-I", CSRC,
         "-c", os.path.join(CSRC, "basis_host.cpp"), "-o", obj_host],
        [nvcc, *NVCC_FLAGS, "-I", INCLUDE, "-I", CSRC, "-c", os.path.join(CSRC, "soap_api.cu"), "-o", obj_api],
        [nvcc, "-shared", "-o", LIB, obj_api, obj_host, "-lquadmath", "-cudart", "static"],
    ]
    for cmd in cmds:
        res = subprocess.run(cmd, capture_output=True, text=True)
        if verbose or res.returncode != 0:
            sys.stderr.write(" ".join(cmd) + "\n" + res.stdout + res.stderr)
        if res.returncode != 0:
            raise RuntimeError("build failed: " + " ".join(cmd))
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose=True))

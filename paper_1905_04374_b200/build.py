"""Builds libgar.so (sm_100a) in-tree with nvcc.  `python -m paper_1905_04374_b200.build`."""
from __future__ import annotations

import os
import shutil
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
CSRC = os.path.join(PKG, "csrc")
OBJ = os.path.join(PKG, "_build")
LIB = os.path.join(PKG, "libgar.so")

# Slot counts the coordinate kernel is compiled for: keep identical to K3_P_LIST in k3_dispatch.cu.
K3_P = list(range(1, 33)) + [36, 40, 44, 48, 52, 56, 60, 64]     # <= 32: theta fixed at compile time

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-I" + os.path.join(ROOT, "include"), "-I" + CSRC]


def _nvcc() -> str:
    exe = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(exe):
        raise RuntimeError("nvcc not found: the CUDA toolkit is needed to build libgar.so")
    return exe


def _units():
    units = [("k1_distances.cu", "k1_distances.o", []),
             ("k1_umma.cu", "k1_umma.o", []),
             ("k2_select.cu", "k2_select.o", []),
             ("k3_dispatch.cu", "k3_dispatch.o", []),
             ("gar_api.cu", "gar_api.o", [])]
    for p in K3_P:
        units.append(("k3_inst.cu", f"k3_inst_{p}.o", [f"-DK3_P={p}", f"-DK3_EXACT={1 if p <= 32 else 0}"]))
    return units


def _newest_header() -> float:
    hdrs = [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".cuh", ".h"))]
    hdrs.append(os.path.join(ROOT, "include", "gar.h"))
    hdrs.append(os.path.abspath(__file__))
    return max(os.path.getmtime(h) for h in hdrs)


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile every translation unit that is out of date and link libgar.so."""
    os.makedirs(OBJ, exist_ok=True)
    nvcc = _nvcc()
    hdr_time = _newest_header()
    jobs = []
    for src, obj, extra in _units():
        s, o = os.path.join(CSRC, src), os.path.join(OBJ, obj)
        if force or not os.path.exists(o) or os.path.getmtime(o) < max(os.path.getmtime(s), hdr_time):
            jobs.append([nvcc, *NVCC_FLAGS, *extra, "-c", s, "-o", o])

    def run(cmd):
        res = subprocess.run(cmd, capture_output=True, text=True)
        if res.returncode != 0:
            raise RuntimeError("nvcc failed: " + " ".join(cmd) + "\n" + res.stdout + res.stderr)
        if verbose and (res.stdout or res.stderr):
            print(res.stdout + res.stderr)

    if jobs:
        with ThreadPoolExecutor(max_workers=min(len(jobs), os.cpu_count() or 4)) as ex:
            list(ex.map(run, jobs))
    objs = [os.path.join(OBJ, obj) for _, obj, _ in _units()]
    if jobs or not os.path.exists(LIB):
        run([nvcc, "-shared", "-o", LIB, *objs, "-gencode", "arch=compute_100a,code=sm_100a"])
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose=True))

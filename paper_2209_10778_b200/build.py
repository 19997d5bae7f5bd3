"""Builds libnfad.so (the C-ABI CUDA library) in-tree with nvcc for sm_100a.

    python -m paper_2209_10778_b200.build          # rebuild if sources are newer
    python -m paper_2209_10778_b200.build --force

Seven translation units: the fp32-storage kernels are compiled with
floating-point contraction OFF (their compensated arithmetic depends on every
fused multiply-add being written out), the 16-bit-storage kernels and the run-time
sequences with it on, the bias-gradient kernels (explicitly rounded intrinsics only),
the extern "C" boundary, the host-memory pipeline and the run-time compiler of FAD sequences (no kernels of their own).  No fast-math, no flush-to-zero, IEEE division:
subnormal inputs and results are part of the contract.
"""
from __future__ import annotations

import glob
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libnfad.so")
OBJ_DIR = os.path.join(HERE, "build")

ARCH = ["-gencode", "arch=compute_100a,code=sm_100a"]
COMMON = ["-O3", "-std=c++17", "-lineinfo", "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden",
          "--ftz=false", "--prec-div=true", "--prec-sqrt=true"]
UNITS = [
    ("nfad_kernels_f32.cu", ["-fmad=false"]),
    ("nfad_kernels_16.cu", ["-fmad=true"]),
    ("nfad_kernels_seq.cu", ["-fmad=true"]),
    ("nfad_kernels_bias.cu", ["-fmad=false"]),
    ("nfad_api.cu", ["-fmad=false"]),
    ("nfad_host.cu", ["-fmad=false"]),
    ("nfad_jit.cu", ["-fmad=false"]),
]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.sep not in cand or os.path.exists(cand)):
            return cand
    raise RuntimeError("nvcc not found")


def _sources():
    return glob.glob(os.path.join(CSRC, "*.cu")) + glob.glob(os.path.join(CSRC, "*.cuh")) + \
        glob.glob(os.path.join(CSRC, "*.h")) + [os.path.join(HERE, "..", "include", "nfad.h"), __file__]


def is_stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    return any(os.path.getmtime(s) > t for s in _sources())


def build_library(force: bool = False, verbose: bool = False) -> str:
    if not force and not is_stale():
        return LIB
    os.makedirs(OBJ_DIR, exist_ok=True)
    nvcc = _nvcc()
    objs = []
    procs = []
    for src, extra in UNITS:
        obj = os.path.join(OBJ_DIR, src.replace(".cu", ".o"))
        cmd = [nvcc, *ARCH, *COMMON, *extra, "-c", os.path.join(CSRC, src), "-o", obj]
        if verbose:
            cmd.insert(1, "-Xptxas=-v")
            print(" ".join(cmd), flush=True)
        procs.append((cmd, subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
        objs.append(obj)
    for cmd, p in procs:
        out, _ = p.communicate()
        if verbose and out:
            print(out)
        if p.returncode != 0:
            raise RuntimeError("nvcc failed:\n" + " ".join(cmd) + "\n" + (out or ""))
    # the extern "C" entry points are the only exported symbols
    link = [nvcc, *ARCH, "-shared", "-o", LIB, *objs, "-Xcompiler", "-fPIC", "-cudart", "static", "-ldl"]
    r = subprocess.run(link, capture_output=True, text=True)
    if r.returncode != 0:
        raise RuntimeError("link failed:\n" + r.stdout + r.stderr)
    return LIB


if __name__ == "__main__":
    print(build_library(force="--force" in sys.argv, verbose="-v" in sys.argv))

"""Builds librabit.so (the C-ABI CUDA library) in-tree with nvcc for sm_100a.

Usage: ``python paper_2602_05367_b200/build.py [--force] [--verbose]`` (run as a script: importing the
package needs the library to exist already).
"""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "librabit.so")
LIB_TRACE = os.path.join(HERE, "librabit_trace.so")          # the same sources with -DRABIT_TRACE (phase stamps)
LIB_CHECKED = os.path.join(HERE, "librabit_checked.so")      # the same sources with -DRABIT_CHECKED (index checks in the decode kernels)
SOURCES = ["rabit_api.cu", "rabit_pack.cu", "rabit_gemv_plain.cu", "rabit_gemv_mma.cu", "rabit_gemv_lut.cu", "rabit_gemv_f16.cu", "rabit_gemm_tc.cu",
           "rabit_noalloc.cu", "rabit_derive.cu", "rabit_selftest.cu"]
NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden", "-shared", "-cudart", "static",
]


def _sources():
    return [os.path.join(CSRC, s) for s in SOURCES if os.path.exists(os.path.join(CSRC, s))]


def needs_build() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = _sources() + [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith(".h")]
    deps.append(os.path.join(HERE, "..", "include", "rabit.h"))
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False, trace: bool = False, checked: bool = False) -> str:
    if not trace and not checked and not force and not needs_build():
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    out = LIB_TRACE if trace else LIB_CHECKED if checked else LIB
    cmd = [nvcc] + NVCC_FLAGS + (["-DRABIT_TRACE"] if trace else []) + (["-DRABIT_CHECKED"] if checked else []) + (["-Xptxas", "-v"] if verbose else []) + ["-o", out] + _sources()
    proc = subprocess.run(cmd, capture_output=True, text=True)
    if verbose or proc.returncode != 0:
        sys.stderr.write(proc.stdout + proc.stderr)
    if proc.returncode != 0:
        raise RuntimeError("nvcc failed building librabit.so")
    return out


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv, trace="--trace" in sys.argv, checked="--checked" in sys.argv))

"""Builds libbbo_mlp_cv.so (the C-ABI CUDA library) in-tree with nvcc for sm_100a.

The fit kernel is a template on the class count; each class count is its own translation
unit (``fit_inst.cu -DBBO_CT=n``) so the objects compile in parallel.
"""
from __future__ import annotations

import concurrent.futures
import os
import shutil
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
OBJ = os.path.join(HERE, "_build")
LIB = os.path.join(HERE, "libbbo_mlp_cv.so")
HEADERS = ["fit_kernel.cuh", "sm100_primitives.cuh", "fit_common.cuh", "aux_kernels.cuh", "device_math.cuh", "fit_launch.h",
           os.path.join("..", "..", "include", "bbo_mlp_cv.h")]
CLASS_COUNTS = list(range(1, 17))
FAST_WIDTHS = list(range(56, 201, 8))   # padded hidden widths with compile-time strides

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a",
    "-O3", "-lineinfo", "-std=c++17",
    "-fmad=false",            # contraction only where the source says fmaf
    "-prec-div=true", "-prec-sqrt=true", "-ftz=false",
    "-Xcompiler", "-fPIC",
]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found; the CUDA library cannot be built")


def _units():
    units = [("bbo_mlp_cv.cu", [], "bbo_mlp_cv.o"), ("fit_dispatch.cu", [], "fit_dispatch.o")]
    units += [("fit_fast.cu", [f"-DBBO_HSC={h}"], f"fit_fast_{h}.o") for h in reversed(FAST_WIDTHS)]
    units += [("fit_inst.cu", [f"-DBBO_CT={c}"], f"fit_inst_{c}.o") for c in CLASS_COUNTS]
    return units


def _deps():
    srcs = ["bbo_mlp_cv.cu", "fit_dispatch.cu", "fit_inst.cu", "fit_fast.cu"] + HEADERS
    return [os.path.join(CSRC, s) for s in srcs] + [os.path.abspath(__file__)]


def needs_build() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    return any(os.path.getmtime(p) > t for p in _deps())


def _compile(nvcc, src, defs, obj, verbose):
    cmd = [nvcc] + NVCC_FLAGS + defs + (["-Xptxas", "-v"] if verbose else [])
    cmd += ["-c", os.path.join(CSRC, src), "-o", os.path.join(OBJ, obj)]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError(f"nvcc failed on {src} {defs}:\n{res.stdout}{res.stderr}")
    return res.stderr


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not needs_build():
        return LIB
    nvcc = _nvcc()
    os.makedirs(OBJ, exist_ok=True)
    units = _units()
    workers = min(len(units), max(1, (os.cpu_count() or 2)))
    with concurrent.futures.ThreadPoolExecutor(workers) as pool:
        logs = list(pool.map(lambda u: _compile(nvcc, u[0], u[1], u[2], verbose), units))
    if verbose:
        sys.stderr.write("".join(logs))
    link = [nvcc, "-shared", "-gencode", "arch=compute_100a,code=sm_100a", "-o", LIB]
    link += [os.path.join(OBJ, u[2]) for u in units]
    res = subprocess.run(link, capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("link failed:\n" + res.stdout + res.stderr)
    return LIB


if __name__ == "__main__":
    print(build(force=True, verbose="-v" in sys.argv))

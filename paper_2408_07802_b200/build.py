"""Builds the library in-tree with nvcc for sm_100a; usable without a GPU (cross-compiles).

Two images come out of the same sources: libkraken.so stores weights, activations and the KV cache as
bfloat16; libkraken_f16.so (compiled with -DKRAKEN_F16=1) stores them as IEEE half, the precision of the
paper's engines (Sec. 4.2).  Same C ABI, same symbols; `kraken_storage_dtype()` tells them apart.
"""
from __future__ import annotations

import concurrent.futures as cf
import os
import shutil
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
OBJ = os.path.join(HERE, "build")
LIB = os.path.join(HERE, "libkraken.so")
LIB_F16 = os.path.join(HERE, "libkraken_f16.so")

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC", "--expt-relaxed-constexpr",
]


def _nvcc() -> str:
    exe = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(exe):
        raise RuntimeError("nvcc not found; the CUDA toolkit is required to build libkraken.so")
    return exe


def _newest_header() -> float:
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".h", ".cuh"))]
    deps.append(os.path.join(HERE, "..", "include", "kraken.h"))
    return max(os.path.getmtime(p) for p in deps)


def lib_path(dtype: str = "bf16") -> str:
    if dtype not in ("bf16", "f16"):
        raise ValueError("storage dtype must be 'bf16' or 'f16'")
    return LIB if dtype == "bf16" else LIB_F16


def build(force: bool = False, verbose: bool = False, dtype: str = "bf16") -> str:
    """Builds one image (dtype 'bf16' or 'f16'); build_all() builds both."""
    lib = lib_path(dtype)
    obj_dir = OBJ if dtype == "bf16" else OBJ + "_f16"
    defs = [] if dtype == "bf16" else ["-DKRAKEN_F16=1"]
    os.makedirs(obj_dir, exist_ok=True)
    srcs = sorted(f for f in os.listdir(CSRC) if f.endswith(".cu"))
    hdr = _newest_header()
    nvcc = _nvcc()
    jobs = []
    for f in srcs:
        src, obj = os.path.join(CSRC, f), os.path.join(obj_dir, f[:-3] + ".o")
        if force or not os.path.exists(obj) or os.path.getmtime(obj) < max(os.path.getmtime(src), hdr):
            cmd = [nvcc, *NVCC_FLAGS, *defs, "-c", src, "-o", obj]
            if verbose:
                cmd.insert(1, "-Xptxas=-v")
            jobs.append(cmd)
    if jobs:
        with cf.ThreadPoolExecutor(max_workers=min(8, len(jobs))) as ex:
            for cmd, res in zip(jobs, ex.map(lambda c: subprocess.run(c, capture_output=True, text=True), jobs)):
                if verbose or res.returncode:
                    sys.stderr.write(res.stdout + res.stderr)
                if res.returncode:
                    raise RuntimeError("nvcc failed: " + " ".join(cmd))
    objs = [os.path.join(obj_dir, f[:-3] + ".o") for f in srcs]
    if jobs or not os.path.exists(lib):
        subprocess.run([nvcc, "-shared", "-o", lib, *objs, "-gencode", "arch=compute_100a,code=sm_100a",
                        "-Xcompiler", "-fPIC"], check=True)
    return lib


def build_all(force: bool = False, verbose: bool = False):
    return [build(force, verbose, "bf16"), build(force, verbose, "f16")]


if __name__ == "__main__":
    for path in build_all(force="--force" in sys.argv, verbose="-v" in sys.argv):
        print(path)

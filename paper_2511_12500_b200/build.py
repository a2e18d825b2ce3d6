"""Build libiris_b200.so in-tree with nvcc for sm_100a (cross-compiles without a GPU)."""
from __future__ import annotations

import os
import subprocess
import sys

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
CSRC = os.path.join(PKG, "csrc")
LIB = os.path.join(PKG, "lib", "libiris_b200.so")
SOURCES = ["heap.cu", "tile_ops.cu", "gemm_all_scatter.cu", "consumer.cu"]
HEADERS = ["iris_internal.h", "iris_device.cuh", "sm100_ptx.cuh"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-std=c++17", "-O3", "-lineinfo", "-Xcompiler", "-fPIC",
              "-Xptxas", "-v", "--expt-relaxed-constexpr"]


def _nvcc() -> str:
    for c in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if c and (os.path.isabs(c) and os.path.exists(c) or not os.path.isabs(c)):
            return c
    return "nvcc"


STAMP = os.path.join(PKG, "lib", "build_flags.txt")


def _flags_line() -> str:
    return " ".join(NVCC_FLAGS + os.environ.get("IRIS_EXTRA_NVCC_FLAGS", "").split())


def _stale() -> bool:
    if not os.path.exists(LIB):
        return True
    try:
        if open(STAMP).read() != _flags_line():   # built with other flags (e.g. a debug macro): not this build
            return True
    except OSError:
        return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, f) for f in SOURCES + HEADERS] + [os.path.join(ROOT, "include", "iris_b200.h"), __file__]
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not _stale():
        return LIB
    os.makedirs(os.path.dirname(LIB), exist_ok=True)
    objdir = os.path.join(PKG, "lib", "obj")
    os.makedirs(objdir, exist_ok=True)
    inc = ["-I", os.path.join(ROOT, "include"), "-I", CSRC]
    procs = []
    for src in SOURCES:
        obj = os.path.join(objdir, src.replace(".cu", ".o"))
        extra = os.environ.get("IRIS_EXTRA_NVCC_FLAGS", "").split()   # e.g. -DIRIS_COMM_TRACE for a debug build
        cmd = [_nvcc(), *NVCC_FLAGS, *extra, *inc, "-c", os.path.join(CSRC, src), "-o", obj]
        procs.append((src, obj, subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
    objs = []
    log = []
    for src, obj, p in procs:
        out, _ = p.communicate()
        log.append(f"== {src}\n{out}")
        if p.returncode != 0:
            sys.stderr.write("\n".join(log))
            raise RuntimeError(f"nvcc failed on {src}")
        objs.append(obj)
    with open(os.path.join(PKG, "lib", "ptxas.log"), "w") as f:
        f.write("\n".join(log))
    if verbose:
        print("\n".join(log))
    tmp = LIB + f".{os.getpid()}.tmp"
    subprocess.check_call([_nvcc(), "-shared", "-o", tmp, *objs, "-cudart", "static"])
    os.replace(tmp, LIB)
    with open(STAMP, "w") as f:
        f.write(_flags_line())
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose=True))

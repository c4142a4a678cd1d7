"""Builds libdabnn_b200.so (sm_100a only) from csrc/ with nvcc, in-tree, beside this file."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libdabnn_b200.so")
SOURCES = ["pack.cu", "bconv.cu", "bconv_tc.cu", "bireal18.cu", "stem_module.cu", "host_api.cu"]
# -fmad=false: no implicit contraction of fp32 mul+add; every fused multiply-add is an explicit fmaf.
NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17", "-fmad=false",
    "-Xcompiler", "-fPIC", "-I", os.path.join(ROOT, "include"), "-I", CSRC,
]


def _stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".cu", ".cuh")) and not f.startswith("ubench")] + [os.path.join(ROOT, "include", "dabnn.h"), __file__]
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not _stale():
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    objs = []
    procs = []
    for src in SOURCES:
        obj = os.path.join(CSRC, src.replace(".cu", ".o"))
        objs.append(obj)
        cmd = [nvcc, *NVCC_FLAGS, *os.environ.get("DABNN_EXTRA_NVCC", "").split(), "-c", os.path.join(CSRC, src), "-o", obj]
        if verbose:
            cmd.insert(1, "-Xptxas=-v")
        procs.append((src, subprocess.Popen(cmd)))
    for src, p in procs:
        if p.wait() != 0:
            raise RuntimeError("nvcc failed on %s" % src)
    tmp = LIB + ".tmp.%d" % os.getpid()
    subprocess.check_call([nvcc, "-shared", "-gencode", "arch=compute_100a,code=sm_100a", "-o", tmp, *objs])
    os.replace(tmp, LIB)
    return LIB


def build_ubench() -> str:
    """Builds the integer-pipe micro-benchmark executable beside the library."""
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    exe = os.path.join(HERE, "ubench_int_pipes")
    src = os.path.join(CSRC, "ubench_int_pipes.cu")
    if not os.path.exists(exe) or os.path.getmtime(exe) < os.path.getmtime(src):
        subprocess.check_call([nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-o", exe, src])
    return exe


if __name__ == "__main__":
    if "--ubench" in sys.argv:
        print(build_ubench())
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))

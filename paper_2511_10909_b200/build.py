"""Builds libmmasim.so in-tree with nvcc for sm_100a (no JIT cache, no pip install)."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libmmasim.so")
SOURCES = ["mmasim_api.cpp", "mmasim_registry.cpp", "mmasim_generic.cu", "mmasim_tfdpa_fast.cu",
           "mmasim_tfdpa_fast_lut8.cu", "mmasim_tfdpa_fast_f16.cu", "mmasim_tfdpa_fast_bf16.cu", "mmasim_trfdpa_f64.cu", "mmasim_efdpa_f64.cu", "mmasim_fp_fast.cu", "mmasim_gst_fast.cu",
           "mmasim_dot_stream.cu", "mmasim_peak.cu", "mmasim_hw_mma.cu", "mmasim_hw_umma.cu", "mmasim_stats.cu"]
HEADERS = ["mmasim_internal.h", "mmasim_device.cuh", "mmasim_tfdpa_fast.cuh", "mmasim_tfdpa_f64.cuh", "mmasim_tfdpa_trop.cuh", os.path.join("..", "..", "include", "mmasim.h")]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "--fmad=false"]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.isabs(cand) and os.path.exists(cand) or not os.path.isabs(cand)):
            return cand
    raise RuntimeError("nvcc not found")


def _stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, s) for s in SOURCES + HEADERS] + [__file__]
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile every source for sm_100a and link libmmasim.so next to this file; returns its path."""
    if not force and not _stale():
        return LIB
    objs = []
    procs = []
    for src in SOURCES:
        obj = os.path.join(CSRC, os.path.splitext(src)[0] + ".o")
        cmd = [_nvcc(), *NVCC_FLAGS, "-x", "cu", "-c", os.path.join(CSRC, src), "-o", obj]
        if verbose:
            cmd.insert(1, "-Xptxas=-v")
        procs.append((src, subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
        objs.append(obj)
    for src, p in procs:
        out, _ = p.communicate()
        if verbose or p.returncode:
            sys.stderr.write(out)
        if p.returncode:
            raise RuntimeError(f"nvcc failed on {src}")
    link = [_nvcc(), "-gencode", "arch=compute_100a,code=sm_100a", "-shared", "-o", LIB, *objs, "-lcudart"]
    subprocess.run(link, check=True)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))

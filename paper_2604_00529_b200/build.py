"""Builds libmxq.so (the CUDA C-ABI library) in-tree with nvcc for sm_100a.

    python -m paper_2604_00529_b200.build [--force] [--debug]

One object per translation unit under ``_build/`` (compiled in parallel), linked into
``paper_2604_00529_b200/libmxq.so``; then ``mxq_abi_timing``, a small C-level caller of the ABI.  A unit is rebuilt when it or any header is newer than
its object.
"""
from __future__ import annotations

import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
OBJ_DIR = os.path.join(ROOT, "_build")
LIB = os.path.join(HERE, "libmxq.so")
TIMING_EXE = os.path.join(HERE, "mxq_abi_timing")      # C-level caller of the ABI (csrc/abi_timing.cu)
UNITS = ["mxq_api", "mxq_quantize", "mxq_slice_scale", "mxq_dequantize", "mxq_fake_quant", "mxq_static_batch", "mxq_slice_scale_multi", "mxq_layout", "mxq_fake_quant_batched"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-std=c++20", "-O3", "-lineinfo",
              "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden"]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.isabs(cand) and os.path.exists(cand) or not os.path.isabs(cand)):
            return cand
    return "nvcc"


def _headers():
    hs = [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".cuh", ".h"))]
    hs.append(os.path.join(ROOT, "include", "mxq.h"))
    return hs


def _stale(target: str, deps) -> bool:
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(d) > t for d in deps)


DEBUG_LIB = os.path.join(HERE, "libmxq_debug.so")      # the same sources with -DMXQ_DEBUG (bounds-checked accesses)


def build(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    """Builds libmxq.so (and mxq_abi_timing); with debug=True builds libmxq_debug.so instead."""
    if debug:
        return _build_library(os.path.join(ROOT, "_build_debug"), DEBUG_LIB, ["-DMXQ_DEBUG"], force, verbose, timing=False)
    return _build_library(OBJ_DIR, LIB, [], force, verbose, timing=True)


def _build_library(obj_dir: str, lib: str, extra, force: bool, verbose: bool, timing: bool) -> str:
    OBJ_DIR, LIB = obj_dir, lib
    os.makedirs(OBJ_DIR, exist_ok=True)
    headers = _headers()
    units = [u for u in UNITS if os.path.exists(os.path.join(CSRC, u + ".cu"))]
    jobs = []
    for u in units:
        src = os.path.join(CSRC, u + ".cu")
        obj = os.path.join(OBJ_DIR, u + ".o")
        if force or _stale(obj, [src] + headers):
            cmd = [_nvcc()] + NVCC_FLAGS + list(extra) + (["-Xptxas", "-v"] if verbose else []) + ["-c", src, "-o", obj]
            jobs.append(cmd)

    def run(cmd):
        r = subprocess.run(cmd, capture_output=True, text=True)
        if r.returncode != 0:
            raise RuntimeError("nvcc failed: %s\n%s\n%s" % (" ".join(cmd), r.stdout, r.stderr))
        return r.stderr

    if jobs:
        with ThreadPoolExecutor(max_workers=min(len(jobs), os.cpu_count() or 1)) as ex:
            for log in ex.map(run, jobs):
                if verbose and log:
                    sys.stderr.write(log)
    objs = [os.path.join(OBJ_DIR, u + ".o") for u in units]
    if force or jobs or _stale(LIB, objs):
        tmp = LIB + ".tmp.%d" % os.getpid()
        run([_nvcc(), "-shared", "-o", tmp] + objs + ["-gencode", "arch=compute_100a,code=sm_100a"])
        os.replace(tmp, LIB)
    timing_src = os.path.join(CSRC, "abi_timing.cu")
    if timing and os.path.exists(timing_src) and (force or _stale(TIMING_EXE, [timing_src, LIB, os.path.join(ROOT, "include", "mxq.h")])):
        tmp = TIMING_EXE + ".tmp.%d" % os.getpid()
        run([_nvcc(), "-O2", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", timing_src, "-o", tmp,
             "-L" + HERE, "-lmxq", "-Xlinker", "-rpath", "-Xlinker", "$ORIGIN"])
        os.replace(tmp, TIMING_EXE)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, debug="--debug" in sys.argv))

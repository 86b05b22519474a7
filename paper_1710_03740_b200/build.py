"""Builds the CUDA shared library in-tree with nvcc for sm_100a.

    python -m paper_1710_03740_b200.build [--force] [--verbose] [--trace]

--trace additionally builds libmpt_trace.so: the same library with the CTA-pair product kernel
instrumented (per-cluster timestamps and cycle counts; see kernel_bench gemm --trace).

Output: paper_1710_03740_b200/libmpt.so (cudart linked statically, so the library
loads on a machine without a GPU; the driver entry point for tensor-map encoding is
looked up at run time).
"""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libmpt.so")
SOURCES = ["update.cu", "softmax_ce.cu", "gemm_simt.cu", "gemm_tc.cu", "gemm_tc2.cu", "gemm_tc3.cu", "gemm_tc4.cu", "lstm.cu", "lstm_api.cu", "lstm_train.cu", "dp_exchange.cu", "wait_selftest.cu", "clock_probe.cu", "mpt_api.cu"]
HEADERS = [os.path.join(CSRC, "mpt_common.cuh"), os.path.join(CSRC, "tc_ptx.cuh"), os.path.join(CSRC, "update_math.cuh"),
           os.path.join(ROOT, "include", "mpt.h")]

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "-lineinfo",
              "-Xcompiler", "-fPIC", "--fmad=true", "-cudart", "static",
              "-I", os.path.join(ROOT, "include"), "-I", CSRC]


def _stale(target, deps):
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(d) > t for d in deps)


def build(force=False, verbose=False):
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    objs = []
    jobs = []
    for src in SOURCES:
        s = os.path.join(CSRC, src)
        o = os.path.join(CSRC, src.replace(".cu", ".o"))
        objs.append(o)
        if force or _stale(o, [s] + HEADERS):
            cmd = [nvcc] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + ["-c", s, "-o", o]
            jobs.append((src, subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
    failed = False
    for src, p in jobs:
        out, _ = p.communicate()
        if p.returncode != 0 or verbose:
            sys.stderr.write("== %s\n%s\n" % (src, out))
        failed |= p.returncode != 0
    if failed:
        raise RuntimeError("nvcc failed")
    if force or jobs or _stale(LIB, objs):
        cmd = [nvcc, "-shared", "-cudart", "static", "-gencode", "arch=compute_100a,code=sm_100a", "-o", LIB] + objs
        subprocess.run(cmd, check=True)
    return LIB


def build_trace():
    """libmpt_trace.so: every object of the normal build except gemm_tc2 and gemm_tc4, which are recompiled with
    -DMPT_GEMM_TRACE."""
    build()
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    traced = ["gemm_tc2.cu", "gemm_tc4.cu"]
    objs = [os.path.join(CSRC, s.replace(".cu", ".o")) for s in SOURCES if s not in traced]
    for src in traced:
        o = os.path.join(CSRC, src.replace(".cu", "_trace.o"))
        subprocess.run([nvcc] + NVCC_FLAGS + ["-DMPT_GEMM_TRACE", "-c", os.path.join(CSRC, src), "-o", o], check=True)
        objs.append(o)
    lib = os.path.join(HERE, "libmpt_trace.so")
    subprocess.run([nvcc, "-shared", "-cudart", "static", "-gencode", "arch=compute_100a,code=sm_100a", "-o", lib] + objs, check=True)
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv))
    if "--trace" in sys.argv:
        print(build_trace())

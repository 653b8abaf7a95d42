"""Builds the CUDA library in-tree: nvcc, sm_100a only, into paper_1901_09290_b200/libpt_b200.so.

``python -m paper_1901_09290_b200.build --trace`` (or ``build(trace=True)``) builds a second library,
libpt_b200_trace.so, with -DPT_DEVICE_TRACE: CTA 0 of the convolution kernels then stamps %globaltimer at the hand-over
points of its roles and the library exports pt_debug_gemm_trace / pt_debug_halo_trace / pt_debug_wgrad_trace, which copy
the stamps (8 roles x 64 entries of nanoseconds) into a host array. It is a tuning aid; the product library never
contains the hooks."""
from __future__ import annotations

import glob
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libpt_b200.so")
NVCC = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-lineinfo", "-std=c++17", "-Xcompiler", "-fPIC",
         "-cudart", "static", "--use_fast_math=false"]


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = sources() + glob.glob(os.path.join(CSRC, "*.h")) + [os.path.join(HERE, "..", "include", "pt.h"), __file__]
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False, trace: bool = False) -> str:
    if trace:
        return _build(os.path.join(HERE, "libpt_b200_trace.so"), os.path.join(HERE, "build", "trace"), ["-DPT_DEVICE_TRACE"], verbose)
    if not force and not _stale():
        return LIB
    return _build(LIB, os.path.join(HERE, "build"), [], verbose)


def _build(lib: str, bdir: str, extra, verbose: bool) -> str:
    objs = []
    procs = []
    os.makedirs(bdir, exist_ok=True)
    flags = [f for f in FLAGS if not f.startswith("--use_fast_math")] + list(extra)
    for src in sources():
        obj = os.path.join(bdir, os.path.basename(src)[:-3] + ".o")
        cmd = [NVCC] + flags + (["-Xptxas", "-v"] if verbose else []) + ["-c", src, "-o", obj]
        procs.append((src, subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
        objs.append(obj)
    failed = False
    for src, p in procs:
        out, _ = p.communicate()
        if p.returncode != 0 or verbose:
            sys.stderr.write(out)
        failed |= p.returncode != 0
    if failed:
        raise RuntimeError("nvcc failed")
    tmp = lib + ".tmp.%d" % os.getpid()
    # (the link step compiles nothing; it names the architecture so that nvcc does not assume, and warn about, its default one)
    subprocess.check_call([NVCC, "-gencode", "arch=compute_100a,code=sm_100a", "-shared", "-cudart", "static", "-o", tmp] + objs +
                          ["-ldl", "-lpthread", "-lrt"])
    os.replace(tmp, lib)
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, trace="--trace" in sys.argv))

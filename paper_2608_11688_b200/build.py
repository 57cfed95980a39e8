"""Builds libapex.so (sm_100a) in-tree with nvcc.  Cross-compiles without a GPU."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libapex.so")
TRACE_LIB = os.path.join(HERE, "libapex_trace.so")   # the same sources with the kernels' time stamps compiled in (trace.py)
SOURCES = ["apex_ctx.cu", "apex_step.cu", "apex_observe.cu", "apex_decode.cu", "kernels_decode.cu", "kernels_router.cu", "kernels_ffn.cu", "kernels_plan.cu", "kernels_ffn_tc.cu", "apex_noalloc.cu", "fit_cdf.cu", "distill.cu"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "--use_fast_math=false"]


def _nvcc() -> str:
    for c in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if c and (os.path.isabs(c) and os.path.exists(c) or not os.path.isabs(c)):
            return c
    return "nvcc"


def _stale(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(HERE, "..", "include", "apex.h")]
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    """Compiles every .cu of the package for sm_100a and links libapex.so.  Returns its path."""
    if not force and not _stale():
        return LIB
    flags = [f for f in NVCC_FLAGS if not f.startswith("--use_fast_math")]
    if verbose:
        flags += ["-Xptxas", "-v"]
    objs = []
    for src in SOURCES:
        obj = os.path.join(CSRC, src.replace(".cu", ".o"))
        cmd = [_nvcc()] + flags + ["-c", os.path.join(CSRC, src), "-o", obj]
        r = subprocess.run(cmd, capture_output=True, text=True)
        if verbose or r.returncode != 0:
            sys.stderr.write(r.stdout + r.stderr)
        if r.returncode != 0:
            raise RuntimeError(f"nvcc failed on {src}")
        objs.append(obj)
    cmd = [_nvcc(), "-shared", "-o", LIB] + objs + ["-gencode", "arch=compute_100a,code=sm_100a"]
    r = subprocess.run(cmd, capture_output=True, text=True)
    if r.returncode != 0:
        sys.stderr.write(r.stdout + r.stderr)
        raise RuntimeError("link failed")
    return LIB


def build_trace(force: bool = False) -> str:
    """libapex_trace.so: every kernel records (kernel id, start, end) of its first block in a device-side log, and the
    expert-FFN kernels per-CTA phase stamps (-DAPEX_TIMELINE).  The log is shared by all translation units, hence
    relocatable device code and one nvcc invocation.  Used by trace.py only; the product library carries no stamps."""
    if not force and not _stale(TRACE_LIB):
        return TRACE_LIB
    flags = [f for f in NVCC_FLAGS if not f.startswith("--use_fast_math")] + ["-DAPEX_TIMELINE", "-rdc=true"]
    cmd = [_nvcc()] + flags + ["-shared", "-o", TRACE_LIB] + [os.path.join(CSRC, f) for f in SOURCES]
    r = subprocess.run(cmd, capture_output=True, text=True)
    if r.returncode != 0:
        sys.stderr.write(r.stdout + r.stderr)
        raise RuntimeError("nvcc failed on the trace build")
    return TRACE_LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
    if "--trace" in sys.argv:
        print(build_trace(force="--force" in sys.argv))

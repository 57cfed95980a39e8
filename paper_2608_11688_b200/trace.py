"""Kernel-level trace of the decode step.

A second build of the library (``build.build_trace()`` -> ``libapex_trace.so``: the same sources with
``-DAPEX_TIMELINE``) makes every kernel record, for its first block, a kernel id and the ``%globaltimer`` values at
entry and at exit in a device-side log of 4096 records; the streaming expert-FFN kernel also stamps the phases of
every CTA.  The product library carries none of this.  Because a process can hold only one of the two libraries,
``use_trace_library()`` must be called before the first context is created.

    python bench.py --trace --resident --layers 8      # prints the spans of one decode token and a summary line

The functions that only format or summarise spans are pure Python (no GPU needed).
"""
from __future__ import annotations

import ctypes as C
from typing import Dict, List, Sequence, Tuple

import numpy as np

from . import binding, build

KERNEL_NAMES = {
    1: "prefetch router (+ candidate selection)",
    2: "candidate selection",
    3: "attention stand-in",
    4: "gate",
    5: "expert FFN, streaming",
    6: "FFN plan (B > 1)",
    7: "gather (B > 1)",
    8: "gate/up GEMM (B > 1)",
    9: "down GEMM (B > 1)",
}
LOG_RECORDS = 4096
# stamps of one CTA of the streaming expert-FFN kernel (index -> meaning); 0, 11, 12 are %globaltimer (ns), the others clock64
FFN_CTA_STAMPS = {0: "entry (ns)", 1: "entry", 4: "dependency wait over", 10: "gate outputs loaded", 2: "plan done",
                  3: "first row consumed", 7: "last row consumed", 8: "partials combined", 9: "exit",
                  11: "dependency wait over (ns)", 12: "exit (ns)"}

Span = Tuple[int, int, int]   # (kernel id, start ns, end ns)


def use_trace_library() -> C.CDLL:
    """Builds (if stale) and loads libapex_trace.so as THE library of this process."""
    path = build.build_trace()
    if binding._lib is not None and getattr(binding._lib, "_name", None) != path:
        raise RuntimeError("another build of the library is already loaded in this process")
    binding.LIB_PATH = path
    lib = binding.load_library(path)
    lib.apex_debug_read_spans.argtypes = [C.c_void_p]
    lib.apex_debug_read_spans.restype = C.c_int
    lib.apex_debug_reset_spans.argtypes = []
    lib.apex_debug_reset_spans.restype = C.c_int
    lib.apex_debug_read_timeline.argtypes = [C.c_void_p, C.c_int]
    lib.apex_debug_read_timeline.restype = C.c_int
    return lib


def reset(lib: C.CDLL) -> None:
    """Empties the span log (call after warm-up, with the device idle)."""
    rc = lib.apex_debug_reset_spans()
    if rc != 0:
        raise RuntimeError(f"apex_debug_reset_spans: CUDA error {rc}")


def read_spans(lib: C.CDLL) -> List[Span]:
    """The recorded spans, ordered by start time (synchronise the device first)."""
    buf = np.zeros(1 + LOG_RECORDS * 3, np.uint64)
    rc = lib.apex_debug_read_spans(buf.ctypes.data)
    if rc != 0:
        raise RuntimeError(f"apex_debug_read_spans: CUDA error {rc}")
    n = min(int(buf[0]), LOG_RECORDS)
    rec = buf[1:1 + 3 * n].reshape(-1, 3).astype(np.int64)
    rec = rec[np.argsort(rec[:, 1], kind="stable")]
    return [(int(k), int(s), int(e)) for k, s, e in rec]


def read_ffn_cta_stamps(lib: C.CDLL, n_ctas: int) -> np.ndarray:
    """[n_ctas][16] stamps of the last streaming expert-FFN launch (see FFN_CTA_STAMPS)."""
    buf = np.zeros(n_ctas * 16, np.uint64)
    rc = lib.apex_debug_read_timeline(buf.ctypes.data, n_ctas * 16)
    if rc != 0:
        raise RuntimeError(f"apex_debug_read_timeline: CUDA error {rc}")
    return buf.reshape(n_ctas, 16).astype(np.int64)


def format_spans(spans: Sequence[Span], limit: int = 64) -> str:
    """One line per span: kernel, start and end relative to the first span, duration, gap to the previous end."""
    if not spans:
        return "(no spans recorded)"
    base = spans[0][1]
    prev_end = base
    lines = ["%-40s %10s %10s %9s %9s" % ("kernel", "start us", "end us", "dur us", "gap us")]
    for k, s, e in spans[:limit]:
        lines.append("%-40s %10.2f %10.2f %9.2f %9.2f" % (KERNEL_NAMES.get(k, f"kernel {k}"), (s - base) / 1e3,
                                                            (e - base) / 1e3, (e - s) / 1e3, (s - prev_end) / 1e3))
        prev_end = max(prev_end, e)
    if len(spans) > limit:
        lines.append(f"... {len(spans) - limit} more")
    return "\n".join(lines)


def summarize(spans: Sequence[Span]) -> Dict[str, dict]:
    """Per kernel: launches, mean / max duration (us); plus the wall span of everything recorded and the busy fraction
    (union of the spans over that wall span)."""
    out: Dict[str, dict] = {}
    by: Dict[int, List[float]] = {}
    for k, s, e in spans:
        by.setdefault(k, []).append((e - s) / 1e3)
    for k in sorted(by):
        v = by[k]
        out[KERNEL_NAMES.get(k, f"kernel {k}")] = {"launches": len(v), "mean_us": float(np.mean(v)), "max_us": float(np.max(v))}
    if spans:
        t0 = min(s for _, s, _ in spans)
        t1 = max(e for _, _, e in spans)
        busy = 0
        cur_s, cur_e = None, None
        for _, s, e in sorted(spans, key=lambda r: r[1]):
            if cur_e is None or s > cur_e:
                if cur_e is not None:
                    busy += cur_e - cur_s
                cur_s, cur_e = s, e
            else:
                cur_e = max(cur_e, e)
        busy += cur_e - cur_s
        out["_all"] = {"wall_us": (t1 - t0) / 1e3, "busy_fraction": busy / max(1, t1 - t0), "spans": len(spans)}
    return out


def ffn_phase_medians(stamps: np.ndarray) -> Dict[str, float]:
    """Median over the CTAs of the cycles between consecutive phase stamps of the streaming expert-FFN kernel."""
    order = [1, 4, 10, 2, 3, 7, 8, 9]
    names = ["entry -> dependency wait over", "-> gate outputs loaded", "-> plan done", "-> first row consumed",
             "-> last row consumed", "-> partials combined", "-> exit"]
    used = stamps[stamps[:, 1] != 0]
    if used.size == 0:
        return {}
    return {n: float(np.median(used[:, b] - used[:, a])) for n, a, b in zip(names, order[:-1], order[1:])}

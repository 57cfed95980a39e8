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
    10: "persistent token kernel (all layers, B = 1)",
}
LOG_RECORDS = 4096
# stamps of one CTA of the streaming expert-FFN kernel (index -> meaning); 0, 11, 12 are %globaltimer (ns), the others clock64
FFN_CTA_STAMPS = {0: "entry (ns)", 1: "entry", 4: "dependency wait over", 10: "gate outputs loaded", 2: "plan done",
                  3: "first row consumed", 7: "last row consumed", 8: "partials combined", 9: "exit",
                  11: "dependency wait over (ns)", 12: "exit (ns)"}

# stamps of one (CTA, layer) of the persistent token kernel, %globaltimer (ns); per CTA the warp that writes last wins
DECODE_STAMPS = {0: "layer start", 15: "previous layer's counter passed (W_p row owners)", 1: "prefetch logit sent",
                 2: "candidate mask out (poster)", 10: "candidate record posted to the host (poster)", 3: "own share of the stand-in landed",
                 14: "stand-in and previous layer's counters passed (W_r row owners)", 4: "gate logit sent", 5: "gate logits complete",
                 6: "execution set and row space planned", 7: "first expert row landed", 8: "last expert row consumed",
                 11: "warps' partial y in shared memory", 12: "cluster's partial y complete", 13: "y added", 9: "layer counted in"}
DECODE_STAMP_ORDER = (15, 1, 2, 10, 3, 14, 4, 5, 6, 7, 8, 11, 12, 13, 9)

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
    lib.apex_debug_read_decode_timeline.argtypes = [C.c_void_p]
    lib.apex_debug_read_decode_timeline.restype = C.c_int
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


def read_decode_stamps(lib: C.CDLL, n_ctas: int, n_layers: int) -> np.ndarray:
    """[n_ctas][n_layers][16] stamps of the last persistent-kernel launch (see DECODE_STAMPS); 0 = not written."""
    buf = np.zeros((160, 64, 16), np.uint64)
    rc = lib.apex_debug_read_decode_timeline(buf.ctypes.data)
    if rc != 0:
        raise RuntimeError(f"apex_debug_read_decode_timeline: CUDA error {rc}")
    return buf[:min(n_ctas, 160), :min(n_layers, 64)].astype(np.int64)


def decode_phase_medians(stamps: np.ndarray) -> Dict[str, float]:
    """Per stamp: median over CTAs and layers (first and last layer left out) of the microseconds since the CTA's own
    layer start; plus the median layer period."""
    if stamps.shape[1] < 3:
        return {}
    out: Dict[str, float] = {}
    inner = stamps[:, 1:-1]
    for i in DECODE_STAMP_ORDER:
        ok = (inner[:, :, i] > 0) & (inner[:, :, 0] > 0)
        if ok.any():
            out[DECODE_STAMPS[i]] = float(np.median((inner[:, :, i] - inner[:, :, 0])[ok])) / 1e3
    start = stamps[:, :, 0]
    ok = (start[:, 1:] > 0) & (start[:, :-1] > 0)
    if ok.any():
        out["layer period"] = float(np.median((start[:, 1:] - start[:, :-1])[ok])) / 1e3
    return out


def format_decode_phases(ph: Dict[str, float]) -> str:
    if not ph:
        return "(no persistent-kernel stamps recorded)"
    lines = ["%-66s %9s" % ("persistent token kernel: event (median over CTAs and layers)", "us")]
    for k, v in ph.items():
        lines.append("%-66s %9.2f" % (k, v))
    return "\n".join(lines)

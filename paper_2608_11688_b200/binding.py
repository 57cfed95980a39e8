"""ctypes binding of libapex.so: the same names as the C entry points, argument marshalling only.

Device buffers are torch CUDA tensors (``data_ptr()``), streams are ``torch.cuda.Stream`` objects
(or None for the current stream).  There is no CPU fallback: loading fails loudly when the
library has not been built.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libapex.so")

APEX_OK, APEX_EINVAL, APEX_ENOMEM, APEX_ECUDA, APEX_ETIMEOUT, APEX_ESTATE, APEX_ENOTIMPL = 0, -1, -2, -3, -4, -5, -6
MODE_EXACT, MODE_STALL_FREE = 0, 1
MODES = {"exact": MODE_EXACT, "stall_free": MODE_STALL_FREE}
FLAG_FP8_EXPERTS = 1
FLAG_SPECULATE = 2
FLAG_FP4_EXPERTS = 4
FLAG_HOST_WAVES = 8
FLAG_LAYER_LAUNCHES = 16
FLAG_SKIP_STANDIN = 32
FLAG_STANDIN_AHEAD = 64
ERR_NAMES = {0: "APEX_OK", -1: "APEX_EINVAL", -2: "APEX_ENOMEM", -3: "APEX_ECUDA", -4: "APEX_ETIMEOUT",
             -5: "APEX_ESTATE", -6: "APEX_ENOTIMPL"}


class ApexConfig(C.Structure):
    _fields_ = [("d", C.c_int32), ("N", C.c_int32), ("k", C.c_int32), ("I", C.c_int32), ("I_shared", C.c_int32),
                ("C", C.c_int32), ("L", C.c_int32), ("max_batch", C.c_int32), ("norm_topk", C.c_int32),
                ("cache_reuse", C.c_int32), ("ctx_len", C.c_int32), ("flags", C.c_int32),
                ("wait_limit_ns", C.c_int64), ("link_gbs", C.c_double)]


class ApexStepStats(C.Structure):
    _fields_ = [(n, C.c_int64) for n in (
        "layer_steps", "tokens", "sum_delta_hat", "sum_delta_star", "sum_ncand", "capped", "routed", "hits_P",
        "hits_R", "covered", "substitutions", "prefetch_copies", "demand_copies", "bytes_copied", "extra_waves",
        "stall_ns", "timeouts", "near_full_prefetch")]

    def as_dict(self):
        return {n: int(getattr(self, n)) for n, _ in self._fields_}


# every symbol include/apex.h declares: name -> (restype, argtypes)
_P = C.c_void_p
_I = C.c_int
SIGNATURES = {
    "apex_create": (_I, [C.POINTER(ApexConfig), C.POINTER(_P)]),
    "apex_destroy": (_I, [_P]),
    "apex_last_error": (C.c_char_p, [_P]),
    "apex_set_router": (_I, [_P, _I, _P, _P]),
    "apex_set_prefetch_router": (_I, [_P, _I, _P, _P]),
    "apex_set_cdf": (_I, [_P, _I, _P, _P]),
    "apex_register_experts": (_I, [_P, _I, _P, C.c_size_t]),
    "apex_set_shared_expert": (_I, [_P, _I, _P]),
    "apex_set_shared_gate": (_I, [_P, _I, _P]),
    "apex_pack_expert": (_I, [_P, _P, _P, _I, _I, _P]),
    "apex_predict": (_I, [_P, _I, _P, _I, _P]),
    "apex_select_candidates": (_I, [_P, _I, _I, C.c_float, _P, _P, _P]),
    "apex_prefetch": (_I, [_P, _I, _I, _P]),
    "apex_attention_standin": (_I, [_P, _I, _P]),
    "apex_route_topk": (_I, [_P, _I, _P, _I, _P, _P, _P]),
    "apex_moe_ffn": (_I, [_P, _I, _I, _P, _I, _P, _P, _P, _P]),
    "apex_moe_ffn_begin": (_I, [_P, _I, _I, _P, _I, _P, _P, _P, _P]),
    "apex_moe_ffn_end": (_I, [_P, _I]),
    "apex_decode_token": (_I, [_P, _P, _P, _I, C.c_float, _I, _P, _P]),
    "apex_decode_token_host": (_I, [_P, _P, _P, _I, C.c_float, _I, _P, _P]),
    "apex_get_stats": (_I, [_P, _I, C.POINTER(ApexStepStats)]),
    "apex_reset_stats": (_I, [_P]),
    "apex_read_prediction": (_I, [_P, _I, _P, _P, _P]),
    "apex_get_last_copies": (_I, [_P, _I, _P, _P, C.POINTER(C.c_int32), C.POINTER(C.c_int32)]),
    "apex_get_slot_table": (_I, [_P, _I, _P, _P, C.POINTER(C.c_int64)]),
    "apex_set_slot_table": (_I, [_P, _I, _P, _P, C.c_int64]),
    "apex_warm_all": (_I, [_P]),
    "apex_test_inject": (_I, [_P, _I]),
    "apex_launch_count": (C.c_int64, [_P]),
    "apex_route_topk_static": (_I, [_P, _P, _P, _I, _I, _I, _I, _P, _P, _P, C.c_char_p, C.c_size_t]),
    "apex_fit_cdf": (_I, [_P, _P, _I, _I, _I, _I, C.c_double, _P, _P, _P, C.c_char_p, C.c_size_t]),
    "apex_distill_router": (_I, [_P, _P, _I, _I, _I, _I, C.c_double, _P, _P, _P, C.c_char_p, C.c_size_t]),
    "apex_slots_create": (_P, [_I, _I, _I]),
    "apex_slots_destroy": (None, [_P]),
    "apex_slots_begin_step": (_I, [_P]),
    "apex_slots_prefetch": (_I, [_P, _P, _P, _I, _I, _P, _P, C.POINTER(C.c_int32)]),
    "apex_slots_demand": (_I, [_P, _P, _I, _I, _P, _P, _P, C.POINTER(C.c_int32)]),
    "apex_slots_touch": (_I, [_P, _P, _I]),
    "apex_slots_get": (_I, [_P, _P, _P, C.POINTER(C.c_int64)]),
    "apex_slots_set": (_I, [_P, _P, _P, C.c_int64]),
}

_lib = None


def load_library(path: str = LIB_PATH) -> C.CDLL:
    """Loads libapex.so and declares every signature.  Raises if the library is missing."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(path):
        raise RuntimeError(f"{path} not found: build it with `python -m paper_2608_11688_b200.build` "
                           "(there is no CPU fallback)")
    lib = C.CDLL(path)
    for name, (res, args) in SIGNATURES.items():
        fn = getattr(lib, name)
        fn.restype = res
        fn.argtypes = args
    _lib = lib
    return lib


class ApexError(RuntimeError):
    def __init__(self, code, msg):
        super().__init__(f"{ERR_NAMES.get(code, code)}: {msg}")
        self.code = code


def _ptr(t) -> Optional[int]:
    """Address of a torch tensor / numpy array, or None."""
    if t is None:
        return None
    if isinstance(t, np.ndarray):
        assert t.flags["C_CONTIGUOUS"]
        return t.ctypes.data
    assert t.is_contiguous()
    return t.data_ptr()


def _stream(s) -> Optional[int]:
    if s is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if isinstance(s, int):
        return s
    return s.cuda_stream


class Apex:
    """One context.  Methods mirror the C entry points one to one (apex_ prefix dropped)."""

    def __init__(self, *, d, N, k, I, C_slots, L=1, I_shared=0, max_batch=1, norm_topk=1, cache_reuse=1,
                 ctx_len=1024, wait_limit_ns=0, flags=0, link_gbs=0.0):
        self.lib = load_library()
        self.cfg = ApexConfig(d=d, N=N, k=k, I=I, I_shared=I_shared, C=C_slots, L=L, max_batch=max_batch,
                              norm_topk=norm_topk, cache_reuse=cache_reuse, ctx_len=ctx_len, flags=flags,
                              wait_limit_ns=wait_limit_ns, link_gbs=float(link_gbs))
        h = C.c_void_p()
        rc = self.lib.apex_create(C.byref(self.cfg), C.byref(h))
        if rc != APEX_OK:
            raise ApexError(rc, self.lib.apex_last_error(None).decode() or "apex_create failed")
        self.h = h
        self._keep = []   # borrowed buffers that must outlive the context

    # -- plumbing
    def _chk(self, rc):
        if rc != APEX_OK:
            raise ApexError(rc, self.lib.apex_last_error(self.h).decode())
        return rc

    def destroy(self):
        if getattr(self, "h", None):
            self.lib.apex_destroy(self.h)
            self.h = None
            self._keep = []

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass

    # -- parameters
    def set_router(self, layer, W_r, b_r=None):
        W = np.ascontiguousarray(W_r, np.float32)
        b = None if b_r is None else np.ascontiguousarray(b_r, np.float32)
        self._chk(self.lib.apex_set_router(self.h, layer, _ptr(W), _ptr(b)))

    def set_prefetch_router(self, layer, W_p, b_p=None):
        W = np.ascontiguousarray(W_p, np.float32)
        b = None if b_p is None else np.ascontiguousarray(b_p, np.float32)
        self._chk(self.lib.apex_set_prefetch_router(self.h, layer, _ptr(W), _ptr(b)))

    def set_cdf(self, layer, w, theta):
        w = np.ascontiguousarray(w, np.float32)
        th = np.ascontiguousarray(theta, np.float32)
        self._chk(self.lib.apex_set_cdf(self.h, layer, _ptr(w), _ptr(th)))

    def register_experts(self, layer, store, stride_bytes=None):
        """store: pinned torch tensor in the store layout, bf16 [N][I][3][d] (uint8 [N][I][3*d+16] with FLAG_FP8_EXPERTS)."""
        self._keep.append(store)
        stride = stride_bytes if stride_bytes is not None else store.stride(0) * store.element_size()
        self._chk(self.lib.apex_register_experts(self.h, layer, _ptr(store), stride))

    def set_shared_expert(self, layer, dev_weights):
        self._keep.append(dev_weights)
        self._chk(self.lib.apex_set_shared_expert(self.h, layer, _ptr(dev_weights)))

    def set_shared_gate(self, layer, w_sg):
        """Gate vector [d] of the layer's shared expert (numpy / tensor, host or device), or None for weight 1."""
        if w_sg is None:
            self._chk(self.lib.apex_set_shared_gate(self.h, layer, None))
            return
        w = np.ascontiguousarray(w_sg, np.float32) if isinstance(w_sg, np.ndarray) else w_sg
        self._chk(self.lib.apex_set_shared_gate(self.h, layer, _ptr(w)))

    # -- the layer-step
    def predict(self, layer, h_dev, B, stream=None):
        self._chk(self.lib.apex_predict(self.h, layer, _ptr(h_dev), B, _stream(stream)))

    def select_candidates(self, layer, B, tau, cand_dev, ncand_dev, stream=None):
        self._chk(self.lib.apex_select_candidates(self.h, layer, B, float(tau), _ptr(cand_dev), _ptr(ncand_dev),
                                                  _stream(stream)))

    def prefetch(self, layer, B, copy_stream=None):
        self._chk(self.lib.apex_prefetch(self.h, layer, B, None if copy_stream is None else _stream(copy_stream)))

    def attention_standin(self, layer, stream=None):
        self._chk(self.lib.apex_attention_standin(self.h, layer, _stream(stream)))

    def route_topk(self, layer, hpost_dev, B, idx_dev, alpha_dev, stream=None):
        self._chk(self.lib.apex_route_topk(self.h, layer, _ptr(hpost_dev), B, _ptr(idx_dev), _ptr(alpha_dev),
                                           _stream(stream)))

    def moe_ffn(self, layer, mode, hpost_dev, B, y_dev, exec_idx_dev=None, exec_gate_dev=None, stream=None):
        m = MODES[mode] if isinstance(mode, str) else mode
        self._chk(self.lib.apex_moe_ffn(self.h, layer, m, _ptr(hpost_dev), B, _ptr(y_dev), _ptr(exec_idx_dev),
                                        _ptr(exec_gate_dev), _stream(stream)))

    def moe_ffn_begin_raw(self, layer, mode_int, hpost_ptr, B, y_ptr, stream_int):
        """apex_moe_ffn_begin with raw addresses (no per-call marshalling): for tight timing loops."""
        rc = self.lib.apex_moe_ffn_begin(self.h, layer, mode_int, hpost_ptr, B, y_ptr, None, None, stream_int)
        if rc != APEX_OK:
            self._chk(rc)

    def moe_ffn_begin(self, layer, mode, hpost_dev, B, y_dev, exec_idx_dev=None, exec_gate_dev=None, stream=None):
        m = MODES[mode] if isinstance(mode, str) else mode
        self._chk(self.lib.apex_moe_ffn_begin(self.h, layer, m, _ptr(hpost_dev), B, _ptr(y_dev), _ptr(exec_idx_dev),
                                              _ptr(exec_gate_dev), _stream(stream)))

    def moe_ffn_end(self, layer):
        self._chk(self.lib.apex_moe_ffn_end(self.h, layer))

    def decode_token(self, h_dev, hpost_dev, B, tau, mode, y_dev, stream=None):
        m = MODES[mode] if isinstance(mode, str) else mode
        self._chk(self.lib.apex_decode_token(self.h, _ptr(h_dev), _ptr(hpost_dev), B, float(tau), m, _ptr(y_dev),
                                             _stream(stream)))

    def decode_token_host(self, h_host, hpost_host, B, tau, mode, y_host, stream=None):
        m = MODES[mode] if isinstance(mode, str) else mode
        self._chk(self.lib.apex_decode_token_host(self.h, _ptr(h_host), _ptr(hpost_host), B, float(tau), m,
                                                  _ptr(y_host), _stream(stream)))

    # -- observation
    def get_stats(self, layer=-1):
        s = ApexStepStats()
        self._chk(self.lib.apex_get_stats(self.h, layer, C.byref(s)))
        return s.as_dict()

    def reset_stats(self):
        self._chk(self.lib.apex_reset_stats(self.h))

    def read_prediction(self, B):
        N = self.cfg.N
        z = np.empty((B, N), np.float32); q = np.empty((B, N), np.float32); pi = np.empty((B, N), np.int32)
        self._chk(self.lib.apex_read_prediction(self.h, B, _ptr(z), _ptr(q), _ptr(pi)))
        return z, q, pi

    def get_last_copies(self, layer):
        N = self.cfg.N
        e = np.empty(4 * N, np.int32); s = np.empty(4 * N, np.int32)
        npf, nd = C.c_int32(), C.c_int32()
        self._chk(self.lib.apex_get_last_copies(self.h, layer, _ptr(e), _ptr(s), C.byref(npf), C.byref(nd)))
        a, b = npf.value, nd.value
        pairs = [(int(e[i]), int(s[i])) for i in range(a + b)]
        return pairs[:a], pairs[a:]

    def get_slot_table(self, layer):
        es = np.empty(self.cfg.N, np.int32); st = np.empty(self.cfg.C, np.int64); clk = C.c_int64()
        self._chk(self.lib.apex_get_slot_table(self.h, layer, _ptr(es), _ptr(st), C.byref(clk)))
        return es, st, clk.value

    def set_slot_table(self, layer, expert_slot, slot_stamp, clock):
        es = np.ascontiguousarray(expert_slot, np.int32); st = np.ascontiguousarray(slot_stamp, np.int64)
        self._chk(self.lib.apex_set_slot_table(self.h, layer, _ptr(es), _ptr(st), int(clock)))

    def warm_all(self):
        self._chk(self.lib.apex_warm_all(self.h))

    def test_inject(self, what):
        self._chk(self.lib.apex_test_inject(self.h, what))

    def launch_count(self):
        return int(self.lib.apex_launch_count(self.h))


def route_topk_static(W_r_dev, b_r_dev, hpost_dev, k, idx_dev, alpha_dev, stream=None):
    """apex_route_topk_static: the gate without a context and without any allocation.  W_r_dev [N][d],
    b_r_dev [N] or None, hpost_dev [B][d] are CUDA tensors; idx_dev [B][k] int32 and alpha_dev [B][N]
    fp32 receive the result.  Raises ApexError with the library's message on failure."""
    lib = load_library()
    N, d = W_r_dev.shape
    B = hpost_dev.shape[0]
    err = C.create_string_buffer(256)
    rc = lib.apex_route_topk_static(_ptr(W_r_dev), _ptr(b_r_dev), _ptr(hpost_dev), N, d, k, B, _ptr(idx_dev),
                                    _ptr(alpha_dev), _stream(stream), err, len(err))
    if rc != APEX_OK:
        raise ApexError(rc, err.value.decode())


def fit_cdf(X_dev, dstar_dev, k, iters=600, lr=0.05, stream=None):
    """apex_fit_cdf: X_dev [T][N] fp64 and dstar_dev [T] int32 CUDA tensors -> (w [N], theta [N-k+1]) fp32 numpy."""
    lib = load_library()
    T, N = X_dev.shape
    w = np.empty(N, np.float32)
    theta = np.empty(N - k + 1, np.float32)
    err = C.create_string_buffer(256)
    rc = lib.apex_fit_cdf(_ptr(X_dev), _ptr(dstar_dev), T, N, k, int(iters), float(lr), _ptr(w), _ptr(theta),
                          _stream(stream), err, len(err))
    if rc != APEX_OK:
        raise ApexError(rc, err.value.decode())
    return w, theta


def distill_router(H_dev, Qr_dev, W0, b0, iters=200, lr=0.01, stream=None):
    """apex_distill_router: H_dev [T][d], Qr_dev [T][N] fp32 CUDA tensors; W0 [N][d], b0 [N] the starting point.
    Returns the trained (W [N][d], b [N]) as fp32 numpy arrays."""
    lib = load_library()
    T, d = H_dev.shape
    N = Qr_dev.shape[1]
    W = np.ascontiguousarray(W0, np.float32).copy()
    b = np.ascontiguousarray(b0, np.float32).copy()
    assert W.shape == (N, d) and b.shape == (N,)
    err = C.create_string_buffer(256)
    rc = lib.apex_distill_router(_ptr(H_dev), _ptr(Qr_dev), T, N, d, int(iters), float(lr), _ptr(W), _ptr(b),
                                 _stream(stream), err, len(err))
    if rc != APEX_OK:
        raise ApexError(rc, err.value.decode())
    return W, b


class Slots:
    """Host-only slot planner (no CUDA call): the state machine behind prefetch / moe_ffn."""

    def __init__(self, N, C_slots, cache_reuse=True):
        self.lib = load_library()
        self.N, self.C = N, C_slots
        self.h = self.lib.apex_slots_create(N, C_slots, int(cache_reuse))
        if not self.h:
            raise ApexError(APEX_EINVAL, "apex_slots_create failed")

    def __del__(self):
        if getattr(self, "h", None):
            self.lib.apex_slots_destroy(self.h)
            self.h = None

    def begin_step(self):
        assert self.lib.apex_slots_begin_step(self.h) == 0

    def prefetch(self, cand_lists):
        B = len(cand_lists)
        stride = max(1, max(len(c) for c in cand_lists))
        cand = np.full((B, stride), -1, np.int32)
        ncand = np.zeros(B, np.int32)
        for b, cl in enumerate(cand_lists):
            cand[b, :len(cl)] = cl
            ncand[b] = len(cl)
        ce = np.empty(self.N, np.int32); cs = np.empty(self.N, np.int32); n = C.c_int32()
        rc = self.lib.apex_slots_prefetch(self.h, _ptr(cand), _ptr(ncand), B, stride, _ptr(ce), _ptr(cs), C.byref(n))
        if rc != 0:
            raise ApexError(rc, "apex_slots_prefetch")
        return [(int(ce[i]), int(cs[i])) for i in range(n.value)]

    def demand(self, K_r_lists):
        B, k = len(K_r_lists), len(K_r_lists[0])
        K = np.ascontiguousarray(K_r_lists, np.int32)
        ce = np.empty(self.N, np.int32); cs = np.empty(self.N, np.int32); cw = np.empty(self.N, np.int32); n = C.c_int32()
        rc = self.lib.apex_slots_demand(self.h, _ptr(K), B, k, _ptr(ce), _ptr(cs), _ptr(cw), C.byref(n))
        if rc != 0:
            raise ApexError(rc, "apex_slots_demand")
        return [(int(ce[i]), int(cs[i]), int(cw[i])) for i in range(n.value)]

    def touch(self, experts):
        e = np.ascontiguousarray(experts, np.int32)
        assert self.lib.apex_slots_touch(self.h, _ptr(e), len(e)) == 0

    def get(self):
        es = np.empty(self.N, np.int32); st = np.empty(self.C, np.int64); clk = C.c_int64()
        assert self.lib.apex_slots_get(self.h, _ptr(es), _ptr(st), C.byref(clk)) == 0
        return es, st, clk.value

    def set(self, expert_slot, slot_stamp, clock):
        es = np.ascontiguousarray(expert_slot, np.int32); st = np.ascontiguousarray(slot_stamp, np.int64)
        return self.lib.apex_slots_set(self.h, _ptr(es), _ptr(st), int(clock))

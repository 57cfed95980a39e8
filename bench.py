#!/usr/bin/env python
"""Benchmark of the MoE decode step with adaptive expert prefetch on B200.

A "step" is one decode token through all layers of the workload: for every layer the prefetch
router, the budget selection, the asynchronous expert prefetch, the stand-in attention window,
the exact gate and the expert FFN (with on-demand correction of misses in exact mode).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--config 1] [--impl ours|reference]

Prints ONE JSON line (rank 0).  N > 1 runs N independent replicas (the path does not shard).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "moe_decode_tokens_per_s"
UNIT = "tokens/s"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
TAU = 0.90

# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) of the per-layer expert-FFN kernel from its ncu
# capture on config 1 (37.809 MB read + 0.045 MB written).  None = not captured.
NCU_TRAFFIC_BYTES = {1: 37_854_500}


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return float(json.load(open(p))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """nvidia-smi clocks and throttle reasons during the timed region."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.idx = gpu_index
        self.proc = None
        self.path = f"/tmp/apex_clocks_{os.getpid()}.csv"

    def start(self):
        try:
            self.f = open(self.path, "w")
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-i", str(self.idx), "-lms", "100"], stdout=self.f, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.f.close()
        sm, mx, reasons = [], [], set()
        for ln in open(self.path):
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        try:
            os.remove(self.path)
        except OSError:
            pass
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm))
        return out


def algorithmic_bytes(cfg, B=1):
    """Per layer-step: routed expert weights + shared FFN + both routers (fp32), and the FFN kernel alone."""
    ffn = cfg.k * cfg.expert_bytes + cfg.shared_bytes + 2 * B * cfg.d * 4
    routers = 2 * cfg.d * cfg.N * 4
    return ffn + routers, ffn


# ------------------------------------------------------------------------------------------------
def build_problem(cfg, device, fp8=False, fp4=False):
    import torch
    from paper_2608_11688_b200 import synth
    routers = [synth.router_weights(cfg, l) for l in range(cfg.L)]
    cdf = [synth.cdf_params(cfg, l) for l in range(cfg.L)]
    if fp4:     # datatype study (Sec. V-G): e2m1 rows with a power-of-two scale per 32 elements
        store = torch.empty((cfg.L, cfg.N, cfg.I, synth.fp4_row_bytes(cfg.d)), dtype=torch.uint8, pin_memory=True)
    elif fp8:   # e4m3 rows with per-row scales
        store = torch.empty((cfg.L, cfg.N, cfg.I, 3 * cfg.d + 16), dtype=torch.uint8, pin_memory=True)
    else:
        store = torch.empty((cfg.L, cfg.N, cfg.I, 3, cfg.d), dtype=torch.bfloat16, pin_memory=True)
    shared = []
    for l in range(cfg.L):
        store[l].copy_(synth.expert_store_fp4(cfg, l, device=device) if fp4 else
                       synth.expert_store_fp8(cfg, l, device=device) if fp8 else synth.expert_store(cfg, l, device=device))
        sh = synth.shared_expert(cfg, l, device=device)
        if sh is not None and (fp4 or fp8):
            sh = synth.quantize_store_fp4(sh) if fp4 else synth.quantize_store_fp8(sh)
        shared.append(sh)
    torch.cuda.synchronize()
    return routers, cdf, store, shared


def make_ctx(cfg, prob, C, max_batch=1, flags=0, link_gbs=0.0, ctx_len=1024, cache_reuse=1):
    from paper_2608_11688_b200 import binding
    routers, cdf, store, shared = prob
    fmt_flag = 0
    if store.dtype != __import__("torch").bfloat16:
        fmt_flag = binding.FLAG_FP8_EXPERTS if store.shape[-1] == 3 * cfg.d + 16 else binding.FLAG_FP4_EXPERTS
    a = binding.Apex(d=cfg.d, N=cfg.N, k=cfg.k, I=cfg.I, C_slots=C, L=cfg.L, I_shared=cfg.I_shared, max_batch=max_batch,
                     flags=fmt_flag | flags, link_gbs=link_gbs, ctx_len=ctx_len, cache_reuse=cache_reuse)
    for l in range(cfg.L):
        W_r, b_r, W_p, b_p = routers[l]
        a.set_router(l, W_r, b_r)
        a.set_prefetch_router(l, W_p, b_p)
        a.set_cdf(l, *cdf[l])
        a.register_experts(l, store[l])
        if shared[l] is not None:
            a.set_shared_expert(l, shared[l])
    return a


def train_auxiliary(cfg, prob, device, n_calib=8192, distill_iters=100, distill_lr=1e-4, fit_iters=600):
    """The paper's two training stages on this GPU (Sec. IV-C): distil the prefetch router of every layer from the
    router (Eq. (10)), then refit the confidence model on the distilled router's rankings (Eq. (11)).  Returns new
    (routers, cdf) lists; the calibration tokens come from the seeded generator's calibration stream.  Teacher
    distributions, rankings and routed sets are the library's own outputs (apex_route_topk; apex_predict +
    apex_read_prediction), taken in batches on a context without expert stores; only the bookkeeping that turns a
    ranking and a routed set into a calibration pair (x = q_p in rank order, delta* = largest rank of a routed expert
    - k, Eq. (3)) is done here.  The step size is small on purpose: a layer has N * (d + 1) parameters and only
    n_calib tokens, and Adam moves every weight by about lr per step whatever its gradient, so a larger step
    overfits the calibration set within a few iterations."""
    import torch
    from paper_2608_11688_b200 import binding, synth
    routers, cdf, store, shared = prob
    MB = 256
    a = binding.Apex(d=cfg.d, N=cfg.N, k=cfg.k, I=cfg.I, C_slots=cfg.k, L=cfg.L, I_shared=cfg.I_shared, max_batch=MB)
    new_routers, new_cdf = [], []
    t_d = t_f = 0.0
    try:
        for l in range(cfg.L):
            W_r, b_r, W_p, b_p = routers[l]
            a.set_router(l, W_r, b_r)
            h, hp = synth.hidden_states(cfg, l, n_calib, 1, calib=True)
            Hd = torch.from_numpy(np.ascontiguousarray(h[:, 0])).to(device)
            Hpd = torch.from_numpy(np.ascontiguousarray(hp[:, 0])).to(device)
            Qr = torch.empty((n_calib, cfg.N), dtype=torch.float32, device=device)      # teacher: alpha = softmax(z_r)
            K_r = torch.empty((n_calib, cfg.k), dtype=torch.int32, device=device)
            for s0 in range(0, n_calib, MB):
                b = min(MB, n_calib - s0)
                a.route_topk(l, Hpd[s0:s0 + b], b, K_r[s0:s0 + b], Qr[s0:s0 + b])
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            W_p2, b_p2 = binding.distill_router(Hd, Qr, W_p, b_p, iters=distill_iters, lr=distill_lr)
            t_d += time.perf_counter() - t0
            # calibration set of the confidence model from the distilled router's own predictions
            a.set_prefetch_router(l, W_p2, b_p2)
            X = np.empty((n_calib, cfg.N), np.float32)
            rank = np.empty((n_calib, cfg.N), np.int64)
            for s0 in range(0, n_calib, MB):
                b = min(MB, n_calib - s0)
                a.predict(l, Hd[s0:s0 + b], b)
                _, q_p, pi = a.read_prediction(b)
                X[s0:s0 + b] = np.take_along_axis(q_p, pi.astype(np.int64), axis=1)
                np.put_along_axis(rank[s0:s0 + b], pi.astype(np.int64), np.broadcast_to(np.arange(cfg.N), pi.shape), axis=1)
            dstar = np.take_along_axis(rank, K_r.cpu().numpy().astype(np.int64), axis=1).max(1) + 1 - cfg.k
            t0 = time.perf_counter()
            w, theta = binding.fit_cdf(torch.from_numpy(X.astype(np.float64)).to(device),
                                       torch.from_numpy(dstar.astype(np.int32)).to(device), cfg.k, iters=fit_iters)
            t_f += time.perf_counter() - t0
            new_routers.append((W_r, b_r, W_p2, b_p2))
            new_cdf.append((w, theta))
    finally:
        a.destroy()
    return new_routers, new_cdf, {"distill_s": t_d, "fit_s": t_f, "calibration_tokens_per_layer": n_calib}


POLICIES = (("no_prefetch", -1.0, None), ("static_k", 0.9, 0), ("static_k+4", 0.9, 4), ("static_k+8", 0.9, 8), ("apex", TAU, None))


def run_policy(cfg, prob, h_dev, hp_dev, y_dev, B, name, tau_p, delta, warmup, steps, link_gbs=0.0, ctx_len=1024, cache_reuse=1):
    """Decode tokens under one prefetch policy of Sec. V-A (same ranking, different budgets); returns a dict."""
    import torch
    ap_ = make_ctx(cfg, prob, cfg.C, max_batch=B, link_gbs=link_gbs, ctx_len=ctx_len, cache_reuse=cache_reuse)
    if delta is not None:      # w = 0 and a step in theta: delta_hat = delta for every token
        nth = cfg.N - cfg.k + 1
        th = np.where(np.arange(nth) >= delta, 50.0, -50.0).astype(np.float32)
        for l in range(cfg.L):
            ap_.set_cdf(l, np.zeros(cfg.N, np.float32), th)
    T_ = h_dev.shape[0]
    n_tok = warmup + steps
    for t in range(warmup):
        ap_.decode_token(h_dev[t % T_], hp_dev[t % T_], B, tau_p, "exact", y_dev)
    torch.cuda.synchronize()
    ap_.reset_stats()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for t in range(warmup, n_tok):
        ap_.decode_token(h_dev[t % T_], hp_dev[t % T_], B, tau_p, "exact", y_dev)
    e1.record()
    torch.cuda.synchronize()
    sp = ap_.get_stats()
    sec = e0.elapsed_time(e1) * 1e-3
    out = {"tokens_per_s": steps * B / sec, "ms_per_token": 1e3 * sec / (steps * B),
           "copies_per_token": (sp["prefetch_copies"] + sp["demand_copies"]) / steps,
           "demand_copies_per_token": sp["demand_copies"] / steps,
           "prefetch_copies_per_token": sp["prefetch_copies"] / steps,
           "overlap_vs_R": sp["hits_R"] / max(1, sp["routed"]),
           "copied_gbs": sp["bytes_copied"] / sec / 1e9}
    ap_.destroy()
    return out


def window_sweep(args, cfg, prob, h_dev, hp_dev, y_dev, B):
    """Study of the overlap condition, Eq. (12): T_prefetch(delta) = delta * S_expert / B_eff + T_queue <= T_attn.  On this
    machine one expert copy over the host link is far longer than the attention window of the paper's context lengths,
    so nothing can be hidden and the policies that move fewer bytes win.  Here the OTHER side of the ratio is moved: the
    stand-in attention is lengthened (through ctx_len) until the window holds 0.5, 1, 2, 4 and 8 expert copies, and the
    policies of Sec. V-A are timed at every window.  Per policy: tokens/s, demand copies per token, the exposed stall
    (time per token minus the all-resident time at the same window) and the stall Eq. (12) allows at best
    (per layer: what the prefetch copies overrun the window by, plus the demand copies, at the measured link rate)."""
    import torch
    from paper_2608_11688_b200 import binding
    d, L = cfg.d, cfg.L
    steps, warmup = max(8, min(args.steps, 16)), 4

    def resident_ms(ctx_len, flags=0):
        a = make_ctx(cfg, prob, cfg.N, max_batch=B, ctx_len=ctx_len, flags=flags)
        a.warm_all()
        sec = time_tokens(a, h_dev, hp_dev, y_dev, B, "exact", warmup, steps)
        a.destroy()
        return 1e3 * sec / steps

    base_ms = resident_ms(1024, flags=binding.FLAG_SKIP_STANDIN)       # the method's own kernels, no window at all
    # link rate and copy time: from a run that keeps the link busy
    ref = run_policy(cfg, prob, h_dev, hp_dev, y_dev, B, "no_prefetch", -1.0, None, warmup, steps)
    link_gbs = ref["copied_gbs"]
    t_copy_us = cfg.expert_bytes / (link_gbs * 1e3)
    # stand-in streaming rate: from two window lengths
    ms_a, ms_b = resident_ms(1024), resident_ms(65536)
    bytes_of = lambda c: (4 * d * d + 2 * c * d) * 2
    us_per_byte = (ms_b - ms_a) * 1e3 / L / (bytes_of(65536) - bytes_of(1024))
    rows = []
    for ratio in (None, 0.5, 1.0, 2.0, 4.0, 8.0):
        if ratio is None:
            ctx_len = 1024
        else:
            want_bytes = ratio * t_copy_us / us_per_byte
            ctx_len = max(1024, int((want_bytes / 2 - 4 * d * d) / (2 * d)))
        res_ms = resident_ms(ctx_len)
        t_attn_us = max(0.0, (res_ms - base_ms) * 1e3 / L)
        row = {"ctx_len": ctx_len, "T_attn_us": t_attn_us, "T_attn_over_copy": t_attn_us / t_copy_us, "all_resident_ms_per_token": res_ms,
               "policies": {}}
        for name, tau_p, delta, reuse in (("no_prefetch", -1.0, None, 1), ("static_k", 0.9, 0, 1), ("static_k+4", 0.9, 4, 1),
                                          ("apex", TAU, None, 1), ("apex_tau0.75", 0.75, None, 1), ("apex_tau0.5", 0.5, None, 1),
                                          ("apex_load_use_evict", TAU, None, 0)):
            r = run_policy(cfg, prob, h_dev, hp_dev, y_dev, B, name, tau_p, delta, warmup, steps, ctx_len=ctx_len, cache_reuse=reuse)
            pre_l, dem_l = r["prefetch_copies_per_token"] / L, r["demand_copies_per_token"] / L
            bound_us = L * (max(0.0, pre_l * t_copy_us - t_attn_us) + dem_l * t_copy_us)
            row["policies"][name] = {"tokens_per_s": r["tokens_per_s"], "ms_per_token": r["ms_per_token"],
                                     "demand_copies_per_token": r["demand_copies_per_token"],
                                     "prefetch_copies_per_token": r["prefetch_copies_per_token"],
                                     "exposed_stall_us_per_token": (r["ms_per_token"] - res_ms) * 1e3,
                                     "eq12_stall_bound_us_per_token": bound_us}
        rows.append(row)
    last = rows[-1]["policies"]
    return {"window_sweep": rows, "expert_copy_us": t_copy_us, "link_gbs": link_gbs, "standin_gbs": 1e-3 / us_per_byte,
            "no_window_ms_per_token": base_ms, "config": f"config{cfg.cfg_id}", "steps": steps, "tau": TAU,
            "apex_over_no_prefetch_at_largest_window": last["apex"]["tokens_per_s"] / last["no_prefetch"]["tokens_per_s"]}


def hidden_inputs(cfg, T, B, device):
    """[T][L][B][d] tensors on the device (h, h')."""
    import torch
    from paper_2608_11688_b200 import synth
    hs = [synth.hidden_states(cfg, l, T, B) for l in range(cfg.L)]
    h = torch.from_numpy(np.stack([x[0] for x in hs], 1))
    hp = torch.from_numpy(np.stack([x[1] for x in hs], 1))
    return h, hp


def time_tokens(apex, h, hp, y, B, mode, warmup, steps, dist_sync=None, host=False):
    """W untimed + K timed decode tokens; returns seconds (CUDA events on the launching stream)."""
    import torch
    T = h.shape[0]
    run = (lambda t: apex.decode_token_host(h[t % T], hp[t % T], B, TAU, mode, y)) if host else \
          (lambda t: apex.decode_token(h[t % T], hp[t % T], B, TAU, mode, y))
    for t in range(warmup):
        run(t)
    torch.cuda.synchronize()
    if dist_sync:
        dist_sync()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for t in range(warmup, warmup + steps):
        run(t)
    e1.record()
    torch.cuda.synchronize()
    if dist_sync:
        dist_sync()
    return e0.elapsed_time(e1) * 1e-3


def time_ffn_kernel(apex, cfg, h, hp, B, tokens):
    """Average device time of one expert-FFN launch, all experts resident.  Per token the prefetch routers
    and the gates of all layers run first; then the L expert-FFN kernels are launched back to back (each reads its own
    layer's experts, so nothing is served from L2) between two CUDA events on the launching stream."""
    import torch
    dev = h.device
    idx = torch.empty((cfg.L, B, cfg.k), dtype=torch.int32, device=dev)
    al = torch.empty((cfg.L, B, cfg.N), dtype=torch.float32, device=dev)
    y = torch.empty((cfg.L, B, cfg.d), dtype=torch.float32, device=dev)
    T = h.shape[0]
    per_launch = []
    stream = torch.cuda.current_stream().cuda_stream
    y_ptr = [y[l].data_ptr() for l in range(cfg.L)]
    cand = torch.empty((B, cfg.N), dtype=torch.int32, device=dev)
    ncand = torch.empty((B,), dtype=torch.int32, device=dev)
    for t in range(tokens + 1):
        hp_ptr = [hp[t % T, l].data_ptr() for l in range(cfg.L)]
        for l in range(cfg.L):      # the steps that precede the expert FFN in a decode step (nothing to copy: all resident)
            apex.predict(l, h[t % T, l], B)
            apex.select_candidates(l, B, TAU, cand, ncand)
            apex.prefetch(l, B)
        for l in range(cfg.L):
            apex.route_topk(l, hp[t % T, l], B, idx[l], al[l])
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for l in range(cfg.L):
            apex.moe_ffn_begin_raw(l, 0, hp_ptr[l], B, y_ptr[l], stream)
        e1.record()
        for l in range(cfg.L):
            apex.moe_ffn_end(l)
        torch.cuda.synchronize()
        if t > 0:                       # first pass is warm-up
            per_launch.append(e0.elapsed_time(e1) / cfg.L)
    return statistics.mean(per_launch) * 1e-3, statistics.median(per_launch) * 1e-3, len(per_launch) * cfg.L


def time_token_kernel(cfg, prob, h, hp, y, tokens, standin):
    """Average device time of one launch of the persistent token kernel (all L layer-steps of a token: prefetch
    router, budget, gate, expert FFN, hand-over between layers), all experts resident, CUDA events on the launching
    stream around `tokens` launches after a warm-up.  standin=False leaves the stand-in attention's bytes out, so the
    launch moves the method's own bytes only."""
    import torch
    from paper_2608_11688_b200 import binding
    a = make_ctx(cfg, prob, cfg.N, flags=0 if standin else binding.FLAG_SKIP_STANDIN)
    try:
        a.warm_all()
        T = h.shape[0]
        n0 = a.launch_count()
        for t in range(4):
            a.decode_token(h[t % T], hp[t % T], 1, TAU, "exact", y)
        per_token = (a.launch_count() - n0) / 4
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for t in range(tokens):
            a.decode_token(h[(4 + t) % T], hp[(4 + t) % T], 1, TAU, "exact", y)
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) * 1e-3 / tokens, per_token
    finally:
        a.destroy()


def other_config_rooflines(dev, peak, peak_kind):
    """The expert-FFN launch of the other configs of the workload table against the same roofline: all experts resident,
    a few layers each (every launch reads its own layer's experts and a token's launches together exceed L2), CUDA
    events on the launching stream.  B = 1: the streaming kernel; B > 1: plan + gather + the two tcgen05 GEMMs, bytes =
    expected distinct experts of B uniformly routed tokens.  `traffic` is null: no ncu capture at these shapes except
    where NCU_TRAFFIC_BYTES has one."""
    import torch
    from paper_2608_11688_b200 import synth
    out = {}
    for cfg_id, layers, batches in ((0, 8, (1,)), (2, 4, (1,)), (3, 2, (1,)), (4, 4, (1, 32, 256))):
        cfg = synth.CONFIGS[cfg_id].scaled(L=layers)
        prob = build_problem(cfg, dev)
        for B in batches:
            h, hp = hidden_inputs(cfg, 4, B, dev)
            h, hp = h.to(dev), hp.to(dev)
            a = make_ctx(cfg, prob, cfg.N, max_batch=B)
            try:
                a.warm_all()
                mean_s, med_s, n_l = time_ffn_kernel(a, cfg, h, hp, B, tokens=6)
            finally:
                a.destroy()
            if B == 1:
                _, bytes_ffn = algorithmic_bytes(cfg, B)
                kernel = "moe_ffn_stream_kernel"
            else:
                distinct = cfg.N * (1.0 - (1.0 - cfg.k / cfg.N) ** B)
                bytes_ffn = distinct * cfg.expert_bytes + cfg.shared_bytes + 2 * B * cfg.d * 4
                kernel = "ffn_plan_kernel + ffn_tc_gather_kernel + ffn_tc_gemm_kernel<1>, <2>"
            ach = bytes_ffn / mean_s / 1e9
            rec = {
                "bound": "hbm", "kernel": kernel, "achieved": ach, "peak": peak, "unit": "GB/s", "frac": ach / peak,
                "peak_kind": f"of {peak_kind}", "traffic": NCU_TRAFFIC_BYTES.get(cfg_id) if B == 1 else None,
                "algorithmic_bytes_per_launch": bytes_ffn, "us_per_launch_mean": mean_s * 1e6, "launches_timed": n_l,
                "layers": layers, "B": B}
            if B == 1:
                # the product path at B = 1: the token kernel over these layers (no stand-in: the method's bytes only)
                y1 = torch.empty((cfg.L, 1, cfg.d), dtype=torch.float32, device=dev)
                sec_tok, per_token = time_token_kernel(cfg, prob, h, hp, y1, 16, standin=False)
                if per_token == 1.0:
                    bytes_step, _ = algorithmic_bytes(cfg, 1)
                    bt = cfg.L * (bytes_step + cfg.d * 4)
                    rec["decode_token_kernel"] = {"us_per_layer_step": sec_tok * 1e6 / cfg.L, "achieved": bt / sec_tok / 1e9,
                                                  "frac": bt / sec_tok / 1e9 / peak, "algorithmic_bytes_per_launch": bt}
            out[f"config{cfg_id}" + (f"_B{B}" if len(batches) > 1 else "")] = rec
            del h, hp
        del prob
        torch.cuda.empty_cache()
    return out


def oracle_tokens_per_s(cfg, prob, n_tokens):
    """The CPU oracle as it stands, timed on the host cores over n_tokens full decode tokens."""
    import torch
    from oracle import apex_oracle as ao
    from paper_2608_11688_b200 import synth
    routers, cdf, store, shared = prob
    caches = [ao.SlotCache(cfg.N, cfg.C) for _ in range(cfg.L)]
    hs = [synth.hidden_states(cfg, l, n_tokens, 1) for l in range(cfg.L)]
    t0 = time.perf_counter()
    for t in range(n_tokens):
        for l in range(cfg.L):
            W_r, b_r, W_p, b_p = routers[l]
            w, theta = cdf[l]

            def experts(e, l=l):
                a = store[l, e].to(torch.float32).numpy()
                return synth.split_store(a)
            sh = None
            if shared[l] is not None:
                s = shared[l].cpu().to(torch.float32).numpy()
                sh = synth.split_store(s)
            ao.layer_step(caches[l], W_p=W_p, b_p=b_p, W_r=W_r, b_r=b_r, w=w, theta=theta, tau=TAU, k=cfg.k,
                          h=hs[l][0][t], h_post=hs[l][1][t], mode="exact", expert_weights=experts, shared=sh)
    dt = time.perf_counter() - t0
    try:
        from threadpoolctl import threadpool_info
        cores = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        cores = 1
    return n_tokens / dt, cores, dt


# ------------------------------------------------------------------------------------------------
def run_reference(args, cfg, rank):
    """--impl reference: the oracle on the host cores, same metric and workload, bounded sample."""
    if rank != 0:
        return
    import torch
    dev = "cuda" if torch.cuda.is_available() else "cpu"
    from paper_2608_11688_b200 import synth
    routers = [synth.router_weights(cfg, l) for l in range(cfg.L)]
    cdf = [synth.cdf_params(cfg, l) for l in range(cfg.L)]
    store = torch.empty((cfg.L, cfg.N, cfg.I, 3, cfg.d), dtype=torch.bfloat16)
    shared = []
    for l in range(cfg.L):
        store[l].copy_(synth.expert_store(cfg, l, device=dev))
        sh = synth.shared_expert(cfg, l, device=dev)
        shared.append(None if sh is None else sh.cpu())
    prob = (routers, cdf, store, shared)
    n = max(1, args.steps)
    for _ in range(min(args.warmup, 1)):
        oracle_tokens_per_s(cfg, prob, 1)
    tps, cores, dt = oracle_tokens_per_s(cfg, prob, n)
    line = {"impl": "reference", "metric": METRIC, "value": tps, "unit": UNIT, "n_gpus": args.gpus, "steps": n,
            "warmup": min(args.warmup, 1), "ms_per_step": 1e3 * dt / n, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": f"config{cfg.cfg_id}:{cfg.name}", "L": cfg.L, "d": cfg.d, "N": cfg.N, "k": cfg.k,
                       "I": cfg.I, "C": cfg.C, "B": 1, "tau": TAU, "mode": "exact"},
            "cpu_baseline": {"value": tps, "unit": UNIT, "cores": cores, "kind": "oracle",
                             "sample": f"{n} decode tokens x {cfg.L} layers, every step of the path in fp64 numpy"},
            "e2e": {"value": tps, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--config", type=int, default=1)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--cpu-baseline-tokens", type=int, default=2)
    ap.add_argument("--skip-extras", action="store_true", help="only the headline leg (used for ncu launch lists)")
    ap.add_argument("--no-other-configs", dest="other_configs", action="store_false",
                    help="leave out the roofline sub-records of configs 0, 2, 3 and 4 (they add about a minute)")
    ap.add_argument("--ffn-only", action="store_true",
                    help="profiling case: all experts resident, gate + expert FFN only, no copy in flight")
    ap.add_argument("--layers", type=int, default=None, help="use only the first LAYERS layers (smaller captures)")
    ap.add_argument("--batch", type=int, default=1, help="tokens per decode step (config 4 sweeps 1, 8, 32, 128, 256)")
    ap.add_argument("--no-policies", dest="policies", action="store_false",
                    help="skip the baselines of the paper's comparison (no prefetch, static top-k, top-(k+4), top-(k+8))")
    ap.add_argument("--policies", dest="policies", action="store_true", help="(default) time those baselines too")
    ap.set_defaults(policies=True)
    ap.add_argument("--resident", action="store_true",
                    help="cache as large as the expert count, warmed up: no host-link copies (kernel launch lists)")
    ap.add_argument("--spec", action="store_true", help="A/B: expert FFN with the speculative first fill (FLAG_SPECULATE)")
    ap.add_argument("--layer-launches", action="store_true",
                    help="A/B: the per-layer kernel sequence instead of the persistent token kernel (FLAG_LAYER_LAUNCHES)")
    ap.add_argument("--standin-ahead", action="store_true",
                    help="A/B: the token kernel requests the stand-in attention's bytes ahead of the previous layer's completion (FLAG_STANDIN_AHEAD)")
    ap.add_argument("--no-standin", action="store_true",
                    help="leave the stand-in attention out of the decode step (FLAG_SKIP_STANDIN): the method's own bytes only")
    ap.add_argument("--fp8", action="store_true",
                    help="datatype study: e4m3 expert store with per-row scales (needs --ffn-only or --skip-extras)")
    ap.add_argument("--link-sweep", action="store_true",
                    help="study: per-token latency of the policies on a throttled host link (every expert copy padded to "
                         "its duration at 8, 16 and 32 GB/s) and on the link as it is")
    ap.add_argument("--window-sweep", action="store_true",
                    help="study: the policies of Sec. V-A with the hiding window (the stand-in attention, through ctx_len) "
                         "lengthened until it holds 0.5, 1, 2, 4 and 8 expert copies -- the regime in which Eq. (12) can hold")
    ap.add_argument("--predictor-noise", type=float, default=1.0,
                    help="study: scales what makes the prefetch router wrong in the synthetic workload (the noise on W_p and "
                         "the part of h' the router cannot see): 1 is the workload of the configs, 0.2 a good predictor.  "
                         "The frozen confidence models were fitted at 1: combine with --train-aux")
    ap.add_argument("--train-aux", action="store_true",
                    help="study: distil the prefetch routers and refit the confidence models on this GPU first "
                         "(a different predictor than the workload's: needs --skip-extras)")
    ap.add_argument("--fp4", action="store_true",
                    help="datatype study: block-scaled e2m1 expert store (needs --ffn-only or --skip-extras)")
    ap.add_argument("--trace", action="store_true",
                    help="debug: run a few decode tokens on the library built with time stamps (trace.py) and print the "
                         "kernel spans of the last two; combine with --resident / --layers / --batch / --config")
    args = ap.parse_args()
    if (args.fp8 or args.fp4) and not (args.ffn_only or args.skip_extras):
        ap.error("--fp8 / --fp4 are study legs: combine them with --ffn-only or --skip-extras")
    if args.train_aux and not (args.skip_extras or args.window_sweep):
        ap.error("--train-aux is a study leg: combine it with --skip-extras or --window-sweep")
    if args.predictor_noise != 1.0 and not (args.skip_extras or args.window_sweep):
        ap.error("--predictor-noise is a study leg: combine it with --skip-extras or --window-sweep")
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))

    from paper_2608_11688_b200 import synth
    cfg = synth.CONFIGS[args.config]
    if args.layers:
        cfg = cfg.scaled(L=args.layers)
    if args.predictor_noise != 1.0:
        cfg = cfg.scaled(sigma_p=cfg.sigma_p * args.predictor_noise, hidden_noise=cfg.hidden_noise * args.predictor_noise)
    if args.impl == "reference":
        args.steps = 2 if args.steps is None else min(args.steps, 4)
        args.warmup = 0 if args.warmup is None else args.warmup
        run_reference(args, cfg, rank)
        return
    args.steps = 48 if args.steps is None else args.steps
    args.warmup = 4 if args.warmup is None else max(3, args.warmup)

    import torch
    from paper_2608_11688_b200 import build
    assert torch.cuda.is_available(), "bench.py needs a CUDA device (there is no CPU fallback)"
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if rank == 0:
        build.build()
    trace_lib = None
    if args.trace:   # before anything loads the product library: a process holds one of the two
        from paper_2608_11688_b200 import trace
        trace_lib = trace.use_trace_library()
    from paper_2608_11688_b200 import replicas
    dist_sync = None
    if world > 1:
        replicas.init("nccl", dev)
        replicas.barrier()
        dist_sync = replicas.barrier
    B = args.batch
    from paper_2608_11688_b200 import binding as _b
    base_flags = (_b.FLAG_SPECULATE if args.spec else 0) | (_b.FLAG_LAYER_LAUNCHES if args.layer_launches else 0) | \
                 (_b.FLAG_SKIP_STANDIN if args.no_standin else 0) | (_b.FLAG_STANDIN_AHEAD if args.standin_ahead else 0)
    prob = build_problem(cfg, dev, fp8=args.fp8, fp4=args.fp4)
    aux_info = None
    if args.train_aux:
        r2, c2, aux_info = train_auxiliary(cfg, prob, dev)
        prob = (r2, c2, prob[2], prob[3])
    # bytes of a stored row relative to bf16
    row_scale = synth.fp4_row_bytes(cfg.d) / (6 * cfg.d) if args.fp4 else (3 * cfg.d + 16) / (6 * cfg.d) if args.fp8 else 1.0
    T = min(cfg.T, args.warmup + args.steps)
    h, hp = hidden_inputs(cfg, T, B, dev)
    h_dev, hp_dev = h.to(dev), hp.to(dev)
    h_pin, hp_pin = h.pin_memory(), hp.pin_memory()
    y_dev = torch.empty((cfg.L, B, cfg.d), dtype=torch.float32, device=dev)
    y_pin = torch.empty((cfg.L, B, cfg.d), dtype=torch.float32).pin_memory()

    if args.trace:
        a = make_ctx(cfg, prob, cfg.N if args.resident else cfg.C, max_batch=B, flags=base_flags)
        if args.resident:
            a.warm_all()
        for t in range(args.warmup):
            a.decode_token(h_dev[t % T], hp_dev[t % T], B, TAU, "exact", y_dev)
        torch.cuda.synchronize()
        trace.reset(trace_lib)
        n_tok = 2
        for t in range(args.warmup, args.warmup + n_tok):
            a.decode_token(h_dev[t % T], hp_dev[t % T], B, TAU, "exact", y_dev)
        torch.cuda.synchronize()
        spans = trace.read_spans(trace_lib)
        per_layer = max(1, len(spans) // (n_tok * cfg.L))
        print(trace.format_spans(spans, limit=3 * per_layer + 2), file=sys.stderr)
        summary = trace.summarize(spans)
        persistent = trace.KERNEL_NAMES[10] in summary
        n_sm = torch.cuda.get_device_properties(dev).multi_processor_count
        phases = trace.ffn_phase_medians(trace.read_ffn_cta_stamps(trace_lib, n_sm)) if (B == 1 and not persistent) else {}
        dec = trace.decode_phase_medians(trace.read_decode_stamps(trace_lib, n_sm, cfg.L)) if persistent else {}
        if persistent:
            print(trace.format_decode_phases(dec), file=sys.stderr)
        print(json.dumps({"trace": summary, "tokens_traced": n_tok, "layers": cfg.L, "B": B,
                          "us_per_layer_step": summary["_all"]["wall_us"] / (n_tok * cfg.L),
                          "ffn_cta_phase_median_cycles": phases, "persistent_kernel_phase_median_us": dec,
                          "config": f"config{cfg.cfg_id}", "resident": bool(args.resident)}), flush=True)
        a.destroy()
        return

    if args.window_sweep:
        print(json.dumps(window_sweep(args, cfg, prob, h_dev, hp_dev, y_dev, B)), flush=True)
        return

    if args.link_sweep:
        import torch
        table = {}
        for bw in (8.0, 16.0, 32.0, 0.0):
            row = {}
            for name, tau_p, delta in (POLICIES[0], POLICIES[1], POLICIES[4]):
                row[name] = run_policy(cfg, prob, h_dev, hp_dev, y_dev, B, name, tau_p, delta, args.warmup, args.steps,
                                       link_gbs=bw)
            table["host link as it is" if bw == 0.0 else f"{bw:.0f} GB/s"] = row
        a3 = make_ctx(cfg, prob, cfg.N, max_batch=B)
        a3.warm_all()
        sec_res = time_tokens(a3, h_dev, hp_dev, y_dev, B, "exact", args.warmup, args.steps)
        a3.destroy()
        print(json.dumps({"link_sweep": table, "all_resident_ms_per_token": 1e3 * sec_res / args.steps,
                          "config": f"config{cfg.cfg_id}", "steps": args.steps, "tau": TAU}), flush=True)
        return

    if args.ffn_only:
        a = make_ctx(cfg, prob, cfg.N, max_batch=B, flags=2 if args.spec else 0)
        a.warm_all()
        mean_s, med_s, n_l = time_ffn_kernel(a, cfg, h_dev, hp_dev, B, tokens=args.steps)
        if B == 1:
            _, bytes_ffn = algorithmic_bytes(cfg, B)
        else:   # expected number of distinct experts touched by B tokens with uniform routing
            distinct = cfg.N * (1.0 - (1.0 - cfg.k / cfg.N) ** B)
            bytes_ffn = distinct * cfg.expert_bytes + cfg.shared_bytes + 2 * B * cfg.d * 4
        bytes_ffn = (bytes_ffn - 2 * B * cfg.d * 4) * row_scale + 2 * B * cfg.d * 4
        flops = 2.0 * 3 * cfg.d * (cfg.k * cfg.I + cfg.I_shared) * B
        print(json.dumps({"ffn_only": True, "B": B, "weights": "e2m1" if args.fp4 else "e4m3" if args.fp8 else "bf16", "us_per_launch_mean": mean_s * 1e6, "us_per_launch_median": med_s * 1e6,
                          "launches": n_l, "GBps_mean": bytes_ffn / mean_s / 1e9, "bytes_per_launch": bytes_ffn,
                          "TFLOPs": flops / mean_s / 1e12}), flush=True)
        a.destroy()
        return

    # ---- headline: config cache size, exact (correctness-preserving) mode, inputs resident in HBM
    apex = make_ctx(cfg, prob, cfg.N if args.resident else cfg.C, max_batch=B, flags=base_flags)
    if args.resident:
        apex.warm_all()
    sampler = ClockSampler(local_rank)
    sampler.start()
    n0 = apex.launch_count()
    sec = time_tokens(apex, h_dev, hp_dev, y_dev, B, "exact", args.warmup, args.steps, dist_sync)
    launches = (apex.launch_count() - n0) * args.steps // (args.warmup + args.steps)
    clocks = sampler.stop()
    st_all = apex.get_stats()
    sec = replicas.max_over_ranks(sec, dev)
    value = world * args.steps * B / sec
    extras = {}
    e2e = None
    roof = None
    cpu = None
    bytes_step, bytes_ffn = algorithmic_bytes(cfg, B)
    peak, peak_kind = measured_peak()
    if not args.skip_extras:
        # ---- end to end: host buffers in, host buffer out, through the C-ABI call
        apex.reset_stats()
        sec_e2e = time_tokens(apex, h_pin, hp_pin, y_pin, B, "exact", args.warmup, args.steps, dist_sync, host=True)
        sec_e2e = replicas.max_over_ranks(sec_e2e, dev)
        st = apex.get_stats()
        per_tok = args.warmup + args.steps
        e2e = {"value": world * args.steps * B / sec_e2e, "unit": UNIT,
               "h2d_bytes_per_step": int(2 * cfg.L * B * cfg.d * 4), "d2h_bytes_per_step": int(cfg.L * B * cfg.d * 4),
               "expert_bytes_copied_per_step": int(st["bytes_copied"] / per_tok)}
        extras["exact"] = {
            "tokens_per_s": args.steps * B / sec, "overlap_vs_P": st["hits_P"] / max(1, st["routed"]),
            "overlap_vs_R": st["hits_R"] / max(1, st["routed"]), "coverage": st["covered"] / max(1, st["tokens"]),
            "mean_delta_hat": st["sum_delta_hat"] / max(1, st["tokens"]),
            "mean_delta_star": st["sum_delta_star"] / max(1, st["tokens"]),
            "copies_per_token": (st["prefetch_copies"] + st["demand_copies"]) / per_tok,
            "demand_copies_per_token": st["demand_copies"] / per_tok,
            "device_flag_wait_us_per_token": st["stall_ns"] / per_tok / 1e3,
            "h2d_expert_gbs": st["bytes_copied"] / per_tok / (sec_e2e / args.steps) / 1e9}
        apex.destroy()
        if rank == 0:
            # ---- stall-free mode
            a2 = make_ctx(cfg, prob, cfg.C, max_batch=B)
            if "stall_free" in cfg.modes:
                sec_sf = time_tokens(a2, h_dev, hp_dev, y_dev, B, "stall_free", args.warmup, args.steps)
                s2 = a2.get_stats()
                extras["stall_free"] = {"tokens_per_s": args.steps * B / sec_sf,
                                        "substitutions_per_token": s2["substitutions"] / (args.warmup + args.steps),
                                        "copies_per_token": s2["prefetch_copies"] / (args.warmup + args.steps)}
            a2.destroy()
            # ---- policy baselines of Sec. V-A under the same harness (same ranking, different budgets)
            if args.policies:
                pol = {}
                for name, tau_p, delta in POLICIES[:4]:
                    pol[name] = run_policy(cfg, prob, h_dev, hp_dev, y_dev, B, name, tau_p, delta, args.warmup, args.steps)
                extras["policies"] = pol
            # ---- all experts resident (C = N): isolates the kernels from the host link
            a3 = make_ctx(cfg, prob, cfg.N, max_batch=B)
            a3.warm_all()
            sec_res = time_tokens(a3, h_dev, hp_dev, y_dev, B, "exact", args.warmup, args.steps)
            extras["all_resident"] = {"tokens_per_s": args.steps * B / sec_res,
                                      "frac_of_8TBs": bytes_step * cfg.L * args.steps / sec_res / 1e9 / NOMINAL_HBM_GBS,
                                      "frac_of_peak": bytes_step * cfg.L * args.steps / sec_res / 1e9 / peak}
            extras["exact"]["exposed_stall_us_per_token"] = (sec / args.steps - sec_res / args.steps) * 1e6
            # ---- the per-layer expert-FFN kernel alone (the kernel behind apex_moe_ffn)
            mean_s, med_s, n_l = time_ffn_kernel(a3, cfg, h_dev, hp_dev, B, tokens=max(2, min(8, args.steps)))
            achieved = bytes_ffn / mean_s / 1e9
            ffn_alone = {"bound": "hbm", "kernel": "moe_ffn_stream_kernel", "achieved": achieved, "peak": peak, "unit": "GB/s",
                         "frac": achieved / peak, "peak_kind": f"of {peak_kind}", "frac_of_8TBs": achieved / NOMINAL_HBM_GBS,
                         "traffic": NCU_TRAFFIC_BYTES.get(cfg.cfg_id), "algorithmic_bytes_per_launch": bytes_ffn,
                         "us_per_launch_mean": mean_s * 1e6, "us_per_launch_median": med_s * 1e6, "launches_timed": n_l}
            a3.destroy()
            roof = ffn_alone
            if B == 1 and not (args.layer_launches or args.fp8 or args.fp4):
                # ---- the dominant kernel of the decode step: the persistent token kernel, one launch = all L layer-steps.
                # Algorithmic bytes per launch: L x (routed expert weights + shared FFN + both routers + h, h', y).
                n_tok = max(8, min(32, args.steps))
                sec_tok, per_token = time_token_kernel(cfg, prob, h_dev, hp_dev, y_dev, n_tok, standin=False)
                if per_token == 1.0:   # (a context that fell back to per-layer launches has no such kernel)
                    bytes_tok = cfg.L * (bytes_step + cfg.d * 4)
                    ach = bytes_tok / sec_tok / 1e9
                    sec_att, _ = time_token_kernel(cfg, prob, h_dev, hp_dev, y_dev, n_tok, standin=True)
                    attn_bytes = (4 * cfg.d * cfg.d + 2 * 1024 * cfg.d) * 2
                    roof = {"bound": "hbm", "kernel": "decode_token_kernel", "achieved": ach, "peak": peak, "unit": "GB/s",
                            "frac": ach / peak, "peak_kind": f"of {peak_kind}", "frac_of_8TBs": ach / NOMINAL_HBM_GBS,
                            "traffic": None, "algorithmic_bytes_per_launch": bytes_tok, "us_per_launch_mean": sec_tok * 1e6,
                            "us_per_layer_step": sec_tok * 1e6 / cfg.L, "launches_timed": n_tok,
                            "launch": f"one token = {cfg.L} layer-steps, all experts resident, stand-in attention left out",
                            "with_standin": {"us_per_launch_mean": sec_att * 1e6, "bytes_per_launch": bytes_tok + cfg.L * attn_bytes,
                                             "achieved": (bytes_tok + cfg.L * attn_bytes) / sec_att / 1e9,
                                             "frac": (bytes_tok + cfg.L * attn_bytes) / sec_att / 1e9 / peak},
                            "per_layer_ffn_kernel_alone": ffn_alone}
            # ---- the same roofline for the FFN launch of the other configs (a few layers each)
            if args.other_configs and world == 1:
                extras["roofline_other_configs"] = other_config_rooflines(dev, peak, f"{peak_kind}")
            # ---- the oracle on the host cores (bounded sample)
            tps, cores, dt = oracle_tokens_per_s(cfg, prob, args.cpu_baseline_tokens)
            cpu = {"value": tps, "unit": UNIT, "cores": cores, "kind": "oracle",
                   "sample": f"{args.cpu_baseline_tokens} decode tokens x {cfg.L} layers ({dt:.1f} s)"}
    else:
        apex.destroy()
    replicas.finish()
    if rank != 0:
        return
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": 1e3 * sec / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "e2m1 weights, fp32 accumulation" if args.fp4 else "e4m3 weights, fp32 accumulation" if args.fp8 else "bf16",
            "data": "synthetic",
            "config": {"workload": f"config{cfg.cfg_id}:{cfg.name}" + (" (e2m1 expert store)" if args.fp4 else " (e4m3 expert store)" if args.fp8 else ""),
                       "L": cfg.L, "d": cfg.d, "N": cfg.N, "k": cfg.k,
                       "I": cfg.I, "C": cfg.N if args.resident else cfg.C, "B": B, "tau": TAU, "mode": "exact", "ctx_len": 1024,
                       "parallelism": "replicas only" if world > 1 else "single GPU",
                       "l2": "inputs larger than L2: each token streams %.0f MB of expert and attention bytes" %
                             ((bytes_step + (4 * cfg.d * cfg.d + 2 * 1024 * cfg.d) * 2) * cfg.L / 1e6)},
            "clocks": clocks, "gpu_launches": int(launches),
            "e2e": e2e, "roofline": roof, "cpu_baseline": cpu, "modes": extras,
            "stats_headline": {"copies_per_token": (st_all["prefetch_copies"] + st_all["demand_copies"]) / (args.warmup + args.steps)}}
    if aux_info is not None:
        line["config"]["workload"] += " (prefetch routers distilled and confidence models refitted on this GPU)"
        line["trained_auxiliary"] = dict(aux_info, overlap_vs_P=st_all["hits_P"] / max(1, st_all["routed"]),
                                         coverage=st_all["covered"] / max(1, st_all["tokens"]),
                                         mean_delta_hat=st_all["sum_delta_hat"] / max(1, st_all["tokens"]),
                                         mean_delta_star=st_all["sum_delta_star"] / max(1, st_all["tokens"]),
                                         demand_copies_per_token=st_all["demand_copies"] / (args.warmup + args.steps))
    print(json.dumps(line), flush=True)


if __name__ == "__main__":
    main()

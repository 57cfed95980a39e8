// C-ABI entry points, part 2: the layer-step -- the host side of the prefetch machinery (slot planning,
// cudaMemcpyAsync on the copy streams, slot-ready flags, demand copies) and the kernel launches.  All arithmetic of
// the path runs in the kernels.
#include "apex_host.hpp"

using namespace apex;

namespace apex {

// Emulated link: measures, once, how long an expert copy from the registered store takes and what a padding
// copy over the host link costs (latency and time per byte), with CUDA events on the copy stream.
int calibrate_link(apex_ctx* ctx, uint8_t* dst, const uint8_t* src, cudaStream_t cs) {
  cudaEvent_t e0, e1;
  CU_TRY(ctx, cudaEventCreate(&e0));
  CU_TRY(ctx, cudaEventCreate(&e1));
  auto time_copy = [&](void* d, const void* s_, size_t n, cudaMemcpyKind kind, double* us) -> int {
    float best = 1e30f;
    for (int rep = 0; rep < 5; ++rep) {
      CU_TRY(ctx, cudaEventRecord(e0, cs));
      CU_TRY(ctx, cudaMemcpyAsync(d, s_, n, kind, cs));
      CU_TRY(ctx, cudaEventRecord(e1, cs));
      CU_TRY(ctx, cudaEventSynchronize(e1));
      float ms = 0.f;
      CU_TRY(ctx, cudaEventElapsedTime(&ms, e0, e1));
      best = ms < best ? ms : best;
    }
    *us = (double)best * 1e3;
    return APEX_OK;
  };
  CU_TRY(ctx, cudaStreamSynchronize(cs));
  double t_small = 0.0, t_large = 0.0;
  const size_t small = 64 * 1024, large = ctx->pad_bytes;
  int r = time_copy(dst, src, ctx->expert_bytes, cudaMemcpyDefault, &ctx->real_copy_us);
  if (r == APEX_OK) r = time_copy(ctx->pad_dst, ctx->pad_src, small, cudaMemcpyHostToDevice, &t_small);
  if (r == APEX_OK) r = time_copy(ctx->pad_dst, ctx->pad_src, large, cudaMemcpyHostToDevice, &t_large);
  cudaEventDestroy(e0);
  cudaEventDestroy(e1);
  if (r != APEX_OK) return r;
  ctx->pad_us_per_byte = (t_large - t_small) / (double)(large - small);
  ctx->pad_lat_us = t_small - (double)small * ctx->pad_us_per_byte;
  if (!(ctx->pad_us_per_byte > 0.0)) return fail(ctx, APEX_ECUDA, "link calibration: padding copies took no time");
  if (ctx->pad_lat_us < 0.0) ctx->pad_lat_us = 0.0;
  ctx->link_calibrated = true;
  return APEX_OK;
}

// One expert copy host store -> slot, followed by the slot-ready flag on the same stream.
int issue_copy(apex_ctx* ctx, int layer, int e, int slot, cudaStream_t cs) {
  if (!ctx->store_base[layer]) return fail(ctx, APEX_ESTATE, "no expert store registered for this layer");
  if (ctx->inject == 1) {
    ctx->inject = 0;
    return fail(ctx, APEX_ECUDA, "injected copy-issue failure");
  }
  const size_t C = ctx->cfg.C;
  uint8_t* dst = ctx->d_cache + ((size_t)layer * C + slot) * ctx->expert_bytes;
  const uint8_t* src = ctx->store_base[layer] + (size_t)e * ctx->store_stride[layer];
  const uint32_t gen = ++ctx->slot_gen[layer][slot];
  if (ctx->cfg.link_gbs > 0.0 && !ctx->link_calibrated) {
    int r = calibrate_link(ctx, dst, src, cs);
    if (r != APEX_OK) return r;
  }
  CU_TRY(ctx, cudaMemcpyAsync(dst, src, ctx->expert_bytes, cudaMemcpyDefault, cs));
  if (ctx->cfg.link_gbs > 0.0) {
    // the copy should have taken expert bytes / link_gbs: pad what is missing with a copy over the host link
    const double target_us = (double)ctx->expert_bytes / (ctx->cfg.link_gbs * 1e3);
    const double missing_us = target_us - ctx->real_copy_us - ctx->pad_lat_us;
    double left_us = missing_us;
    for (int guard = 0; left_us > 0.0 && guard < 64; ++guard) {  // as many padding copies as it takes
      size_t pad = (size_t)(left_us / ctx->pad_us_per_byte);
      pad = pad > ctx->pad_bytes ? ctx->pad_bytes : (pad & ~(size_t)255);
      if (!pad) break;
      CU_TRY(ctx, cudaMemcpyAsync(ctx->pad_dst, ctx->pad_src, pad, cudaMemcpyHostToDevice, cs));
      left_us -= ctx->pad_lat_us + (double)pad * ctx->pad_us_per_byte;
    }
  }
  uint32_t* flag = ctx->d_slot_ready + (size_t)layer * C + slot;
  if (ctx->inject == 2) {
    ctx->inject = 0;
    ctx->withheld_flag = flag;
    ctx->withheld_gen = gen;
    ctx->withheld_stream = cs;
  } else {
    int r = stream_write32(ctx, cs, flag, gen);
    if (r != APEX_OK) return r;
  }
  ctx->phys_expert[layer][slot] = e;
  ctx->host_stats[layer].bytes_copied += (int64_t)ctx->expert_bytes;
  return APEX_OK;
}

int release_withheld(apex_ctx* ctx) {
  if (!ctx->withheld_flag) return APEX_OK;
  uint32_t* srcv = ctx->gen_src + (ctx->gen_src_pos++ % ctx->gen_src_len);
  *srcv = ctx->withheld_gen;
  CU_TRY(ctx, cudaMemcpyAsync(ctx->withheld_flag, srcv, sizeof(uint32_t), cudaMemcpyHostToDevice, ctx->withheld_stream));
  ctx->withheld_flag = nullptr;
  return APEX_OK;
}

SlotSnapshot make_snapshot(apex_ctx* ctx, int layer) {
  SlotSnapshot s;
  const auto& es = ctx->tables[layer].expert_slot();
  s.resident_mask = 0;
  for (int e = 0; e < APEX_MAX_EXPERTS; ++e) {
    const int slot = e < ctx->cfg.N ? es[e] : -1;
    s.expert_slot[e] = (int8_t)slot;
    s.need_gen[e] = slot >= 0 ? ctx->slot_gen[layer][slot] : 0u;
    if (slot >= 0) s.resident_mask |= (1ull << e);
  }
  return s;
}

int check_device_status(apex_ctx* ctx) {
  if (mhdr(ctx)->status != 0) {
    mhdr(ctx)->status = 0;
    release_withheld(ctx);
    // If it was a wait for a demand copy inside the kernel, launches may not be asynchronous here (the copy is issued
    // after the launch returns): from now on misses are corrected by further launches instead.
    ctx->host_waves = true;
    ctx->dec_dirty = true;  // a persistent decode launch that gave up leaves its counters short
    return fail(ctx, APEX_ETIMEOUT, "a device-side wait on a slot-ready flag or a demand copy ran out");
  }
  return APEX_OK;
}

}  // namespace apex

namespace {


int begin_predict(apex_ctx* ctx, int layer, const float* h_dev, int B, RouterParams* p) {
  if (!h_dev || B < 1 || B > ctx->cfg.max_batch) return fail(ctx, APEX_EINVAL, "apex_predict: bad h or B");
  const size_t N = ctx->cfg.N, d = ctx->cfg.d;
  if (ctx->step[layer].pending) return fail(ctx, APEX_ESTATE, "the previous expert FFN of this layer has not been completed");
  ctx->tables[layer].begin_step();
  ctx->last_copies[layer].clear();
  ctx->step[layer] = apex_ctx::StepState{};
  ctx->step[layer].B = B;
  *p = RouterParams{};
  p->W = ctx->d_Wp + (size_t)layer * N * d;
  p->bias = ctx->has_bp[layer] ? ctx->d_bp + (size_t)layer * N : nullptr;
  p->x = h_dev;
  p->z_out = ctx->d_zp;
  p->q_out = ctx->d_qp;
  p->pi_out = ctx->d_pi;
  p->topk_out = B == 1 ? ctx->d_spec + (size_t)layer * APEX_MAX_TOPK : nullptr;  // the FFN's speculative first fill
  p->N = (int)N; p->d = (int)d; p->B = B; p->k = ctx->cfg.k; p->C = ctx->cfg.C;
  return APEX_OK;
}

int fill_select(apex_ctx* ctx, int layer, int B, float tau, int32_t* cand_dev, int32_t* ncand_dev, SelectParams* p) {
  if (!cand_dev || !ncand_dev) return fail(ctx, APEX_EINVAL, "null output");
  if (!ctx->has_cdf[layer]) return fail(ctx, APEX_ESTATE, "no confidence model set for this layer");
  if (!(tau == tau)) return fail(ctx, APEX_EINVAL, "tau is NaN");
  const int N = ctx->cfg.N, k = ctx->cfg.k;
  *p = SelectParams{};
  p->q = ctx->d_qp;
  p->pi = ctx->d_pi;
  p->w = ctx->d_w + (size_t)layer * N;
  p->theta = ctx->d_theta + (size_t)layer * (N - k + 1);
  p->cand_out = cand_dev;
  p->ncand_out = ncand_dev;
  p->ncand_keep = ctx->d_ncand;
  p->mbox_cand = mbox_i32(ctx, ctx->ml.off_cand);
  p->mbox_ncand = mbox_i32(ctx, ctx->ml.off_ncand);
  p->mbox_seq = &mhdr(ctx)->sel_seq;
  p->mbox_rec = const_cast<uint32_t*>(mbox_sel_rec(ctx));
  p->seq_value = ++ctx->sel_seq;
  if (B > 1) ctx->sel_done += (unsigned long long)B;
  p->done_counter = ctx->d_counters + 0;
  p->done_target = ctx->sel_done;
  p->stats = ctx->d_stats + layer;
  p->force = tau <= 0.f ? 1 : (tau >= 1.f ? 2 : 0);
  p->t_tau = p->force ? 0.f : (float)std::log((double)tau / (1.0 - (double)tau));
  p->N = N; p->k = k; p->C = ctx->cfg.C; p->B = B;
  return APEX_OK;
}

// S1-S3 in one launch (used by apex_decode_token): the leader warp of the prefetch-router kernel
// goes on with the budget selection of its token.
int predict_select_fused(apex_ctx* ctx, int layer, const float* h_dev, int B, float tau, int32_t* cand_dev,
                         int32_t* ncand_dev, cudaStream_t cs) {
  RouterParams p;
  int r = begin_predict(ctx, layer, h_dev, B, &p);
  if (r != APEX_OK) return r;
  if ((r = fill_select(ctx, layer, B, tau, cand_dev, ncand_dev, &p.sel)) != APEX_OK) return r;
  p.fuse_select = 1;
  CU_TRY(ctx, launch_router(p, cs));
  ctx->last_was_ffn = false;
  ctx->last_pred_layer = layer;
  ctx->last_stream = cs;
  ++ctx->launches;
  ctx->pred_stream = cs;
  ctx->step[layer].predicted = true;
  ctx->step[layer].selected = true;
  ctx->host_stats[layer].layer_steps += 1;
  return APEX_OK;
}

}  // namespace

extern "C" {

int apex_predict(apex_ctx* ctx, int layer, const float* h_dev, int B, void* stream) {
  CHECK_CTX(ctx);
  CHECK_LAYER(ctx, layer);
  RouterParams p;
  int r = begin_predict(ctx, layer, h_dev, B, &p);
  if (r != APEX_OK) return r;
  CU_TRY(ctx, launch_router(p, (cudaStream_t)stream));
  ctx->last_was_ffn = false;
  ctx->last_pred_layer = layer;
  ctx->last_stream = (cudaStream_t)stream;
  ++ctx->launches;
  ctx->pred_stream = (cudaStream_t)stream;
  ctx->step[layer].predicted = true;
  ctx->host_stats[layer].layer_steps += 1;
  return APEX_OK;
}

int apex_select_candidates(apex_ctx* ctx, int layer, int B, float tau, int32_t* cand_dev, int32_t* ncand_dev, void* stream) {
  CHECK_CTX(ctx);
  CHECK_LAYER(ctx, layer);
  auto& st = ctx->step[layer];
  if (!st.predicted || st.B != B) return fail(ctx, APEX_ESTATE, "apex_select_candidates needs apex_predict of the same layer-step and B");
  SelectParams p;
  int r = fill_select(ctx, layer, B, tau, cand_dev, ncand_dev, &p);
  if (r != APEX_OK) return r;
  CU_TRY(ctx, launch_select(p, (cudaStream_t)stream));
  ctx->last_was_ffn = false;
  ctx->last_pred_layer = layer;
  ctx->last_stream = (cudaStream_t)stream;
  ++ctx->launches;
  st.selected = true;
  return APEX_OK;
}

int apex_prefetch(apex_ctx* ctx, int layer, int B, void* copy_stream) {
  CHECK_CTX(ctx);
  CHECK_LAYER(ctx, layer);
  auto& st = ctx->step[layer];
  if (!st.selected || st.B != B) return fail(ctx, APEX_ESTATE, "apex_prefetch needs apex_select_candidates of the same layer-step and B");
  if (st.prefetched) return fail(ctx, APEX_ESTATE, "apex_prefetch called twice in one layer-step");
  for (int i = 0; i < ctx->n_copy_streams; ++i)
    ctx->cur_copy_streams[i] = copy_stream ? (cudaStream_t)copy_stream : ctx->copy_streams[i];
  const int C = ctx->cfg.C;
  const int32_t* ncand = mbox_i32(ctx, ctx->ml.off_ncand);
  const int32_t* cand = mbox_i32(ctx, ctx->ml.off_cand);
  std::vector<SlotCopy> copies;
  std::vector<SlotCopy> ordered;
  if (B == 1) {
    // one 16-byte record {mask lo, mask hi, ncand, seq}; the ranked list beside it is advisory
    volatile uint32_t* rec = mbox_sel_rec(ctx);
    if (!host_wait_seq(ctx, rec + 3, ctx->sel_seq)) return fail(ctx, APEX_ETIMEOUT, "apex_prefetch: candidate set did not arrive");
    const uint64_t mask = ((uint64_t)rec[1] << 32) | rec[0];
    const int n = (int)rec[2];
    int32_t list[APEX_MAX_EXPERTS];
    int m = 0;
    for (int e = 0; e < ctx->cfg.N; ++e)
      if ((mask >> e) & 1) list[m++] = e;
    if (m != n || n > C) return fail(ctx, APEX_ESTATE, "candidate record is inconsistent");
    int32_t nn = n;
    if (!ctx->tables[layer].plan_prefetch(list, &nn, 1, APEX_MAX_EXPERTS, &copies)) return fail(ctx, APEX_ESTATE, "no evictable slot");
    ordered = copies;
    // issue most likely first if the ranked list (written without a fence) is the same set
    int pos[APEX_MAX_EXPERTS];
    for (int e = 0; e < APEX_MAX_EXPERTS; ++e) pos[e] = -1;
    uint64_t seen = 0;
    bool valid = true;
    for (int j = 0; j < n && valid; ++j) {
      const int e = cand[j];
      if (e < 0 || e >= ctx->cfg.N || ((seen >> e) & 1) || !((mask >> e) & 1)) valid = false;
      else { seen |= 1ull << e; pos[e] = j; }
    }
    if (valid && copies.size() > 1)
      std::stable_sort(ordered.begin(), ordered.end(), [&](const SlotCopy& a, const SlotCopy& b) { return pos[a.expert] < pos[b.expert]; });
  } else {
    if (!host_wait_seq(ctx, &mhdr(ctx)->sel_seq, ctx->sel_seq))
      return fail(ctx, APEX_ETIMEOUT, "apex_prefetch: candidate lists did not arrive");
    if (!ctx->tables[layer].plan_prefetch(cand, ncand, B, C, &copies)) return fail(ctx, APEX_ESTATE, "no evictable slot");
    ordered = copies;
  }
  for (size_t i = 0; i < ordered.size(); ++i) {
    const auto& c = ordered[i];
    int r = issue_copy(ctx, layer, c.expert, c.slot, ctx->stream_of_slot(c.slot));
    if (r != APEX_OK) {
      // The plan has already installed every candidate in the table.  What was not copied must not stay there as
      // resident (the expert FFN would multiply by the previous occupant's bytes): those slots are left empty and
      // the call can be repeated.
      for (size_t j = i; j < ordered.size(); ++j) ctx->tables[layer].drop(ordered[j].expert);
      ctx->host_stats[layer].prefetch_copies += (int64_t)i;
      for (const auto& cc : copies)
        if (ctx->tables[layer].expert_slot()[cc.expert] >= 0) ctx->last_copies[layer].push_back(cc);
      return r;
    }
  }
  ctx->host_stats[layer].prefetch_copies += (int64_t)copies.size();
  ctx->last_copies[layer].insert(ctx->last_copies[layer].end(), copies.begin(), copies.end());
  st.prefetched = true;
  return APEX_OK;
}

int apex_attention_standin(apex_ctx* ctx, int layer, void* stream) {
  CHECK_CTX(ctx);
  CHECK_LAYER(ctx, layer);
  AttnParams p{};
  p.buf = reinterpret_cast<const uint4*>(ctx->d_attn + (size_t)(layer % ctx->attn_layers) * ctx->attn_bytes);
  p.n_vec = ctx->attn_bytes / 16;
  p.sink = ctx->d_attn_sink;
  // The attention block of a layer reads the layer's input, not the prefetch router's output: when the kernel
  // just before it on this stream is this layer-step's prefetch stage, the two may run side by side (Sec. IV-A:
  // prediction and prefetch are hidden under attention).  Anything else in front of it is waited for first.
  p.wait_first = (ctx->last_stream == (cudaStream_t)stream && ctx->last_pred_layer == layer) ? 0 : 1;
  CU_TRY(ctx, launch_attention(p, ctx->n_sm, (cudaStream_t)stream));
  ctx->last_was_ffn = false;
  ctx->last_pred_layer = -1;
  ctx->last_stream = (cudaStream_t)stream;
  ++ctx->launches;
  return APEX_OK;
}

int apex_route_topk(apex_ctx* ctx, int layer, const float* hpost_dev, int B, int32_t* idx_dev, float* alpha_dev, void* stream) {
  CHECK_CTX(ctx);
  CHECK_LAYER(ctx, layer);
  if (!hpost_dev || !idx_dev || !alpha_dev || B < 1 || B > ctx->cfg.max_batch) return fail(ctx, APEX_EINVAL, "apex_route_topk: bad argument");
  auto& st = ctx->step[layer];
  if (st.pending) return fail(ctx, APEX_ESTATE, "the previous expert FFN of this layer has not been completed");
  if (st.predicted && st.B != B) return fail(ctx, APEX_ESTATE, "B differs from apex_predict of this layer-step");
  if (!st.predicted) {  // gate used on its own (no prefetch stage): still one layer-step
    ctx->tables[layer].begin_step();
    ctx->last_copies[layer].clear();
    st = apex_ctx::StepState{};
    st.B = B;
    ctx->host_stats[layer].layer_steps += 1;
  }
  const size_t N = ctx->cfg.N, d = ctx->cfg.d;
  RouterParams p{};
  p.W = ctx->d_Wr + (size_t)layer * N * d;
  p.bias = ctx->has_br[layer] ? ctx->d_br + (size_t)layer * N : nullptr;
  p.x = hpost_dev;
  p.z_out = ctx->d_zr + (size_t)layer * ctx->cfg.max_batch * N;
  p.q_out = alpha_dev;
  p.pi_out = nullptr;
  p.topk_out = idx_dev;
  p.N = (int)N; p.d = (int)d; p.B = B; p.k = ctx->cfg.k; p.C = ctx->cfg.C;
  p.pi_pred = st.selected ? ctx->d_pi : nullptr;
  p.ncand_pred = st.selected ? ctx->d_ncand : nullptr;
  p.stats = ctx->d_stats + layer;
  CU_TRY(ctx, launch_router(p, (cudaStream_t)stream));
  ctx->last_was_ffn = false;
  ctx->last_pred_layer = -1;
  ctx->last_stream = (cudaStream_t)stream;
  ++ctx->launches;
  st.routed = true;
  st.route_stream = (cudaStream_t)stream;
  st.idx_dev = idx_dev;
  st.alpha_dev = alpha_dev;
  return APEX_OK;
}

}  // extern "C"

namespace {

constexpr long long kSpecDelayAfterGateNs = 1000;

// Every launch of the streaming kernel gets its own row-ticket counter out of a ring of 64; the
// launch also clears the counter that will be used 32 launches later.
cudaError_t launch_stream(apex_ctx* ctx, FfnParams p, cudaStream_t cs) {
  const uint32_t id = ctx->ffn_launch_id++;
  // y may be zeroed before the dependency wait when the kernel in front of this one on the stream does not touch it:
  // any kernel of this library that is not an expert-FFN launch, or an FFN launch that wrote another buffer.
  const uintptr_t y_lo = (uintptr_t)p.y, y_hi = y_lo + (size_t)p.B * p.d * sizeof(float);
  const bool prev_ffn_disjoint = ctx->last_was_ffn && (y_hi <= ctx->last_ffn_y_lo || ctx->last_ffn_y_hi <= y_lo);
  p.zero_early = (ctx->last_stream == cs && (!ctx->last_was_ffn || prev_ffn_disjoint)) ? 1 : 0;
  ctx->last_ffn_y_lo = y_lo;
  ctx->last_ffn_y_hi = y_hi;
  // With APEX_FLAG_SPECULATE: after the gate kernel the speculative first fill is held back until the gate has fetched
  // its input; between two FFN launches there is nothing to spare.
  p.spec_delay_ns = ctx->last_was_ffn ? 0 : kSpecDelayAfterGateNs;
  ctx->last_was_ffn = true;
  ctx->last_pred_layer = -1;
  ctx->last_stream = cs;
  p.ticket = ctx->d_tickets + (id & 63u);
  p.ticket_reset = ctx->d_tickets + ((id + 32u) & 63u);
  // (one CTA per SM also right behind the gate kernel: leaving the gate's SMs out of the grid was measured and is
  // slower, 998 against 970-984 tokens/s all resident)
  const int n_ctas = ffn_grid_ctas(ctx->n_sm);
  if (!p.accumulate) {  // every CTA zeroes a slice of y and counts itself in
    ctx->zero_done += (unsigned long long)n_ctas;
    p.zero_target = ctx->zero_done;
  }
  return launch_ffn(p, n_ctas, cs);
}


// B > 1: plan kernel, then either the tensor-core grouped GEMM or the streaming kernel per pair.
int launch_batched(apex_ctx* ctx, int layer, const FfnParams& p, cudaStream_t cs) {
  CU_TRY(ctx, launch_ffn_plan(p, cs));
  ctx->last_was_ffn = false;
  ctx->last_pred_layer = -1;
  ctx->last_stream = cs;
  ++ctx->launches;
  if (ctx->tc_ok && p.B >= kTcMinBatch) {
    TcParams t{};
    t.f = p;
    t.grp = ctx->d_grp;
    t.xg = ctx->d_xg;
    t.act = ctx->d_act;
    t.act_stride = ctx->act_stride;
    t.act_plane = ctx->act_plane;
    t.layer_slot0 = layer * ctx->cfg.C;
    CU_TRY(ctx, launch_ffn_tc(t, ctx->tc_shared_maps[layer], ctx->n_sm, cs));
    ctx->last_was_ffn = true;
    ctx->last_ffn_y_lo = (uintptr_t)p.y;
    ctx->last_ffn_y_hi = (uintptr_t)p.y + (size_t)p.B * p.d * sizeof(float);
    ctx->last_pred_layer = -1;
    ctx->launches += 3;
  } else {
    CU_TRY(ctx, launch_stream(ctx, p, cs));
    ++ctx->launches;
  }
  return APEX_OK;
}

// First half of apex_moe_ffn: launches the expert FFN of a layer-step.  B == 1 in exact mode is one
// launch that also waits, inside the kernel, for experts the host has to fetch on demand; otherwise
// the launch covers the experts that are resident and ffn_finalize adds further launches.
int ffn_launch(apex_ctx* ctx, int layer, int mode, const float* hpost_dev, int B, float* y_dev, int32_t* exec_idx_dev,
               float* exec_gate_dev, cudaStream_t cs) {
  auto& st = ctx->step[layer];
  if (!st.routed || st.B != B) return fail(ctx, APEX_ESTATE, "apex_moe_ffn needs apex_route_topk of the same layer-step and B");
  if (!hpost_dev || !y_dev) return fail(ctx, APEX_EINVAL, "null h' or y");
  if (mode != APEX_MODE_EXACT && mode != APEX_MODE_STALL_FREE) return fail(ctx, APEX_EINVAL, "unknown mode");
  if (ctx->cfg.I_shared > 0 && !ctx->shared_dev[layer]) return fail(ctx, APEX_ESTATE, "shared expert not set for this layer");
  const int N = ctx->cfg.N, k = ctx->cfg.k, C = ctx->cfg.C;
  FfnParams& p = ctx->ffn_params[layer];
  p = FfnParams{};
  p.hpost = hpost_dev;
  p.y = y_dev;
  p.idx = st.idx_dev;
  p.alpha = st.alpha_dev;
  p.z_r = ctx->d_zr + (size_t)layer * ctx->cfg.max_batch * N;
  p.exec_idx = exec_idx_dev;
  p.exec_gate = exec_gate_dev;
  p.cache = ctx->d_cache + (size_t)layer * C * ctx->expert_bytes;
  p.shared_w = ctx->shared_dev[layer];
  p.shared_gate = ctx->shared_gate_on[layer] ? ctx->shared_gate_dev[layer] : nullptr;
  p.slot_ready = ctx->d_slot_ready + (size_t)layer * C;
  p.plan_exec_idx = ctx->d_plan_exec_idx;
  p.plan_exec_gate = ctx->d_plan_exec_gate;
  p.pair_tok = ctx->d_pair_tok;
  p.pair_gate = ctx->d_pair_gate;
  p.pair_expert = ctx->d_pair_expert;
  p.n_pairs = ctx->d_n_pairs;
  p.grp = ctx->d_grp;
  p.mbox_exec = mbox_exec(ctx, layer);
  p.mbox_kr = mbox_kr(ctx, layer);
  p.mbox_rec = const_cast<uint32_t*>(mbox_exec_rec(ctx, layer));
  p.mbox_seq = mbox_exec_seq(ctx, layer);
  p.mbox_status = &mhdr(ctx)->status;
  p.seq_value = ++ctx->exec_seq[layer];
  p.stats = ctx->d_stats + layer;
  p.zero_counter = ctx->d_counters + 1;
  p.snap = make_snapshot(ctx, layer);
  p.slot_stride = ctx->expert_bytes;
  p.wait_limit_ns = ctx->cfg.wait_limit_ns;
  p.d = ctx->cfg.d; p.N = N; p.k = k; p.I = ctx->cfg.I; p.I_shared = ctx->cfg.I_shared; p.B = B; p.C = C;
  p.mode = mode; p.norm_topk = ctx->cfg.norm_topk; p.accumulate = 0;
  p.run_shared = ctx->cfg.I_shared > 0 ? 1 : 0;
  p.post_exec = 1;
  p.fmt = ctx->fmt;
  p.demand = ctx->d_demand + (size_t)layer * N;
  ctx->launch_tag = ctx->launch_tag % 0xfffffeu + 1u;
  p.demand_tag = ctx->launch_tag;
  p.demand_in_kernel = (mode == APEX_MODE_EXACT && B == 1 && !ctx->host_waves) ? 1 : 0;
  p.run_mask = p.demand_in_kernel ? ~0ull : p.snap.resident_mask;
  // Speculative first fill (opt-in): the kernel may start streaming the experts the prefetch router ranked
  // first before the gate's decision is visible.  Allowed when that ranking is certainly complete by
  // then: predicted in this step, its candidate record already seen by the host (apex_prefetch), and
  // the gate kernel (which waits for everything before it) between the two on this same stream.
  p.spec = (B == 1 && st.predicted && st.prefetched && ctx->pred_stream == cs && st.route_stream == cs &&
            (ctx->cfg.flags & APEX_FLAG_SPECULATE))
               ? ctx->d_spec + (size_t)layer * APEX_MAX_TOPK
               : nullptr;
  if (B > 1) {
    int r = launch_batched(ctx, layer, p, cs);
    if (r != APEX_OK) return r;
  } else {
    CU_TRY(ctx, launch_stream(ctx, p, cs));
    ++ctx->launches;
  }
  st.pending = true;
  st.pend_mode = mode;
  st.pend_tag = p.demand_tag;
  st.pend_stream = cs;
  return APEX_OK;
}

// Second half: host work that needs the gate's decision (LRU stamps, demand copies, further waves).
int ffn_finalize(apex_ctx* ctx, int layer) {
  auto& st = ctx->step[layer];
  if (!st.pending) return APEX_OK;
  st.pending = false;
  const int B = st.B, N = ctx->cfg.N, k = ctx->cfg.k;
  cudaStream_t cs = st.pend_stream;
  auto& tab = ctx->tables[layer];
  const FfnParams& p = ctx->ffn_params[layer];
  // the FFN's plan step posts the routed and the execution sets of this layer-step
  std::vector<int32_t> kr_one, ex_one;  // B = 1: the sets arrive as masks, each with its sequence number in one 16-byte record
  const int32_t* K_r = mbox_kr(ctx, layer);
  const int32_t* ex_list = mbox_exec(ctx, layer);
  if (B == 1) {
    volatile uint32_t* rec = mbox_exec_rec(ctx, layer);
    if (!host_wait_seq(ctx, rec + 2, ctx->exec_seq[layer]) || !host_wait_seq(ctx, rec + 6, ctx->exec_seq[layer]))
      return fail(ctx, APEX_ETIMEOUT, "apex_moe_ffn: K_r did not arrive");
    const uint64_t kr_mask = ((uint64_t)rec[1] << 32) | rec[0], ex_mask = ((uint64_t)rec[5] << 32) | rec[4];
    for (int e = 0; e < N; ++e) {
      if ((kr_mask >> e) & 1) kr_one.push_back(e);
      if ((ex_mask >> e) & 1) ex_one.push_back(e);
    }
    kr_one.resize(k, -1);
    ex_one.resize(k, -1);
    K_r = kr_one.data();
    ex_list = ex_one.data();
  } else if (!host_wait_seq(ctx, mbox_exec_seq(ctx, layer), ctx->exec_seq[layer])) {
    return fail(ctx, APEX_ETIMEOUT, "apex_moe_ffn: K_r did not arrive");
  }
  if (st.pend_mode == APEX_MODE_EXACT) {
    std::vector<SlotCopy> copies;
    uint64_t need = 0;
    const std::vector<int32_t> slot_expert_before = tab.slot_expert();
    if (!tab.plan_demand(K_r, B, k, &copies, &need)) return fail(ctx, APEX_ESTATE, "no evictable slot");
    if (p.demand_in_kernel) {
      // the running kernel waits for these experts: copy, then publish (tag, slot)
      for (size_t i = 0; i < copies.size(); ++i) {
        const auto& c = copies[i];
        const int prev = slot_expert_before[c.slot];
        int r = APEX_OK;
        if (c.wave != 1 || (prev >= 0 && ((need >> prev) & 1))) r = fail(ctx, APEX_ESTATE, "demand plan would evict an expert in use");
        if (r == APEX_OK) r = issue_copy(ctx, layer, c.expert, c.slot, ctx->stream_of_slot(c.slot));
        if (r == APEX_OK)
          r = stream_write32(ctx, ctx->stream_of_slot(c.slot), ctx->d_demand + (size_t)layer * ctx->cfg.N + c.expert,
                             (st.pend_tag << 8) | (uint32_t)c.slot);
        if (r != APEX_OK) {
          // experts whose copy was not issued (or not published) leave the table again; the running kernel's wait
          // for them runs out and y stays incomplete: the caller sees the error and may repeat the expert FFN
          for (size_t j = i; j < copies.size(); ++j) tab.drop(copies[j].expert);
          return r;
        }
      }
    } else {
      int n_waves = 0;
      for (const auto& c : copies) n_waves = c.wave > n_waves ? c.wave : n_waves;
      // The plan above covers every wave; replay it wave by wave so that each launch gets the table
      // as it stands when that wave runs.
      std::vector<int32_t> cur_slot_expert = slot_expert_before;
      SlotSnapshot cur = p.snap;
      for (int w = 1; w <= n_waves; ++w) {
        // a victim that an earlier launch of this step may still be reading: order the copy after it
        bool hazard = false;
        uint64_t chunk = 0;
        for (const auto& c : copies)
          if (c.wave == w) {
            chunk |= (1ull << c.expert);
            const int prev = cur_slot_expert[c.slot];
            if (prev >= 0 && ((need >> prev) & 1)) hazard = true;
          }
        if (hazard) {
          CU_TRY(ctx, cudaEventRecord(ctx->ev_wave, cs));
          for (int i = 0; i < ctx->n_copy_streams; ++i)
            if (i == 0 || ctx->cur_copy_streams[i] != ctx->cur_copy_streams[0])
              CU_TRY(ctx, cudaStreamWaitEvent(ctx->cur_copy_streams[i], ctx->ev_wave, 0));
        }
        for (size_t ci = 0; ci < copies.size(); ++ci) {
          const auto& c = copies[ci];
          if (c.wave == w) {
            int r = issue_copy(ctx, layer, c.expert, c.slot, ctx->stream_of_slot(c.slot));
            if (r != APEX_OK) {
              // (the plan lists the copies wave by wave) nothing from here on was copied: un-install it.  An expert of
              // an earlier wave whose slot a later wave was going to reuse is no longer in the table either way.
              for (size_t j = ci; j < copies.size(); ++j) tab.drop(copies[j].expert);
              return r;
            }
            const int prev = cur_slot_expert[c.slot];
            if (prev >= 0) {
              cur.expert_slot[prev] = -1;
              cur.resident_mask &= ~(1ull << prev);
            }
            cur_slot_expert[c.slot] = c.expert;
            cur.expert_slot[c.expert] = (int8_t)c.slot;
            cur.need_gen[c.expert] = ctx->slot_gen[layer][c.slot];
            cur.resident_mask |= (1ull << c.expert);
          }
        }
        FfnParams q = p;
        q.snap = cur;
        q.run_mask = chunk;
        q.accumulate = 1;
        q.run_shared = 0;
        q.post_exec = 0;
        if (B > 1) {
          int r = launch_batched(ctx, layer, q, cs);
          if (r != APEX_OK) return r;
        } else {
          CU_TRY(ctx, launch_stream(ctx, q, cs));
          ++ctx->launches;
        }
        ctx->host_stats[layer].extra_waves += 1;
      }
    }
    ctx->host_stats[layer].demand_copies += (int64_t)copies.size();
    ctx->last_copies[layer].insert(ctx->last_copies[layer].end(), copies.begin(), copies.end());
  } else {
    for (int i = 0; i < B * k; ++i) tab.touch(ex_list[i]);
  }
  st.routed = false;  // the layer-step is complete
  st.predicted = false;
  st.selected = false;
  return check_device_status(ctx);
}

}  // namespace

extern "C" {

int apex_moe_ffn(apex_ctx* ctx, int layer, int mode, const float* hpost_dev, int B, float* y_dev, int32_t* exec_idx_dev,
                 float* exec_gate_dev, void* stream) {
  CHECK_CTX(ctx);
  CHECK_LAYER(ctx, layer);
  int r = ffn_launch(ctx, layer, mode, hpost_dev, B, y_dev, exec_idx_dev, exec_gate_dev, (cudaStream_t)stream);
  if (r != APEX_OK) return r;
  return ffn_finalize(ctx, layer);
}

int apex_moe_ffn_begin(apex_ctx* ctx, int layer, int mode, const float* hpost_dev, int B, float* y_dev, int32_t* exec_idx_dev,
                       float* exec_gate_dev, void* stream) {
  CHECK_CTX(ctx);
  CHECK_LAYER(ctx, layer);
  return ffn_launch(ctx, layer, mode, hpost_dev, B, y_dev, exec_idx_dev, exec_gate_dev, (cudaStream_t)stream);
}

int apex_moe_ffn_end(apex_ctx* ctx, int layer) {
  CHECK_CTX(ctx);
  CHECK_LAYER(ctx, layer);
  if (!ctx->step[layer].pending) return fail(ctx, APEX_ESTATE, "apex_moe_ffn_end without apex_moe_ffn_begin");
  return ffn_finalize(ctx, layer);
}

// Pipelined over layers: the host work that needs the gate's decision of layer l-1 (LRU stamps,
// demand copies) is done after the kernels of layer l have been queued, so that on the hit path
// the GPU never waits for the host.
int apex_decode_token(apex_ctx* ctx, const float* h_dev, const float* hpost_dev, int B, float tau, int mode, float* y_dev,
                      void* stream) {
  CHECK_CTX(ctx);
  if (!h_dev || !hpost_dev || !y_dev || B < 1 || B > ctx->cfg.max_batch) return fail(ctx, APEX_EINVAL, "apex_decode_token: bad argument");
  if (decode_persistent_usable(ctx, B))  // one persistent kernel over all layers
    return decode_token_persistent(ctx, h_dev, hpost_dev, tau, mode, y_dev, (cudaStream_t)stream);
  const size_t step = (size_t)B * ctx->cfg.d;
  const size_t MB = ctx->cfg.max_batch, k = ctx->cfg.k, N = ctx->cfg.N;
  const bool standin = !(ctx->cfg.flags & APEX_FLAG_SKIP_STANDIN);
  int r;
  for (int l = 0; l < ctx->cfg.L; ++l) {
    int32_t* idx = ctx->d_idx + (size_t)l * MB * k;
    float* alpha = ctx->d_alpha + (size_t)l * MB * N;
    const bool prefetching = !(tau < 0.f);  // tau < 0: the conventional scheme, expert loading on the critical path
    if (prefetching &&
        (r = predict_select_fused(ctx, l, h_dev + l * step, B, tau, ctx->d_cand, ctx->d_cand_ncand, (cudaStream_t)stream)) != APEX_OK)
      return r;
    if (standin && (r = apex_attention_standin(ctx, l, stream)) != APEX_OK) return r;
    if ((r = apex_route_topk(ctx, l, hpost_dev + l * step, B, idx, alpha, stream)) != APEX_OK) return r;
    if (l > 0 && (r = ffn_finalize(ctx, l - 1)) != APEX_OK) return r;
    if (prefetching && (r = apex_prefetch(ctx, l, B, nullptr)) != APEX_OK) return r;
    if ((r = ffn_launch(ctx, l, mode, hpost_dev + l * step, B, y_dev + l * step, ctx->d_exec_idx, ctx->d_exec_gate,
                        (cudaStream_t)stream)) != APEX_OK)
      return r;
  }
  return ffn_finalize(ctx, ctx->cfg.L - 1);
}

int apex_decode_token_host(apex_ctx* ctx, const float* h_host, const float* hpost_host, int B, float tau, int mode,
                           float* y_host, void* stream) {
  CHECK_CTX(ctx);
  if (!h_host || !hpost_host || !y_host || B < 1 || B > ctx->cfg.max_batch) return fail(ctx, APEX_EINVAL, "apex_decode_token_host: bad argument");
  const size_t n = (size_t)ctx->cfg.L * ctx->cfg.max_batch * ctx->cfg.d;
  if (!ctx->d_h_stage) {
    CU_TRY(ctx, dev_alloc(&ctx->d_h_stage, n));
    CU_TRY(ctx, dev_alloc(&ctx->d_hp_stage, n));
    CU_TRY(ctx, dev_alloc(&ctx->d_y_stage, n));
  }
  cudaStream_t cs = (cudaStream_t)stream;
  const size_t bytes = (size_t)ctx->cfg.L * B * ctx->cfg.d * sizeof(float);
  CU_TRY(ctx, cudaMemcpyAsync(ctx->d_h_stage, h_host, bytes, cudaMemcpyHostToDevice, cs));
  CU_TRY(ctx, cudaMemcpyAsync(ctx->d_hp_stage, hpost_host, bytes, cudaMemcpyHostToDevice, cs));
  int r = apex_decode_token(ctx, ctx->d_h_stage, ctx->d_hp_stage, B, tau, mode, ctx->d_y_stage, stream);
  if (r != APEX_OK) return r;
  CU_TRY(ctx, cudaMemcpyAsync(y_host, ctx->d_y_stage, bytes, cudaMemcpyDeviceToHost, cs));
  CU_TRY(ctx, cudaStreamSynchronize(cs));
  return check_device_status(ctx);
}

// ---------------------------------------------------------------------------------------------

}  // extern "C"

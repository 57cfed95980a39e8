// Host half of the persistent decode path (B = 1): one cooperative launch per token, then the host follows the kernel
// layer by layer through the records it posts -- plans and issues the prefetch copies (S5), publishes a layer's new slot
// table when it changed, issues demand copies for missing routed experts (S8) and keeps the recency stamps.  The
// sequence of table operations per layer-step is that of apex_predict / apex_prefetch / apex_moe_ffn, so tables, copy
// lists and counters come out the same.  No arithmetic of the path runs here.
#include "apex_host.hpp"

using namespace apex;

namespace apex {

// Allocations of the persistent path; called once from apex_create.  On any failure the path is left unavailable
// (dec_clusters = 0) and apex_decode_token keeps to the per-layer kernel sequence.
int decode_setup(apex_ctx* ctx) {
  ctx->dec_clusters = 0;
  if (ctx->cfg.N > kDecCluster * kDecWarps) return APEX_OK;
  if (ctx->cfg.flags & APEX_FLAG_LAYER_LAUNCHES) return APEX_OK;
  const int n = decode_max_clusters(ctx->cfg.d, ctx->fmt);
  if (n < 1) return APEX_OK;
  const size_t L = ctx->cfg.L;
  CU_TRY(ctx, dev_alloc(&ctx->d_dec_tab, L));
  CU_TRY(ctx, cudaHostAlloc(reinterpret_cast<void**>(&ctx->dec_tab_stage), 2 * L * sizeof(SlotSnapshot), cudaHostAllocPortable));
  CU_TRY(ctx, cudaHostAlloc(reinterpret_cast<void**>(&ctx->dec_snap), L * sizeof(DecodeHostSnap), cudaHostAllocMapped | cudaHostAllocPortable));
  CU_TRY(ctx, cudaHostAlloc(reinterpret_cast<void**>(&ctx->dec_mbox), L * sizeof(DecodeMbox), cudaHostAllocMapped | cudaHostAllocPortable));
  memset(ctx->dec_snap, 0, L * sizeof(DecodeHostSnap));
  memset(ctx->dec_mbox, 0, L * sizeof(DecodeMbox));
  CU_TRY(ctx, dev_alloc(&ctx->d_dec_bar, 2 * L));
  CU_TRY(ctx, cudaMemset(ctx->d_dec_bar, 0, 2 * L * sizeof(unsigned long long)));
  CU_TRY(ctx, dev_alloc(&ctx->d_dec_snap, L));
  CU_TRY(ctx, cudaMemset(ctx->d_dec_snap, 0, L * sizeof(DecodeHostSnap)));
  CU_TRY(ctx, dev_alloc(&ctx->d_dec_opt, L));
  CU_TRY(ctx, cudaMemset(ctx->d_dec_opt, 0, L));
  CU_TRY(ctx, cudaHostAlloc(reinterpret_cast<void**>(&ctx->dec_opt_stage), 2 * L, cudaHostAllocPortable));
  ctx->dec_opt_host.assign(L, 0);
  ctx->dec_opt_last.assign(L, 0);
  CU_TRY(ctx, dev_alloc(&ctx->d_dec_cand, 2 * L));
  CU_TRY(ctx, cudaMemset(ctx->d_dec_cand, 0, 2 * L * sizeof(unsigned long long)));
  CU_TRY(ctx, dev_alloc(&ctx->d_dec_abort, 4));
  CU_TRY(ctx, cudaMemset(ctx->d_dec_abort, 0, 4 * sizeof(unsigned int)));
  CU_TRY(ctx, dev_alloc(&ctx->d_shared_ptrs, L));
  CU_TRY(ctx, cudaMemset(ctx->d_shared_ptrs, 0, L * sizeof(void*)));
  CU_TRY(ctx, dev_alloc(&ctx->d_shared_gate_ptrs, L));
  CU_TRY(ctx, cudaMemset(ctx->d_shared_gate_ptrs, 0, L * sizeof(void*)));
  ctx->dec_tab_last.assign(L, SlotSnapshot{});
  ctx->dec_tab_valid = false;
  ctx->dec_clusters = n;
  return APEX_OK;
}

void decode_teardown(apex_ctx* ctx) {
  if (ctx->d_dec_tab) cudaFree(ctx->d_dec_tab);
  if (ctx->dec_tab_stage) cudaFreeHost(ctx->dec_tab_stage);
  if (ctx->dec_snap) cudaFreeHost(ctx->dec_snap);
  if (ctx->dec_mbox) cudaFreeHost(ctx->dec_mbox);
  if (ctx->d_dec_bar) cudaFree(ctx->d_dec_bar);
  if (ctx->d_dec_abort) cudaFree(ctx->d_dec_abort);
  if (ctx->d_dec_cand) cudaFree(ctx->d_dec_cand);
  if (ctx->d_dec_opt) cudaFree(ctx->d_dec_opt);
  if (ctx->d_dec_snap) cudaFree(ctx->d_dec_snap);
  if (ctx->dec_opt_stage) cudaFreeHost(ctx->dec_opt_stage);
  if (ctx->d_shared_ptrs) cudaFree(ctx->d_shared_ptrs);
  if (ctx->d_shared_gate_ptrs) cudaFree(ctx->d_shared_gate_ptrs);
}

bool decode_persistent_usable(const apex_ctx* ctx, int B) {
  return B == 1 && ctx->dec_clusters > 0 && !ctx->host_waves;
}

namespace {

// Tells the running kernel to stop waiting (the host cannot deliver what it waits for).
void raise_device_abort(apex_ctx* ctx) {
  stream_write32(ctx, ctx->cur_copy_streams[0], ctx->d_dec_abort, 1u);
  ctx->dec_dirty = true;
}

// The token cannot be completed.  If the kernel itself gave up first (a wait of its own ran out), that is the error to
// report, with everything that goes with it (withheld test flag released, later tokens on the per-layer path).
int fail_token(apex_ctx* ctx, int code, const char* what) {
  raise_device_abort(ctx);
  if (mhdr(ctx)->status != 0) return check_device_status(ctx);
  return fail(ctx, code, what);
}

}  // namespace

int decode_token_persistent(apex_ctx* ctx, const float* h_dev, const float* hpost_dev, float tau, int mode, float* y_dev,
                            cudaStream_t cs) {
  const int L = ctx->cfg.L, N = ctx->cfg.N, k = ctx->cfg.k, C = ctx->cfg.C, d = ctx->cfg.d;
  if (mode != APEX_MODE_EXACT && mode != APEX_MODE_STALL_FREE) return fail(ctx, APEX_EINVAL, "unknown mode");
  if (!(tau == tau)) return fail(ctx, APEX_EINVAL, "tau is NaN");
  const bool prefetching = !(tau < 0.f);
  for (int l = 0; l < L; ++l) {
    if (ctx->step[l].pending) return fail(ctx, APEX_ESTATE, "the previous expert FFN of a layer has not been completed");
    if (prefetching && !ctx->has_cdf[l]) return fail(ctx, APEX_ESTATE, "no confidence model set for a layer");
    if (ctx->cfg.I_shared > 0 && !ctx->shared_dev[l]) return fail(ctx, APEX_ESTATE, "shared expert not set for a layer");
  }
  for (int i = 0; i < ctx->n_copy_streams; ++i) ctx->cur_copy_streams[i] = ctx->copy_streams[i];

  // A launch that gave up leaves counters short and the abort word set: start over.
  if (ctx->dec_dirty) {
    CU_TRY(ctx, cudaDeviceSynchronize());
    CU_TRY(ctx, cudaMemset(ctx->d_dec_bar, 0, 2 * (size_t)L * sizeof(unsigned long long)));
    CU_TRY(ctx, cudaMemset(ctx->d_dec_abort, 0, 4 * sizeof(unsigned int)));
    ctx->dec_epoch = 0;
    ctx->dec_dirty = false;
  }
  // Slot tables as they stand now; uploaded when any of them differs from what the device holds.
  {
    SlotSnapshot* stage = ctx->dec_tab_stage + (size_t)ctx->dec_stage_sel * L;
    bool changed = !ctx->dec_tab_valid;
    for (int l = 0; l < L; ++l) {
      SlotSnapshot s{};
      s = make_snapshot(ctx, l);
      if (changed || memcmp(&s, &ctx->dec_tab_last[l], sizeof s) != 0) {
        changed = true;
        ctx->dec_tab_last[l] = s;
      }
      stage[l] = s;
    }
    // ... and where the host expects a layer's table to stay as it is in this step (its previous step copied nothing)
    uint8_t* ostage = ctx->dec_opt_stage + (size_t)ctx->dec_stage_sel * L;
    const bool opt_changed = ctx->dec_opt_host != ctx->dec_opt_last;
    if (changed) {
      CU_TRY(ctx, cudaMemcpyAsync(ctx->d_dec_tab, stage, (size_t)L * sizeof(SlotSnapshot), cudaMemcpyHostToDevice, cs));
      ctx->dec_tab_valid = true;
    }
    if (opt_changed) {
      memcpy(ostage, ctx->dec_opt_host.data(), L);
      CU_TRY(ctx, cudaMemcpyAsync(ctx->d_dec_opt, ostage, L, cudaMemcpyHostToDevice, cs));
      ctx->dec_opt_last = ctx->dec_opt_host;
    }
    if (changed || opt_changed) ctx->dec_stage_sel ^= 1;
  }
  CU_TRY(ctx, cudaMemsetAsync(y_dev, 0, (size_t)L * d * sizeof(float), cs));

  const uint32_t seq = ++ctx->dec_seq;
  ctx->launch_tag = ctx->launch_tag % 0xfffffeu + 1u;
  const uint32_t tag = ctx->launch_tag;
  const int G = ctx->dec_clusters * kDecCluster;
  ++ctx->dec_epoch;

  DecodeParams p{};
  p.h = h_dev;
  p.hpost = hpost_dev;
  p.y = y_dev;
  p.W_p = ctx->d_Wp; p.b_p = ctx->d_bp; p.W_r = ctx->d_Wr; p.b_r = ctx->d_br;
  p.w = ctx->d_w; p.theta = ctx->d_theta;
  p.cache = ctx->d_cache;
  p.shared_w = ctx->cfg.I_shared > 0 ? ctx->d_shared_ptrs : nullptr;
  p.shared_gate = ctx->cfg.I_shared > 0 ? ctx->d_shared_gate_ptrs : nullptr;
  p.slot_ready = ctx->d_slot_ready;
  p.demand = ctx->d_demand;
  p.tab = ctx->d_dec_tab;
  p.opt = ctx->d_dec_opt;
  p.snap = ctx->dec_snap;
  p.snap_dev = ctx->d_dec_snap;
  p.mbox = ctx->dec_mbox;
  p.mbox_status = &mhdr(ctx)->status;
  p.stats = ctx->d_stats;
  p.zp_out = ctx->d_zp; p.qp_out = ctx->d_qp; p.pi_out = ctx->d_pi;
  p.zr_out = ctx->d_zr; p.alpha_out = ctx->d_alpha; p.idx_out = ctx->d_idx;
  p.zr_stride = (size_t)ctx->cfg.max_batch * N;
  p.idx_stride = (size_t)ctx->cfg.max_batch * k;
  p.ncand_keep = ctx->d_ncand; p.cand_dev = ctx->d_cand; p.ncand_dev = ctx->d_cand_ncand;
  p.cand_rec = ctx->d_dec_cand;
  p.bar = ctx->d_dec_bar;
  p.bar_target = ctx->dec_epoch * (unsigned long long)G;
  p.abort_flag = ctx->d_dec_abort;
  p.attn = ctx->d_attn; p.attn_bytes = ctx->attn_bytes; p.attn_layers = (int)ctx->attn_layers;
  p.run_attn = (ctx->cfg.flags & APEX_FLAG_SKIP_STANDIN) ? 0 : 1;
  p.fmt = ctx->fmt;
  // (quantised rows are shorter than a vector of y: the cross-warp reduction then uses the start of the ring, so
  // nothing is requested ahead of it)
  p.standin_ahead = ((ctx->cfg.flags & APEX_FLAG_STANDIN_AHEAD) && ctx->fmt == 0) ? 1 : 0;
  p.seq = seq;
  p.demand_tag = tag;
  p.force = !prefetching ? 0 : (tau <= 0.f ? 1 : (tau >= 1.f ? 2 : 0));
  p.t_tau = (prefetching && !p.force) ? (float)std::log((double)tau / (1.0 - (double)tau)) : 0.f;
  p.prefetching = prefetching ? 1 : 0;
  p.slot_stride = ctx->expert_bytes;
  p.wait_limit_ns = ctx->cfg.wait_limit_ns;
  p.d = d; p.N = N; p.k = k; p.I = ctx->cfg.I; p.I_shared = ctx->cfg.I_shared; p.C = C; p.L = L;
  p.mode = mode; p.norm_topk = ctx->cfg.norm_topk; p.cache_reuse = ctx->cfg.cache_reuse; p.n_sm = ctx->n_sm;
  CU_TRY(ctx, launch_decode(p, ctx->dec_clusters, cs));
  ++ctx->launches;
  ctx->last_was_ffn = false;
  ctx->last_pred_layer = -1;
  ctx->last_stream = cs;
  ctx->pred_stream = cs;

  // ---- follow the kernel layer by layer
  for (int l = 0; l < L; ++l) {
    auto& tab = ctx->tables[l];
    DecodeMbox* mb = ctx->dec_mbox + l;
    tab.begin_step();
    ctx->last_copies[l].clear();
    ctx->step[l] = apex_ctx::StepState{};
    ctx->host_stats[l].layer_steps += 1;
    if (prefetching) {
      volatile uint32_t* rec = mb->sel_rec;
      if (!host_wait_seq(ctx, rec + 3, seq)) return fail_token(ctx, APEX_ETIMEOUT, "apex_decode_token: a candidate set did not arrive");
      const uint64_t mask = ((uint64_t)rec[1] << 32) | rec[0];
      const int n = (int)rec[2];
      int32_t list[APEX_MAX_EXPERTS];
      int m = 0;
      for (int e = 0; e < N; ++e)
        if ((mask >> e) & 1) list[m++] = e;
      if (m != n || n > C) return fail_token(ctx, APEX_ESTATE, "candidate record is inconsistent");
      std::vector<SlotCopy> copies;
      int32_t nn = n;
      if (!tab.plan_prefetch(list, &nn, 1, APEX_MAX_EXPERTS, &copies)) return fail_token(ctx, APEX_ESTATE, "no evictable slot");
      std::vector<SlotCopy> ordered = copies;
      if (copies.size() > 1) {  // most likely first, if the advisory ranked list names the same set
        int pos[APEX_MAX_EXPERTS];
        for (int e = 0; e < APEX_MAX_EXPERTS; ++e) pos[e] = -1;
        uint64_t seen = 0;
        bool valid = true;
        for (int j = 0; j < n && valid; ++j) {
          const int e = mb->cand[j];
          if (e < 0 || e >= N || ((seen >> e) & 1) || !((mask >> e) & 1)) valid = false;
          else { seen |= 1ull << e; pos[e] = j; }
        }
        if (valid) std::stable_sort(ordered.begin(), ordered.end(), [&](const SlotCopy& a, const SlotCopy& b) { return pos[a.expert] < pos[b.expert]; });
      }
      for (size_t i = 0; i < ordered.size(); ++i) {
        int r = issue_copy(ctx, l, ordered[i].expert, ordered[i].slot, ctx->stream_of_slot(ordered[i].slot));
        if (r != APEX_OK) {
          for (size_t j = i; j < ordered.size(); ++j) tab.drop(ordered[j].expert);
          raise_device_abort(ctx);
          return r;
        }
      }
      ctx->host_stats[l].prefetch_copies += (int64_t)copies.size();
      ctx->last_copies[l].insert(ctx->last_copies[l].end(), copies.begin(), copies.end());
      ctx->dec_opt_host[l] = (copies.empty() && ctx->cfg.cache_reuse) ? 1 : 0;  // next token: expect the same again
      if (!copies.empty() || !ctx->cfg.cache_reuse) {
        // the table of this layer changed: the kernel is (or will be) waiting for the new snapshot
        DecodeHostSnap* hs = ctx->dec_snap + l;
        hs->tab = make_snapshot(ctx, l);
        __atomic_store_n(&hs->seq, seq, __ATOMIC_RELEASE);
      }
    }
    // routed and execution set of this layer-step
    volatile uint32_t* kr = mb->kr_rec;
    volatile uint32_t* ex = mb->exec_rec;
    if (!host_wait_seq(ctx, kr + 2, seq) || !host_wait_seq(ctx, ex + 2, seq)) return fail_token(ctx, APEX_ETIMEOUT, "apex_decode_token: K_r did not arrive");
    const uint64_t kr_mask = ((uint64_t)kr[1] << 32) | kr[0], ex_mask = ((uint64_t)ex[1] << 32) | ex[0];
    if (mode == APEX_MODE_EXACT) {
      int32_t K_r[APEX_MAX_TOPK];
      int m = 0;
      for (int e = 0; e < N && m < k; ++e)
        if ((kr_mask >> e) & 1) K_r[m++] = e;
      for (; m < k; ++m) K_r[m] = -1;
      std::vector<SlotCopy> copies;
      uint64_t need = 0;
      const std::vector<int32_t> slot_expert_before = tab.slot_expert();
      if (!tab.plan_demand(K_r, 1, k, &copies, &need)) return fail_token(ctx, APEX_ESTATE, "no evictable slot");
      for (size_t i = 0; i < copies.size(); ++i) {
        const auto& c = copies[i];
        const int prev = slot_expert_before[c.slot];
        int r = APEX_OK;
        if (c.wave != 1 || (prev >= 0 && ((need >> prev) & 1))) r = fail(ctx, APEX_ESTATE, "demand plan would evict an expert in use");
        if (r == APEX_OK) r = issue_copy(ctx, l, c.expert, c.slot, ctx->stream_of_slot(c.slot));
        if (r == APEX_OK)
          r = stream_write32(ctx, ctx->stream_of_slot(c.slot), ctx->d_demand + (size_t)l * N + c.expert, (tag << 8) | (uint32_t)c.slot);
        if (r != APEX_OK) {
          for (size_t j = i; j < copies.size(); ++j) tab.drop(copies[j].expert);
          raise_device_abort(ctx);
          return r;
        }
      }
      ctx->host_stats[l].demand_copies += (int64_t)copies.size();
      ctx->last_copies[l].insert(ctx->last_copies[l].end(), copies.begin(), copies.end());
    } else {
      for (int e = 0; e < N; ++e)
        if ((ex_mask >> e) & 1) tab.touch(e);
    }
  }
  return check_device_status(ctx);
}

}  // namespace apex

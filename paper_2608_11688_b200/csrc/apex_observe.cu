// C-ABI entry points, part 3: observation and test support (counters, slot table snapshot and restore, warm-up,
// host-side fault hooks) and the host-only slot planner.
#include "apex_host.hpp"

using namespace apex;

extern "C" {

static void add_dev_stats(apex_step_stats* o, const DevStats& s, int n_sm) {
  o->tokens += (int64_t)s.tokens;
  o->sum_delta_hat += (int64_t)s.sum_delta_hat;
  o->sum_delta_star += (int64_t)s.sum_delta_star;
  o->sum_ncand += (int64_t)s.sum_ncand;
  o->capped += (int64_t)s.capped;
  o->routed += (int64_t)s.routed;
  o->hits_P += (int64_t)s.hits_P;
  o->hits_R += (int64_t)s.hits_R;
  o->covered += (int64_t)s.covered;
  o->substitutions += (int64_t)s.substitutions;
  o->stall_ns += (int64_t)(s.stall_ns / (unsigned long long)(n_sm > 0 ? n_sm : 1));
  o->timeouts += (int64_t)s.timeouts;
  o->near_full_prefetch += (int64_t)s.near_full;
}

int apex_get_stats(apex_ctx* ctx, int layer, apex_step_stats* out) {
  CHECK_CTX(ctx);
  if (!out || layer < -1 || layer >= ctx->cfg.L) return fail(ctx, APEX_EINVAL, "apex_get_stats: bad argument");
  CU_TRY(ctx, cudaDeviceSynchronize());
  std::vector<DevStats> ds(ctx->cfg.L);
  CU_TRY(ctx, cudaMemcpy(ds.data(), ctx->d_stats, ds.size() * sizeof(DevStats), cudaMemcpyDeviceToHost));
  memset(out, 0, sizeof *out);
  for (int l = 0; l < ctx->cfg.L; ++l) {
    if (layer >= 0 && l != layer) continue;
    const apex_step_stats& h = ctx->host_stats[l];
    out->layer_steps += h.layer_steps;
    out->prefetch_copies += h.prefetch_copies;
    out->demand_copies += h.demand_copies;
    out->bytes_copied += h.bytes_copied;
    out->extra_waves += h.extra_waves;
    add_dev_stats(out, ds[l], ctx->n_sm);
  }
  return APEX_OK;
}

int apex_reset_stats(apex_ctx* ctx) {
  CHECK_CTX(ctx);
  CU_TRY(ctx, cudaDeviceSynchronize());
  CU_TRY(ctx, cudaMemset(ctx->d_stats, 0, ctx->cfg.L * sizeof(DevStats)));
  for (auto& h : ctx->host_stats) h = apex_step_stats{};
  return APEX_OK;
}

int apex_read_prediction(apex_ctx* ctx, int B, float* z_p, float* q_p, int32_t* pi) {
  CHECK_CTX(ctx);
  if (B < 1 || B > ctx->cfg.max_batch) return fail(ctx, APEX_EINVAL, "bad B");
  CU_TRY(ctx, cudaStreamSynchronize(ctx->pred_stream));
  const size_t n = (size_t)B * ctx->cfg.N;
  if (z_p) CU_TRY(ctx, cudaMemcpy(z_p, ctx->d_zp, n * sizeof(float), cudaMemcpyDeviceToHost));
  if (q_p) CU_TRY(ctx, cudaMemcpy(q_p, ctx->d_qp, n * sizeof(float), cudaMemcpyDeviceToHost));
  if (pi) CU_TRY(ctx, cudaMemcpy(pi, ctx->d_pi, n * sizeof(int32_t), cudaMemcpyDeviceToHost));
  return APEX_OK;
}

int apex_get_last_copies(apex_ctx* ctx, int layer, int32_t* expert, int32_t* slot, int32_t* n_prefetch, int32_t* n_demand) {
  CHECK_CTX(ctx);
  CHECK_LAYER(ctx, layer);
  int np = 0, nd = 0, i = 0;
  for (const auto& c : ctx->last_copies[layer]) {
    if (expert) expert[i] = c.expert;
    if (slot) slot[i] = c.slot;
    ++i;
    if (c.wave == 0) ++np; else ++nd;
  }
  if (n_prefetch) *n_prefetch = np;
  if (n_demand) *n_demand = nd;
  return APEX_OK;
}

int apex_get_slot_table(apex_ctx* ctx, int layer, int32_t* expert_slot, int64_t* slot_stamp, int64_t* clock) {
  CHECK_CTX(ctx);
  CHECK_LAYER(ctx, layer);
  ctx->tables[layer].get(expert_slot, slot_stamp, clock);
  return APEX_OK;
}

int apex_set_slot_table(apex_ctx* ctx, int layer, const int32_t* expert_slot, const int64_t* slot_stamp, int64_t clock) {
  CHECK_CTX(ctx);
  CHECK_LAYER(ctx, layer);
  if (!expert_slot || !slot_stamp) return fail(ctx, APEX_EINVAL, "null table");
  if (!ctx->tables[layer].set(expert_slot, slot_stamp, clock)) return fail(ctx, APEX_EINVAL, "inconsistent slot table");
  // slots whose bytes belong to another expert are refilled
  CU_TRY(ctx, cudaDeviceSynchronize());
  for (int e = 0; e < ctx->cfg.N; ++e) {
    const int s = expert_slot[e];
    if (s >= 0 && ctx->phys_expert[layer][s] != e) {
      int r = issue_copy(ctx, layer, e, s, ctx->stream_of_slot(s));
      if (r != APEX_OK) return r;
    }
  }
  return APEX_OK;
}

int apex_warm_all(apex_ctx* ctx) {
  CHECK_CTX(ctx);
  if (ctx->cfg.C != ctx->cfg.N) return fail(ctx, APEX_ESTATE, "apex_warm_all needs C == N");
  std::vector<int32_t> es(ctx->cfg.N);
  std::vector<int64_t> stamp(ctx->cfg.C, 0);
  for (int e = 0; e < ctx->cfg.N; ++e) es[e] = e;
  for (int l = 0; l < ctx->cfg.L; ++l) {
    int r = apex_set_slot_table(ctx, l, es.data(), stamp.data(), ctx->tables[l].clock());
    if (r != APEX_OK) return r;
  }
  for (int i = 0; i < ctx->n_copy_streams; ++i) CU_TRY(ctx, cudaStreamSynchronize(ctx->cur_copy_streams[i]));
  return APEX_OK;
}

int apex_test_inject(apex_ctx* ctx, int what) {
  CHECK_CTX(ctx);
  if (what < 0 || what > 2) return fail(ctx, APEX_EINVAL, "unknown injection");
  ctx->inject = what;
  return APEX_OK;
}

int64_t apex_launch_count(const apex_ctx* ctx) { return ctx ? ctx->launches : -1; }

// ---- host-only slot planner ---------------------------------------------------------------------

struct apex_slots {
  SlotTable t;
  apex_slots(int N, int C, bool r) : t(N, C, r) {}
};

apex_slots* apex_slots_create(int N, int C, int cache_reuse) {
  if (N < 1 || N > APEX_MAX_EXPERTS || C < 1 || C > N) return nullptr;
  return new (std::nothrow) apex_slots(N, C, cache_reuse != 0);
}
void apex_slots_destroy(apex_slots* s) { delete s; }
int apex_slots_begin_step(apex_slots* s) {
  if (!s) return APEX_EINVAL;
  s->t.begin_step();
  return APEX_OK;
}
int apex_slots_prefetch(apex_slots* s, const int32_t* cand, const int32_t* ncand, int B, int stride, int32_t* copy_expert,
                        int32_t* copy_slot, int32_t* n_copies) {
  if (!s || !cand || !ncand || !n_copies || B < 1) return APEX_EINVAL;
  std::vector<SlotCopy> cp;
  if (!s->t.plan_prefetch(cand, ncand, B, stride, &cp)) return APEX_ESTATE;
  for (size_t i = 0; i < cp.size(); ++i) {
    if (copy_expert) copy_expert[i] = cp[i].expert;
    if (copy_slot) copy_slot[i] = cp[i].slot;
  }
  *n_copies = (int32_t)cp.size();
  return APEX_OK;
}
int apex_slots_demand(apex_slots* s, const int32_t* K_r, int B, int k, int32_t* copy_expert, int32_t* copy_slot,
                      int32_t* wave_of_copy, int32_t* n_copies) {
  if (!s || !K_r || !n_copies || B < 1 || k < 1) return APEX_EINVAL;
  std::vector<SlotCopy> cp;
  if (!s->t.plan_demand(K_r, B, k, &cp)) return APEX_ESTATE;
  for (size_t i = 0; i < cp.size(); ++i) {
    if (copy_expert) copy_expert[i] = cp[i].expert;
    if (copy_slot) copy_slot[i] = cp[i].slot;
    if (wave_of_copy) wave_of_copy[i] = cp[i].wave;
  }
  *n_copies = (int32_t)cp.size();
  return APEX_OK;
}
int apex_slots_touch(apex_slots* s, const int32_t* experts, int n) {
  if (!s || (!experts && n > 0)) return APEX_EINVAL;
  for (int i = 0; i < n; ++i) s->t.touch(experts[i]);
  return APEX_OK;
}
int apex_slots_get(const apex_slots* s, int32_t* expert_slot, int64_t* slot_stamp, int64_t* clock) {
  if (!s) return APEX_EINVAL;
  s->t.get(expert_slot, slot_stamp, clock);
  return APEX_OK;
}
int apex_slots_set(apex_slots* s, const int32_t* expert_slot, const int64_t* slot_stamp, int64_t clock) {
  if (!s || !expert_slot || !slot_stamp) return APEX_EINVAL;
  return s->t.set(expert_slot, slot_stamp, clock) ? APEX_OK : APEX_EINVAL;
}

}  // extern "C"

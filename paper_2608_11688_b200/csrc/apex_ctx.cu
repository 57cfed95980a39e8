// C-ABI entry points, part 1: context creation and destruction, parameters (routers, confidence model, expert
// stores).  No arithmetic of the path runs here.
#include "apex_host.hpp"

using namespace apex;

extern "C" {

namespace {
// A kernel launch that does not return before the kernel has finished (CUDA_LAUNCH_BLOCKING, or a tool injected
// into the CUDA runtime that serialises kernels) cannot be combined with a kernel that waits for the launching
// thread's next action.
bool launches_may_block() {
  const char* a = getenv("APEX_ASYNC_LAUNCHES");  // the caller vouches for asynchronous launches (e.g. a profiler capture of
  if (a && *a && strcmp(a, "0") != 0) return false;  // a run that cannot miss: every expert resident)
  const char* b = getenv("CUDA_LAUNCH_BLOCKING");
  if (b && *b && strcmp(b, "0") != 0) return true;
  for (const char* name : {"CUDA_INJECTION64_PATH", "CUDA_INJECTION32_PATH", "NV_COMPUTE_PROFILER_PERFWORKS_DIR",
                           "NV_NSIGHT_INJECTION_PORT_BASE", "NSIGHT_CUDA_DEBUGGER", "CUDA_DEBUGGER_SOFTWARE_PREEMPTION"}) {
    const char* v = getenv(name);
    if (v && *v) return true;
  }
  return false;
}
}  // namespace

int apex_create(const apex_config* cfg, apex_ctx** out) {
  create_error().clear();
  if (!cfg || !out) {
    create_error() = "apex_create: null argument";
    return APEX_EINVAL;
  }
  *out = nullptr;
  const apex_config& c = *cfg;
  if (c.N < 1 || c.N > APEX_MAX_EXPERTS || c.k < 1 || c.k > APEX_MAX_TOPK || c.k > c.N || c.C < c.k || c.C > c.N ||
      c.L < 1 || c.I < 1 || c.I_shared < 0 || c.max_batch < 1 || c.max_batch > APEX_MAX_BATCH || !ffn_shape_supported(c.d) ||
      c.ctx_len < 0) {
    create_error() = "apex_create: shape outside the limits of this build (see apex.h)";
    return APEX_EINVAL;
  }
  if (!(c.link_gbs >= 0.0)) {
    create_error() = "apex_create: link_gbs must be >= 0";
    return APEX_EINVAL;
  }
  // the kernels index (token, expert, intermediate index) rows with 31 bits
  if ((long long)c.max_batch * (c.k + 1) * (long long)(c.I > c.I_shared ? c.I : c.I_shared) >= (1ll << 30)) {
    create_error() = "apex_create: max_batch * (k + 1) * I does not fit the kernels' row index";
    return APEX_EINVAL;
  }
  apex_ctx* ctx = new (std::nothrow) apex_ctx();
  if (!ctx) return APEX_ENOMEM;
  ctx->cfg = c;
  ctx->host_waves = (c.flags & APEX_FLAG_HOST_WAVES) != 0 || launches_may_block();
  if (ctx->cfg.wait_limit_ns <= 0) ctx->cfg.wait_limit_ns = 2000000000ll;
  if (ctx->cfg.ctx_len == 0) ctx->cfg.ctx_len = 1024;
  const size_t L = c.L, N = c.N, C = c.C, d = c.d, MB = c.max_batch, k = c.k;
  const bool fp8 = (c.flags & APEX_FLAG_FP8_EXPERTS) != 0, fp4 = (c.flags & APEX_FLAG_FP4_EXPERTS) != 0;
  if ((fp8 && fp4) || ((fp8 || fp4) && !ffn_quantised_shape_supported(c.d))) {
    delete ctx;
    create_error() = "apex_create: the quantised expert stores exclude each other and need d in {512, 1024, 1536, 2048, 4096}";
    return APEX_EINVAL;
  }
  ctx->fmt = fp4 ? 2 : (fp8 ? 1 : 0);
  const size_t row_bytes = ffn_row_bytes(ctx->fmt, c.d);
  ctx->expert_bytes = row_bytes * (size_t)c.I;
  ctx->shared_bytes = row_bytes * (size_t)c.I_shared;

  auto bail = [&](int code, const char* what, cudaError_t e) {
    fail(ctx, code, what, e);
    create_error() = ctx->err;
    apex_destroy(ctx);
    return code;
  };
#define CR(expr)                                                                  \
  do {                                                                            \
    cudaError_t _e = (expr);                                                      \
    if (_e != cudaSuccess)                                                        \
      return bail(_e == cudaErrorMemoryAllocation ? APEX_ENOMEM : APEX_ECUDA, #expr, _e); \
  } while (0)

  CR(cudaGetDevice(&ctx->device));
  CR(cudaDeviceGetAttribute(&ctx->n_sm, cudaDevAttrMultiProcessorCount, ctx->device));
  CR(dev_alloc(&ctx->d_Wr, L * N * d));
  CR(dev_alloc(&ctx->d_Wp, L * N * d));
  CR(dev_alloc(&ctx->d_br, L * N));
  CR(dev_alloc(&ctx->d_bp, L * N));
  CR(dev_alloc(&ctx->d_w, L * N));
  CR(dev_alloc(&ctx->d_theta, L * (N - k + 1)));
  CR(cudaMemset(ctx->d_br, 0, L * N * sizeof(float)));
  CR(cudaMemset(ctx->d_bp, 0, L * N * sizeof(float)));
  CR(cudaMemset(ctx->d_w, 0, L * N * sizeof(float)));
  CR(cudaMemset(ctx->d_theta, 0, L * (N - k + 1) * sizeof(float)));
  ctx->has_br.assign(L, 0);
  ctx->has_bp.assign(L, 0);
  ctx->has_cdf.assign(L, 0);
  CR(dev_alloc(&ctx->d_cache, L * C * ctx->expert_bytes));
  CR(dev_alloc(&ctx->d_slot_ready, L * C));
  CR(cudaMemset(ctx->d_slot_ready, 0, L * C * sizeof(uint32_t)));
  CR(dev_alloc(&ctx->d_zp, MB * N));
  CR(dev_alloc(&ctx->d_qp, MB * N));
  CR(dev_alloc(&ctx->d_zr, L * MB * N));
  CR(dev_alloc(&ctx->d_demand, L * N));
  CR(cudaMemset(ctx->d_demand, 0, L * N * sizeof(uint32_t)));
  CR(dev_alloc(&ctx->d_pi, MB * N));
  CR(dev_alloc(&ctx->d_ncand, MB));
  CR(dev_alloc(&ctx->d_stats, L));
  CR(cudaMemset(ctx->d_stats, 0, L * sizeof(DevStats)));
  CR(dev_alloc(&ctx->d_tickets, 64));
  CR(cudaMemset(ctx->d_tickets, 0, 64 * sizeof(unsigned int)));
  CR(dev_alloc(&ctx->d_spec, L * APEX_MAX_TOPK));
  CR(cudaMemset(ctx->d_spec, 0xff, L * APEX_MAX_TOPK * sizeof(int32_t)));
  CR(dev_alloc(&ctx->d_counters, 2));
  CR(cudaMemset(ctx->d_counters, 0, 2 * sizeof(unsigned long long)));
  const size_t max_pairs = MB * (k + 1);
  CR(dev_alloc(&ctx->d_plan_exec_idx, MB * k));
  CR(dev_alloc(&ctx->d_plan_exec_gate, MB * k));
  CR(dev_alloc(&ctx->d_pair_tok, max_pairs));
  CR(dev_alloc(&ctx->d_pair_gate, max_pairs));
  CR(dev_alloc(&ctx->d_pair_expert, max_pairs));
  CR(dev_alloc(&ctx->d_n_pairs, 4));
  CR(dev_alloc(&ctx->d_grp, 4 + 3 * (N + 1)));
  CR(dev_alloc(&ctx->d_cand, MB * C));
  CR(dev_alloc(&ctx->d_idx, L * MB * k));
  CR(dev_alloc(&ctx->d_exec_idx, MB * k));
  CR(dev_alloc(&ctx->d_alpha, L * MB * N));
  CR(dev_alloc(&ctx->d_exec_gate, MB * k));
  CR(dev_alloc(&ctx->d_cand_ncand, MB));
  // batched tensor-core path: scratch and tensor maps (only for contexts that will see large batches)
  if (MB >= kTcMinBatch && tc_shape_supported(c.d, c.I, c.I_shared, ctx->fmt)) {
    const size_t rows = max_pairs + 256;
    const size_t i_max = (size_t)(c.I > c.I_shared ? c.I : c.I_shared);
    ctx->act_stride = (int)i_max;
    CR(dev_alloc(&ctx->d_xg, rows * d));
    ctx->act_plane = rows * i_max;
    CR(dev_alloc(&ctx->d_act, 2 * rows * i_max));
    CR(cudaMemset(ctx->d_xg, 0, rows * d * 2));
    CR(cudaMemset(ctx->d_act, 0, 2 * rows * i_max * 2));
    ctx->tc_ok = tc_make_store_maps(ctx->fmt, ctx->tc_maps.w_gateup, ctx->tc_maps.w_down, ctx->tc_maps.sc_gateup, ctx->tc_maps.sc_down,
                                    ctx->d_cache, c.d, c.I, L * C, ctx->expert_bytes) &&
                 tc_make_rows_map(ctx->tc_maps.xg, ctx->d_xg, c.d, rows, d) &&
                 tc_make_rows_map(ctx->tc_maps.act, ctx->d_act, (int)i_max, rows, i_max) &&
                 tc_make_rows_map(ctx->tc_maps.act_lo, ctx->d_act + ctx->act_plane, (int)i_max, rows, i_max);
    ctx->tc_shared_maps.assign(L, ctx->tc_maps);
  }
  ctx->attn_bytes = (4 * d * d + 2 * (size_t)ctx->cfg.ctx_len * d) * 2;
  ctx->attn_layers = L < 8 ? L : 8;
  CR(dev_alloc(&ctx->d_attn, ctx->attn_bytes * ctx->attn_layers));
  CR(cudaMemset(ctx->d_attn, 0, ctx->attn_bytes * ctx->attn_layers));
  CR(dev_alloc(&ctx->d_attn_sink, 4));

  // mapped mailbox
  MailboxLayout& ml = ctx->ml;
  size_t off = sizeof(MailboxHeader);
  ml.off_exec_seq = off;  off += L * sizeof(uint32_t);
  off = (off + 15) & ~(size_t)15;
  ml.off_sel_rec = off;   off += 16;
  ml.off_exec_rec = off;  off += L * 32;   // per layer: routed-set record, execution-set record (B = 1)
  ml.off_ncand = off; off += MB * sizeof(int32_t);
  ml.off_cand = off;  off += MB * C * sizeof(int32_t);
  ml.kr_stride = MB * k * sizeof(int32_t);
  ml.off_kr = off;    off += L * ml.kr_stride;
  ml.off_exec = off;  off += L * ml.kr_stride;
  ml.bytes = off;
  ctx->exec_seq.assign(L, 0u);
  CR(cudaHostAlloc(reinterpret_cast<void**>(&ctx->mbox), ml.bytes, cudaHostAllocMapped | cudaHostAllocPortable));
  memset(ctx->mbox, 0, ml.bytes);
  ctx->gen_src_len = 1 << 16;
  CR(cudaHostAlloc(reinterpret_cast<void**>(&ctx->gen_src), ctx->gen_src_len * sizeof(uint32_t), cudaHostAllocPortable));

  if (c.link_gbs > 0.0) {  // one emulated link: copies one after the other, each padded to its target duration
    ctx->n_copy_streams = 1;
    ctx->pad_bytes = ctx->expert_bytes > (4u << 20) ? ctx->expert_bytes : (size_t)(4u << 20);
    CR(cudaHostAlloc(reinterpret_cast<void**>(&ctx->pad_src), ctx->pad_bytes, cudaHostAllocDefault));
    memset(ctx->pad_src, 0, ctx->pad_bytes);
    CR(cudaMalloc(reinterpret_cast<void**>(&ctx->pad_dst), ctx->pad_bytes));
  }
  for (int i = 0; i < ctx->n_copy_streams; ++i) {
    CR(cudaStreamCreateWithFlags(&ctx->copy_streams[i], cudaStreamNonBlocking));
    ctx->cur_copy_streams[i] = ctx->copy_streams[i];
  }
  CR(cudaEventCreateWithFlags(&ctx->ev_wave, cudaEventDisableTiming));
  CR(cudaEventCreateWithFlags(&ctx->ev_in, cudaEventDisableTiming));
#undef CR
  {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qr;
    if (cudaGetDriverEntryPoint("cuStreamWriteValue32", &fn, cudaEnableDefault, &qr) == cudaSuccess &&
        qr == cudaDriverEntryPointSuccess)
      ctx->fn_write_value32 = fn;
    cudaGetLastError();
  }
  ctx->tables.reserve(L);
  for (size_t l = 0; l < L; ++l) ctx->tables.emplace_back((int)N, (int)C, c.cache_reuse != 0);
  ctx->store_base.assign(L, nullptr);
  ctx->store_stride.assign(L, 0);
  ctx->shared_dev.assign(L, nullptr);
  ctx->shared_gate_dev.assign(L, nullptr);
  ctx->shared_gate_on.assign(L, 0);
  ctx->slot_gen.assign(L, std::vector<uint32_t>(C, 0u));
  ctx->phys_expert.assign(L, std::vector<int32_t>(C, -1));
  ctx->last_copies.assign(L, {});
  ctx->host_stats.assign(L, apex_step_stats{});
  ctx->step.assign(L, apex_ctx::StepState{});
  ctx->ffn_params.assign(L, FfnParams{});
  {
    const int r = decode_setup(ctx);
    if (r != APEX_OK) {
      create_error() = ctx->err;
      apex_destroy(ctx);
      return r;
    }
  }
  *out = ctx;
  return APEX_OK;
}

int apex_destroy(apex_ctx* ctx) {
  if (!ctx) return APEX_EINVAL;
  cudaDeviceSynchronize();
  cudaGetLastError();
  void* dev[] = {ctx->d_Wr, ctx->d_br, ctx->d_Wp, ctx->d_bp, ctx->d_w, ctx->d_theta, ctx->d_cache, ctx->d_slot_ready, ctx->d_zp,
                 ctx->d_qp, ctx->d_zr, ctx->d_demand, ctx->d_pi, ctx->d_ncand, ctx->d_stats, ctx->d_counters, ctx->d_tickets, ctx->d_spec, ctx->d_plan_exec_idx,
                 ctx->d_plan_exec_gate, ctx->d_pair_tok, ctx->d_pair_gate, ctx->d_pair_expert, ctx->d_n_pairs, ctx->d_grp, ctx->d_xg, ctx->d_act, ctx->d_cand,
                 ctx->d_idx, ctx->d_exec_idx, ctx->d_alpha, ctx->d_exec_gate, ctx->d_cand_ncand, ctx->d_attn, ctx->d_attn_sink,
                 ctx->d_h_stage, ctx->d_hp_stage, ctx->d_y_stage};
  for (void* p : dev)
    if (p) cudaFree(p);
  decode_teardown(ctx);
  for (float* g : ctx->shared_gate_dev)
    if (g) cudaFree(g);
  if (ctx->mbox) cudaFreeHost(ctx->mbox);
  if (ctx->pad_src) cudaFreeHost(ctx->pad_src);
  if (ctx->pad_dst) cudaFree(ctx->pad_dst);
  if (ctx->gen_src) cudaFreeHost(ctx->gen_src);
  for (cudaStream_t cs : ctx->copy_streams)
    if (cs) cudaStreamDestroy(cs);
  if (ctx->ev_wave) cudaEventDestroy(ctx->ev_wave);
  if (ctx->ev_in) cudaEventDestroy(ctx->ev_in);
  delete ctx;
  return APEX_OK;
}

const char* apex_last_error(const apex_ctx* ctx) { return ctx ? ctx->err.c_str() : create_error().c_str(); }

int apex_set_router(apex_ctx* ctx, int layer, const float* W, const float* b) {
  CHECK_CTX(ctx);
  CHECK_LAYER(ctx, layer);
  if (!W) return fail(ctx, APEX_EINVAL, "W_r is null");
  const size_t N = ctx->cfg.N, d = ctx->cfg.d;
  CU_TRY(ctx, cudaMemcpy(ctx->d_Wr + (size_t)layer * N * d, W, N * d * sizeof(float), cudaMemcpyHostToDevice));
  if (b) CU_TRY(ctx, cudaMemcpy(ctx->d_br + (size_t)layer * N, b, N * sizeof(float), cudaMemcpyHostToDevice));
  ctx->has_br[layer] = b ? 1 : 0;
  return APEX_OK;
}

int apex_set_prefetch_router(apex_ctx* ctx, int layer, const float* W, const float* b) {
  CHECK_CTX(ctx);
  CHECK_LAYER(ctx, layer);
  if (!W) return fail(ctx, APEX_EINVAL, "W_p is null");
  const size_t N = ctx->cfg.N, d = ctx->cfg.d;
  CU_TRY(ctx, cudaMemcpy(ctx->d_Wp + (size_t)layer * N * d, W, N * d * sizeof(float), cudaMemcpyHostToDevice));
  if (b) CU_TRY(ctx, cudaMemcpy(ctx->d_bp + (size_t)layer * N, b, N * sizeof(float), cudaMemcpyHostToDevice));
  ctx->has_bp[layer] = b ? 1 : 0;
  return APEX_OK;
}

int apex_set_cdf(apex_ctx* ctx, int layer, const float* w, const float* theta) {
  CHECK_CTX(ctx);
  CHECK_LAYER(ctx, layer);
  if (!w || !theta) return fail(ctx, APEX_EINVAL, "w or theta is null");
  const size_t N = ctx->cfg.N, nth = ctx->cfg.N - ctx->cfg.k + 1;
  for (size_t i = 1; i < nth; ++i)
    if (!(theta[i] >= theta[i - 1])) return fail(ctx, APEX_EINVAL, "theta must be non-decreasing");
  CU_TRY(ctx, cudaMemcpy(ctx->d_w + (size_t)layer * N, w, N * sizeof(float), cudaMemcpyHostToDevice));
  CU_TRY(ctx, cudaMemcpy(ctx->d_theta + (size_t)layer * nth, theta, nth * sizeof(float), cudaMemcpyHostToDevice));
  ctx->has_cdf[layer] = 1;
  return APEX_OK;
}

int apex_register_experts(apex_ctx* ctx, int layer, const void* base, size_t stride) {
  CHECK_CTX(ctx);
  CHECK_LAYER(ctx, layer);
  if (!base || stride < ctx->expert_bytes || (stride & 15) || ((uintptr_t)base & 15))
    return fail(ctx, APEX_EINVAL, "expert store: null base, stride below 3*I*d*2 or not 16-byte aligned");
  // Pinned host memory only.  Copies from it run on the copy engines beside the kernels that wait for them;
  // a copy from pageable memory is staged and synchronous, and a device-to-device copy was seen not to make
  // progress while the expert-FFN kernel waited for it.
  cudaPointerAttributes attr{};
  if (cudaPointerGetAttributes(&attr, base) != cudaSuccess || attr.type != cudaMemoryTypeHost) {
    cudaGetLastError();
    return fail(ctx, APEX_EINVAL, "expert store: the base must be pinned (page-locked) host memory");
  }
  ctx->store_base[layer] = static_cast<const uint8_t*>(base);
  ctx->store_stride[layer] = stride;
  return APEX_OK;
}

int apex_set_shared_expert(apex_ctx* ctx, int layer, const void* dev_weights) {
  CHECK_CTX(ctx);
  CHECK_LAYER(ctx, layer);
  if (ctx->cfg.I_shared <= 0) return fail(ctx, APEX_EINVAL, "the context was created with I_shared = 0");
  if (!dev_weights || ((uintptr_t)dev_weights & 15)) return fail(ctx, APEX_EINVAL, "shared expert: null or unaligned");
  ctx->shared_dev[layer] = static_cast<const uint8_t*>(dev_weights);
  if (ctx->d_shared_ptrs)
    CU_TRY(ctx, cudaMemcpy(ctx->d_shared_ptrs + layer, &dev_weights, sizeof(void*), cudaMemcpyHostToDevice));
  if (ctx->tc_ok) {
    TcMaps& m = ctx->tc_shared_maps[layer];
    if (!tc_make_store_maps(ctx->fmt, m.ws_gateup, m.ws_down, m.ssc_gateup, m.ssc_down, dev_weights, ctx->cfg.d, ctx->cfg.I_shared, 1,
                            ctx->shared_bytes))
      return fail(ctx, APEX_ECUDA, "tensor map for the shared expert could not be encoded");
  }
  return APEX_OK;
}

int apex_set_shared_gate(apex_ctx* ctx, int layer, const float* w_sg) {
  CHECK_CTX(ctx);
  CHECK_LAYER(ctx, layer);
  if (ctx->cfg.I_shared <= 0) return fail(ctx, APEX_EINVAL, "the context was created with I_shared = 0");
  float* dst = ctx->shared_gate_dev[layer];
  if (!w_sg) {  // back to weight 1 (the vector stays allocated for a later call)
    const float* none = nullptr;
    if (ctx->d_shared_gate_ptrs)
      CU_TRY(ctx, cudaMemcpy(ctx->d_shared_gate_ptrs + layer, &none, sizeof(void*), cudaMemcpyHostToDevice));
    ctx->shared_gate_on[layer] = 0;
    return APEX_OK;
  }
  if (!dst) {
    CU_TRY(ctx, cudaMalloc(reinterpret_cast<void**>(&dst), (size_t)ctx->cfg.d * sizeof(float)));
    ctx->shared_gate_dev[layer] = dst;
  }
  CU_TRY(ctx, cudaMemcpy(dst, w_sg, (size_t)ctx->cfg.d * sizeof(float), cudaMemcpyDefault));
  if (ctx->d_shared_gate_ptrs)
    CU_TRY(ctx, cudaMemcpy(ctx->d_shared_gate_ptrs + layer, &dst, sizeof(void*), cudaMemcpyHostToDevice));
  ctx->shared_gate_on[layer] = 1;
  return APEX_OK;
}

int apex_pack_expert(const void* gate, const void* up, const void* down, int d, int I, void* dst) {
  if (!gate || !up || !down || !dst || d < 1 || I < 1) return APEX_EINVAL;
  const uint16_t* dn = static_cast<const uint16_t*>(down);
  uint16_t* o = static_cast<uint16_t*>(dst);
  const uint16_t* g = static_cast<const uint16_t*>(gate);
  const uint16_t* u = static_cast<const uint16_t*>(up);
  for (int i = 0; i < I; ++i) {
    uint16_t* row = o + (size_t)i * 3 * d;
    memcpy(row, g + (size_t)i * d, (size_t)d * 2);
    memcpy(row + d, u + (size_t)i * d, (size_t)d * 2);
    for (int j = 0; j < d; ++j) row[2 * (size_t)d + j] = dn[(size_t)j * I + i];
  }
  return APEX_OK;
}

// ---------------------------------------------------------------------------------------------

}  // extern "C"

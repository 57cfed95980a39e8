// Expert FFN over the HBM slot cache: y = sum_{e in K~} g_e W_down,e ( silu(W_gate,e h') * (W_up,e h') )
// (Sec. III-A weighted sum of expert outputs; Sec. IV-E execution modes; Algorithm 1).
//
// The step is bandwidth-bound at decode batch sizes: every weight byte is used once per token.
// Layout: a slot holds gate[I][d], up[I][d], downT[I][d] (bf16), so intermediate index i owns three
// d-vectors and one pass suffices:  a_i = g_e * silu(gate_i . h') * (up_i . h'),  y += a_i * downT_i.
//
// Kernel: persistent, one CTA per SM.  The (pair, i) row space -- a pair is (token, expert) -- is
// cut into equal contiguous ranges, one per CTA.  A producer thread streams row triples into a
// shared-memory ring with bulk asynchronous copies (TMA, mbarrier completion); eight consumer warps
// take ring entries round-robin, do the two dot products with warp-shuffle reductions and
// accumulate the down projection in registers (fp32).  Partial y vectors are reduced across the
// warps of the CTA in shared memory and added to y with vector atomics.
#include <cuda_bf16.h>

#include "apex_internal.hpp"

namespace apex {

// Debug builds (-DAPEX_TIMELINE) record per-CTA time stamps of the streaming kernel.
#ifdef APEX_TIMELINE
__device__ unsigned long long g_timeline[1024 * 16];
#define TL(slot)                                                                      \
  do {                                                                                \
    g_timeline[blockIdx.x * 16 + (slot)] = (slot) == 0 ? globaltimer_ns_raw() : (unsigned long long)clock64(); \
  } while (0)
__device__ __forceinline__ unsigned long long globaltimer_ns_raw() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
#else
#define TL(slot) do { } while (0)
#endif

constexpr int kConsumerWarps = 8;
constexpr int kFfnThreads = (kConsumerWarps + 1) * 32;
constexpr int kMaxStages = 32;
constexpr int kSmemBudget = 224 * 1024;  // ring bytes; static tables fit in what is left of the 227 KB per-CTA limit
constexpr int kSmallPairs = APEX_MAX_TOPK + 1;

__host__ __device__ constexpr int ring_stages(uint32_t entry_bytes) {
  int n = kSmemBudget / (int)entry_bytes;
  if (n > kMaxStages) n = kMaxStages;
  return n / kConsumerWarps * kConsumerWarps;
}

// ---------------------------------------------------------------- PTX helpers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ unsigned long long globaltimer_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
// Bounded wait: returns false when the time limit ran out or another thread of the CTA gave up
// (the caller records it and stops working).
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, const volatile int* abort_flag, long long limit_ns) {
  if (mbar_try_wait(bar, parity)) return true;
  const unsigned long long t0 = globaltimer_ns();
  for (uint32_t it = 1;; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((it & 255u) == 0u) {
      if (*abort_flag) return false;
      if ((long long)(globaltimer_ns() - t0) > limit_ns) return false;
    }
  }
}
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   smem_u32(dst)),
               "l"(src), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}
__device__ __forceinline__ uint32_t ld_acquire_sys(const uint32_t* p) {
  uint32_t v;
  asm volatile("ld.acquire.sys.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ unsigned long long ld_acquire_gpu_u64(const unsigned long long* p) {
  unsigned long long v;
  asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ float bf16lo(uint32_t v) { return __uint_as_float(v << 16); }
__device__ __forceinline__ float bf16hi(uint32_t v) { return __uint_as_float(v & 0xffff0000u); }

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// ---------------------------------------------------------------- execution set of one token (S6)
// One warp.  Lanes own experts lane and lane+32.  Exact mode: K~ = K_r.  Stall-free mode
// (Algorithm 1 with K_p := resident set): keep K_r that is resident, replace the |M| missing ones by
// the |M| best remaining resident experts.  "Best" is by router weight alpha = softmax(z_r); the
// order of alpha is the order of the logits, so the comparison is done on z_r (value descending,
// index ascending).  Gates: alpha_e / sum over K~ (norm_topk) or alpha_e.
// Returns the execution mask; pos/gate describe this lane's experts.
struct TokenPlan {
  unsigned long long exec_mask;
  unsigned long long kr_mask;
  float g0, g1;  // gates of experts lane, lane+32 (0 if not executed)
};

__device__ __forceinline__ TokenPlan plan_token(const int32_t* __restrict__ idx, const float* __restrict__ z_r,
                                                const float* __restrict__ alpha, int N, int k, int mode,
                                                int norm_topk, unsigned long long resident, int lane) {
  unsigned lo = 0, hi = 0;
  if (lane < k) {
    const int e = idx[lane];
    if (e < 32)
      lo = 1u << e;
    else
      hi = 1u << (e - 32);
  }
  lo = __reduce_or_sync(0xffffffffu, lo);
  hi = __reduce_or_sync(0xffffffffu, hi);
  const unsigned long long kr = ((unsigned long long)hi << 32) | lo;
  unsigned long long exec = kr;
  if (mode == APEX_MODE_STALL_FREE && (kr & ~resident) != 0ull) {
    const unsigned long long keep = kr & resident;
    const int n_missing = __popcll(kr & ~resident);
    const unsigned long long cand = resident & ~kr;
    const int e0 = lane, e1 = lane + 32;
    const float z0 = e0 < N ? z_r[e0] : 0.f, z1 = e1 < N ? z_r[e1] : 0.f;
    int r0 = 0, r1 = 0;
    unsigned long long rest = cand;
    while (rest) {
      const int f = __ffsll((long long)rest) - 1;
      rest &= rest - 1;
      const float zf = __shfl_sync(0xffffffffu, f < 32 ? z0 : z1, f & 31);
      r0 += (zf > z0 || (zf == z0 && f < e0)) ? 1 : 0;
      r1 += (zf > z1 || (zf == z1 && f < e1)) ? 1 : 0;
    }
    const bool s0 = ((cand >> e0) & 1) && r0 < n_missing;
    const bool s1 = e1 < 64 && ((cand >> e1) & 1) && r1 < n_missing;
    const unsigned b0 = __ballot_sync(0xffffffffu, s0), b1 = __ballot_sync(0xffffffffu, s1);
    exec = keep | (((unsigned long long)b1 << 32) | b0);
  }
  const int e0 = lane, e1 = lane + 32;
  const bool x0 = (exec >> e0) & 1, x1 = (exec >> e1) & 1;
  const float a0 = x0 ? alpha[e0] : 0.f, a1 = x1 ? alpha[e1] : 0.f;
  float denom = 1.f;
  if (norm_topk) denom = warp_sum(a0 + a1);
  TokenPlan tp;
  tp.exec_mask = exec;
  tp.kr_mask = kr;
  tp.g0 = a0 / denom;
  tp.g1 = a1 / denom;
  return tp;
}

// Writes the per-token outputs of the plan (ascending expert index).
__device__ __forceinline__ void store_token_plan(const TokenPlan& tp, int lane, int k, int32_t* exec_idx, float* exec_gate,
                                                 int32_t* mbox_exec) {
  const int e0 = lane, e1 = lane + 32;
  if ((tp.exec_mask >> e0) & 1) {
    const int pos = __popcll(tp.exec_mask & ((1ull << e0) - 1ull));
    if (pos < k) {
      if (exec_idx) exec_idx[pos] = e0;
      if (exec_gate) exec_gate[pos] = tp.g0;
      if (mbox_exec) mbox_exec[pos] = e0;
    }
  }
  if ((tp.exec_mask >> e1) & 1) {
    const int pos = __popcll(tp.exec_mask & ((1ull << e1) - 1ull));
    if (pos < k) {
      if (exec_idx) exec_idx[pos] = e1;
      if (exec_gate) exec_gate[pos] = tp.g1;
      if (mbox_exec) mbox_exec[pos] = e1;
    }
  }
}

// ---------------------------------------------------------------- batched plan (B > 1)
// One CTA.  Warps plan tokens; then thread e gathers the tokens that execute expert e, so the pair
// list is sorted by (expert, token).  Shared-expert pairs (expert id N) follow.
__global__ void __launch_bounds__(1024) ffn_plan_kernel(const FfnParams p) {
  __shared__ unsigned long long s_exec[APEX_MAX_BATCH];
  __shared__ int s_count[APEX_MAX_EXPERTS + 1];
  __shared__ int s_off[APEX_MAX_EXPERTS + 2];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarp = blockDim.x >> 5;
  const int N = p.N, k = p.k, B = p.B;
  int my_subst = 0;
  for (int b = warp; b < B; b += nwarp) {
    const TokenPlan tp = plan_token(p.idx + (size_t)b * k, p.z_r + (size_t)b * N, p.alpha + (size_t)b * N, N, k, p.mode,
                                    p.norm_topk, p.snap.resident_mask, lane);
    store_token_plan(tp, lane, k, p.plan_exec_idx + (size_t)b * k, p.plan_exec_gate + (size_t)b * k,
                     p.post_exec ? p.mbox_exec + (size_t)b * k : nullptr);
    if (p.post_exec) {
      const int e0 = lane, e1 = lane + 32;
      if ((tp.exec_mask >> e0) & 1) {
        const int pos = __popcll(tp.exec_mask & ((1ull << e0) - 1ull));
        if (p.exec_idx) p.exec_idx[(size_t)b * k + pos] = e0;
        if (p.exec_gate) p.exec_gate[(size_t)b * k + pos] = tp.g0;
      }
      if ((tp.exec_mask >> e1) & 1) {
        const int pos = __popcll(tp.exec_mask & ((1ull << e1) - 1ull));
        if (p.exec_idx) p.exec_idx[(size_t)b * k + pos] = e1;
        if (p.exec_gate) p.exec_gate[(size_t)b * k + pos] = tp.g1;
      }
      my_subst += __popcll(tp.exec_mask & ~tp.kr_mask);
    }
    if (lane == 0) s_exec[b] = tp.exec_mask;
  }
  if (p.post_exec && lane == 0 && my_subst && p.stats) atomicAdd(&p.stats->substitutions, (unsigned long long)my_subst);
  __syncthreads();
  const int e = threadIdx.x;
  if (e < N) {
    int c = 0;
    if ((p.run_mask >> e) & 1)
      for (int b = 0; b < B; ++b) c += (int)((s_exec[b] >> e) & 1);
    s_count[e] = c;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    int acc = 0;
    for (int f = 0; f < N; ++f) {
      s_off[f] = acc;
      acc += s_count[f];
    }
    s_off[N] = acc;  // routed pairs
    const int n_pairs = acc + (p.run_shared ? B : 0);
    p.n_pairs[0] = n_pairs;
  }
  __syncthreads();
  if (e < N && s_count[e] > 0) {
    int o = s_off[e];
    for (int b = 0; b < B; ++b) {
      if ((s_exec[b] >> e) & 1) {
        const int pos = __popcll(s_exec[b] & ((1ull << e) - 1ull));
        p.pair_tok[o] = b;
        p.pair_expert[o] = e;
        p.pair_gate[o] = p.plan_exec_gate[(size_t)b * k + pos];
        ++o;
      }
    }
  }
  if (p.run_shared) {
    const int base = s_off[N];
    for (int b = threadIdx.x; b < B; b += blockDim.x) {
      p.pair_tok[base + b] = b;
      p.pair_expert[base + b] = N;
      p.pair_gate[base + b] = 1.f;
    }
  }
  if (p.post_exec) {
    __threadfence_system();
    __syncthreads();
    if (threadIdx.x == 0) {
      __threadfence_system();
      *p.mbox_seq = p.seq_value;
    }
  }
}

cudaError_t launch_ffn_plan(const FfnParams& p, cudaStream_t s) {
  ffn_plan_kernel<<<1, 1024, 0, s>>>(p);
  return cudaGetLastError();
}

// ---------------------------------------------------------------- the streaming FFN kernel
struct PairView {
  const int32_t* tok;
  const float* gate;
  const int32_t* expert;
  int n_pairs;
  int n_routed;  // pairs before the shared-expert pairs
};

__device__ __forceinline__ long long pair_row_off(const PairView& v, int pidx, int I, int I_shared) {
  return pidx <= v.n_routed ? (long long)pidx * I : (long long)v.n_routed * I + (long long)(pidx - v.n_routed) * I_shared;
}
// pair that contains row r
__device__ __forceinline__ int pair_of_row(const PairView& v, long long r, int I, int I_shared) {
  const long long routed_rows = (long long)v.n_routed * I;
  return r < routed_rows ? (int)(r / I) : v.n_routed + (int)((r - routed_rows) / I_shared);
}

template <int NCH, bool H_REGS>
__global__ void __launch_bounds__(kFfnThreads, 1) moe_ffn_stream_kernel(const FfnParams p) {
  extern __shared__ __align__(128) uint8_t smem[];
  __shared__ int32_t s_tok[kSmallPairs], s_exp[kSmallPairs];
  __shared__ float s_gate[kSmallPairs];
  __shared__ int s_np[2];
  __shared__ int s_abort;
  __shared__ uint64_t s_full[kMaxStages], s_empty[kMaxStages];

  constexpr int d = NCH * 256;
  constexpr uint32_t row_bytes = d * 2;
  constexpr uint32_t entry_bytes = 3 * row_bytes;
  // The ring depth is a multiple of the consumer-warp count, so a stage is always consumed by the
  // same warp: a warp can then never wait on a stage's next phase before it has consumed the current
  // one (a parity wait cannot tell "one phase ahead" from "done").
  constexpr int NS = ring_stages(entry_bytes);
  static_assert(NS >= kConsumerWarps && NS % kConsumerWarps == 0, "ring depth must be a multiple of the consumer warps");

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int N = p.N, k = p.k, I = p.I, B = p.B;
  const int G = gridDim.x, cta = blockIdx.x;

  if (tid == 0) {
    TL(0);
    TL(1);
    s_abort = 0;
    for (int s = 0; s < NS; ++s) {
      mbar_init(&s_full[s], 1);
      mbar_init(&s_empty[s], 1);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }

  // ---- zero this CTA's slice of y (first launch of a layer-step only)
  if (!p.accumulate) {
    const size_t n4 = (size_t)B * d / 4;
    const size_t per = (n4 + G - 1) / G;
    const size_t lo = per * cta, hi = lo + per < n4 ? lo + per : n4;
    float4* y4 = reinterpret_cast<float4*>(p.y);
    for (size_t i = lo + tid; i < hi; i += kFfnThreads) y4[i] = make_float4(0.f, 0.f, 0.f, 0.f);
  }

  // ---- plan
  PairView pv;
  if (B == 1) {
    if (warp == 0) {
      const TokenPlan tp = plan_token(p.idx, p.z_r, p.alpha, N, k, p.mode, p.norm_topk, p.snap.resident_mask, lane);
      if (cta == 0 && p.post_exec) {
        store_token_plan(tp, lane, k, p.exec_idx, p.exec_gate, p.mbox_exec);
        if (lane == 0 && p.stats) {
          const int ns = __popcll(tp.exec_mask & ~tp.kr_mask);
          if (ns) atomicAdd(&p.stats->substitutions, (unsigned long long)ns);
        }
        __threadfence_system();
        __syncwarp();
        if (lane == 0) {
          __threadfence_system();
          *p.mbox_seq = p.seq_value;
        }
      }
      const unsigned long long run = tp.exec_mask & p.run_mask;
      const int e0 = lane, e1 = lane + 32;
      if ((run >> e0) & 1) {
        const int pos = __popcll(run & ((1ull << e0) - 1ull));
        s_tok[pos] = 0;
        s_exp[pos] = e0;
        s_gate[pos] = tp.g0;
      }
      if ((run >> e1) & 1) {
        const int pos = __popcll(run & ((1ull << e1) - 1ull));
        s_tok[pos] = 0;
        s_exp[pos] = e1;
        s_gate[pos] = tp.g1;
      }
      if (lane == 0) {
        const int nr = __popcll(run);
        if (p.run_shared) {
          s_tok[nr] = 0;
          s_exp[nr] = N;
          s_gate[nr] = 1.f;
        }
        s_np[0] = nr + (p.run_shared ? 1 : 0);
        s_np[1] = nr;
      }
    }
    __syncthreads();
    pv.tok = s_tok;
    pv.gate = s_gate;
    pv.expert = s_exp;
    pv.n_pairs = s_np[0];
    pv.n_routed = s_np[1];
  } else {
    __syncthreads();
    pv.tok = p.pair_tok;
    pv.gate = p.pair_gate;
    pv.expert = p.pair_expert;
    pv.n_pairs = p.n_pairs[0];
    pv.n_routed = pv.n_pairs - (p.run_shared ? B : 0);
  }
  if (!p.accumulate && tid == 0) {
    __threadfence();
    atomicAdd(p.zero_counter, 1ull);
  }

  if (tid == 0) TL(2);  // plan done
  const long long total_rows = pair_row_off(pv, pv.n_pairs, I, p.I_shared);
  const long long r_begin = total_rows * cta / G, r_end = total_rows * (cta + 1) / G;
  const int n_my = (int)(r_end - r_begin);

  float acc[NCH * 8];
#pragma unroll
  for (int i = 0; i < NCH * 8; ++i) acc[i] = 0.f;

  if (warp == kConsumerWarps) {
    // ================= producer: one thread issues every copy of this CTA
    if (lane == 0 && n_my > 0) {
      int pidx = pair_of_row(pv, r_begin, I, p.I_shared);
      long long pair_end = pair_row_off(pv, pidx + 1, I, p.I_shared);
      int cur_e = -1;
      const uint8_t* base = nullptr;
      size_t mat_bytes = 0;
      unsigned long long waited = 0;
      bool ok = true;
      for (int q = 0; q < n_my && ok; ++q) {
        const long long r = r_begin + q;
        while (r >= pair_end) {
          ++pidx;
          pair_end = pair_row_off(pv, pidx + 1, I, p.I_shared);
        }
        const int e = pv.expert[pidx];
        if (e != cur_e) {
          cur_e = e;
          if (e < N) {
            const int slot = p.snap.expert_slot[e];
            if (slot < 0) {  // the host never asks for an expert without a slot; refuse rather than read out of range
              ok = false;
              break;
            }
            const uint32_t need = p.snap.need_gen[e];
            const uint32_t* flag = p.slot_ready + slot;
            if ((int32_t)(ld_acquire_sys(flag) - need) < 0) {
              const unsigned long long t0 = globaltimer_ns();
              while ((int32_t)(ld_acquire_sys(flag) - need) < 0) {
                if ((long long)(globaltimer_ns() - t0) > p.wait_limit_ns) {
                  ok = false;
                  break;
                }
                __nanosleep(64);
              }
              waited += globaltimer_ns() - t0;
            }
            asm volatile("fence.proxy.async;" ::: "memory");
            base = p.cache + (size_t)slot * p.slot_stride;
            mat_bytes = (size_t)I * row_bytes;
          } else {
            base = p.shared_w;
            mat_bytes = (size_t)p.I_shared * row_bytes;
          }
          if (!ok) break;
        }
        const long long i = r - pair_row_off(pv, pidx, I, p.I_shared);
        const int s = q % NS;
        if (q >= NS) {
          if (!mbar_wait(&s_empty[s], (uint32_t)((q / NS - 1) & 1), &s_abort, p.wait_limit_ns)) {
            ok = false;
            break;
          }
        }
        uint8_t* dst = smem + (size_t)s * entry_bytes;
        const uint8_t* src = base + (size_t)i * row_bytes;
        if (q == 0) TL(3);  // first copy issued
        mbar_expect_tx(&s_full[s], entry_bytes);
        bulk_g2s(dst, src, row_bytes, &s_full[s]);
        bulk_g2s(dst + row_bytes, src + mat_bytes, row_bytes, &s_full[s]);
        bulk_g2s(dst + 2 * row_bytes, src + 2 * mat_bytes, row_bytes, &s_full[s]);
      }
      TL(4);  // last copy issued
      if (waited && p.stats) atomicAdd(&p.stats->stall_ns, waited);
      if (!ok) {
        // a wait ran out: tell the consumers to stop, and the host
        atomicExch(&s_abort, 1);
        if (p.stats) atomicAdd(&p.stats->timeouts, 1ull);
        *p.mbox_status = 1u;
        __threadfence_system();
      }
    }
  } else {
    // ================= consumers
    float hreg[H_REGS ? NCH * 8 : 1];
    bool zero_seen = p.accumulate != 0;  // batched case: y must be zero before the first atomic add
    auto wait_zeroed = [&]() {
      if (zero_seen) return;
      const unsigned long long t0 = globaltimer_ns();
      while (ld_acquire_gpu_u64(p.zero_counter) < p.zero_target) {
        if ((long long)(globaltimer_ns() - t0) > p.wait_limit_ns) {
          *p.mbox_status = 1u;
          break;
        }
        __nanosleep(32);
      }
      zero_seen = true;
    };
    int cur_tok = -1, pidx = 0;
    long long pair_end = -1;
    float gate = 0.f;
    const float* hrow = p.hpost;
    if (n_my > 0) pidx = pair_of_row(pv, r_begin, I, p.I_shared) - 1, pair_end = r_begin;  // forces a lookup
    for (int q = warp; q < n_my; q += kConsumerWarps) {
      const long long r = r_begin + q;
      if (r >= pair_end) {
        while (r >= pair_end) {
          ++pidx;
          pair_end = pair_row_off(pv, pidx + 1, I, p.I_shared);
        }
        gate = pv.gate[pidx];
        const int t = pv.tok[pidx];
        if (t != cur_tok) {
          if (cur_tok >= 0) {
            // batched case: this warp moves to another token, flush its partial sums
            wait_zeroed();
            float4* y4 = reinterpret_cast<float4*>(p.y + (size_t)cur_tok * d);
#pragma unroll
            for (int c = 0; c < NCH; ++c) {
              const int col4 = (c * 32 + lane) * 2;
              atomicAdd(y4 + col4, make_float4(acc[c * 8 + 0], acc[c * 8 + 1], acc[c * 8 + 2], acc[c * 8 + 3]));
              atomicAdd(y4 + col4 + 1, make_float4(acc[c * 8 + 4], acc[c * 8 + 5], acc[c * 8 + 6], acc[c * 8 + 7]));
            }
#pragma unroll
            for (int i2 = 0; i2 < NCH * 8; ++i2) acc[i2] = 0.f;
          }
          cur_tok = t;
          hrow = p.hpost + (size_t)t * d;
          if (H_REGS) {
#pragma unroll
            for (int c = 0; c < NCH; ++c) {
              const float4 a = __ldg(reinterpret_cast<const float4*>(hrow) + (c * 32 + lane) * 2);
              const float4 b2 = __ldg(reinterpret_cast<const float4*>(hrow) + (c * 32 + lane) * 2 + 1);
              hreg[c * 8 + 0] = a.x; hreg[c * 8 + 1] = a.y; hreg[c * 8 + 2] = a.z; hreg[c * 8 + 3] = a.w;
              hreg[c * 8 + 4] = b2.x; hreg[c * 8 + 5] = b2.y; hreg[c * 8 + 6] = b2.z; hreg[c * 8 + 7] = b2.w;
            }
          }
        }
      }
      const int s = q % NS;
      if (!mbar_wait(&s_full[s], (uint32_t)((q / NS) & 1), &s_abort, p.wait_limit_ns)) {
        atomicExch(&s_abort, 1);
        break;
      }
      if (*(volatile int*)&s_abort) break;
      if (lane == 0 && q == 0) TL(5);                       // first row landed
      if (lane == 0 && q == n_my - 1) TL(6);                // last row landed
      const uint4* gs = reinterpret_cast<const uint4*>(smem + (size_t)s * entry_bytes);
      const uint4* us = gs + row_bytes / 16;
      const uint4* ds = us + row_bytes / 16;
      float g = 0.f, u = 0.f;
#pragma unroll
      for (int c = 0; c < NCH; ++c) {
        const uint4 gv = gs[c * 32 + lane];
        const uint4 uv = us[c * 32 + lane];
        float h0, h1, h2, h3, h4, h5, h6, h7;
        if (H_REGS) {
          h0 = hreg[c * 8 + 0]; h1 = hreg[c * 8 + 1]; h2 = hreg[c * 8 + 2]; h3 = hreg[c * 8 + 3];
          h4 = hreg[c * 8 + 4]; h5 = hreg[c * 8 + 5]; h6 = hreg[c * 8 + 6]; h7 = hreg[c * 8 + 7];
        } else {
          const float4 a = __ldg(reinterpret_cast<const float4*>(hrow) + (c * 32 + lane) * 2);
          const float4 b2 = __ldg(reinterpret_cast<const float4*>(hrow) + (c * 32 + lane) * 2 + 1);
          h0 = a.x; h1 = a.y; h2 = a.z; h3 = a.w; h4 = b2.x; h5 = b2.y; h6 = b2.z; h7 = b2.w;
        }
        g = fmaf(bf16lo(gv.x), h0, g); g = fmaf(bf16hi(gv.x), h1, g);
        g = fmaf(bf16lo(gv.y), h2, g); g = fmaf(bf16hi(gv.y), h3, g);
        g = fmaf(bf16lo(gv.z), h4, g); g = fmaf(bf16hi(gv.z), h5, g);
        g = fmaf(bf16lo(gv.w), h6, g); g = fmaf(bf16hi(gv.w), h7, g);
        u = fmaf(bf16lo(uv.x), h0, u); u = fmaf(bf16hi(uv.x), h1, u);
        u = fmaf(bf16lo(uv.y), h2, u); u = fmaf(bf16hi(uv.y), h3, u);
        u = fmaf(bf16lo(uv.z), h4, u); u = fmaf(bf16hi(uv.z), h5, u);
        u = fmaf(bf16lo(uv.w), h6, u); u = fmaf(bf16hi(uv.w), h7, u);
      }
      g = warp_sum(g);
      u = warp_sum(u);
      const float a = gate * (g / (1.f + expf(-g))) * u;
#pragma unroll
      for (int c = 0; c < NCH; ++c) {
        const uint4 dv = ds[c * 32 + lane];
        acc[c * 8 + 0] = fmaf(a, bf16lo(dv.x), acc[c * 8 + 0]);
        acc[c * 8 + 1] = fmaf(a, bf16hi(dv.x), acc[c * 8 + 1]);
        acc[c * 8 + 2] = fmaf(a, bf16lo(dv.y), acc[c * 8 + 2]);
        acc[c * 8 + 3] = fmaf(a, bf16hi(dv.y), acc[c * 8 + 3]);
        acc[c * 8 + 4] = fmaf(a, bf16lo(dv.z), acc[c * 8 + 4]);
        acc[c * 8 + 5] = fmaf(a, bf16hi(dv.z), acc[c * 8 + 5]);
        acc[c * 8 + 6] = fmaf(a, bf16lo(dv.w), acc[c * 8 + 6]);
        acc[c * 8 + 7] = fmaf(a, bf16hi(dv.w), acc[c * 8 + 7]);
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&s_empty[s]);
    }
    if (B > 1 && cur_tok >= 0) {
      // batched case: every warp adds its own partial sums (y was zeroed by all CTAs: wait for that)
      wait_zeroed();
      float4* y4 = reinterpret_cast<float4*>(p.y + (size_t)cur_tok * d);
#pragma unroll
      for (int c = 0; c < NCH; ++c) {
        const int col4 = (c * 32 + lane) * 2;
        atomicAdd(y4 + col4, make_float4(acc[c * 8 + 0], acc[c * 8 + 1], acc[c * 8 + 2], acc[c * 8 + 3]));
        atomicAdd(y4 + col4 + 1, make_float4(acc[c * 8 + 4], acc[c * 8 + 5], acc[c * 8 + 6], acc[c * 8 + 7]));
      }
    }
  }

  if (B > 1) return;

  // ---- B == 1: reduce the eight partial vectors in shared memory, then one vector atomic per float4
  __syncthreads();  // every ring entry has been consumed; the ring is free
  if (tid == 0) TL(7);
  float* red = reinterpret_cast<float*>(smem);
  if (warp < kConsumerWarps) {
    float4* dst = reinterpret_cast<float4*>(red + (size_t)warp * d);
#pragma unroll
    for (int c = 0; c < NCH; ++c) {
      const int col4 = (c * 32 + lane) * 2;
      dst[col4] = make_float4(acc[c * 8 + 0], acc[c * 8 + 1], acc[c * 8 + 2], acc[c * 8 + 3]);
      dst[col4 + 1] = make_float4(acc[c * 8 + 4], acc[c * 8 + 5], acc[c * 8 + 6], acc[c * 8 + 7]);
    }
  } else if (lane == 0 && !p.accumulate) {
    const unsigned long long t0 = globaltimer_ns();
    while (ld_acquire_gpu_u64(p.zero_counter) < p.zero_target) {
      if ((long long)(globaltimer_ns() - t0) > p.wait_limit_ns) {
        *p.mbox_status = 1u;
        break;
      }
      __nanosleep(32);
    }
  }
  __syncthreads();
  if (tid == 0) TL(8);
  if (n_my > 0 && !s_abort) {
    float4* y4 = reinterpret_cast<float4*>(p.y);
    for (int col4 = tid; col4 < d / 4; col4 += kFfnThreads) {
      float4 sacc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int w = 0; w < kConsumerWarps; ++w) {
        const float4 v = reinterpret_cast<const float4*>(red + (size_t)w * d)[col4];
        sacc.x += v.x; sacc.y += v.y; sacc.z += v.z; sacc.w += v.w;
      }
      atomicAdd(y4 + col4, sacc);
    }
  }
  if (tid == 0) TL(9);
}

#ifdef APEX_TIMELINE
extern "C" int apex_debug_read_timeline(unsigned long long* host, int n) {
  return (int)cudaMemcpyFromSymbol(host, g_timeline, sizeof(unsigned long long) * n);
}
#endif

template <int NCH>
static cudaError_t launch_ffn_t(const FfnParams& p, int n_sm, cudaStream_t s) {
  constexpr bool HR = NCH <= 8;
  constexpr uint32_t entry = 3 * NCH * 256 * 2;
  constexpr int NS = ring_stages(entry);
  const size_t smem = (size_t)NS * entry;
  static bool configured = false;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(moe_ffn_stream_kernel<NCH, HR>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    configured = true;
  }
  moe_ffn_stream_kernel<NCH, HR><<<n_sm, kFfnThreads, smem, s>>>(p);
  return cudaGetLastError();
}

bool ffn_shape_supported(int d) {
  switch (d) {
    case 256: case 512: case 768: case 1024: case 1536: case 2048: case 3072: case 4096:
      return true;
  }
  return false;
}

cudaError_t ffn_configure(int) { return cudaSuccess; }

cudaError_t launch_ffn(const FfnParams& p, int n_sm, cudaStream_t s) {
  switch (p.d) {
    case 256: return launch_ffn_t<1>(p, n_sm, s);
    case 512: return launch_ffn_t<2>(p, n_sm, s);
    case 768: return launch_ffn_t<3>(p, n_sm, s);
    case 1024: return launch_ffn_t<4>(p, n_sm, s);
    case 1536: return launch_ffn_t<6>(p, n_sm, s);
    case 2048: return launch_ffn_t<8>(p, n_sm, s);
    case 3072: return launch_ffn_t<12>(p, n_sm, s);
    case 4096: return launch_ffn_t<16>(p, n_sm, s);
  }
  return cudaErrorInvalidValue;
}

}  // namespace apex

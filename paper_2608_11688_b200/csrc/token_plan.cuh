// Execution set of one token (S6) and small warp helpers, shared by the batch-1 streaming kernel (every warp plans
// its CTA's token itself) and the batched plan kernel.
#ifndef APEX_TOKEN_PLAN_CUH
#define APEX_TOKEN_PLAN_CUH

#include "apex_internal.hpp"

namespace apex {

__device__ __forceinline__ unsigned long long warp_max_u64(unsigned long long v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const unsigned long long w = __shfl_xor_sync(0xffffffffu, v, o);
    v = w > v ? w : v;
  }
  return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
// Weight of a gated shared expert for one token: sigmoid(w_sg . h'), by a whole warp (every lane gets the value).
// d is a multiple of 128; lane-strided float4 loads, fused multiply-adds in ascending index order, xor tree.
__device__ __forceinline__ float shared_gate_weight(const float* __restrict__ w_sg, const float* __restrict__ hpost, int d, int lane) {
  float z = 0.f;
  for (int i = lane * 4; i < d; i += 128) {
    const float4 a = __ldg(reinterpret_cast<const float4*>(w_sg + i));
    const float4 b = __ldg(reinterpret_cast<const float4*>(hpost + i));
    z = fmaf(a.x, b.x, z);
    z = fmaf(a.y, b.y, z);
    z = fmaf(a.z, b.z, z);
    z = fmaf(a.w, b.w, z);
  }
  z = warp_sum(z);
  return 1.f / (1.f + expf(-z));
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

struct TokenLoads {
  int my_idx;          // idx[lane] for lane < k, else -1
  float al0, al1;      // alpha of experts lane, lane+32
  float z0, z1;        // logits of experts lane, lane+32 (stall-free mode only)
};
__device__ __forceinline__ TokenLoads load_token(const int32_t* __restrict__ idx, const float* __restrict__ z_r,
                                                 const float* __restrict__ alpha, int N, int k, int mode, int lane) {
  TokenLoads t;
  const int e0 = lane, e1 = lane + 32;
  t.my_idx = lane < k ? idx[lane] : -1;
  t.al0 = e0 < N ? alpha[e0] : 0.f;
  t.al1 = e1 < N ? alpha[e1] : 0.f;
  t.z0 = t.z1 = 0.f;
  if (mode == APEX_MODE_STALL_FREE) {
    t.z0 = e0 < N ? z_r[e0] : 0.f;
    t.z1 = e1 < N ? z_r[e1] : 0.f;
  }
  return t;
}
// Execution set from the routed set (Alg. 1 in stall-free mode; K~ = K_r otherwise).  z0, z1: logits of experts lane,
// lane + 32 (read in stall-free mode only).
__device__ __forceinline__ unsigned long long exec_set(unsigned long long kr, int mode, unsigned long long resident, float z0,
                                                       float z1, int lane) {
  const int e0 = lane, e1 = lane + 32;
  unsigned long long exec = kr;
  if (mode == APEX_MODE_STALL_FREE && (kr & ~resident) != 0ull) {
    const unsigned long long keep = kr & resident;
    const int n_missing = __popcll(kr & ~resident);
    const unsigned long long cand = resident & ~kr;
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
    const bool s1 = ((cand >> e1) & 1) && r1 < n_missing;
    const unsigned b0 = __ballot_sync(0xffffffffu, s0), b1 = __ballot_sync(0xffffffffu, s1);
    exec = keep | (((unsigned long long)b1 << 32) | b0);
  }
  return exec;
}
// Gates of the executed experts: alpha_e / sum over K~ (norm_topk) or alpha_e; 0 for the others.
__device__ __forceinline__ void exec_gates(unsigned long long exec, float al0, float al1, int norm_topk, int lane, float* g0,
                                           float* g1) {
  const bool x0 = (exec >> lane) & 1, x1 = (exec >> (lane + 32)) & 1;
  const float a0 = x0 ? al0 : 0.f, a1 = x1 ? al1 : 0.f;
  float denom = 1.f;
  if (norm_topk) denom = warp_sum(a0 + a1);
  *g0 = a0 / denom;
  *g1 = a1 / denom;
}
__device__ __forceinline__ TokenPlan plan_token(const TokenLoads& t, int mode, int norm_topk, unsigned long long resident,
                                                int lane) {
  const int my_idx = t.my_idx;
  unsigned lo = 0, hi = 0;
  if (my_idx >= 0) {
    if (my_idx < 32)
      lo = 1u << my_idx;
    else
      hi = 1u << (my_idx - 32);
  }
  lo = __reduce_or_sync(0xffffffffu, lo);
  hi = __reduce_or_sync(0xffffffffu, hi);
  TokenPlan tp;
  tp.kr_mask = ((unsigned long long)hi << 32) | lo;
  tp.exec_mask = exec_set(tp.kr_mask, mode, resident, t.z0, t.z1, lane);
  exec_gates(tp.exec_mask, t.al0, t.al1, norm_topk, lane, &tp.g0, &tp.g1);
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

__device__ __forceinline__ int nth_set_bit64(unsigned long long m, int n) {
  for (int i = 0; i < n; ++i) m &= m - 1;
  return __ffsll((long long)m) - 1;
}

}  // namespace apex

#endif  // APEX_TOKEN_PLAN_CUH

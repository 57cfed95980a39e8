// Device code shared by the router kernels and the persistent decode kernel: the fixed-order warp reductions, the
// budget selection of one token (Eq. (8), (9), (1)) and the per-token epilogue of a router (softmax, ranking, top-k,
// metrics of Eq. (2), (3)).
#ifndef APEX_ROUTER_COMMON_CUH
#define APEX_ROUTER_COMMON_CUH

#include "apex_internal.hpp"

#ifndef RTL
#define RTL(i) do { } while (0)
#endif

namespace apex {

__device__ __forceinline__ float warp_sum_tree(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max_tree(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ int warp_max_int(int v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = max(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// One cluster per token.  CTA r of the cluster owns experts r*wpc .. r*wpc+wpc-1, one warp per
// expert; the logits are gathered in the leader CTA's shared memory through distributed shared
// memory, and the leader's first warp does softmax, ranking, top-k and (for the gate) the
// per-step metrics of Eq. (2)-(3).
// Budget selection for one token by one warp (Eq. (8), (9) in the logit domain; Eq. (1)).
// Lane l holds positions l and l+32 of the ranked list E: pj = expert at that position, x = its
// prefetch probability (so x is the prefetch distribution in descending order).
//   s = w.x   (lane partial: position l then l+32 with fused multiply-adds, then the xor tree)
//   delta_hat = first delta with theta_delta - s >= logit(tau), capped to C - k
//   K_p = first k + delta_hat experts of E
// The budget itself (uniform over the warp): returns delta_hat after the cap, *uncapped receives it before.
// w0, w1: w at positions lane, lane + 32; th0, th1: theta at lane, lane + 32 (anything where there is none).
__device__ __forceinline__ int select_budget_vals(float w0, float w1, float th0, float th1, float t_tau, int force, int N, int k,
                                                  int C, int lane, float x0, float x1, int* uncapped) {
  float part = 0.f;
  if (lane < N) part = fmaf(w0, x0, part);
  if (lane + 32 < N) part = fmaf(w1, x1, part);
  const float sdot = warp_sum_tree(part);
  const int nth = N - k + 1;
  const bool pass0 = lane < nth && (th0 - sdot >= t_tau);
  const bool pass1 = lane + 32 < nth && (th1 - sdot >= t_tau);
  const unsigned m0 = __ballot_sync(0xffffffffu, pass0), m1 = __ballot_sync(0xffffffffu, pass1);
  int d_hat = m0 ? (__ffs(m0) - 1) : (m1 ? 32 + __ffs(m1) - 1 : N - k);
  if (force == 1) d_hat = 0;
  if (force == 2) d_hat = N - k;
  *uncapped = d_hat;
  return min(d_hat, C - k);
}
__device__ __forceinline__ int select_budget(const float* __restrict__ w, const float* __restrict__ theta, float t_tau, int force,
                                             int N, int k, int C, int lane, float x0, float x1, int* uncapped) {
  const int nth = N - k + 1;
  const float w0 = lane < N ? __ldg(w + lane) : 0.f, w1 = lane + 32 < N ? __ldg(w + lane + 32) : 0.f;
  const float th0 = lane < nth ? __ldg(theta + lane) : 0.f, th1 = lane + 32 < nth ? __ldg(theta + lane + 32) : 0.f;
  return select_budget_vals(w0, w1, th0, th1, t_tau, force, N, k, C, lane, x0, x1, uncapped);
}

__device__ __forceinline__ void select_token(const SelectParams& p, int b, int lane, int pj0, int pj1, float x0, float x1) {
  const int N = p.N, k = p.k, C = p.C;
  int uncapped;
  const int d_hat = select_budget(p.w, p.theta, p.t_tau, p.force, N, k, C, lane, x0, x1, &uncapped);
  const int ncand = k + d_hat;
  // candidates in rank order, padded with -1
  const bool in0 = lane < ncand, in1 = lane + 32 < ncand;
  if (lane < C) {
    const int v = in0 ? pj0 : -1;
    p.cand_out[(size_t)b * C + lane] = v;
    p.mbox_cand[(size_t)b * C + lane] = v;
  }
  if (lane + 32 < C) {
    const int v = in1 ? pj1 : -1;
    p.cand_out[(size_t)b * C + lane + 32] = v;
    p.mbox_cand[(size_t)b * C + lane + 32] = v;
  }
  // the candidate set as a 64-bit mask
  unsigned lo = 0, hi = 0;
  if (in0) { if (pj0 < 32) lo |= 1u << pj0; else hi |= 1u << (pj0 - 32); }
  if (in1) { if (pj1 < 32) lo |= 1u << pj1; else hi |= 1u << (pj1 - 32); }
  lo = __reduce_or_sync(0xffffffffu, lo);
  hi = __reduce_or_sync(0xffffffffu, hi);
  if (lane == 0) {
    p.ncand_out[b] = ncand;
    p.ncand_keep[b] = ncand;
    p.mbox_ncand[b] = ncand;
    if (p.stats) {
      atomicAdd(&p.stats->tokens, 1ull);
      atomicAdd(&p.stats->sum_delta_hat, (unsigned long long)d_hat);
      atomicAdd(&p.stats->sum_ncand, (unsigned long long)ncand);
      atomicAdd(&p.stats->capped, (unsigned long long)(uncapped > d_hat ? 1 : 0));
      atomicAdd(&p.stats->near_full, (unsigned long long)(2 * ncand > N ? 1 : 0));
    }
  }
  if (p.B == 1) {
    // one token: the host needs only the set.  Mask, count and sequence number travel in ONE aligned
    // 16-byte store, so no system-scope fence sits on the kernel's critical path.  (The ranked list
    // above is advisory for the host: it is used for the issue order only if it matches the mask.)
    if (lane == 0) {
      asm volatile("st.global.v4.u32 [%0], {%1, %2, %3, %4};" ::"l"(p.mbox_rec), "r"(lo), "r"(hi), "r"((unsigned)ncand),
                   "r"(p.seq_value)
                   : "memory");
    }
    return;
  }
  __threadfence_system();
  __syncwarp();
  if (lane == 0) {
    const unsigned long long old = atomicAdd(p.done_counter, 1ull);
    if (old + 1 == p.done_target) {
      __threadfence_system();
      *p.mbox_seq = p.seq_value;
    }
  }
}


// Softmax, ranking, top-k and the per-token outputs of one token by one warp (lanes own experts lane and lane+32),
// from the token's N logits in shared memory; then either the budget selection (prefetch router, fused launch) or
// the metrics of Eq. (2), (3) against the prefetch stage (gate).  qs, pis, posp: this warp's scratch, 64 entries each.
// Softmax over the N logits in shared memory and the rank of this lane's two experts (e0 = lane, e1 = lane + 32):
// rank = number of experts ordered before it by (value descending, index ascending).
struct RankedLogits {
  float z0, z1;  // logits (most negative float where the lane has no expert)
  float q0, q1;  // softmax
  int r0, r1;    // ranks
};
// the two halves of softmax_and_rank, for callers that need the ranks before the probabilities
__device__ __forceinline__ void rank_lane_logits(const float* zs, int N, int lane, RankedLogits* R) {
  const int e0 = lane, e1 = lane + 32;
  const float NEG = -3.402823466e38f;
  R->z0 = e0 < N ? zs[e0] : NEG;
  R->z1 = e1 < N ? zs[e1] : NEG;
  R->r0 = 0;
  R->r1 = 0;
#pragma unroll 8
  for (int f = 0; f < N; ++f) {
    const float zf = zs[f];
    R->r0 += (zf > R->z0 || (zf == R->z0 && f < e0)) ? 1 : 0;
    R->r1 += (zf > R->z1 || (zf == R->z1 && f < e1)) ? 1 : 0;
  }
}
__device__ __forceinline__ void softmax_lane_logits(int N, int lane, RankedLogits* R) {
  const int e0 = lane, e1 = lane + 32;
  const float m = warp_max_tree(fmaxf(R->z0, R->z1));
  const float x0 = e0 < N ? expf(R->z0 - m) : 0.f;
  const float x1 = e1 < N ? expf(R->z1 - m) : 0.f;
  const float sum = warp_sum_tree(x0 + x1);
  R->q0 = x0 / sum;
  R->q1 = x1 / sum;
}
__device__ __forceinline__ RankedLogits softmax_and_rank(const float* zs, int N, int lane) {
  RankedLogits R;
  rank_lane_logits(zs, N, lane, &R);
  softmax_lane_logits(N, lane, &R);
  return R;
}

__device__ __forceinline__ void router_epilogue(const RouterParams& p, int b, int lane, const float* zs, float* qs, int* pis,
                                                int* posp) {
  const int N = p.N, k = p.k;
  const int e0 = lane, e1 = lane + 32;
  const RankedLogits R = softmax_and_rank(zs, N, lane);
  const float z0 = R.z0, z1 = R.z1, q0 = R.q0, q1 = R.q1;
  const int r0 = R.r0, r1 = R.r1;
  const size_t row = (size_t)b * N;
  if (e0 < N) {
    p.z_out[row + e0] = z0;
    p.q_out[row + e0] = q0;
    if (p.pi_out) p.pi_out[row + r0] = e0;
    if (p.topk_out && r0 < k) p.topk_out[(size_t)b * k + r0] = e0;
  }
  if (e1 < N) {
    p.z_out[row + e1] = z1;
    p.q_out[row + e1] = q1;
    if (p.pi_out) p.pi_out[row + r1] = e1;
    if (p.topk_out && r1 < k) p.topk_out[(size_t)b * k + r1] = e1;
  }
  RTL(4);
  if (p.fuse_select) {
    // prefetch router and budget selection in one launch: the ranked list goes through shared memory
    if (e0 < N) { qs[e0] = q0; pis[r0] = e0; }
    if (e1 < N) { qs[e1] = q1; pis[r1] = e1; }
    __syncwarp();
    const int pj0 = lane < N ? pis[lane] : -1, pj1 = lane + 32 < N ? pis[lane + 32] : -1;
    const float x0 = pj0 >= 0 ? qs[pj0] : 0.f, x1 = pj1 >= 0 ? qs[pj1] : 0.f;
    select_token(p.sel, b, lane, pj0, pj1, x0, x1);
    RTL(5);
    return;
  }
  if (!p.topk_out || !p.stats) return;

  // ---- gate epilogue: metrics of this token against the prefetch stage (Eq. (2), (3))
  const bool in0 = e0 < N && r0 < k, in1 = e1 < N && r1 < k;
  {
    int dstar = 0, hitsP = 0, have_pred = 0;
    if (p.pi_pred) {
      have_pred = 1;
      if (e0 < N) posp[__ldg(p.pi_pred + row + e0)] = e0;  // position of expert pi[j] in E is j
      if (e1 < N) posp[__ldg(p.pi_pred + row + e1)] = e1;
      __syncwarp();
      const int nc = __ldg(p.ncand_pred + b);
      const int pos0 = in0 ? posp[e0] : -1, pos1 = in1 ? posp[e1] : -1;
      dstar = warp_max_int(max(pos0, pos1)) + 1 - k;
      hitsP = __popc(__ballot_sync(0xffffffffu, in0 && pos0 < nc)) + __popc(__ballot_sync(0xffffffffu, in1 && pos1 < nc));
    }
    if (lane == 0) {
      atomicAdd(&p.stats->routed, (unsigned long long)k);
      if (have_pred) {
        atomicAdd(&p.stats->sum_delta_star, (unsigned long long)dstar);
        atomicAdd(&p.stats->hits_P, (unsigned long long)hitsP);
        atomicAdd(&p.stats->covered, (unsigned long long)(hitsP == k ? 1 : 0));
      }
    }
  }
  RTL(5);
}

}  // namespace apex

#endif  // APEX_ROUTER_COMMON_CUH

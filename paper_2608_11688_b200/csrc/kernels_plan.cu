// ffn_plan_kernel: the execution sets of a batched step (B > 1) and the (expert, token) pair list sorted by expert,
// for the tensor-core grouped GEMMs and for the per-pair streaming kernel.
#include <cooperative_groups.h>

#include "apex_internal.hpp"
#include "ptx.cuh"
#include "timeline.cuh"
#include "token_plan.cuh"

namespace cg = cooperative_groups;

namespace apex {

// ---------------------------------------------------------------- batched plan (B > 1)
// A cluster of ceil(B / 32) CTAs (at most 8) of 32 warps.  Phase A: every warp of the cluster plans one token (planning
// a token costs a warp 2-3 us of dependent latency, so eight tokens per warp on one SM were 16 us at B = 256) and puts
// its execution mask and gates into the leader CTA's shared memory through distributed shared memory.  Phase B, leader
// CTA only: warp w owns experts w and w+32 and gathers the tokens that execute them with ballots, so the pair list is
// sorted by (expert, token).  Shared-expert pairs (expert id N) follow.
constexpr int kPlanMaxCtas = APEX_MAX_BATCH / 32;
static_assert(kPlanMaxCtas <= 8, "one token per warp needs a cluster of at most 8 CTAs");

#ifdef APEX_TIMELINE
#define PTL(i) do { if (threadIdx.x == 0) g_timeline[1000 * 16 + (i)] = globaltimer_ns_raw(); } while (0)
#else
#define PTL(i) do { } while (0)
#endif

__global__ void __launch_bounds__(1024) ffn_plan_kernel(const FfnParams p) {
  constexpr int TOK_PER_WARP = 1;
  cg::cluster_group cluster = cg::this_cluster();
  const unsigned crank = cluster.block_rank();
  __shared__ unsigned long long s_exec[APEX_MAX_BATCH];
  __shared__ float s_pgate[APEX_MAX_BATCH][APEX_MAX_TOPK];  // gate of the j-th executed expert of each token
  __shared__ float s_sgate[APEX_MAX_BATCH];                 // weight of the shared expert for each token (gated variant)
  __shared__ int s_count[APEX_MAX_EXPERTS + 1];
  __shared__ int s_off[APEX_MAX_EXPERTS + 2];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarp = blockDim.x >> 5;
  const int N = p.N, k = p.k, B = p.B;
  int my_subst = 0, my_hits = 0;
  // the leader's copies of the per-token results
  unsigned long long* l_exec = cluster.map_shared_rank(&s_exec[0], 0);
  float* l_pgate = cluster.map_shared_rank(&s_pgate[0][0], 0);
  float* l_sgate = cluster.map_shared_rank(&s_sgate[0], 0);
  SPAN_BEGIN();
  PTL(0);
  TokenLoads tls[TOK_PER_WARP];
#pragma unroll
  for (int j = 0; j < TOK_PER_WARP; ++j) {
    const int b = (int)crank * nwarp + warp + j * nwarp * (int)cluster.num_blocks();
    if (b < B) tls[j] = load_token(p.idx + (size_t)b * k, p.z_r + (size_t)b * N, p.alpha + (size_t)b * N, N, k, p.mode, lane);
  }
#pragma unroll
  for (int j = 0; j < TOK_PER_WARP; ++j) {
    const int b = (int)crank * nwarp + warp + j * nwarp * (int)cluster.num_blocks();
    if (b >= B) break;
    const TokenLoads& tl = tls[j];
    const TokenPlan tp = plan_token(tl, p.mode, p.norm_topk, p.snap.resident_mask, lane);
    store_token_plan(tp, lane, k, p.plan_exec_idx + (size_t)b * k, p.plan_exec_gate + (size_t)b * k, nullptr);
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
      my_hits += __popcll(tp.kr_mask & p.snap.resident_mask);
    }
    if (lane == 0) l_exec[b] = tp.exec_mask;
    if (p.run_shared && p.shared_gate) {
      const float sg = shared_gate_weight(p.shared_gate, p.hpost + (size_t)b * p.d, p.d, lane);
      if (lane == 0) l_sgate[b] = sg;
    }
    {
      const int e0 = lane, e1 = lane + 32;
      if ((tp.exec_mask >> e0) & 1) {
        const int pos = __popcll(tp.exec_mask & ((1ull << e0) - 1ull));
        if (pos < APEX_MAX_TOPK) l_pgate[b * APEX_MAX_TOPK + pos] = tp.g0;
      }
      if ((tp.exec_mask >> e1) & 1) {
        const int pos = __popcll(tp.exec_mask & ((1ull << e1) - 1ull));
        if (pos < APEX_MAX_TOPK) l_pgate[b * APEX_MAX_TOPK + pos] = tp.g1;
      }
    }
  }
  if (p.post_exec && lane == 0 && my_subst && p.stats) atomicAdd(&p.stats->substitutions, (unsigned long long)my_subst);
  if (p.post_exec && lane == 0 && my_hits && p.stats) atomicAdd(&p.stats->hits_R, (unsigned long long)my_hits);
  cluster.sync();  // every token's mask and gates are in the leader's shared memory
  if (crank != 0) return;
  PTL(1);
  // ---- phase B, counts: warp w counts the tokens of experts w and w + 32
  for (int e = warp; e < N; e += nwarp) {
    int c = 0;
    if ((p.run_mask >> e) & 1)
      for (int b0 = 0; b0 < B; b0 += 32) {
        const int b = b0 + lane;
        c += __popc(__ballot_sync(0xffffffffu, b < B && ((s_exec[b] >> e) & 1)));
      }
    if (lane == 0) s_count[e] = c;
  }
  __syncthreads();
  PTL(2);
  if (warp == 0) {
    // exclusive prefix over the experts (lane owns experts lane and lane + 32), then the group table
    // of the tensor-core path: one group per executed expert, then the shared expert
    const int c0 = lane < N ? s_count[lane] : 0, c1 = lane + 32 < N ? s_count[lane + 32] : 0;
    int i0 = c0, i1 = c1;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int u0 = __shfl_up_sync(0xffffffffu, i0, o), u1 = __shfl_up_sync(0xffffffffu, i1, o);
      if (lane >= o) {
        i0 += u0;
        i1 += u1;
      }
    }
    const int tot0 = __shfl_sync(0xffffffffu, i0, 31), acc = tot0 + __shfl_sync(0xffffffffu, i1, 31);
    const int off0 = i0 - c0, off1 = tot0 + i1 - c1;
    if (lane < N) s_off[lane] = off0;
    if (lane + 32 < N) s_off[lane + 32] = off1;
    const unsigned g0m = __ballot_sync(0xffffffffu, c0 > 0), g1m = __ballot_sync(0xffffffffu, c1 > 0);
    const int ng_routed = __popc(g0m) + __popc(g1m);
    if (c0 > 0) {
      const int gi = __popc(g0m & ((1u << lane) - 1u));
      p.grp[4 + 3 * gi] = lane;
      p.grp[5 + 3 * gi] = off0;
      p.grp[6 + 3 * gi] = c0;
    }
    if (c1 > 0) {
      const int gi = __popc(g0m) + __popc(g1m & ((1u << lane) - 1u));
      p.grp[4 + 3 * gi] = lane + 32;
      p.grp[5 + 3 * gi] = off1;
      p.grp[6 + 3 * gi] = c1;
    }
    if (lane == 0) {
      s_off[N] = acc;  // routed pairs
      p.n_pairs[0] = acc + (p.run_shared ? B : 0);
      p.grp[0] = ng_routed;
      if (p.run_shared) {
        p.grp[4 + 3 * ng_routed] = N;
        p.grp[5 + 3 * ng_routed] = acc;
        p.grp[6 + 3 * ng_routed] = B;
      }
      p.grp[1] = ng_routed + (p.run_shared ? 1 : 0);
    }
  }
  __syncthreads();
  PTL(3);
  // ---- phase B, placement: token b of expert e goes to s_off[e] + (number of earlier tokens of e)
  for (int e = warp; e < N; e += nwarp) {
    if (s_count[e] == 0) continue;
    int o = s_off[e];
    for (int b0 = 0; b0 < B; b0 += 32) {
      const int b = b0 + lane;
      const bool has = b < B && ((s_exec[b] >> e) & 1);
      const unsigned m = __ballot_sync(0xffffffffu, has);
      if (has) {
        const int at = o + __popc(m & ((1u << lane) - 1u));
        const int pos = __popcll(s_exec[b] & ((1ull << e) - 1ull));
        p.pair_tok[at] = b;
        p.pair_expert[at] = e;
        p.pair_gate[at] = s_pgate[b][pos];
      }
      o += __popc(m);
    }
  }
  if (p.run_shared) {
    const int base = s_off[N];
    for (int b = threadIdx.x; b < B; b += blockDim.x) {
      p.pair_tok[base + b] = b;
      p.pair_expert[base + b] = N;
      p.pair_gate[base + b] = p.shared_gate ? s_sgate[b] : 1.f;
    }
  }
  PTL(4);
  // The routed and the execution sets go to the host mailbox last, as whole lines from consecutive
  // threads (a 4-byte store per lane and token from inside the planning loop cost 2 us per token).
  if (p.post_exec) {
    for (int t = threadIdx.x; t < B * k; t += blockDim.x) {
      const int b = t / k, j = t - b * k;
      const unsigned long long m = s_exec[b];
      p.mbox_exec[t] = j < __popcll(m) ? nth_set_bit64(m, j) : -1;
      p.mbox_kr[t] = p.idx[t];
    }
  }
  if (p.post_exec) {
    // the barrier orders every thread's mailbox stores before thread 0's system-scope fence
    // (fences are cumulative), which orders them before the sequence number
    __syncthreads();
    PTL(5);
    if (threadIdx.x == 0) {
      __threadfence_system();
      *p.mbox_seq = p.seq_value;
    }
  }
  PTL(6);
  SPAN_END(6);
}

cudaError_t launch_ffn_plan(const FfnParams& p, cudaStream_t s) {
  int n_cta = (p.B + 31) / 32;
  n_cta = n_cta < 1 ? 1 : (n_cta > kPlanMaxCtas ? kPlanMaxCtas : n_cta);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(n_cta, 1, 1);
  cfg.blockDim = dim3(1024, 1, 1);
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = n_cta;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, ffn_plan_kernel, p);
}

}  // namespace apex

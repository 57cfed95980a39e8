// Router kernels: the prefetch router and the exact gate share one GEMV + softmax + ranking kernel
// (Sec. IV-D: the prefetch router mirrors the original router), plus the budget selection of
// Eq. (8)-(9) and the stand-in attention stream that provides the hiding window of Eq. (12).
//
// Reduction order (fixed, so results are reproducible run to run): a dot product of length d is
// split over the 32 lanes of one warp; lane l accumulates float4 columns l, l+32, l+64, ... in
// ascending order with fused multiply-adds (x, y, z, w of each float4 in that order), then the 32
// partial sums are combined by a 5-step xor-shuffle tree (offsets 16, 8, 4, 2, 1).
#include <cooperative_groups.h>

#include <mutex>

#include "apex_internal.hpp"
#include "ptx.cuh"

namespace apex {
#ifdef APEX_TIMELINE
__device__ long long g_router_tl[16];
#define RTL(i) do { if (blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0) g_router_tl[i] = clock64(); } while (0)
extern "C" int apex_debug_read_router_tl(long long* host) { return (int)cudaMemcpyFromSymbol(host, g_router_tl, sizeof(long long) * 16); }
#else
#define RTL(i) do { } while (0)
#endif
}  // namespace apex

#include "router_common.cuh"

namespace cg = cooperative_groups;

namespace apex {

constexpr int kRouterMaxVec = 32;  // float4 per lane of one weight row: d <= 4096


__global__ void __launch_bounds__(256) router_kernel(const RouterParams p) {
  SPAN_BEGIN();
  cg::cluster_group cluster = cg::this_cluster();
  const unsigned crank = cluster.block_rank();
  const int b = blockIdx.y;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  __shared__ float zs[APEX_MAX_EXPERTS];
  __shared__ float qs[APEX_MAX_EXPERTS];
  __shared__ int pis[APEX_MAX_EXPERTS];
  __shared__ int posp[APEX_MAX_EXPERTS];
  __shared__ float4 xs[kRouterMaxVec * 32];

  // The router weights are parameters, not results of the preceding kernel: this warp's row is
  // loaded into registers before the dependency wait, so its DRAM latency hides behind that kernel.
  const int e = (int)crank * p.warps_per_cta + warp;
  const bool active = warp < p.warps_per_cta && e < p.N;
  const int nv = p.d >> 2;
  float4 wreg[kRouterMaxVec];
  float bias_e = 0.f;
  if (active) {
    const float4* __restrict__ Wrow = reinterpret_cast<const float4*>(p.W + (size_t)e * p.d);
#pragma unroll
    for (int i = 0; i < kRouterMaxVec; ++i) {
      const int c = i * 32 + lane;
      if (c < nv) wreg[i] = __ldg(Wrow + c);
    }
    if (p.bias) bias_e = __ldg(p.bias + e);
  }
  RTL(0);
  pdl_wait();               // everything queued before this kernel is complete: x may be read
  pdl_launch_dependents();  // the next kernel may begin its own prologue
  RTL(1);

  // x is staged in shared memory by the whole CTA in one round of loads
  {
    const float4* __restrict__ xv = reinterpret_cast<const float4*>(p.x + (size_t)b * p.d);
    for (int c = threadIdx.x; c < nv; c += blockDim.x) xs[c] = __ldg(xv + c);
  }
  __syncthreads();
  if (active) {
    float acc = 0.f;
#pragma unroll
    for (int i = 0; i < kRouterMaxVec; ++i) {
      const int c = i * 32 + lane;
      if (c < nv) {
        const float4 x = xs[c];
        acc = fmaf(wreg[i].x, x.x, acc);
        acc = fmaf(wreg[i].y, x.y, acc);
        acc = fmaf(wreg[i].z, x.z, acc);
        acc = fmaf(wreg[i].w, x.w, acc);
      }
    }
    acc = warp_sum_tree(acc);
    if (lane == 0) {
      const float z = acc + bias_e;
      float* dst = cluster.map_shared_rank(zs, 0);
      dst[e] = z;
    }
  }
  RTL(2);
  cluster.sync();
  RTL(3);
  if (crank != 0 || warp != 0) return;

  // ---- leader warp
  router_epilogue(p, b, lane, zs, qs, pis, posp);
  SPAN_END((p.fuse_select || !p.topk_out || !p.stats) ? 1 : 4);
}

// The same for a batch (B > 1).  A cluster keeps its weight rows in registers and walks over groups of
// kRouterTok tokens: the group's hidden states (1 to kRouterTok tokens, chosen by the launcher) are staged in shared memory once, every warp takes the dot
// products of its expert's row with all of them (per token the arithmetic and its order are those of
// router_kernel), the logits go to the leader CTA, one cluster barrier per group, and warp t of the leader
// CTA finishes token t of the group.  The logits are double-buffered: a buffer is written again two groups
// later, after the barrier of the group in between, which the leader's warps reach only when they are done
// reading it.  W_r is read once per cluster instead of once per token.
constexpr int kRouterTok = 8;  // tokens per group = warps of a CTA

__global__ void __launch_bounds__(256) router_batched_kernel(const RouterParams p) {
  SPAN_BEGIN();
  cg::cluster_group cluster = cg::this_cluster();
  const unsigned crank = cluster.block_rank();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  __shared__ float zs[2][kRouterTok][APEX_MAX_EXPERTS];
  __shared__ float qs[kRouterTok][APEX_MAX_EXPERTS];
  __shared__ int pis[kRouterTok][APEX_MAX_EXPERTS];
  __shared__ int posp[kRouterTok][APEX_MAX_EXPERTS];
  extern __shared__ float4 xs_dyn[];  // [kRouterTok][d / 4]

  const int e = (int)crank * p.warps_per_cta + warp;
  const bool active = warp < p.warps_per_cta && e < p.N;
  const int nv = p.d >> 2;
  float4 wreg[kRouterMaxVec];
  float bias_e = 0.f;
  if (active) {
    const float4* __restrict__ Wrow = reinterpret_cast<const float4*>(p.W + (size_t)e * p.d);
#pragma unroll
    for (int i = 0; i < kRouterMaxVec; ++i) {
      const int c = i * 32 + lane;
      // volatile: under this kernel's register pressure the compiler would otherwise sink the loads into the
      // token loop, behind the dependency wait and once per group
      if (c < nv)
        asm volatile("ld.global.nc.v4.f32 {%0, %1, %2, %3}, [%4];"
                     : "=f"(wreg[i].x), "=f"(wreg[i].y), "=f"(wreg[i].z), "=f"(wreg[i].w)
                     : "l"(Wrow + c));
    }
    if (p.bias) bias_e = __ldg(p.bias + e);
  }
  RTL(0);
  pdl_wait();
  pdl_launch_dependents();
  RTL(1);

  const int tpg = p.tok_per_group;  // tokens per group, 1..kRouterTok
  const int n_groups = (p.B + tpg - 1) / tpg;
  int buf = 0;
  for (int g = blockIdx.y; g < n_groups; g += gridDim.y, buf ^= 1) {
    const int b0 = g * tpg;
    const int nt = p.B - b0 < tpg ? p.B - b0 : tpg;
    {
      // the group's rows of x are contiguous: one linear copy.  (Every warp of this CTA passed the cluster
      // barrier of the previous group after its last read of xs.)
      // Asynchronous 16-byte copies, all in flight at once: a loop of load-then-store would pay the memory
      // latency once per trip (up to 32 trips per thread).
      const float4* __restrict__ xv = reinterpret_cast<const float4*>(p.x + (size_t)b0 * p.d);
      for (int c = threadIdx.x; c < nt * nv; c += blockDim.x)
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(xs_dyn + c)), "l"(xv + c) : "memory");
      asm volatile("cp.async.wait_all;" ::: "memory");
    }
    __syncthreads();
    RTL(2);
    if (active) {
      float acc[kRouterTok];
#pragma unroll
      for (int t = 0; t < kRouterTok; ++t) acc[t] = 0.f;
      if (nt == kRouterTok) {  // full group: no per-token predicate inside the unrolled loops
#pragma unroll
        for (int i = 0; i < kRouterMaxVec; ++i) {
          const int c = i * 32 + lane;
          if (c < nv) {
#pragma unroll
            for (int t = 0; t < kRouterTok; ++t) {
              const float4 x = xs_dyn[t * nv + c];
              acc[t] = fmaf(wreg[i].x, x.x, acc[t]);
              acc[t] = fmaf(wreg[i].y, x.y, acc[t]);
              acc[t] = fmaf(wreg[i].z, x.z, acc[t]);
              acc[t] = fmaf(wreg[i].w, x.w, acc[t]);
            }
          }
        }
      }
      float mine = 0.f;  // lane t delivers token t
      if (nt == kRouterTok) {
#pragma unroll
        for (int t = 0; t < kRouterTok; ++t) {
          const float v = warp_sum_tree(acc[t]);
          if (lane == t) mine = v;
        }
      } else {  // partial group: token by token
        for (int t = 0; t < nt; ++t) {
          float a = 0.f;
#pragma unroll
          for (int i = 0; i < kRouterMaxVec; ++i) {
            const int c = i * 32 + lane;
            if (c < nv) {
              const float4 x = xs_dyn[t * nv + c];
              a = fmaf(wreg[i].x, x.x, a);
              a = fmaf(wreg[i].y, x.y, a);
              a = fmaf(wreg[i].z, x.z, a);
              a = fmaf(wreg[i].w, x.w, a);
            }
          }
          a = warp_sum_tree(a);
          if (lane == t) mine = a;
        }
      }
      if (lane < nt) {
        float* dst = cluster.map_shared_rank(&zs[0][0][0], 0);
        dst[(buf * kRouterTok + lane) * APEX_MAX_EXPERTS + e] = mine + bias_e;
      }
    }
    RTL(3);
    cluster.sync();
    RTL(4);
    if (crank == 0 && warp < nt) router_epilogue(p, b0 + warp, lane, zs[buf][warp], qs[warp], pis[warp], posp[warp]);
  }
  RTL(6);
  SPAN_END((p.fuse_select || !p.topk_out || !p.stats) ? 1 : 4);
}

cudaError_t launch_router(const RouterParams& p, cudaStream_t s) {
  // cluster size: power of two, up to 8 CTAs of up to 8 warps
  int csize = 1;
  while (csize < 8 && csize * 8 < p.N) csize <<= 1;
  RouterParams q = p;
  q.warps_per_cta = (p.N + csize - 1) / csize;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(csize, p.B, 1);
  cfg.blockDim = dim3(256, 1, 1);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = s;
  const bool batched = p.B > 1;
  if (batched) {
    // one cluster per group of tokens, at most as many clusters as fit the GPU at one CTA per SM (the weight
    // rows in registers allow no more); further groups are walked by the same clusters
    static int n_sm_of[kMaxDevices];
    static bool configured[kMaxDevices];
    static std::mutex setup_mutex;  // contexts of several host threads (and the context-free gate) share this set-up
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    int n_sm = 0;
    {
      std::lock_guard<std::mutex> lock(setup_mutex);
      if (!configured[dev]) {
        if ((e = cudaDeviceGetAttribute(&n_sm_of[dev], cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
        if ((e = cudaFuncSetAttribute(router_batched_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      kRouterTok * kRouterMaxVec * 32 * (int)sizeof(float4))) != cudaSuccess)
          return e;
        configured[dev] = true;
      }
      n_sm = n_sm_of[dev];
    }
    int resident = n_sm / csize;
    if (resident < 1) resident = 1;
    // small batches spread over the clusters (a token per cluster while they last); large ones fill the groups,
    // because a group costs a barrier and a round of shared-memory reads of all its tokens per warp
    int tpg = (p.B + resident - 1) / resident;
    tpg = tpg > kRouterTok ? kRouterTok : tpg;
    q.tok_per_group = tpg;
    const int n_groups = (p.B + tpg - 1) / tpg;
    cfg.gridDim = dim3(csize, n_groups < resident ? n_groups : resident, 1);
    cfg.dynamicSmemBytes = (size_t)tpg * p.d * sizeof(float);
  }
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = csize;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  return batched ? cudaLaunchKernelEx(&cfg, router_batched_kernel, q) : cudaLaunchKernelEx(&cfg, router_kernel, q);
}

// One warp per token: x_j = q_p[pi[j]] (the prefetch distribution in descending order),
// s = w.x, delta_hat = first delta with theta_delta - s >= logit(tau)  (Eq. (8), (9) in the logit
// domain), capped to C - k; K_p = first k + delta_hat experts of E (Eq. (1)).
__global__ void __launch_bounds__(128) select_kernel(const SelectParams p) {
  SPAN_BEGIN();
  pdl_wait();
  pdl_launch_dependents();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int b = blockIdx.x * (blockDim.x >> 5) + warp;
  if (b >= p.B) return;
  const int N = p.N;
  const size_t row = (size_t)b * N;
  int pj0 = -1, pj1 = -1;
  float x0 = 0.f, x1 = 0.f;
  if (lane < N) {
    pj0 = __ldg(p.pi + row + lane);
    x0 = __ldg(p.q + row + pj0);
  }
  if (lane + 32 < N) {
    pj1 = __ldg(p.pi + row + lane + 32);
    x1 = __ldg(p.q + row + pj1);
  }
  select_token(p, b, lane, pj0, pj1, x0, x1);
  SPAN_END(2);
}

cudaError_t launch_select(const SelectParams& p, cudaStream_t s) {
  const int wpb = 4;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((p.B + wpb - 1) / wpb, 1, 1);
  cfg.blockDim = dim3(wpb * 32, 1, 1);
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, select_kernel, p);
}

// Streams attn_bytes once (the weight and KV bytes an attention block of this shape reads).  The
// xor of everything read is stored only if it equals one fixed pattern, which keeps the loads live.
__global__ void __launch_bounds__(512) attention_standin_kernel(const AttnParams p) {
  SPAN_BEGIN();
  if (p.wait_first) pdl_wait();
  pdl_launch_dependents();
  const size_t stride = (size_t)gridDim.x * blockDim.x;
  uint4 a = make_uint4(0, 0, 0, 0);
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < p.n_vec; i += stride) {
    const uint4 v = __ldcs(p.buf + i);
    a.x ^= v.x;
    a.y ^= v.y;
    a.z ^= v.z;
    a.w ^= v.w;
  }
  if (a.x == 0x12345678u && a.y == 0x9abcdef0u && a.z == 0x0fedcba9u && a.w == 0x87654321u) p.sink[0] = 1.f;
  // Streamed beside the preceding kernel: wait for it now, so that whoever waits for this kernel has, as
  // always, everything before it on the stream complete.
  if (!p.wait_first) pdl_wait();
  SPAN_END(3);
}

cudaError_t launch_attention(const AttnParams& p, int n_sm, cudaStream_t s) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(n_sm * 2, 1, 1);
  cfg.blockDim = dim3(512, 1, 1);
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, attention_standin_kernel, p);
}

}  // namespace apex

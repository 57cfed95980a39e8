// Persistent decode kernel: all L layer-steps of one token (B = 1) in ONE cooperative launch, so that no kernel
// launch, no grid completion and no host round trip sits between the steps of the hit path (Sec. IV-D:
// predict + budget before attention, prefetch during attention, exact gate after it, then the chosen
// execution mode of Sec. IV-E; the overlap condition is Eq. (12)).
//
// Grid: clusters of eight CTAs, as many as the GPU holds at one CTA per SM (15 on a B200: 120 CTAs stream a layer's
// expert bytes as fast as 148 do).  Every CTA has eight warps, and every warp streams rows through its own stages of
// a shared-memory ring with bulk asynchronous copies (TMA, mbarrier completion), exactly as the per-layer streaming
// kernel does.  A warp's stream is ONE sequence over all layers; per layer, in this order,
//
//   [its share of the attention stand-in's bytes]  [its rows of the expert FFN]
//
// The stand-in's chunks of a layer are requested when the previous layer's y is complete (the attention block's window
// of Eq. (12) opens when its input exists).  With APEX_FLAG_STANDIN_AHEAD they are requested as far ahead as the ring
// allows instead -- a warp starts them as soon as its last expert rows of the previous layer have been requested, so
// they arrive while that layer's tail, the reduction of y and the hand-over are still going on; faster, but the window
// then overlaps the previous layer.  (Consumption stays in order, and everything derived from h or h' waits for the
// counters below.)  The router rows do not go through the ring: narrow ones (d <= 1024) are held in registers from the
// start of the layer, wide ones are prefetched into L2 and read when the dot product is taken (see load_row).
//
//   prefetch router (S1-S3): CTA r of a cluster owns experts 8r .. 8r+7, one warp per expert.  Its dot product with h
//     (reduction order of router_kernel: lane-strided fused multiply-adds, then the xor tree -- the logits are
//     bit-identical to the per-layer kernels') waits for the previous layer's y to be complete (device counter) and is
//     sent through distributed shared memory with st.async, which also counts the bytes on the receiver's mbarrier.
//     Only the first cluster does this, and only its last CTA (the "poster", whose warp 0 carries neither stand-in
//     chunks nor expert rows) receives the logits and derives softmax, ranking, budget and candidate set, posts the
//     record the host plans the prefetch copies from, and leaves the candidate mask in device memory for everybody else.
//   attention stand-in: the bytes that define the hiding window of Eq. (12), streamed by everybody.
//   exact gate (S4): the same exchange with W_r and h', to all eight CTAs of every cluster, after ALL CTAs have
//     finished the stand-in (device counter): a real attention block would only then have produced h'.  The ranks are
//     counted once per CTA (the comparisons split over its warps, summed in shared memory); every warp then derives
//     K_r, alpha and the execution set (S6) itself, so no further exchange is needed before the expert rows are requested.
//   expert FFN (S7, S8): rows split over the CTAs by weight (the first cluster and the poster take fewer); slot-ready
//     flags, demand words and every other wait are bounded as in the per-layer kernel.  Partial y vectors are reduced
//     over the warps in shared memory, then over the cluster (CTA r sums slice r of the eight partial vectors through
//     distributed shared memory) and added to y with vector atomics; then the CTA counts itself in on the layer's counter.
//
// Slot tables: the kernel holds the table of every layer as it stood when the token was launched.  If a layer's
// candidates are all resident in it (and slots persist), nothing changes and the kernel never waits for the host;
// otherwise the host publishes the new snapshot of that layer in mapped memory after it has issued the copies, and
// the kernel picks it up before it plans the expert rows.  Missing routed experts (exact mode) are waited for through
// the demand words, as in the per-layer kernel.
//
// Every wait is bounded by the context's limit and by a device-wide abort flag: whoever gives up raises it, and
// everybody else then leaves its own waits within microseconds, drains its copies and runs to the end (the
// cluster-wide barrier at the end is reached by all).
#include <cuda_bf16.h>

#include "apex_internal.hpp"
#include "ptx.cuh"
#include "router_common.cuh"
#include "ffn_rows.cuh"
#include "token_plan.cuh"

namespace apex {

namespace {

constexpr int kDecMaxStages = 64;
// Shared memory of a CTA: 227 KB, of which the kernel's static variables take 5 KB (a d = 1536 bf16 ring of 24 stages fills
// the rest to the byte: the tests check that the token kernel is what ran) and the CTA's partial y 4 d bytes.
constexpr int kDecSmemTotal = 227 * 1024, kDecSmemStatic = 5120;

__host__ __device__ constexpr int dec_ring_stages(uint32_t entry_bytes, int d) {
  int n = (kDecSmemTotal - kDecSmemStatic - 4 * d) / (int)entry_bytes;
  if (n > kDecMaxStages) n = kDecMaxStages;
  return n / kDecWarps * kDecWarps;
}

#ifdef APEX_TIMELINE
// per CTA and layer (the warp that writes last wins): 0 layer start, 1 W_p logit sent, 2 candidate mask out (poster),
// 3 own attention share landed, 4 W_r logit sent, 5 gate logits complete, 6 plan done, 7 first expert row landed, 8 last
// row consumed, 9 layer counted in, 10 candidate record posted (poster), 11 warps' partial y in shared memory, 12 cluster's
// partial y complete, 13 y added, 14 both counters passed (W_r), 15 previous layer's counter passed (W_p)
__device__ unsigned long long g_dec_tl[160][64][16];
#define DTL(i) do { if (lane == 0 && blockIdx.x < 160 && l < 64) g_dec_tl[blockIdx.x][l][(i)] = globaltimer_ns(); } while (0)
#else
#define DTL(i) do { } while (0)
#endif

__device__ __forceinline__ float dbf16lo(uint32_t v) { return __uint_as_float(v << 16); }
__device__ __forceinline__ float dbf16hi(uint32_t v) { return __uint_as_float(v & 0xffff0000u); }

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_barrier() {
  asm volatile("barrier.cluster.arrive.release.aligned;\nbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// one 32-bit value into the shared memory of CTA `rank` of this cluster; the receiver's mbarrier counts its 4 bytes
__device__ __forceinline__ void st_async_remote(void* local_dst, uint64_t* local_bar, uint32_t rank, float value) {
  uint32_t ra, rb;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(ra) : "r"(smem_u32(local_dst)), "r"(rank));
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(rb) : "r"(smem_u32(local_bar)), "r"(rank));
  asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.b32 [%0], %1, [%2];" ::"r"(ra), "r"(__float_as_uint(value)),
               "r"(rb)
               : "memory");
}
__device__ __forceinline__ void red_release_gpu_u64(unsigned long long* p, unsigned long long v) {
  asm volatile("red.release.gpu.global.add.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
__device__ __forceinline__ uint32_t ld_acquire_gpu_u32(const uint32_t* p) {
  uint32_t v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ unsigned ld_volatile_u32(const unsigned* p) {
  unsigned v;
  asm volatile("ld.volatile.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

// Sum of the row weights of CTAs 0 .. cta-1.  16 per CTA; with the prefetch stage running, 14 for the CTAs of the first
// cluster and 11 for its last CTA (the poster).
__device__ __forceinline__ long long row_weight_prefix(int cta, bool prefetching) {
  if (!prefetching) return 16ll * cta;
  if (cta < kDecCluster) return 14ll * cta;
  return 14ll * (kDecCluster - 1) + 11ll + 16ll * (cta - kDecCluster);
}

}  // namespace

// NCH = d / 256; H_REGS: h' of the layer in registers; FMT: storage format of the expert rows (ffn_rows.cuh).
template <int NCH, bool H_REGS, int FMT>
__global__ void __launch_bounds__(kDecThreads, 1) decode_token_kernel(const DecodeParams p) {
  extern __shared__ __align__(128) uint8_t smem[];
  __shared__ uint64_t s_full[kDecMaxStages];
  __shared__ uint64_t s_xbar[2];   // logits of the prefetch router / of the gate have arrived from the whole cluster
  __shared__ uint64_t s_pbar;      // warp 0 has derived the candidate set of this layer
  __shared__ uint64_t s_rbar;      // every warp has added its share of the gate's rank counts
  __shared__ unsigned s_rank[APEX_MAX_EXPERTS / 4];  // rank of each expert's gate logit, four 8-bit counts to a word (zero between layers)
  __shared__ float s_zp[APEX_MAX_EXPERTS], s_zr[APEX_MAX_EXPERTS];
  __shared__ float s_q[APEX_MAX_EXPERTS];              // warp 0: prefetch probabilities by expert
  __shared__ int s_pi[1][APEX_MAX_EXPERTS];            // warp 0: expert by rank
  __shared__ int s_posp[APEX_MAX_EXPERTS];             // position of each expert in the prefetch ranking (warp 0)
  __shared__ int s_pos[kDecWarps][APEX_MAX_TOPK];      // expert at each position of the row space (a copy per warp)
  __shared__ int s_exp[kDecMaxStages];
  __shared__ unsigned long long s_cand_mask;
  __shared__ int s_abort;
  __shared__ unsigned int s_attn_done;
  __shared__ int8_t s_slot[kDecWarps][APEX_MAX_EXPERTS];  // per warp: slot of every expert of this layer (-1 none)
  __shared__ int s_red_stage[kDecWarps];  // the stage that holds each warp's partial y during the reduction (-1: none)

  constexpr int d = NCH * 256;
  constexpr uint32_t row_bytes = fmt_vec_bytes(FMT, d);      // one vector of a row
  constexpr uint32_t entry_bytes = fmt_entry_bytes(FMT, d);  // gate_i | up_i | downT_i (| scales)
  constexpr int NS = dec_ring_stages(entry_bytes, d);
  constexpr int NSW = NS / kDecWarps;
  constexpr int NV = d / 128;                  // float4 per lane of a router row
  constexpr int SLICE4 = d / 4 / kDecCluster;  // float4 columns of y a CTA adds for its cluster
  static_assert(NS >= kDecWarps, "ring too small");
  static_assert(NS * entry_bytes >= kDecWarps * d * 4, "ring must also hold the cross-warp reduction buffer");
  static_assert(SLICE4 >= 1 && SLICE4 <= kDecThreads, "one thread per float4 of the cluster slice");
  float4* part4 = reinterpret_cast<float4*>(smem + (size_t)NS * entry_bytes);  // this CTA's partial y (behind the ring)

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int N = p.N, k = p.k, I = p.I, L = p.L;
  const int G = gridDim.x, cta = blockIdx.x;
  const uint32_t crank = cluster_ctarank();
  const bool poster = cta == kDecCluster - 1;  // the CTA that writes global outputs, counters and the host's records

  SPAN_BEGIN();
  if (tid == 0) {
    s_abort = 0;
    s_attn_done = 0u;
    mbar_init(&s_xbar[0], 1);
    mbar_init(&s_xbar[1], 1);
    mbar_init(&s_pbar, 1);
    mbar_init(&s_rbar, kDecWarps);
  }
  if (tid < APEX_MAX_EXPERTS / 4) s_rank[tid] = 0u;
  if (tid < NS) mbar_init(&s_full[tid], 1);
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  __syncthreads();
  cluster_barrier();  // nobody sends into a CTA whose barriers are not initialised yet

  // the router row this warp owns in every layer (CTA r of the cluster: experts 8r .. 8r+7)
  const int my_e = (int)crank * kDecWarps + warp;
  const bool has_row = my_e < N;
  const bool wp_cluster = cta < kDecCluster;  // the cluster that computes the prefetch router

  // attention stand-in: chunks of one ring entry, split evenly over the CTAs, a CTA's chunks dealt out to its warps
  const size_t attn_bytes = p.run_attn ? p.attn_bytes : 0;
  const int n_chunks = (int)((attn_bytes + entry_bytes - 1) / entry_bytes);
  const int ch_per = n_chunks / G, ch_extra = n_chunks - ch_per * G;
  const int ch_lo = cta * ch_per + (cta < ch_extra ? cta : ch_extra);
  const int ch_n = ch_per + (cta < ch_extra ? 1 : 0);
  // (the poster's warp 0 takes none while the prefetch stage runs: it has the candidate selection to do as soon as the
  // prefetch logits arrive, and everybody's gate waits until every warp has counted its chunks)
  const bool poster_w0_free = (cta == kDecCluster - 1) && p.prefetching;
  const int ch_warps = poster_w0_free ? kDecWarps - 1 : kDecWarps;
  const int ch_warp = poster_w0_free ? warp - 1 : warp;
  const int ch_mine = (ch_warp >= 0 && ch_n > ch_warp) ? (ch_n - ch_warp + ch_warps - 1) / ch_warps : 0;
  // Segment 1 of a layer in the ring: the warp's chunks of the stand-in.  The router rows do not go through the ring:
  // a warp loads its row of W_p and of W_r straight into registers at the start of the layer (parameters: nothing to
  // wait for), so the rows are there when the counters allow the dot products.
  const bool has_wp = p.prefetching && has_row && wp_cluster, has_wr = has_row;
  const int J = ch_mine;

  // expert rows: which warps of this CTA take rows (the poster's warp 0 does not while the prefetch stage runs)
  const int row_warps = (poster && p.prefetching) ? kDecWarps - 1 : kDecWarps;
  const int row_warp = (poster && p.prefetching) ? warp - 1 : warp;  // index among them, -1: none

  // Row range of this CTA and the rows of this warp for the usual row space (k executed experts and the shared expert):
  // the same in every layer, so the divisions are done once; lane j < NSW also keeps where the warp's row j lies
  // (position in the row space, intermediate index) for the first ring fill.
  const int std_total = k * I + ((p.shared_w && p.I_shared > 0) ? p.I_shared : 0);
  const unsigned std_pre_all = (unsigned)row_weight_prefix(G, p.prefetching != 0);
  const int std_lo = (int)((unsigned long long)std_total * (unsigned)row_weight_prefix(cta, p.prefetching != 0) / std_pre_all);
  const int std_S = (int)((unsigned long long)std_total * (unsigned)row_weight_prefix(cta + 1, p.prefetching != 0) / std_pre_all) - std_lo;
  int ff_pidx = k, ff_i = 0;
  {
    const int r = std_lo + row_warp + row_warps * lane;
    if (r < k * I) {
      ff_pidx = r / I;
      ff_i = r - ff_pidx * I;
    } else {
      ff_i = r - k * I;
    }
  }

  int n_iss = 0, n_con = 0;  // copies this warp has started / consumed since the kernel began (uniform over the warp)
  int il = 0, iq = 0;        // the next segment-1 job to start: layer il, job iq
  bool ok = true;            // false once a wait of this warp ran out
  unsigned long long waited = 0;

  auto gave_up = [&]() {  // a wait ran out: tell the CTA, the other CTAs and the host
    ok = false;
    atomicExch(&s_abort, 1);
    atomicExch(p.abort_flag, 1u);
    *p.mbox_status = 1u;
  };
  auto stop_requested = [&]() -> bool {
    if (*(volatile int*)&s_abort) return true;
    if (ld_volatile_u32(p.abort_flag)) {
      atomicExch(&s_abort, 1);
      return true;
    }
    return false;
  };
  // warp-uniform: has a thread of this CTA given up (or learnt that another CTA did)?
  auto cta_stopped = [&]() -> bool { return __any_sync(0xffffffffu, *(volatile int*)&s_abort != 0); };
  // bounded wait on a shared-memory barrier that also leaves when anybody has given up
  auto wait_bar = [&](uint64_t* bar, uint32_t parity) -> bool {
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = globaltimer_ns();
    for (uint32_t it = 1;; ++it) {
      if (mbar_try_wait(bar, parity)) return true;
      if ((it & 127u) == 0u) {
        if (stop_requested()) return false;
        if ((long long)(globaltimer_ns() - t0) > p.wait_limit_ns) return false;
      }
    }
  };
  // bounded wait for a device-wide counter (one lane calls it).  Hundreds of warps wait for the same word while the
  // CTAs are still adding to it: poll gently.
  auto wait_counter = [&](const unsigned long long* ctr, unsigned long long target) -> bool {
    if (ld_acquire_gpu_u64(ctr) >= target) return true;
    const unsigned long long t0 = globaltimer_ns();
    for (uint32_t it = 1;; ++it) {
      __nanosleep(40);
      if (ld_acquire_gpu_u64(ctr) >= target) return true;
      if ((it & 15u) == 0u) {
        if (stop_requested()) return false;
        if ((long long)(globaltimer_ns() - t0) > p.wait_limit_ns) return false;
      }
    }
  };
  // lane 0: start the copy of `bytes` from src as this warp's next stage entry
  auto start_copy = [&](const void* src, uint32_t bytes) {
    const int s = warp + kDecWarps * (n_iss % NSW);
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // the stage may have been read or written by threads before
    mbar_expect_tx(&s_full[s], bytes);
    bulk_g2s(smem + (size_t)s * entry_bytes, src, bytes, &s_full[s]);
  };
  // all lanes: start segment-1 jobs, in order, of layers up to layer_limit while fewer than max_in_flight copies of this
  // warp are outstanding
  auto start_seg1 = [&](int layer_limit, int max_in_flight) {
    while (il < L && il <= layer_limit && n_iss - n_con < max_in_flight) {
      if (iq >= J) {
        ++il;
        iq = 0;
        continue;
      }
      if (lane == 0) {
        const size_t c = (size_t)ch_lo + ch_warp + (size_t)ch_warps * iq;
        const size_t off = c * entry_bytes;
        const size_t left = attn_bytes - off;
        start_copy(p.attn + (size_t)(il % p.attn_layers) * p.attn_bytes + off, left < entry_bytes ? (uint32_t)left : entry_bytes);
      }
      ++iq;
      ++n_iss;
    }
  };
  // all lanes: wait for this warp's oldest copy; returns its stage (or -1 when the wait was given up)
  auto wait_copy = [&]() -> int {
    const int s = warp + kDecWarps * (n_con % NSW);
    const bool landed = wait_bar(&s_full[s], (uint32_t)((n_con / NSW) & 1));
    if (!__all_sync(0xffffffffu, landed)) {
      if (lane == 0 && ok && !stop_requested()) gave_up();
      ok = false;
      return -1;
    }
    return s;
  };
  // A router row in registers: lane l holds float4 columns l, l + 32, ... (the order of router_kernel's reduction).
  // Up to d = 1024 (8 float4 per lane and row) both rows are fetched at the start of the layer.  Wider rows are
  // prefetched into L2 there instead: two rows of d = 2048 in registers spilled and cost 17 % of the layer-step
  // (configs 2 and 4: 36.8 -> 29.8 and 42.3 -> 35.1 us without them), and even the 96 registers of two d = 1536 rows,
  // which fit, cost the row loop more than the loads' latency costs the logits (config 1 without the stand-in:
  // 19.3 -> 17.2 us per layer-step).  The prefetch router's wide row is read when its dot product is taken; the gate's
  // row of d = 1536 comes into registers right before the wait for the attention window (the latency passes during the
  // wait; + 3 % with the stand-in), and is read with x where there is no window to wait for.
  constexpr int NVRP = NV <= 8 ? NV : 1;   // prefetch-router row
  constexpr int NVRR = NV <= 12 ? NV : 1;  // gate row (9 to 12 float4 per lane: loaded late, see below; wider: not held)
  constexpr bool WR_LATE = NV > 8 && NV <= 12;       // the gate row is fetched right before the wait for the attention window
  auto load_row = [&](const float* __restrict__ W_row, auto& wr) {
    constexpr int NVR = (int)(sizeof(wr) / sizeof(float4));
    constexpr bool ROW_REGS = NVR > 1 || NV == 1;
    if (!ROW_REGS) return;
    const float4* rp = reinterpret_cast<const float4*>(W_row);
#pragma unroll
    for (int i = 0; i < NVR; ++i)  // volatile: keep the loads here, ahead of the waits
      asm volatile("ld.global.nc.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(wr[i].x), "=f"(wr[i].y), "=f"(wr[i].z), "=f"(wr[i].w) : "l"(rp + i * 32 + lane));
  };
  // dot product of the row with x (reduction order of router_kernel), plus bias; sent to CTAs [rank_lo, rank_hi) of the cluster
  auto row_logit = [&](const float* __restrict__ W_row, const auto& wr, bool held, const float* __restrict__ x, float bias, float* zs,
                       uint64_t* xbar, int rank_lo, int rank_hi) {
    constexpr int NVR = (int)(sizeof(wr) / sizeof(float4));
    constexpr bool ROW_REGS = NVR > 1 || NV == 1;
    const float4* __restrict__ xv = reinterpret_cast<const float4*>(x);
    const float4* __restrict__ rp = reinterpret_cast<const float4*>(W_row);
    float acc = 0.f;
    if (ROW_REGS && held) {
      float4 xr[NVR];
#pragma unroll
      for (int i = 0; i < NVR; ++i) xr[i] = __ldg(xv + i * 32 + lane);
#pragma unroll
      for (int i = 0; i < NVR; ++i) {
        acc = fmaf(wr[i].x, xr[i].x, acc);
        acc = fmaf(wr[i].y, xr[i].y, acc);
        acc = fmaf(wr[i].z, xr[i].z, acc);
        acc = fmaf(wr[i].w, xr[i].w, acc);
      }
    } else {
#pragma unroll 8
      for (int i = 0; i < NV; ++i) {
        const float4 wv = __ldg(rp + i * 32 + lane);
        const float4 v = __ldg(xv + i * 32 + lane);
        acc = fmaf(wv.x, v.x, acc);
        acc = fmaf(wv.y, v.y, acc);
        acc = fmaf(wv.z, v.z, acc);
        acc = fmaf(wv.w, v.w, acc);
      }
    }
    acc = warp_sum_tree(acc);
    const float z = acc + bias;
    if (lane >= rank_lo && lane < rank_hi) st_async_remote(&zs[my_e], xbar, (uint32_t)lane, z);
  };
  auto prefetch_l2 = [&](const void* ptr) { asm volatile("prefetch.global.L2 [%0];" ::"l"(ptr)); };

  float sgate = 1.f;      // value of the shared expert's gate for layer sgate_layer (gated variant only)
  int sgate_layer = -1;
  for (int l = 0; l < L; ++l) {
    __syncwarp();
    const bool running = ok && !cta_stopped();  // per warp: skip the work, keep the barriers
    DTL(0);
    const uint32_t lpar = (uint32_t)(l & 1);
    if (tid == 0 && !*(volatile int*)&s_abort) {  // arm this layer's exchange barriers: N logits of 4 bytes each
      if (p.prefetching && poster) mbar_expect_tx(&s_xbar[0], (uint32_t)N * 4u);
      mbar_expect_tx(&s_xbar[1], (uint32_t)N * 4u);
    }
    const float* hl = p.h + (size_t)l * d;
    const float* hpl = p.hpost + (size_t)l * d;
    const unsigned long long* bar_prev_ffn = l > 0 ? p.bar + 2 * (l - 1) : nullptr;
    unsigned long long* bar_ffn = p.bar + 2 * l;
    unsigned long long* bar_attn = p.bar + 2 * l + 1;

    // slot table of this layer as it stood at launch, and the ready flags of its slots (none of this comes from
    // earlier work of this kernel); lanes own experts lane and lane + 32
    const SlotSnapshot* tab = p.tab + l;
    int sl0 = lane < N ? tab->expert_slot[lane] : -1, sl1 = lane + 32 < N ? tab->expert_slot[lane + 32] : -1;
    uint32_t need0 = lane < N ? tab->need_gen[lane] : 0u, need1 = lane + 32 < N ? tab->need_gen[lane + 32] : 0u;
    unsigned long long resident = tab->resident_mask;
    const uint32_t* slot_ready = p.slot_ready + (size_t)l * p.C;
    uint32_t f0 = sl0 >= 0 ? ld_relaxed_sys(slot_ready + sl0) : 0u;
    uint32_t f1 = sl1 >= 0 ? ld_relaxed_sys(slot_ready + sl1) : 0u;
    // parameters of this layer this warp will need: fetched now, used after the waits
    float bias_p = 0.f, bias_r = 0.f;
    float4 wp_row[NVRP], wr_row[NVRR];
    const float* Wp_row = p.W_p + ((size_t)l * N + (has_row ? my_e : 0)) * d;
    const float* Wr_row = p.W_r + ((size_t)l * N + (has_row ? my_e : 0)) * d;
    if (has_wp) load_row(Wp_row, wp_row);
    if (has_wr && !has_wp && !WR_LATE) load_row(Wr_row, wr_row);  // (a warp with both rows fetches W_r after its W_p dot product)
    if (has_row) {
      if (has_wp) bias_p = __ldg(p.b_p + (size_t)l * N + my_e);
      bias_r = __ldg(p.b_r + (size_t)l * N + my_e);
      // x of the two dot products: brought into L2 ahead of time (in a model the previous layer has just written it there)
      if ((lane & 7) == 0) {
#pragma unroll
        for (int i = 0; i < NV; ++i) {
          if (has_wp) prefetch_l2(reinterpret_cast<const float4*>(hl) + i * 32 + lane);
          prefetch_l2(reinterpret_cast<const float4*>(hpl) + i * 32 + lane);
          // ... and so are the router rows that are not held in registers
          if (NVRP == 1 && NV > 1 && has_wp) prefetch_l2(reinterpret_cast<const float4*>(Wp_row) + i * 32 + lane);
          if (NVRR == 1 && NV > 1) prefetch_l2(reinterpret_cast<const float4*>(Wr_row) + i * 32 + lane);
        }
      }
    }
    float cw0 = 0.f, cw1 = 0.f, cth0 = 0.f, cth1 = 0.f;  // poster's warp 0: confidence model of this layer
    if (poster && warp == 0 && p.prefetching) {
      const float* wl = p.w + (size_t)l * N;
      const float* thl = p.theta + (size_t)l * (N - k + 1);
      if (lane < N) cw0 = __ldg(wl + lane);
      if (lane + 32 < N) cw1 = __ldg(wl + lane + 32);
      if (lane < N - k + 1) cth0 = __ldg(thl + lane);
      if (lane + 32 < N - k + 1) cth1 = __ldg(thl + lane + 32);
    }

    // ------------------------------------------------------------ segment 1: attention share, W_p row, W_r row
    bool pref_done = !(p.prefetching && poster && warp == 0);  // poster's warp 0: the candidate set of this layer is out
    int ncand_p = 0;                                           // poster's warp 0: k + delta_hat of this layer
    // the poster's warp 0: softmax, ranking, budget, candidate set from the exchanged prefetch logits
    auto prefetch_epilogue = [&]() {
      const RankedLogits R = softmax_and_rank(s_zp, N, lane);
      const int e0 = lane, e1 = lane + 32;
      if (e0 < N) { s_q[e0] = R.q0; s_pi[0][R.r0] = e0; s_posp[e0] = R.r0; }
      if (e1 < N) { s_q[e1] = R.q1; s_pi[0][R.r1] = e1; s_posp[e1] = R.r1; }
      __syncwarp();
      const int pj0 = lane < N ? s_pi[0][lane] : -1, pj1 = lane + 32 < N ? s_pi[0][lane + 32] : -1;
      const float x0 = pj0 >= 0 ? s_q[pj0] : 0.f, x1 = pj1 >= 0 ? s_q[pj1] : 0.f;
      // the budget and the candidate mask, first of all for every other CTA (device memory) ...
      int uncapped;
      const int d_hat = select_budget_vals(cw0, cw1, cth0, cth1, p.t_tau, p.force, N, k, p.C, lane, x0, x1, &uncapped);
      ncand_p = k + d_hat;
      unsigned lo = 0, hi = 0;
      if (lane < ncand_p) { if (pj0 < 32) lo |= 1u << pj0; else hi |= 1u << (pj0 - 32); }
      if (lane + 32 < ncand_p) { if (pj1 < 32) lo |= 1u << pj1; else hi |= 1u << (pj1 - 32); }
      lo = __reduce_or_sync(0xffffffffu, lo);
      hi = __reduce_or_sync(0xffffffffu, hi);
      if (lane == 0) {
        p.cand_rec[2 * l] = ((unsigned long long)hi << 32) | lo;
        asm volatile("st.release.gpu.global.u64 [%0], %1;" ::"l"(p.cand_rec + 2 * l + 1), "l"((unsigned long long)p.seq) : "memory");
      }
      DTL(2);
      // ... then the outputs of S1-S3, the counters and the record the host plans the copies from (one 16-byte store
      // to mapped memory; kept behind the release above, which would otherwise have to wait for it)
      if (e0 < N) { p.zp_out[e0] = R.z0; p.qp_out[e0] = R.q0; p.pi_out[R.r0] = e0; }
      if (e1 < N) { p.zp_out[e1] = R.z1; p.qp_out[e1] = R.q1; p.pi_out[R.r1] = e1; }
      SelectParams sp;
      sp.w = p.w + (size_t)l * N;
      sp.theta = p.theta + (size_t)l * (N - k + 1);
      sp.cand_out = p.cand_dev;
      sp.ncand_out = p.ncand_dev;
      sp.ncand_keep = p.ncand_keep;
      sp.mbox_cand = p.mbox[l].cand;
      sp.mbox_ncand = reinterpret_cast<int32_t*>(&p.mbox[l].pad[0]);
      sp.mbox_rec = p.mbox[l].sel_rec;
      sp.seq_value = p.seq;
      sp.stats = p.stats + l;
      sp.t_tau = p.t_tau;
      sp.force = p.force;
      sp.N = N; sp.k = k; sp.C = p.C; sp.B = 1;
      select_token(sp, 0, lane, pj0, pj1, x0, x1);
      DTL(10);
      pref_done = true;

    };
    bool attn_counted = false;
    auto count_attention = [&]() {  // this warp's share of the stand-in has landed; the last warp counts the CTA in
      if (attn_counted) return;
      attn_counted = true;
      DTL(3);
      if (lane == 0 && p.run_attn) {
        const unsigned old = atomicAdd(&s_attn_done, 1u);
        if ((old + 1u) % kDecWarps == 0u) red_release_gpu_u64(bar_attn, 1ull);
      }
    };
    // The stand-in is this layer's attention block: its window opens when the previous layer's y is complete.  (With
    // standin_ahead the chunks were requested earlier, while the previous layer was still finishing: the window then
    // overlaps that layer's tail -- including any wait for its experts -- which is not what Eq. (12) describes.)
    if ((J > 0 || has_wp) && running && bar_prev_ffn) {
      bool go = true;
      if (lane == 0) go = wait_counter(bar_prev_ffn, p.bar_target);
      go = __shfl_sync(0xffffffffu, go ? 1 : 0, 0) != 0;
      if (!go) {
        if (lane == 0 && !stop_requested()) gave_up();
        ok = false;
      }
      DTL(15);
    }
    if (ok && running) start_seg1(l, NSW);  // this layer's chunks: on their way while the prefetch logit is computed
    // prefetch router first of all: the sooner the candidate set is out, the more of the window the copies can use
    if (has_wp && running && ok) {
      row_logit(Wp_row, wp_row, true, hl, bias_p, s_zp, &s_xbar[0], kDecCluster - 1, kDecCluster);  // to the poster only
      DTL(1);
      if (has_wr && !WR_LATE) load_row(Wr_row, wr_row);
    }
    {
      int q_con = 0;
      while (q_con < J && ok && running) {
        start_seg1(l, NSW);
        const int s = wait_copy();
        if (s < 0) break;
        __syncwarp();
        ++q_con;
        ++n_con;
      }
    }
    count_attention();
    // the poster's warp 0: the candidate set, as soon as the prefetch logits are complete (after it has counted its
    // share of the stand-in: everybody's gate waits for that count)
    if (!pref_done && ok && !cta_stopped()) {
      if (__all_sync(0xffffffffu, wait_bar(&s_xbar[0], lpar))) prefetch_epilogue();
      else {
        if (lane == 0 && !stop_requested()) gave_up();
        ok = false;
      }
    }
    // exact gate: this warp's logit, once the whole stand-in has been streamed (a real attention block would only then
    // have produced h') and the previous layer's y is complete
    if (has_wr && ok && !cta_stopped()) {
      // (a wide gate row comes into registers only now, from L2: its latency passes while the counters are waited for,
      // and the registers were free for the stand-in's segment and are free again for the expert rows)
      if (WR_LATE && p.run_attn) load_row(Wr_row, wr_row);  // (without a window to wait for, the row is read with x)
      bool go = true;
      if (lane == 0) {
        if (p.run_attn) go = wait_counter(bar_attn, p.bar_target);
        if (go && bar_prev_ffn) go = wait_counter(bar_prev_ffn, p.bar_target);
      }
      go = __shfl_sync(0xffffffffu, go ? 1 : 0, 0) != 0;
      if (!go) {
        if (lane == 0 && !stop_requested()) gave_up();
        ok = false;
      } else {
        DTL(14);
        row_logit(Wr_row, wr_row, !WR_LATE || p.run_attn != 0, hpl, bias_r, s_zr, &s_xbar[1], 0, kDecCluster);
        DTL(4);
      }
    }
    // h' for the expert rows (the router rows' registers are free again)
    float hreg[H_REGS ? NCH * 8 : 1];
    if (H_REGS) {
#pragma unroll
      for (int c = 0; c < NCH; ++c) {
        const float4 a = __ldg(reinterpret_cast<const float4*>(hpl) + (c * 32 + lane) * 2);
        const float4 b2 = __ldg(reinterpret_cast<const float4*>(hpl) + (c * 32 + lane) * 2 + 1);
        hreg[c * 8 + 0] = a.x; hreg[c * 8 + 1] = a.y; hreg[c * 8 + 2] = a.z; hreg[c * 8 + 3] = a.w;
        hreg[c * 8 + 4] = b2.x; hreg[c * 8 + 5] = b2.y; hreg[c * 8 + 6] = b2.z; hreg[c * 8 + 7] = b2.w;
      }
    }
    // ------------------------------------------------------------ gate: routed set, execution set, row space
    // First what the copies need (ranks -> K_r -> K~ -> positions), then the copies are started, and only then the
    // probabilities and gates are derived, while the first rows are on their way.
    //
    // Which slot table?  The one the kernel was launched with is this step's table unless the host changes it, which it
    // does only if a candidate of this step is not resident (it then publishes the new table).  Whether that is so is
    // known once the poster's candidate mask has arrived -- a few microseconds after the gate on the hit path.  Where
    // the host expects no change for this layer (opt[l]: the layer's previous step copied nothing) the warp does not
    // wait for the mask: it plans with the launch-time table and starts streaming, checks the mask when it arrives, and
    // in the rare case that the table did change it drops what it has accumulated and repeats the layer's rows with the
    // published table.  It never waits for a flag or a demand copy on an unconfirmed table.
    unsigned long long kr_mask = 0ull, run = 0ull, ready_mask = 0ull;
    float g0 = 0.f, g1 = 0.f;
    RankedLogits Rg;
    Rg.z0 = Rg.z1 = Rg.q0 = Rg.q1 = 0.f;
    Rg.r0 = Rg.r1 = 0;
    bool planned = false;
    bool verified = !p.prefetching;  // the table this warp plans with is known to be this step's
    bool changed = false;            // ... and it is not the launch-time table: the host's snapshot has been taken
    bool cand_known = !p.prefetching;  // warp 0: the poster's mask has been passed on to this CTA's warps
    // warp 0, all lanes: pass the poster's candidate mask on to the CTA.  blocking: wait for it (bounded); otherwise take
    // it only if `seen` (a value of the record's sequence word loaded earlier) shows that it is there.
    auto relay_cand_mask = [&](bool blocking, unsigned long long seen) {
      if (cand_known) return;
      const unsigned long long* seqw = p.cand_rec + 2 * l + 1;
      bool got = seen == (unsigned long long)p.seq;
      bool fail_ = false;
      if (!got && blocking) {
        if (lane == 0) {
          const unsigned long long t0 = globaltimer_ns();
          got = ld_acquire_gpu_u64(seqw) == (unsigned long long)p.seq;
          for (uint32_t it = 1; !got; ++it) {
            if ((it & 7u) == 0u && (stop_requested() || (long long)(globaltimer_ns() - t0) > p.wait_limit_ns)) break;
            __nanosleep(40);
            got = ld_acquire_gpu_u64(seqw) == (unsigned long long)p.seq;
          }
          fail_ = !got;
        }
        got = __shfl_sync(0xffffffffu, got ? 1 : 0, 0) != 0;
        fail_ = __shfl_sync(0xffffffffu, fail_ ? 1 : 0, 0) != 0;
      }
      if (fail_) {
        if (lane == 0 && !stop_requested()) gave_up();
        ok = false;
        return;
      }
      if (got) {
        if (lane == 0) {
          (void)ld_acquire_gpu_u64(seqw);  // orders the read of the mask behind the sequence word
          s_cand_mask = *(volatile const unsigned long long*)(p.cand_rec + 2 * l);
          mbar_arrive(&s_pbar);  // release: the other warps read the mask after waiting for this barrier
        }
        cand_known = true;
      }
    };
    // all lanes: the candidate mask is there (s_pbar complete): take this step's table.  Returns false when a wait ran out.
    auto confirm_table = [&]() -> bool {
      verified = true;
      const unsigned long long cand = s_cand_mask;
      if (p.cache_reuse && (cand & ~resident) == 0ull) return true;  // every candidate was resident: nothing changes
      // The host publishes the new table in mapped host memory.  ONE warp of the grid reads it there and passes it on
      // through device memory: a poll of host memory is a read over the host link, and a thousand warps polling would
      // take the link away from the very copies they are waiting for.
      const DecodeHostSnap* hs = p.snap + l;
      DecodeHostSnap* ds_ = p.snap_dev + l;
      bool got = true;
      if (cta == 0 && warp == 0) {
        if (lane == 0 && ld_acquire_sys(&hs->seq) != p.seq) {
          const unsigned long long t0 = globaltimer_ns();
          for (uint32_t it = 1; ld_acquire_sys(&hs->seq) != p.seq; ++it) {
            if ((it & 3u) == 0u && (stop_requested() || (long long)(globaltimer_ns() - t0) > p.wait_limit_ns)) {
              got = false;
              break;
            }
            __nanosleep(400);
          }
        }
        got = __shfl_sync(0xffffffffu, got ? 1 : 0, 0) != 0;
        if (got) {
          const volatile SlotSnapshot* vt = &hs->tab;
          if (lane < N) { ds_->tab.expert_slot[lane] = vt->expert_slot[lane]; ds_->tab.need_gen[lane] = vt->need_gen[lane]; }
          if (lane + 32 < N) { ds_->tab.expert_slot[lane + 32] = vt->expert_slot[lane + 32]; ds_->tab.need_gen[lane + 32] = vt->need_gen[lane + 32]; }
          if (lane == 0) ds_->tab.resident_mask = vt->resident_mask;
          __threadfence();
          __syncwarp();
          if (lane == 0) asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(&ds_->seq), "r"(p.seq) : "memory");
        }
      }
      if (got && lane == 0 && ld_acquire_gpu_u32(&ds_->seq) != p.seq) {
        const unsigned long long t0 = globaltimer_ns();
        for (uint32_t it = 1; ld_acquire_gpu_u32(&ds_->seq) != p.seq; ++it) {
          if ((it & 3u) == 0u && (stop_requested() || (long long)(globaltimer_ns() - t0) > p.wait_limit_ns)) {
            got = false;
            break;
          }
          __nanosleep(200);
        }
        waited += globaltimer_ns() - t0;
      }
      got = __shfl_sync(0xffffffffu, got ? 1 : 0, 0) != 0;
      if (!got) {
        if (lane == 0 && !stop_requested()) gave_up();
        ok = false;
        return false;
      }
      (void)ld_acquire_gpu_u32(&ds_->seq);  // every lane: its reads of the table come after the sequence word
      const volatile SlotSnapshot* vt = &ds_->tab;
      sl0 = lane < N ? vt->expert_slot[lane] : -1;
      sl1 = lane + 32 < N ? vt->expert_slot[lane + 32] : -1;
      need0 = lane < N ? vt->need_gen[lane] : 0u;
      need1 = lane + 32 < N ? vt->need_gen[lane + 32] : 0u;
      resident = vt->resident_mask;
      f0 = sl0 >= 0 ? ld_relaxed_sys(slot_ready + sl0) : 0u;
      f1 = sl1 >= 0 ? ld_relaxed_sys(slot_ready + sl1) : 0u;
      changed = true;
      return true;
    };
    auto wait_and_confirm = [&]() -> bool {  // blocking form
      if (warp == 0) relay_cand_mask(true, 0ull);
      if (!ok) return false;
      if (!__all_sync(0xffffffffu, wait_bar(&s_pbar, lpar))) {
        if (lane == 0 && !stop_requested()) gave_up();
        ok = false;
        return false;
      }
      return confirm_table();
    };
    auto derive_sets = [&]() {  // from the current table: which slots are ready, which experts are executed
      const bool r0 = sl0 >= 0 && (int32_t)(f0 - need0) >= 0, r1 = sl1 >= 0 && (int32_t)(f1 - need1) >= 0;
      ready_mask = ((unsigned long long)__ballot_sync(0xffffffffu, r1) << 32) | __ballot_sync(0xffffffffu, r0);
      run = exec_set(kr_mask, p.mode, resident, Rg.z0, Rg.z1, lane);
    };
    const bool optimistic = p.prefetching && p.cache_reuse && p.opt[l] != 0;
    if (ok && !cta_stopped()) {
      if (!__all_sync(0xffffffffu, wait_bar(&s_xbar[1], lpar))) {
        if (lane == 0 && !stop_requested()) gave_up();
        ok = false;
      } else {
        DTL(5);
        // Ranks by counting, the count shared by the CTA's warps: warp w compares every logit with the logits of experts
        // w, w + 8, ... only and adds its counts up in shared memory (each warp ranking all N logits by itself was
        // 0.8 us of every warp's path to the first row).
        const int e0 = lane, e1 = lane + 32;
        {
          const float NEG = -3.402823466e38f;
          Rg.z0 = e0 < N ? s_zr[e0] : NEG;
          Rg.z1 = e1 < N ? s_zr[e1] : NEG;
          int c0 = 0, c1 = 0;
          for (int f = warp; f < N; f += kDecWarps) {
            const float zf = s_zr[f];
            c0 += (zf > Rg.z0 || (zf == Rg.z0 && f < e0)) ? 1 : 0;
            c1 += (zf > Rg.z1 || (zf == Rg.z1 && f < e1)) ? 1 : 0;
          }
          unsigned* rk = s_rank;  // counts stay below N <= 64: no carry between the bytes of a word
          if (e0 < N && c0) atomicAdd(rk + (e0 >> 2), (unsigned)c0 << (8 * (e0 & 3)));
          if (e1 < N && c1) atomicAdd(rk + (e1 >> 2), (unsigned)c1 << (8 * (e1 & 3)));
          __syncwarp();
          if (lane == 0) mbar_arrive(&s_rbar);
          if (!__all_sync(0xffffffffu, wait_bar(&s_rbar, lpar))) {
            if (lane == 0 && !stop_requested()) gave_up();
            ok = false;
          }
          Rg.r0 = e0 < N ? (int)((rk[e0 >> 2] >> (8 * (e0 & 3))) & 0xffu) : N;
          Rg.r1 = e1 < N ? (int)((rk[e1 >> 2] >> (8 * (e1 & 3))) & 0xffu) : N;
        }
        kr_mask = ((unsigned long long)__ballot_sync(0xffffffffu, e1 < N && Rg.r1 < k) << 32) | __ballot_sync(0xffffffffu, e0 < N && Rg.r0 < k);
        if (poster && warp == 0 && lane == 0) {  // K_r does not depend on the table: the host gets it at once
          asm volatile("st.global.v4.u32 [%0], {%1, %2, %3, %4};" ::"l"(p.mbox[l].kr_rec), "r"((uint32_t)kr_mask),
                       "r"((uint32_t)(kr_mask >> 32)), "r"(p.seq), "r"(0u)
                       : "memory");
          if (p.mode == APEX_MODE_EXACT)  // ... and in this mode neither does the execution set
            asm volatile("st.global.v4.u32 [%0], {%1, %2, %3, %4};" ::"l"(p.mbox[l].exec_rec), "r"((uint32_t)kr_mask),
                         "r"((uint32_t)(kr_mask >> 32)), "r"(p.seq), "r"(0u)
                         : "memory");
        }
        if (!verified && !optimistic) wait_and_confirm();
        if (ok) {
          derive_sets();
          if (!verified && (run & ~ready_mask) != 0ull) {  // something to wait for: only on the confirmed table
            if (wait_and_confirm() && changed) derive_sets();
          }
          planned = ok;
        }
      }
    }
    const uint8_t* shared_w = (p.shared_w && p.I_shared > 0) ? p.shared_w[l] : nullptr;
    const uint32_t* demand = p.demand + (size_t)l * N;
    const uint8_t* cache_l = p.cache + (size_t)l * p.C * p.slot_stride;
    // (the slot of an expert lives in the lane that owns it: looked up with a shuffle by the whole warp)
    auto slot_of = [&](int e) -> int { return __shfl_sync(0xffffffffu, e < 32 ? sl0 : sl1, e & 31); };
    auto need_of = [&](int e) -> uint32_t { return __shfl_sync(0xffffffffu, e < 32 ? need0 : need1, e & 31); };
    float acc[NCH * 8];
    bool go_rows = false;
    bool outputs_done = false;
    int dm_e = -1, dm_slot = -1;  // lane 0: last expert that had to be waited for on demand
    for (int pass = 0; pass < 2; ++pass) {
      // row space of the expert FFN: executed experts in ascending index, then the shared expert
      const int n_routed = __popcll(run);
      const int total_rows = planned ? n_routed * I + (shared_w ? p.I_shared : 0) : 0;
      // Rows are dealt out by weight: the first cluster also runs the prefetch router and its last CTA (the poster)
      // the candidate selection on warp 0, so they take fewer rows and the poster's warp 0 none -- otherwise
      // everybody would wait for them at the end of the layer.
      int range_lo = std_lo, S = std_S;
      const bool std_rows = total_rows == std_total;
      if (!std_rows) {  // fewer experts executed than k (or no plan): the range is worked out for this row count
        range_lo = (int)((unsigned long long)total_rows * (unsigned)row_weight_prefix(cta, p.prefetching != 0) / std_pre_all);
        S = (int)((unsigned long long)total_rows * (unsigned)row_weight_prefix(cta + 1, p.prefetching != 0) / std_pre_all) - range_lo;
      }
      const int n_mine = (row_warp >= 0 && S > row_warp) ? (S - row_warp + row_warps - 1) / row_warps : 0;
      if (planned) {
        if (lane < APEX_MAX_TOPK) s_pos[warp][lane] = lane < n_routed ? nth_set_bit64(run, lane) : -1;
        if (lane < N) s_slot[warp][lane] = (int8_t)sl0;
        if (lane + 32 < N) s_slot[warp][lane + 32] = (int8_t)sl1;
        __syncwarp();
      }
      if (pass == 0) DTL(6);

      // ---------------------------------------------------------- segment 2: the expert rows
#pragma unroll
      for (int i = 0; i < NCH * 8; ++i) acc[i] = 0.f;
      go_rows = planned && ok && !cta_stopped();
      bool redo = false;
      {
        int q_iss = 0, q_con = 0;
        const int Jr = go_rows ? n_mine : 0;
        bool gates_done = false;
        // First ring fill when every executed expert is resident and ready (the usual case): one copy per lane, all
        // started at once.  Otherwise (a flag or a demand copy to wait for) the copies are started one by one below.
        if (Jr > 0 && (run & ~ready_mask) == 0ull && n_iss == n_con) {
          const int fill = Jr < NSW ? Jr : NSW;
          if (lane < fill) {
            int pidx = ff_pidx, i = ff_i;
            if (!std_rows) {
              const int r = range_lo + row_warp + row_warps * lane;
              if (r < n_routed * I) {
                pidx = r / I;
                i = r - pidx * I;
              } else {
                pidx = n_routed;
                i = r - n_routed * I;
              }
            }
            const int e = pidx < n_routed ? s_pos[warp][pidx] : N;
            const uint8_t* base = e < N ? cache_l + (size_t)s_slot[warp][e] * p.slot_stride : shared_w;
            const int st = warp + kDecWarps * ((n_iss + lane) % NSW);
            s_exp[st] = e;
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            mbar_expect_tx(&s_full[st], entry_bytes);
            bulk_g2s(smem + (size_t)st * entry_bytes, base + (size_t)i * entry_bytes, entry_bytes, &s_full[st]);
          }
          q_iss = fill;
          n_iss += fill;
          __syncwarp();
        }
        while (q_con < Jr || (go_rows && !gates_done)) {
          // warp 0, while the table is unconfirmed: look for the poster's mask (the load is issued here and its value
          // used at the end of the iteration, so its latency hides behind a row)
          unsigned long long seen = 0ull;
          if (!cand_known && warp == 0 && lane == 0) seen = *(volatile const unsigned long long*)(p.cand_rec + 2 * l + 1);
          // start copies while this warp has free stages (whole warp: the slot lookup is a shuffle)
          while (q_iss < Jr && n_iss - n_con < NSW && ok && !redo) {
            const int r = range_lo + row_warp + row_warps * q_iss;
            int pidx, i;
            if (r < n_routed * I) {
              pidx = r / I;
              i = r - pidx * I;
            } else {
              pidx = n_routed;
              i = r - n_routed * I;
            }
            const int e = pidx < n_routed ? s_pos[warp][pidx] : N;
            const uint8_t* base = shared_w;
            if (e < N) {
              int slot = slot_of(e);
              const uint32_t need = need_of(e);
              bool good = true;
              if (lane == 0) {
                if (slot < 0) {
                  // not resident when the table was taken: the host fetches it on demand and publishes (tag, slot)
                  // after the copy -- asynchronous miss correction inside the launch (exact mode only)
                  if (e == dm_e) {
                    slot = dm_slot;
                  } else {
                    const uint32_t* wd = demand + e;
                    uint32_t v = ld_acquire_sys(wd);
                    if ((v >> 8) != p.demand_tag) {
                      const unsigned long long t0 = globaltimer_ns();
                      for (uint32_t it = 1; ((v = ld_acquire_sys(wd)) >> 8) != p.demand_tag; ++it) {
                        if ((it & 3u) == 0u && (stop_requested() || (long long)(globaltimer_ns() - t0) > p.wait_limit_ns)) {
                          good = false;
                          break;
                        }
                        __nanosleep(128);
                      }
                      waited += globaltimer_ns() - t0;
                    }
                    slot = (int)(v & 0xffu);
                    if (good && slot >= p.C) good = false;  // a published slot outside the cache: refuse
                    if (good) {
                      dm_e = e;
                      dm_slot = slot;
                      asm volatile("fence.proxy.async;" ::: "memory");
                    }
                  }
                } else if (!((ready_mask >> e) & 1ull)) {
                  const uint32_t* flag = slot_ready + slot;
                  const unsigned long long t0 = globaltimer_ns();
                  for (uint32_t it = 1; (int32_t)(ld_acquire_sys(flag) - need) < 0; ++it) {
                    if ((it & 3u) == 0u && (stop_requested() || (long long)(globaltimer_ns() - t0) > p.wait_limit_ns)) {
                      good = false;
                      break;
                    }
                    __nanosleep(64);
                  }
                  waited += globaltimer_ns() - t0;
                  if (good) asm volatile("fence.proxy.async;" ::: "memory");
                }
              }
              good = __shfl_sync(0xffffffffu, good ? 1 : 0, 0) != 0;
              slot = __shfl_sync(0xffffffffu, slot, 0);
              if (!good) {
                if (lane == 0 && !stop_requested()) gave_up();
                ok = false;
                break;
              }
              if (slot >= 0 && slot_of(e) >= 0) ready_mask |= 1ull << e;
              base = cache_l + (size_t)slot * p.slot_stride;
            }
            if (lane == 0) {
              s_exp[warp + kDecWarps * (n_iss % NSW)] = e;
              start_copy(base + (size_t)i * entry_bytes, entry_bytes);
            }
            ++q_iss;
            ++n_iss;
          }
          // every row of this layer has been requested (and the table is confirmed: no repeat can follow): go on with
          // the next layer's first segment (one stage stays free for the reduction of y)
          if (p.standin_ahead && q_iss >= Jr && ok && verified && !redo) start_seg1(l + 1, NSW - 1);
          __syncwarp();  // s_exp of the copies just started is visible to the whole warp
          if (!ok) break;
          if (!gates_done) {
            // the first rows are in flight: probabilities, gates and (poster) the outputs of S4
            gates_done = true;
            if (pass == 0) softmax_lane_logits(N, lane, &Rg);
            exec_gates(run, lane < N ? Rg.q0 : 0.f, lane + 32 < N ? Rg.q1 : 0.f, p.norm_topk, lane, &g0, &g1);
            if (poster && warp == 0 && !outputs_done) {
              outputs_done = true;
              const int e0 = lane, e1 = lane + 32;
              const size_t zo = (size_t)l * p.zr_stride;
              if (e0 < N) { p.zr_out[zo + e0] = Rg.z0; p.alpha_out[zo + e0] = Rg.q0; if (Rg.r0 < k) p.idx_out[(size_t)l * p.idx_stride + Rg.r0] = e0; }
              if (e1 < N) { p.zr_out[zo + e1] = Rg.z1; p.alpha_out[zo + e1] = Rg.q1; if (Rg.r1 < k) p.idx_out[(size_t)l * p.idx_stride + Rg.r1] = e1; }
              const bool in0 = e0 < N && Rg.r0 < k, in1 = e1 < N && Rg.r1 < k;
              int dstar = 0, hitsP = 0;
              if (p.prefetching) {
                const int pos0 = in0 ? s_posp[e0] : -1, pos1 = in1 ? s_posp[e1] : -1;
                dstar = warp_max_int(max(pos0, pos1)) + 1 - k;
                hitsP = __popc(__ballot_sync(0xffffffffu, in0 && pos0 < ncand_p)) + __popc(__ballot_sync(0xffffffffu, in1 && pos1 < ncand_p));
              }
              if (lane == 0) {
                DevStats* st = p.stats + l;
                atomicAdd(&st->routed, (unsigned long long)k);
                if (p.prefetching) {
                  atomicAdd(&st->sum_delta_star, (unsigned long long)dstar);
                  atomicAdd(&st->hits_P, (unsigned long long)hitsP);
                  atomicAdd(&st->covered, (unsigned long long)(hitsP == k ? 1 : 0));
                }
              }
            }
            if (q_con >= q_iss && q_iss >= Jr) break;
          }
          if (q_con < q_iss) {
            const int s = wait_copy();
            if (s < 0) break;
            if (q_con == 0 && pass == 0) DTL(7);
            if (!redo) {
              const int e = s_exp[s];
              float gate = __shfl_sync(0xffffffffu, e < 32 ? g0 : g1, e & 31);
              if (e >= N) {  // the shared expert: weight 1, or its gate's value (once per warp and layer)
                gate = 1.f;
                const float* wsg = p.shared_gate ? p.shared_gate[l] : nullptr;
                if (wsg) {
                  if (sgate_layer != l) {
                    sgate = shared_gate_weight(wsg, hpl, d, lane);
                    sgate_layer = l;
                  }
                  gate = sgate;
                }
              }
              const uint8_t* gs = smem + (size_t)s * entry_bytes;
              const uint8_t* us = gs + row_bytes;
              const uint8_t* ds = us + row_bytes;
              if constexpr (FMT != kFmtBf16) {
                // quantised rows: decoded eight weights at a time; e4m3 scales multiply the two dot products and the
                // gated intermediate once per row, e2m1 block scales a lane's eight-element partial sums
                float g = 0.f, u = 0.f;
#pragma unroll
                for (int c = 0; c < NCH; ++c) {
                  float gw[8], uw[8], hh[8];
                  load8<FMT>(gs, c * 32 + lane, gw);
                  load8<FMT>(us, c * 32 + lane, uw);
                  if (H_REGS) {
#pragma unroll
                    for (int m = 0; m < 8; ++m) hh[m] = hreg[c * 8 + m];
                  } else {
                    const float4 a = __ldg(reinterpret_cast<const float4*>(hpl) + (c * 32 + lane) * 2);
                    const float4 b2 = __ldg(reinterpret_cast<const float4*>(hpl) + (c * 32 + lane) * 2 + 1);
                    hh[0] = a.x; hh[1] = a.y; hh[2] = a.z; hh[3] = a.w; hh[4] = b2.x; hh[5] = b2.y; hh[6] = b2.z; hh[7] = b2.w;
                  }
                  float pg = 0.f, pu = 0.f;
#pragma unroll
                  for (int m = 0; m < 8; ++m) pg = fmaf(gw[m], hh[m], pg);
#pragma unroll
                  for (int m = 0; m < 8; ++m) pu = fmaf(uw[m], hh[m], pu);
                  if (FMT == kFmtMxfp4) {
                    const uint8_t* sc = ds + row_bytes;  // gate | up | downT block scales, d/32 bytes each
                    g = fmaf(block_scale(sc, c * 32 + lane), pg, g);
                    u = fmaf(block_scale(sc + d / 32, c * 32 + lane), pu, u);
                  } else {
                    g += pg;
                    u += pu;
                  }
                }
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) {
                  const float g2 = __shfl_xor_sync(0xffffffffu, g, o), u2 = __shfl_xor_sync(0xffffffffu, u, o);
                  g += g2;
                  u += u2;
                }
                float down_scale = 1.f;
                if (FMT == kFmtE4m3) {
                  const float* sc = reinterpret_cast<const float*>(ds + row_bytes);
                  g *= sc[0];
                  u *= sc[1];
                  down_scale = sc[2];
                }
                const float a = gate * g * __fdividef(1.f, 1.f + __expf(-g)) * u * down_scale;
#pragma unroll
                for (int c = 0; c < NCH; ++c) {
                  float dw[8];
                  load8<FMT>(ds, c * 32 + lane, dw);
                  const float ac = FMT == kFmtMxfp4 ? a * block_scale(ds + row_bytes + 2 * (d / 32), c * 32 + lane) : a;
#pragma unroll
                  for (int m = 0; m < 8; ++m) acc[c * 8 + m] = fmaf(ac, dw[m], acc[c * 8 + m]);
                }
              } else {
              // four partial sums per dot product: independent chains instead of one of 8 * NCH dependent multiply-adds
              float gp[4] = {0.f, 0.f, 0.f, 0.f}, up[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
              for (int c = 0; c < NCH; ++c) {
                const uint4 gv = reinterpret_cast<const uint4*>(gs)[c * 32 + lane];
                const uint4 uv = reinterpret_cast<const uint4*>(us)[c * 32 + lane];
                float hh[8];
                if (H_REGS) {
#pragma unroll
                  for (int m = 0; m < 8; ++m) hh[m] = hreg[c * 8 + m];
                } else {
                  const float4 a = __ldg(reinterpret_cast<const float4*>(hpl) + (c * 32 + lane) * 2);
                  const float4 b2 = __ldg(reinterpret_cast<const float4*>(hpl) + (c * 32 + lane) * 2 + 1);
                  hh[0] = a.x; hh[1] = a.y; hh[2] = a.z; hh[3] = a.w; hh[4] = b2.x; hh[5] = b2.y; hh[6] = b2.z; hh[7] = b2.w;
                }
                gp[0] = fmaf(dbf16lo(gv.x), hh[0], gp[0]); gp[1] = fmaf(dbf16hi(gv.x), hh[1], gp[1]);
                gp[2] = fmaf(dbf16lo(gv.y), hh[2], gp[2]); gp[3] = fmaf(dbf16hi(gv.y), hh[3], gp[3]);
                gp[0] = fmaf(dbf16lo(gv.z), hh[4], gp[0]); gp[1] = fmaf(dbf16hi(gv.z), hh[5], gp[1]);
                gp[2] = fmaf(dbf16lo(gv.w), hh[6], gp[2]); gp[3] = fmaf(dbf16hi(gv.w), hh[7], gp[3]);
                up[0] = fmaf(dbf16lo(uv.x), hh[0], up[0]); up[1] = fmaf(dbf16hi(uv.x), hh[1], up[1]);
                up[2] = fmaf(dbf16lo(uv.y), hh[2], up[2]); up[3] = fmaf(dbf16hi(uv.y), hh[3], up[3]);
                up[0] = fmaf(dbf16lo(uv.z), hh[4], up[0]); up[1] = fmaf(dbf16hi(uv.z), hh[5], up[1]);
                up[2] = fmaf(dbf16lo(uv.w), hh[6], up[2]); up[3] = fmaf(dbf16hi(uv.w), hh[7], up[3]);
              }
              float g = (gp[0] + gp[1]) + (gp[2] + gp[3]), u = (up[0] + up[1]) + (up[2] + up[3]);
#pragma unroll
              for (int o = 16; o > 0; o >>= 1) {  // the two reductions side by side
                const float g2 = __shfl_xor_sync(0xffffffffu, g, o), u2 = __shfl_xor_sync(0xffffffffu, u, o);
                g += g2;
                u += u2;
              }
              // SiLU with the fast exponential and reciprocal: relative error about 1e-6, far inside the output tolerance,
              // and a fifth of the row's dependent latency less than expf and an IEEE division
              const float a = gate * g * __fdividef(1.f, 1.f + __expf(-g)) * u;
#pragma unroll
              for (int c = 0; c < NCH; ++c) {
                const uint4 dv = reinterpret_cast<const uint4*>(ds)[c * 32 + lane];
                acc[c * 8 + 0] = fmaf(a, dbf16lo(dv.x), acc[c * 8 + 0]); acc[c * 8 + 1] = fmaf(a, dbf16hi(dv.x), acc[c * 8 + 1]);
                acc[c * 8 + 2] = fmaf(a, dbf16lo(dv.y), acc[c * 8 + 2]); acc[c * 8 + 3] = fmaf(a, dbf16hi(dv.y), acc[c * 8 + 3]);
                acc[c * 8 + 4] = fmaf(a, dbf16lo(dv.z), acc[c * 8 + 4]); acc[c * 8 + 5] = fmaf(a, dbf16hi(dv.z), acc[c * 8 + 5]);
                acc[c * 8 + 6] = fmaf(a, dbf16lo(dv.w), acc[c * 8 + 6]); acc[c * 8 + 7] = fmaf(a, dbf16hi(dv.w), acc[c * 8 + 7]);
              }
              }
            }
            __syncwarp();  // every lane has read stage s: it may be refilled
            ++q_con;
            ++n_con;
          }
          // the table is still unconfirmed: has the candidate mask arrived?
          if (!verified) {
            if (warp == 0) relay_cand_mask(false, __shfl_sync(0xffffffffu, seen, 0));
            if (!ok) break;
            if (__all_sync(0xffffffffu, mbar_try_wait(&s_pbar, lpar))) {
              if (!confirm_table()) break;
              if (changed) redo = true;  // the rows in flight are let land, nothing more is started, the layer's rows are repeated
            }
          }
          if (redo && q_con >= q_iss) break;
        }
      }
      if (pass == 0 && go_rows && ok && !verified) {  // (a warp with few rows can be done before the mask is there)
        if (wait_and_confirm() && changed) redo = true;
      }
      if (!(redo && ok && pass == 0)) break;
      derive_sets();  // the published table: which slots are ready, which experts are executed; then once more
    }
    if (poster && warp == 0 && planned && ok) {
      // what depends on the table: the execution set of the stall-free mode for the host, and the counters of S6
      if (lane == 0) {
        if (p.mode != APEX_MODE_EXACT)
          asm volatile("st.global.v4.u32 [%0], {%1, %2, %3, %4};" ::"l"(p.mbox[l].exec_rec), "r"((uint32_t)run), "r"((uint32_t)(run >> 32)),
                       "r"(p.seq), "r"(0u)
                       : "memory");
        DevStats* st = p.stats + l;
        const int ns = __popcll(run & ~kr_mask);
        if (ns) atomicAdd(&st->substitutions, (unsigned long long)ns);
        atomicAdd(&st->hits_R, (unsigned long long)__popcll(kr_mask & resident));
      }
    }
    if (p.standin_ahead && go_rows && ok) start_seg1(l + 1, NSW - 1);
    DTL(8);
    if (lane == 0 && waited && planned) {
      atomicAdd(&p.stats[l].stall_ns, waited * (unsigned long long)p.n_sm / (unsigned long long)G);  // the host divides by the SM count
      waited = 0;
    }

    // ------------------------------------------------------------ y: warps -> CTA -> cluster -> memory; count the CTA in
    // A warp's partial vector goes to the stage it would use next: free, because at most NSW - 1 of its copies (the
    // next layer's, started ahead) are outstanding.  After a failed wait nothing is written (the CTA contributes zeros).
    // (A quantised row is shorter than a vector of y: the warps' vectors then lie side by side at the start of the ring,
    // written once every warp of the CTA has consumed its rows; no copies are started ahead in that case.)
    constexpr bool RED_IN_STAGE = entry_bytes >= (uint32_t)d * 4u;
    const bool warp_good = go_rows && ok && (RED_IN_STAGE ? (n_iss - n_con) <= NSW - 1 : n_iss == n_con);
    if (lane == 0) s_red_stage[warp] = warp_good ? (RED_IN_STAGE ? warp + kDecWarps * (n_iss % NSW) : warp) : -1;
    if (!RED_IN_STAGE) __syncthreads();
    if (warp_good) {
      float4* dst = reinterpret_cast<float4*>(RED_IN_STAGE ? smem + (size_t)(warp + kDecWarps * (n_iss % NSW)) * entry_bytes
                                                           : smem + (size_t)warp * d * 4);
#pragma unroll
      for (int c = 0; c < NCH; ++c) {
        const int col4 = (c * 32 + lane) * 2;
        dst[col4] = make_float4(acc[c * 8 + 0], acc[c * 8 + 1], acc[c * 8 + 2], acc[c * 8 + 3]);
        dst[col4 + 1] = make_float4(acc[c * 8 + 4], acc[c * 8 + 5], acc[c * 8 + 6], acc[c * 8 + 7]);
      }
    }
    __syncthreads();
    if (tid < APEX_MAX_EXPERTS / 4) s_rank[tid] = 0u;  // every warp has read this layer's ranks; the next layer adds to zeros
    DTL(11);
    // the peers of this cluster have read this CTA's partial sums of the previous layer
    if (l > 0) asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
    for (int col4 = tid; col4 < d / 4; col4 += kDecThreads) {
      float4 sacc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int w = 0; w < kDecWarps; ++w) {
        const int st = s_red_stage[w];
        if (st >= 0) {
          const float4 v = reinterpret_cast<const float4*>(RED_IN_STAGE ? smem + (size_t)st * entry_bytes : smem + (size_t)st * d * 4)[col4];
          sacc.x += v.x; sacc.y += v.y; sacc.z += v.z; sacc.w += v.w;
        }
      }
      part4[col4] = sacc;
    }
    cluster_barrier();  // every CTA's partial y is complete (and the stages that held the warps' vectors are free again)
    DTL(12);
    if (p.standin_ahead && ok && !cta_stopped()) start_seg1(l + 1, NSW);
    if (tid < SLICE4) {
      // CTA r of the cluster adds columns [r * d/8, (r+1) * d/8) of the cluster's eight partial vectors to y
      const int col4 = (int)crank * SLICE4 + tid;
      float4 sacc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (uint32_t r = 0; r < (uint32_t)kDecCluster; ++r) {
        uint32_t ra;
        asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(ra) : "r"(smem_u32(part4 + col4)), "r"(r));
        float4 v;
        asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(ra) : "memory");
        sacc.x += v.x; sacc.y += v.y; sacc.z += v.z; sacc.w += v.w;
      }
      atomicAdd(reinterpret_cast<float4*>(p.y + (size_t)l * d) + col4, sacc);
    }
    __syncthreads();
    DTL(13);
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");  // done reading the peers' partial sums
    if (tid == 0) red_release_gpu_u64(bar_ffn, 1ull);  // this CTA's part of y[l] is in memory
    DTL(9);
  }

  // nothing may be in flight into this CTA's shared memory when it leaves
  while (n_con < n_iss) {
    const int s = warp + kDecWarps * (n_con % NSW);
    mbar_wait(&s_full[s], (uint32_t)((n_con / NSW) & 1), nullptr, p.wait_limit_ns);
    ++n_con;
  }
  if (lane == 0 && !ok) atomicAdd(&p.stats[0].timeouts, 1ull);
  if (tid == 0 && *(volatile int*)&s_abort) __threadfence_system();
  __syncthreads();
  if (L > 0) asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
  cluster_barrier();  // nobody leaves while a peer may still send into (or read from) its shared memory
  SPAN_END(10);
}

#ifdef APEX_TIMELINE
extern "C" int apex_debug_read_decode_timeline(unsigned long long* host) {
  return (int)cudaMemcpyFromSymbol(host, g_dec_tl, sizeof(g_dec_tl));
}
#endif

// ---------------------------------------------------------------- host side
namespace {

template <int NCH, int FMT = 0>
cudaError_t launch_decode_t(const DecodeParams& p, int n_clusters, cudaStream_t s, int* max_clusters_out) {
  constexpr bool HR = NCH <= 8;
  constexpr uint32_t entry = fmt_entry_bytes(FMT, NCH * 256);
  constexpr int NS = dec_ring_stages(entry, NCH * 256);
  const size_t smem = (size_t)NS * entry + (size_t)NCH * 256 * sizeof(float);  // ring, then the CTA's partial y
  static bool configured[kMaxDevices] = {};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  if (!configured[dev]) {
    e = cudaFuncSetAttribute(decode_token_kernel<NCH, HR, FMT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    configured[dev] = true;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.blockDim = dim3(kDecThreads, 1, 1);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = kDecCluster;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeCooperative;  // all CTAs resident together: they wait for one another
  attr[1].val.cooperative = 1;
  cfg.attrs = attr;
  if (max_clusters_out) {
    cfg.gridDim = dim3(kDecCluster, 1, 1);
    cfg.numAttrs = 1;
    int n = 0;
    e = cudaOccupancyMaxActiveClusters(&n, decode_token_kernel<NCH, HR, FMT>, &cfg);
    *max_clusters_out = e == cudaSuccess ? n : 0;
    return e;
  }
  cfg.gridDim = dim3(kDecCluster * n_clusters, 1, 1);
  cfg.numAttrs = 2;
  return cudaLaunchKernelEx(&cfg, decode_token_kernel<NCH, HR, FMT>, p);
}

template <int FMT>
cudaError_t dispatch_quantised(const DecodeParams& p, int n_clusters, cudaStream_t s, int* max_clusters_out) {
  switch (p.d) {  // the widths the quantised row decoders are built for
    case 512: return launch_decode_t<2, FMT>(p, n_clusters, s, max_clusters_out);
    case 1024: return launch_decode_t<4, FMT>(p, n_clusters, s, max_clusters_out);
    case 1536: return launch_decode_t<6, FMT>(p, n_clusters, s, max_clusters_out);
    case 2048: return launch_decode_t<8, FMT>(p, n_clusters, s, max_clusters_out);
    case 4096: return launch_decode_t<16, FMT>(p, n_clusters, s, max_clusters_out);
  }
  return cudaErrorInvalidValue;
}

cudaError_t dispatch(const DecodeParams& p, int n_clusters, cudaStream_t s, int* max_clusters_out) {
  if (p.fmt == kFmtE4m3) return dispatch_quantised<kFmtE4m3>(p, n_clusters, s, max_clusters_out);
  if (p.fmt == kFmtMxfp4) return dispatch_quantised<kFmtMxfp4>(p, n_clusters, s, max_clusters_out);
  switch (p.d) {
    case 256: return launch_decode_t<1>(p, n_clusters, s, max_clusters_out);
    case 512: return launch_decode_t<2>(p, n_clusters, s, max_clusters_out);
    case 768: return launch_decode_t<3>(p, n_clusters, s, max_clusters_out);
    case 1024: return launch_decode_t<4>(p, n_clusters, s, max_clusters_out);
    case 1536: return launch_decode_t<6>(p, n_clusters, s, max_clusters_out);
    case 2048: return launch_decode_t<8>(p, n_clusters, s, max_clusters_out);
    case 3072: return launch_decode_t<12>(p, n_clusters, s, max_clusters_out);
    case 4096: return launch_decode_t<16>(p, n_clusters, s, max_clusters_out);
  }
  return cudaErrorInvalidValue;
}

}  // namespace

int decode_max_clusters(int d, int fmt) {
  DecodeParams p{};
  p.d = d;
  p.fmt = fmt;
  int n = 0;
  if (dispatch(p, 0, nullptr, &n) != cudaSuccess) {
    cudaGetLastError();
    return 0;
  }
  return n;
}

cudaError_t launch_decode(const DecodeParams& p, int n_clusters, cudaStream_t s) { return dispatch(p, n_clusters, s, nullptr); }

}  // namespace apex

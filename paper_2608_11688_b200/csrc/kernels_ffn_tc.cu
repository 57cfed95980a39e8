// Batched expert FFN on the 5th-generation tensor cores (tcgen05 + TMEM), for decode steps with many
// tokens (Sec. V-B: several concurrent requests are decoded as one batch).
//
// With B tokens per step an expert serves several tokens, so its weights should be read once and
// applied to all of them: a grouped GEMM, one group per executed expert (plus the shared expert).
// The step is still HBM-bound (a few tens of flop per weight byte at most), so the kernels are
// organised around streaming the weights once; the tensor cores only keep arithmetic off the
// critical path.  "Swap-AB": the weight rows are the MMA's M dimension (128 per tile), the group's
// tokens are N (16..256), so a small token count does not waste a 128-row tile.
//
//   gather     X_g[pair][d] (bf16) = h'[token of pair]   (pairs are sorted by expert); zero y
//   gate/up    G, U [128 x n] = W_gate/up[128 rows of I x d] . X_g^T       accumulators in TMEM
//              a = g_pair * silu(G) * U  (fp32) is kept as TWO bf16 planes, a_hi = bf16(a) and
//              a_lo = bf16(a - a_hi), so feeding it back to the tensor cores loses 2^-17, not 2^-9
//                                                                            -> global scratch (L2)
//   down       D [128 cols of d x 2n] = downT[I x 128]^T . [a_hi ; a_lo]^T   (downT is MN-major; both planes
//              y[token][col] += D[:, j] + D[:, n + j]          fp32 atomics      in one MMA: N = 2n)
//              (at most 64 tokens per unit here; larger groups are split; the shared expert's longer K is cut
//              into chunks of I rows so that all units are about equally long)
//
// Measured on B200: an MMA with M = 128, K = 16 costs about 35-40 ns to issue whatever N is (it streams a
// 128 x 16 slice of A), so small-N "swap-AB" MMAs are bound by their count, not by their flops: eight per
// 64-wide K tile was the pace of both kernels until the two planes of the down projection were merged into
// one instruction.  Accumulators are double-buffered in TMEM (2 x 256 columns), so the epilogue of one unit
// overlaps the MMAs of the next.
//
// Operands reach shared memory through TMA tensor maps with the 128-byte swizzle and are consumed
// by tcgen05.mma through shared-memory descriptors (K-major for gate, up, X, A; MN-major for downT).
// One CTA per SM, three roles: two warps issue TMA loads (alternating K tiles; a single issuing
// thread cannot keep up with 16 KB tiles), one thread issues MMAs, four warps run the epilogue out
// of TMEM.  Every wait is bounded.
//
// Quantised stores (e4m3 codes with a scale per row vector, e2m1 codes with a power-of-two scale per 32
// elements) take the same path with one more role: the producers bring the raw code bytes (and, for e2m1,
// the scale bytes) of a K tile into a staging area of the stage, eight converter warps expand them to bf16
// in the swizzled operand layout the MMA descriptors expect, and the MMAs run as for a bf16 store.  Both code
// sets are exact in bf16 (3 and 1 mantissa bits), and so is an e2m1 value times its power-of-two scale, so
// the tensor cores see the dequantised weights exactly; the per-vector fp32 scales of an e4m3 row are not
// exact in bf16 and are applied in fp32 instead: gate and up scales to the accumulators, the down scale
// folded into the intermediate before it is split into its two bf16 planes.  HBM sees 1 or 0.53 bytes per
// weight; the expansion costs shared-memory bandwidth and ALU work that the streaming leaves idle.
#include <cuda.h>
#include <cuda_fp16.h>
#include <cuda_bf16.h>

#include "apex_internal.hpp"
#include "ptx.cuh"

namespace apex {

namespace {

constexpr int kProducerWarps = 2;  // TMA producers: K tile t is loaded by warp t mod 2
constexpr int kMmaWarp = kProducerWarps;
constexpr int kCvWarp0 = kProducerWarps + 1 + 4;  // first of the converter warps (quantised stores only)
constexpr int kCvThreads = 256;   // eight warps: two per scheduler, so one warp's shared-memory latency hides behind the other's arithmetic
// producers, MMA + TMEM owner, four epilogue warps; for a quantised store the converter warps as well
__host__ __device__ constexpr int tc_threads(int qf) { return (kProducerWarps + 1 + 4) * 32 + (qf ? kCvThreads : 0); }
__host__ __device__ constexpr int tc_tiles_per_stage(int phase, int qf) { return (phase == 2 && qf == 0) ? 2 : 1; }
// bytes of raw codes (and e2m1 scale bytes: 16 per row) a pipeline stage stages for the converters
__host__ __device__ constexpr int tc_raw_bytes(int phase, int qf) {
  return qf == 1 ? (phase == 1 ? 2 * 128 * 64 : 64 * 128) : qf == 2 ? (phase == 1 ? 2 * 128 * 32 + 2 * 128 * 16 : 64 * 64 + 64 * 16) : 0;
}
constexpr int kKTile = 64;       // K elements per pipeline stage (128 bytes: one swizzle span)
constexpr int kXRowsPerLoad = 8;    // rows per B-tile box: one 8-row swizzle atom, so a small group does not fetch rows it has no token for

__device__ __forceinline__ void tma_load_4d(void* dst, const CUtensorMap* map, int c0, int c1, int c2, int c3, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];" ::"r"(smem_u32(dst)),
      "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
      : "memory");
}
__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, int c0, int c1, uint64_t* bar) {
  asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];" ::"r"(smem_u32(dst)),
               "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1)
               : "memory");
}
__device__ __forceinline__ void tma_load_3d(void* dst, const CUtensorMap* map, int c0, int c1, int c2, uint64_t* bar) {
  asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];" ::"r"(smem_u32(dst)),
               "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2)
               : "memory");
}
// Expanding codes to bf16 with conversion instructions runs at a quarter of the plain ALU rate and was the pace of the
// whole kernel; the converters therefore build the bf16 bit patterns with integer operations and one bf16 multiply:
// a code's exponent and mantissa bits, placed at the top of a bf16's mantissa and the bottom of its exponent field,
// read as the code's value times 2^(code bias - 127), subnormal codes included (they become bf16 subnormals, which
// the multiply does not flush); the multiply by a power of two puts the exponent right and is exact.
__device__ __forceinline__ uint32_t mul_bf16x2(uint32_t a, uint32_t b) {
  uint32_t o;
  asm("mul.rn.bf16x2 %0, %1, %2;" : "=r"(o) : "r"(a), "r"(b));
  return o;
}
// four e4m3 codes (s eeee mmm, bias 7) -> four bf16 values
__device__ __forceinline__ void e4m3x4_to_bf16(uint32_t c, uint32_t& o0, uint32_t& o1) {
  const uint32_t k = 0x7B807B80u;                       // 2^120, twice
  const uint32_t r0 = __byte_perm(c, 0u, 0x1404u);      // codes 0, 1 in the high byte of each half
  const uint32_t r1 = __byte_perm(c, 0u, 0x3424u);      // codes 2, 3
  o0 = mul_bf16x2((r0 & 0x80008000u) | ((r0 >> 4) & 0x07f007f0u), k);
  o1 = mul_bf16x2((r1 & 0x80008000u) | ((r1 >> 4) & 0x07f007f0u), k);
}
// eight e2m1 codes (s ee m, bias 1; the even element in the low nibble of its byte) times the block scale
// 2^(sb - 127) (sb = 0: zero) -> eight bf16 values
__device__ __forceinline__ uint4 e2m1x8_to_bf16(uint32_t c, uint32_t sb) {
  uint32_t o[4];
  if (sb <= 128u) {
    // code bits as a bf16 read as value * 2^-126; times 2^126 * 2^(sb - 127) = 2^(sb - 1): one multiply
    const uint32_t m1 = sb ? (sb + 126u) << 7 : 0u;
    const uint32_t m = m1 | (m1 << 16);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const uint32_t t = __byte_perm(c, 0u, 0x4440u + j) * 4097u;   // low nibble at bits 0..3, high nibble at bits 16..19
      o[j] = mul_bf16x2(((t & 0x00080008u) << 12) | ((t & 0x00070007u) << 6), m);
    }
  } else {
    // scales above 2 (never produced for weights of ordinary size): through the conversion instructions
    const float scale = __uint_as_float(sb << 23);
    uint32_t h[4];
    asm("{\n.reg .b8 b0, b1, b2, b3;\n"
        "mov.b32 {b0, b1, b2, b3}, %4;\n"
        "cvt.rn.f16x2.e2m1x2 %0, b0;\n"
        "cvt.rn.f16x2.e2m1x2 %1, b1;\n"
        "cvt.rn.f16x2.e2m1x2 %2, b2;\n"
        "cvt.rn.f16x2.e2m1x2 %3, b3;\n}"
        : "=r"(h[0]), "=r"(h[1]), "=r"(h[2]), "=r"(h[3])
        : "r"(c));
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&h[j]));
      const __nv_bfloat162 b = __floats2bfloat162_rn(f.x * scale, f.y * scale);
      o[j] = *reinterpret_cast<const uint32_t*>(&b);
    }
  }
  return make_uint4(o[0], o[1], o[2], o[3]);
}
// shared-memory matrix descriptor, 128-byte swizzle (layout type 2), version 1
__device__ __forceinline__ uint64_t umma_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr >> 4) & 0x3FFF);
  d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFF) << 16;
  d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFF) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}
// instruction descriptor: bf16 x bf16 -> fp32, M x N, optional MN-major A
__device__ __forceinline__ uint32_t umma_idesc(int M, int N, int a_mn_major) {
  uint32_t d = 0;
  d |= 1u << 4;    // D fp32
  d |= 1u << 7;    // A bf16
  d |= 1u << 10;   // B bf16
  d |= (uint32_t)a_mn_major << 15;
  d |= (uint32_t)(N >> 3) << 17;
  d |= (uint32_t)(M >> 4) << 24;
  return d;
}
__device__ __forceinline__ void umma(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile("{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\ntcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}" ::"r"(tmem_d),
               "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
               : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
        "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]),
        "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]),
        "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

#ifdef APEX_TIMELINE
__device__ unsigned long long g_tc_tl[2][148][128];
#define TCTL(ph, i) do { if ((i) < 128) g_tc_tl[(ph) - 1][blockIdx.x][(i)] = globaltimer_ns(); } while (0)
// per K tile (the first 96 of a CTA): loads issued, raw bytes landed, operand buffer free, tiles converted; stage free
// (producer), operands complete (MMA thread), MMAs issued
__device__ unsigned long long g_cv_tl[2][148][96][8];
#define CVTL(ph, it, i) do { if ((it) < 96u) g_cv_tl[(ph) - 1][blockIdx.x][(it)][(i)] = globaltimer_ns(); } while (0)
#else
#define TCTL(ph, i) do { } while (0)
#define CVTL(ph, it, i) do { } while (0)
#endif

struct Group {
  int expert, pair_off, n_tok;
};
// One unit of work of a GEMM CTA: the (part of a) group, the M block and the K-tile range.
struct UnitDesc {
  int expert, pair_off, n_tok, blk, kt_begin, kt_end;
};
constexpr int kUnitChunk = 32;  // unit descriptors held in shared memory at a time
__device__ __forceinline__ Group load_group(const int32_t* grp, int g) {
  Group r;
  r.expert = grp[4 + 3 * g];
  r.pair_off = grp[5 + 3 * g];
  r.n_tok = grp[6 + 3 * g];
  return r;
}

}  // namespace

// ---------------------------------------------------------------- gather + zero
__global__ void __launch_bounds__(256) ffn_tc_gather_kernel(const TcParams p) {
  SPAN_BEGIN();
  pdl_wait();               // the plan kernel's pair list is complete from here on
  pdl_launch_dependents();  // the next kernel may start its prologue
  const int n_pairs = p.f.n_pairs[0];
  const int d = p.f.d;
  if (!p.f.accumulate) {
    float4* y4 = reinterpret_cast<float4*>(p.f.y);
    const size_t n4 = (size_t)p.f.B * d / 4;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += (size_t)gridDim.x * blockDim.x)
      y4[i] = make_float4(0.f, 0.f, 0.f, 0.f);
  }
  for (int pr = blockIdx.x; pr < n_pairs; pr += gridDim.x) {
    const int t = p.f.pair_tok[pr];
    const float4* src = reinterpret_cast<const float4*>(p.f.hpost + (size_t)t * d);
    uint2* dst = reinterpret_cast<uint2*>(p.xg + (size_t)pr * d);
    for (int c = threadIdx.x; c < d / 4; c += blockDim.x) {
      const float4 v = __ldg(src + c);
      __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y), hi = __floats2bfloat162_rn(v.z, v.w);
      uint2 o;
      o.x = *reinterpret_cast<uint32_t*>(&lo);
      o.y = *reinterpret_cast<uint32_t*>(&hi);
      dst[c] = o;
    }
  }
  SPAN_END(7);
}

// ---------------------------------------------------------------- the two GEMM kernels
// PHASE 1: gate/up.  A tiles: gate and up rows [128 x 64] (K-major), B tile: X_g rows [<=256 x 64].
// PHASE 2: down.     A tile: downT [64 k-rows x 128 cols] as two 64-column atoms (MN-major), B tile: the group's rows of
//                    a_hi, then of a_lo [2 x <=64 x 64].
//
// QF: storage format of the weights (0 bf16, 1 e4m3, 2 e2m1).  For QF != 0, tm_w / tm_ws cover the raw row bytes of
// the slots / the shared expert (boxes of one K tile's code bytes) and tm_sc / tm_ssc the same bytes with 16-byte boxes
// (the e2m1 scale bytes); a stage is [A tiles, bf16, written by the converters][B planes][raw bytes, written by TMA].
template <int PHASE, int QF>
__global__ void __launch_bounds__(tc_threads(QF), 1)
ffn_tc_gemm_kernel(const __grid_constant__ CUtensorMap tm_w, const __grid_constant__ CUtensorMap tm_ws,
                   const __grid_constant__ CUtensorMap tm_sc, const __grid_constant__ CUtensorMap tm_ssc,
                   const __grid_constant__ CUtensorMap tm_b, const __grid_constant__ CUtensorMap tm_b2, const TcParams p) {
  SPAN_BEGIN();
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  constexpr int A_BYTES = PHASE == 1 ? 2 * 128 * 128 : 2 * 64 * 128;  // gate+up tiles | two downT atoms
  constexpr int PLANES = PHASE == 1 ? 1 : 2;                          // X | a_hi and a_lo
  constexpr int MAX_STAGES = 8;
  // Tokens per unit (NMAX), hence the size of a B tile and the pipeline depth, are chosen per launch:
  // small batches get deep pipelines (more weight bytes in flight), large groups are cut into parts.
  const int NMAX = PHASE == 1 ? p.nmax1 : p.nmax2;
  const int B_PLANE = NMAX * 128;
  constexpr int RAW_BYTES = tc_raw_bytes(PHASE, QF);
  // K tiles per stage.  The down projection of a bf16 store puts two in a stage (each laid out as a stage of one): its
  // tiles are small (16 KB of weights) and cheap in MMAs (four), so the fixed cost of a stage -- a barrier round trip,
  // a commit, the producer's turn -- weighed as much as the tile itself (672 ns per tile, 3.5 TB/s while it streamed).
  constexpr int KPS = tc_tiles_per_stage(PHASE, QF);
  const int HALF_BYTES = A_BYTES + PLANES * B_PLANE;
  const int STAGE_BYTES = KPS * HALF_BYTES + RAW_BYTES;
  const int NSTAGE = PHASE == 1 ? p.nstage1 : p.nstage2;
  __shared__ uint64_t full[MAX_STAGES], empty[MAX_STAGES], rawfull[MAX_STAGES], tmem_full[2], tmem_empty[2];
  __shared__ uint32_t tmem_base_s;
  __shared__ int s_abort;
  __shared__ UnitDesc s_unit[kUnitChunk];
  __shared__ unsigned long long s_ready_mask;  // experts whose slot was seen ready in the prologue
  __shared__ int s_ustart[APEX_MAX_EXPERTS + 3];  // first unit of each group
  __shared__ int32_t s_grp[4 + 3 * (APEX_MAX_EXPERTS + 1)];

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int N = p.f.N, d = p.f.d, I = p.f.I, I_s = p.f.I_shared;
  const int32_t* grp = p.grp;

  if (tid == 0) {
    s_abort = 0;
    for (int s = 0; s < MAX_STAGES; ++s) {
      mbar_init(&full[s], QF ? 1 + kCvThreads / 32 : 1);  // the producer's arrival (B tile bytes) and one per converter warp
      mbar_init(&empty[s], 1);
      mbar_init(&rawfull[s], 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(&tmem_full[b], 1);
      mbar_init(&tmem_empty[b], 128);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_w) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_ws) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_b) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_b2) : "memory");
    if (QF == 2) {
      asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_sc) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_ssc) : "memory");
    }
  }
  if (warp == kMmaWarp) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_s)), "r"(512) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  // Slot-ready flags of all resident experts in one round of loads (neither the flags nor the snapshot come from the
  // preceding kernel): the producers then skip the per-unit check, a system-scope load and a proxy fence on their path
  // at every unit boundary, for every expert already seen ready here.
  if (warp == 0) {
    bool r0 = false, r1 = false;
    const int e0 = lane, e1 = lane + 32;
    if (e0 < N) {
      const int sl = p.f.snap.expert_slot[e0];
      if (sl >= 0) r0 = (int32_t)(ld_acquire_sys(p.f.slot_ready + sl) - p.f.snap.need_gen[e0]) >= 0;
    }
    if (e1 < N) {
      const int sl = p.f.snap.expert_slot[e1];
      if (sl >= 0) r1 = (int32_t)(ld_acquire_sys(p.f.slot_ready + sl) - p.f.snap.need_gen[e1]) >= 0;
    }
    const unsigned m0 = __ballot_sync(0xffffffffu, r0), m1 = __ballot_sync(0xffffffffu, r1);
    if (lane == 0) s_ready_mask = ((unsigned long long)m1 << 32) | m0;
    asm volatile("fence.proxy.async;" ::: "memory");  // the tensor-map loads that follow the barrier read what the flags cover
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_s;
  // everything above (barriers, TMEM, tensor-map prefetch, flags) is independent of the preceding kernel
  pdl_wait();
  pdl_launch_dependents();

  // the group table goes to shared memory once: a global load per unit would sit on every role's path
  for (int i = tid; i < 4 + 3 * (N + 1); i += (int)blockDim.x) s_grp[i] = grp[i];
  __syncthreads();
  const int n_rg = s_grp[0], n_g = s_grp[1];
  const int blocks_r = PHASE == 1 ? I / 128 : d / 128;                       // M blocks of a routed group
  const int blocks_s = PHASE == 1 ? (I_s > 0 ? I_s / 128 : 0) : d / 128;     // ... of the shared group
  const int kdim_r = PHASE == 1 ? d : I, kdim_s = PHASE == 1 ? d : I_s;
  // A group of n tokens is cut into ceil(n / NMAX) parts; a unit is (group, M block, part), parts
  // fastest so that the CTAs that share a weight block run at the same time (second reader hits L2).
  // The shared expert's down projection has a longer K (I_s) than a routed expert's (I): it is cut into
  // chunks of I rows, each a unit of its own (partial sums meet in y through the atomics), so that all
  // units of a launch are about equally long and the round-robin assignment stays balanced.
  const int kchunks_s = (PHASE == 2 && I_s > I) ? (I_s + I - 1) / I : 1;
  if (tid == 0) {
    int acc = 0;
    for (int g = 0; g < n_g; ++g) {
      s_ustart[g] = acc;
      const int parts = (s_grp[6 + 3 * g] + NMAX - 1) / NMAX;
      acc += (g < n_rg ? blocks_r : blocks_s * kchunks_s) * parts;
    }
    s_ustart[n_g] = acc;
  }
  __syncthreads();
  const int n_units = s_ustart[n_g];

  uint32_t it_load = 0, it_mma = 0, it_cv = 0;  // running K-tile counters of the producers, the MMA thread and the converters
  uint32_t unit_no = 0;              // units done by this CTA (phase of the TMEM barriers)
  // The units of this CTA (uu = blockIdx.x, + gridDim.x, ...) are described once, kUnitChunk at a time and a thread
  // per unit: group lookup and index arithmetic are then off every role's path at the unit boundaries, where that
  // cold code cost each role more than a microsecond per unit.
  for (int chunk0 = blockIdx.x; chunk0 < n_units; chunk0 += (int)gridDim.x * kUnitChunk) {
    if (tid < kUnitChunk) {
      // units are taken from the end of the list: the shared expert's (the widest token tiles, the longest epilogues)
      // come first, so that their epilogues overlap later units instead of forming the tail of the launch
      const int uf = chunk0 + tid * (int)gridDim.x;
      const int uu = n_units - 1 - uf;
      UnitDesc ud = {};
      if (uf < n_units) {
        int g = 0;
        while (uu >= s_ustart[g + 1]) ++g;
        Group gr = load_group(s_grp, g);
        const int parts = (gr.n_tok + NMAX - 1) / NMAX;
        const int local = uu - s_ustart[g];
        const bool shared = gr.expert >= N;
        const int kch = shared ? kchunks_s : 1;
        const int blk = local / (parts * kch), kc = (local / parts) % kch, sub = local % parts;
        const int kdim = shared ? kdim_s : kdim_r;
        ud.expert = gr.expert;
        ud.pair_off = gr.pair_off + sub * NMAX;
        ud.n_tok = gr.n_tok - sub * NMAX < NMAX ? gr.n_tok - sub * NMAX : NMAX;
        ud.blk = blk;
        ud.kt_begin = kch > 1 ? kc * (I / kKTile) : 0;  // K tiles of this unit
        ud.kt_end = kch > 1 ? (ud.kt_begin + I / kKTile < kdim / kKTile ? ud.kt_begin + I / kKTile : kdim / kKTile) : kdim / kKTile;
      }
      s_unit[tid] = ud;
    }
    __syncthreads();
  for (int uj = 0; uj < kUnitChunk && chunk0 + uj * (int)gridDim.x < n_units && !*(volatile int*)&s_abort; ++uj) {
    const UnitDesc ud = s_unit[uj];
    Group gr;
    gr.expert = ud.expert;
    gr.pair_off = ud.pair_off;
    gr.n_tok = ud.n_tok;
    const bool shared = gr.expert >= N;
    const int blk = ud.blk, kt_begin = ud.kt_begin, kt_end = ud.kt_end;
    const int n_pad = (gr.n_tok + 15) & ~15;                                  // MMA N
    const int n_loads = (gr.n_tok + kXRowsPerLoad - 1) / kXRowsPerLoad;       // 32-row boxes of the B tile

    if (warp < kProducerWarps) {
      // ================= TMA producers: the whole warp walks the K tiles; lane 0 owns the barriers and
      // each load of a stage is issued by a different lane (one thread sustains only about one bulk
      // copy per 570 cycles)
      int slot = 0;
      bool ok = true;
      if (!shared) {
        slot = p.f.snap.expert_slot[gr.expert];
        if (slot < 0) ok = false;
        if (ok && lane == 0 && !((s_ready_mask >> gr.expert) & 1ull)) {
          const uint32_t need = p.f.snap.need_gen[gr.expert];
          const uint32_t* flag = p.f.slot_ready + slot;
          if ((int32_t)(ld_acquire_sys(flag) - need) < 0) {
            const unsigned long long t0 = globaltimer_ns();
            while ((int32_t)(ld_acquire_sys(flag) - need) < 0) {
              if ((long long)(globaltimer_ns() - t0) > p.f.wait_limit_ns) {
                ok = false;
                break;
              }
              __nanosleep(64);
            }
            if (p.f.stats) atomicAdd(&p.f.stats->stall_ns, (globaltimer_ns() - t0) * (unsigned long long)gridDim.x / 4ull);
          }
          asm volatile("fence.proxy.async;" ::: "memory");
        }
        ok = __all_sync(0xffffffffu, ok);
        slot += p.layer_slot0;  // the tensor map covers the slots of all layers
      }
      const CUtensorMap* wmap = shared ? &tm_ws : &tm_w;
      constexpr int planes = PLANES;
      for (int kt = kt_begin; kt < kt_end && ok; kt += KPS, ++it_load) {
        if ((int)(it_load % kProducerWarps) != warp) continue;  // the other producer warp's stage
        const int s = it_load % NSTAGE;
        if (lane == 0) {
          if (it_load >= (uint32_t)NSTAGE && !mbar_wait(&empty[s], ((it_load / NSTAGE) - 1) & 1, &s_abort, p.f.wait_limit_ns)) ok = false;
          CVTL(PHASE, it_load, 4);
          if (ok) {
            mbar_expect_tx(&full[s], KPS * ((QF ? 0 : A_BYTES) + planes * n_loads * kXRowsPerLoad * 128));
            if (QF) mbar_expect_tx(&rawfull[s], RAW_BYTES);
          }
        }
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        uint8_t* st0 = smem + (size_t)s * STAGE_BYTES;
        // the weight loads first; then op n_wops + r*planes + pl: 8-row box r of B plane pl
        constexpr int n_wops = QF == 0 ? 2 : QF == 1 ? (PHASE == 1 ? 2 : 1) : (PHASE == 1 ? 4 : 2);
        const int n_ops = n_wops + planes * n_loads;
        uint8_t* raw = st0 + A_BYTES + planes * B_PLANE;
        const int kt0 = kt;
        for (int opx = lane; opx < KPS * n_ops; opx += 32) {
          const int half = KPS > 1 ? opx / n_ops : 0, op = KPS > 1 ? opx - half * n_ops : opx;
          const int kt = kt0 + half;                      // (shadows the stage's first tile)
          uint8_t* st = st0 + (size_t)half * HALF_BYTES;
          if (op < n_wops) {
            if (QF == 0) {
              if (PHASE == 1) tma_load_4d(st + op * 128 * 128, wmap, kt * kKTile, op, blk * 128, slot, &full[s]);   // gate | up rows
              else tma_load_4d(st + op * 64 * 128, wmap, blk * 128 + op * 64, 2, kt * kKTile, slot, &full[s]);      // downT, 64 columns
            } else if (QF == 1) {  // row: gate | up | downT codes (d bytes each), then the scales
              if (PHASE == 1) tma_load_3d(raw + op * 128 * 64, wmap, op * d + kt * kKTile, blk * 128, slot, &rawfull[s]);
              else tma_load_3d(raw, wmap, 2 * d + blk * 128, kt * kKTile, slot, &rawfull[s]);
            } else {  // row: gate | up | downT codes (d/2 bytes each), then their scale bytes (d/32 each)
              const CUtensorMap* smap = shared ? &tm_ssc : &tm_sc;
              if (PHASE == 1) {
                if (op < 2) tma_load_3d(raw + op * 128 * 32, wmap, op * (d / 2) + kt * (kKTile / 2), blk * 128, slot, &rawfull[s]);
                else tma_load_3d(raw + 2 * 128 * 32 + (op - 2) * 128 * 16, smap, 3 * (d / 2) + (op - 2) * (d / 32) + ((kt * 2) & ~15), blk * 128,
                                 slot, &rawfull[s]);
              } else {
                if (op == 0) tma_load_3d(raw, wmap, d + blk * 64, kt * kKTile, slot, &rawfull[s]);
                else tma_load_3d(raw + 64 * 64, smap, 3 * (d / 2) + 2 * (d / 32) + ((blk * 4) & ~15), kt * kKTile, slot, &rawfull[s]);
              }
            }
          } else {
            // B rows of this stage: the tokens' rows of plane 0, padded to n_pad, then those of plane 1
            const int r = (op - n_wops) / planes, pl = (op - n_wops) % planes;
            tma_load_2d(st + A_BYTES + pl * n_pad * 128 + r * kXRowsPerLoad * 128, pl ? &tm_b2 : &tm_b, kt * kKTile,
                        gr.pair_off + r * kXRowsPerLoad, &full[s]);
          }
        }
        __syncwarp();
        if (lane == 0) CVTL(PHASE, it_load, 0);
      }
      if (!ok && lane == 0) {
        atomicExch(&s_abort, 1);
        *p.f.mbox_status = 1u;
        if (p.f.stats) atomicAdd(&p.f.stats->timeouts, 1ull);
      }
    } else if (warp == kMmaWarp) {
      // ================= MMA issuer
      if (lane == 0) {
        bool ok = true;
        // two accumulator buffers of 256 TMEM columns: this unit's MMAs run while the epilogue warps
        // still read the previous unit's
        const uint32_t buf = unit_no & 1u;
        TCTL(PHASE, unit_no * 16 + 15);
        if (unit_no >= 2) ok = mbar_wait(&tmem_empty[buf], ((unit_no >> 1) - 1) & 1, &s_abort, p.f.wait_limit_ns);
        tc_fence_after();
        TCTL(PHASE, unit_no * 16);
        const uint32_t tacc = tmem_base + buf * 256u;
        // An MMA costs about 128 cycles whatever N is (it streams a 128 x 16 slice of A), so the down
        // projection multiplies both planes of the intermediate in one instruction: N = 2 * n_pad.
        const uint32_t idesc = umma_idesc(128, PHASE == 2 ? 2 * n_pad : n_pad, PHASE == 2 ? 1 : 0);
        const uint64_t desc_a0 = PHASE == 1 ? umma_desc(smem_u32(smem), 16, 1024) : umma_desc(smem_u32(smem), 64 * 128, 1024);
        const uint64_t desc_b0 = umma_desc(smem_u32(smem) + A_BYTES, 16, 1024);
        for (int kt = kt_begin; kt < kt_end && ok; kt += KPS, ++it_mma) {
          const int s = it_mma % NSTAGE;
          if (!mbar_wait(&full[s], (it_mma / NSTAGE) & 1, &s_abort, p.f.wait_limit_ns)) {
            ok = false;
            break;
          }
          if (kt - kt_begin < 10) TCTL(PHASE, unit_no * 16 + 1 + kt - kt_begin);
          CVTL(PHASE, it_mma, 5);
          tc_fence_after();
          // descriptors differ from the stage-0, k-step-0 ones only in the start-address field (address >> 4, the low
          // 14 bits; the sums below stay inside the CTA's shared memory, so nothing carries into the next field)
          const uint64_t soff = (uint64_t)((uint32_t)s * (uint32_t)STAGE_BYTES >> 4);
#pragma unroll
          for (int half = 0; half < KPS; ++half) {
          const uint64_t hoff = soff + (uint64_t)((uint32_t)half * (uint32_t)HALF_BYTES >> 4);
          const uint64_t da = desc_a0 + hoff, db = desc_b0 + hoff;
#pragma unroll
          for (int ks = 0; ks < kKTile / 16; ++ks) {
            const uint32_t acc = (kt > kt_begin || half > 0 || ks > 0) ? 1u : 0u;
            const uint64_t bdesc = db + (uint64_t)(ks * 2);   // 32 bytes per k-step
            if (PHASE == 1) {
              umma(tacc, da + (uint64_t)(ks * 2), bdesc, idesc, acc);                           // G
              umma(tacc + 128, da + (uint64_t)(128 * 128 / 16 + ks * 2), bdesc, idesc, acc);    // U
            } else {
              umma(tacc, da + (uint64_t)(ks * 128), bdesc, idesc, acc);  // 2 KB per k-step; columns [0, n_pad): a_hi, [n_pad, 2 n_pad): a_lo
            }
          }
          }
          umma_commit(&empty[s]);  // the stage is free once these MMAs have read it
          CVTL(PHASE, it_mma, 6);
        }
        TCTL(PHASE, unit_no * 16 + 11);
        if (ok) umma_commit(&tmem_full[buf]);
        else atomicExch(&s_abort, 1);
        TCTL(PHASE, unit_no * 16 + 14);
      }
    } else if (QF != 0 && warp >= kCvWarp0) {
      // ================= converters: raw codes of a stage -> bf16 operand tiles in the 128-byte-swizzled layout
      // (a tile row is 128 bytes = 64 values; its 16-byte chunk j sits at chunk j ^ (row mod 8))
      const int ct = tid - kCvWarp0 * 32;
      bool ok = true;
      for (int kt = kt_begin; kt < kt_end && ok; kt += KPS, ++it_cv) {
        const int s = it_cv % NSTAGE;
        ok = __all_sync(0xffffffffu, mbar_wait(&rawfull[s], (it_cv / NSTAGE) & 1, &s_abort, p.f.wait_limit_ns));
        if (ct == 0) CVTL(PHASE, it_cv, 1);
        if (!ok) break;
        uint8_t* st = smem + (size_t)s * STAGE_BYTES;
        const uint8_t* raw = st + A_BYTES + PLANES * B_PLANE;
        if (QF == 1 && PHASE == 1) {
          // two tiles [128 rows][64 codes]: chunk q of 16 codes -> two chunks of 8 bf16
#pragma unroll
          for (int q = ct; q < 1024; q += kCvThreads) {
            const int tile = q >> 9, row = (q & 511) >> 2, c = q & 3;
            const uint4 v = *reinterpret_cast<const uint4*>(raw + q * 16);
            uint4 o0, o1;
            e4m3x4_to_bf16(v.x, o0.x, o0.y);
            e4m3x4_to_bf16(v.y, o0.z, o0.w);
            e4m3x4_to_bf16(v.z, o1.x, o1.y);
            e4m3x4_to_bf16(v.w, o1.z, o1.w);
            uint8_t* dst = st + tile * (128 * 128) + row * 128;
            *reinterpret_cast<uint4*>(dst + (((2 * c) ^ (row & 7)) << 4)) = o0;
            *reinterpret_cast<uint4*>(dst + (((2 * c + 1) ^ (row & 7)) << 4)) = o1;
          }
        } else if (QF == 1) {
          // [64 k-rows][128 codes] -> two 64-column atoms, MN-major
#pragma unroll
          for (int q = ct; q < 512; q += kCvThreads) {
            const int kk = q >> 3, cc = q & 7;
            const uint4 v = *reinterpret_cast<const uint4*>(raw + q * 16);
            uint4 o0, o1;
            e4m3x4_to_bf16(v.x, o0.x, o0.y);
            e4m3x4_to_bf16(v.y, o0.z, o0.w);
            e4m3x4_to_bf16(v.z, o1.x, o1.y);
            e4m3x4_to_bf16(v.w, o1.z, o1.w);
            uint8_t* dst = st + (cc >> 2) * (64 * 128) + kk * 128;
            const int jc = (cc & 3) * 2;
            *reinterpret_cast<uint4*>(dst + ((jc ^ (kk & 7)) << 4)) = o0;
            *reinterpret_cast<uint4*>(dst + (((jc + 1) ^ (kk & 7)) << 4)) = o1;
          }
        } else if (PHASE == 1) {
          // two tiles [128 rows][32 bytes = 64 codes]: a 16-byte chunk is one 32-element scale block
          const uint8_t* rsc = raw + 2 * 128 * 32;
#pragma unroll
          for (int q = ct; q < 512; q += kCvThreads) {
            const int tile = q >> 8, row = (q & 255) >> 1, half = q & 1;
            const uint4 v = *reinterpret_cast<const uint4*>(raw + q * 16);
            const uint32_t sc = rsc[tile * (128 * 16) + row * 16 + ((kt * 2) & 15) + half];
            uint8_t* dst = st + tile * (128 * 128) + row * 128;
            const int jc = half * 4;
            *reinterpret_cast<uint4*>(dst + (((jc + 0) ^ (row & 7)) << 4)) = e2m1x8_to_bf16(v.x, sc);
            *reinterpret_cast<uint4*>(dst + (((jc + 1) ^ (row & 7)) << 4)) = e2m1x8_to_bf16(v.y, sc);
            *reinterpret_cast<uint4*>(dst + (((jc + 2) ^ (row & 7)) << 4)) = e2m1x8_to_bf16(v.z, sc);
            *reinterpret_cast<uint4*>(dst + (((jc + 3) ^ (row & 7)) << 4)) = e2m1x8_to_bf16(v.w, sc);
          }
        } else {
          // [64 k-rows][64 bytes = 128 codes]: chunk cb of a row is the scale block of columns 32 cb .. 32 cb + 31
          const uint8_t* rsc = raw + 64 * 64;
#pragma unroll
          for (int q = ct; q < 256; q += kCvThreads) {
            const int kk = q >> 2, cb = q & 3;
            const uint4 v = *reinterpret_cast<const uint4*>(raw + q * 16);
            const uint32_t sc = rsc[kk * 16 + ((blk * 4) & 15) + cb];
            uint8_t* dst = st + (cb >> 1) * (64 * 128) + kk * 128;
            const int jc = (cb & 1) * 4;
            *reinterpret_cast<uint4*>(dst + (((jc + 0) ^ (kk & 7)) << 4)) = e2m1x8_to_bf16(v.x, sc);
            *reinterpret_cast<uint4*>(dst + (((jc + 1) ^ (kk & 7)) << 4)) = e2m1x8_to_bf16(v.y, sc);
            *reinterpret_cast<uint4*>(dst + (((jc + 2) ^ (kk & 7)) << 4)) = e2m1x8_to_bf16(v.z, sc);
            *reinterpret_cast<uint4*>(dst + (((jc + 3) ^ (kk & 7)) << 4)) = e2m1x8_to_bf16(v.w, sc);
          }
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // the MMAs read these tiles through the async proxy
        __syncwarp();
        if (lane == 0) mbar_arrive(&full[s]);
        if (ct == 0) CVTL(PHASE, it_cv, 3);
      }
      if (!ok && lane == 0) atomicExch(&s_abort, 1);
    } else {
      // ================= epilogue: warp w owns TMEM lanes 32*(w%4) .. +31
      const int quad = warp & 3;
      const int row = quad * 32 + lane;  // row of the 128-row tile
      const uint32_t buf = unit_no & 1u;
      if (__all_sync(0xffffffffu, mbar_wait(&tmem_full[buf], (unit_no >> 1) & 1, &s_abort, p.f.wait_limit_ns))) {
        tc_fence_after();
        if (warp == kMmaWarp + 1 && lane == 0) TCTL(PHASE, unit_no * 16 + 12);
        for (int c0 = 0; c0 < gr.n_tok; c0 += 32) {
          uint32_t a[32];
          const uint32_t taddr = tmem_base + buf * 256u + ((uint32_t)(quad * 32) << 16) + (uint32_t)c0;
          tmem_ld32(taddr, a);
          uint32_t b2[32];
          tmem_ld32(taddr + (PHASE == 1 ? 128 : n_pad), b2);   // U | the a_lo half of the down product
          asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
          if (PHASE == 1) {
            const int i = blk * 128 + row;
            float sg = 1.f, su = 1.f, sd = 1.f;
            if (QF == 1) {  // the row's three fp32 scales follow its 3 d code bytes
              const uint8_t* wb = shared ? p.f.shared_w : p.f.cache + (size_t)p.f.snap.expert_slot[gr.expert] * p.f.slot_stride;
              const float* sc = reinterpret_cast<const float*>(wb + (size_t)i * (3u * d + 16u) + 3u * d);
              sg = __ldg(sc);
              su = __ldg(sc + 1);
              sd = __ldg(sc + 2);
            }
#pragma unroll
            for (int j = 0; j < 32; ++j) {
              if (c0 + j < gr.n_tok) {
                const float gq = sg * __uint_as_float(a[j]), uq = su * __uint_as_float(b2[j]);
                const float w = __ldg(p.f.pair_gate + gr.pair_off + c0 + j);
                const float v = w * (gq / (1.f + expf(-gq))) * uq * sd;
                const __nv_bfloat16 hi = __float2bfloat16(v);
                const size_t at = (size_t)(gr.pair_off + c0 + j) * p.act_stride + i;
                p.act[at] = hi;
                p.act[p.act_plane + at] = __float2bfloat16(v - __bfloat162float(hi));
              }
            }
          } else {
            const int col = blk * 128 + row;
#pragma unroll
            for (int j = 0; j < 32; ++j) {
              if (c0 + j < gr.n_tok) {
                const int t = __ldg(p.f.pair_tok + gr.pair_off + c0 + j);
                atomicAdd(p.f.y + (size_t)t * d + col, __uint_as_float(a[j]) + __uint_as_float(b2[j]));
              }
            }
          }
        }
      }
      tc_fence_before();
      if (warp == kMmaWarp + 1 && lane == 0) TCTL(PHASE, unit_no * 16 + 13);
      mbar_arrive(&tmem_empty[unit_no & 1u]);
    }
    ++unit_no;
    if (*(volatile int*)&s_abort) break;
  }
    __syncthreads();  // every role is done with this chunk's descriptors (after an abort the later chunks fall through)
  }
  tc_fence_before();
  __syncthreads();
  if (warp == kMmaWarp) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512) : "memory");
  SPAN_END(PHASE == 1 ? 8 : 9);
}

#ifdef APEX_TIMELINE
extern "C" int apex_debug_read_tc_timeline(unsigned long long* host) {
  return (int)cudaMemcpyFromSymbol(host, g_tc_tl, sizeof(g_tc_tl));
}
extern "C" int apex_debug_read_tc_converter_timeline(unsigned long long* host) {
  return (int)cudaMemcpyFromSymbol(host, g_cv_tl, sizeof(g_cv_tl));
}
#endif

// ---------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qr;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qr) == cudaSuccess && qr == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
    cudaGetLastError();
  }
  return fn;
}

// Weights of n_slots consecutive slots, each [I][3][d] bf16: dims (d, 3, I, n_slots); box (64, 1, box_rows, 1).
bool tc_make_weight_map(void* out, const void* base, int d, int I, size_t n_slots, size_t slot_bytes, int box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[4] = {(cuuint64_t)d, 3, (cuuint64_t)I, (cuuint64_t)n_slots};
  cuuint64_t strides[3] = {(cuuint64_t)d * 2, (cuuint64_t)d * 6, (cuuint64_t)slot_bytes};
  cuuint32_t box[4] = {64, 1, (cuuint32_t)box_rows, 1};
  cuuint32_t es[4] = {1, 1, 1, 1};
  return fn(reinterpret_cast<CUtensorMap*>(out), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, es,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Row-major bf16 matrix [rows][cols] with row stride `stride_elems`: dims (cols, rows); box (64, 32).
bool tc_make_rows_map(void* out, const void* base, int cols, size_t rows, size_t stride_elems) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)stride_elems * 2};
  cuuint32_t box[2] = {64, kXRowsPerLoad};
  cuuint32_t es[2] = {1, 1};
  return fn(reinterpret_cast<CUtensorMap*>(out), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, es,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Raw bytes of n_slots consecutive slots of a quantised store, each [I][row_bytes]: dims (row_bytes, I, n_slots);
// box (box_bytes, box_rows, 1), no swizzle (the converters read the staging area with plain loads).
bool tc_make_raw_map(void* out, const void* base, size_t row_bytes, int I, size_t n_slots, size_t slot_bytes, int box_bytes, int box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[3] = {(cuuint64_t)row_bytes, (cuuint64_t)I, (cuuint64_t)n_slots};
  cuuint64_t strides[2] = {(cuuint64_t)row_bytes, (cuuint64_t)slot_bytes};
  cuuint32_t box[3] = {(cuuint32_t)box_bytes, (cuuint32_t)box_rows, 1};
  cuuint32_t es[3] = {1, 1, 1};
  return fn(reinterpret_cast<CUtensorMap*>(out), CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, const_cast<void*>(base), dims, strides, box, es,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// The weight maps of one store (the slots of all layers, or one shared expert) for the storage format.
bool tc_make_store_maps(int fmt, void* gateup, void* down, void* sc_gateup, void* sc_down, const void* base, int d, int I, size_t n_slots,
                        size_t slot_bytes) {
  if (fmt == 0)
    return tc_make_weight_map(gateup, base, d, I, n_slots, slot_bytes, 128) && tc_make_weight_map(down, base, d, I, n_slots, slot_bytes, 64);
  const size_t rb = ffn_row_bytes(fmt, d);
  if (fmt == 1)  // a K tile of 64 codes is 64 bytes of a gate / up row; 128 columns of a downT row are 128 bytes
    return tc_make_raw_map(gateup, base, rb, I, n_slots, slot_bytes, 64, 128) && tc_make_raw_map(down, base, rb, I, n_slots, slot_bytes, 128, 64);
  return tc_make_raw_map(gateup, base, rb, I, n_slots, slot_bytes, 32, 128) && tc_make_raw_map(down, base, rb, I, n_slots, slot_bytes, 64, 64) &&
         tc_make_raw_map(sc_gateup, base, rb, I, n_slots, slot_bytes, 16, 128) && tc_make_raw_map(sc_down, base, rb, I, n_slots, slot_bytes, 16, 64);
}

bool tc_shape_supported(int d, int I, int I_shared, int fmt) {
  if (d % 128 != 0 || I % 128 != 0 || I_shared % 128 != 0) return false;
  if (fmt == 1) return d % 256 == 0;   // code offsets of a row stay 16-byte aligned
  if (fmt == 2) return d % 512 == 0;   // ... and so do the scale bytes of each vector (d / 32 of them)
  return true;
}

namespace {
template <int QF>
cudaError_t launch_tc_gemms(const TcParams& p, const TcMaps& m, cudaLaunchConfig_t& cfg, size_t ring1, size_t ring2, size_t st1, size_t st2) {
  const CUtensorMap* w1 = reinterpret_cast<const CUtensorMap*>(m.w_gateup);
  const CUtensorMap* ws1 = reinterpret_cast<const CUtensorMap*>(p.f.shared_w ? m.ws_gateup : m.w_gateup);
  const CUtensorMap* w2 = reinterpret_cast<const CUtensorMap*>(m.w_down);
  const CUtensorMap* ws2 = reinterpret_cast<const CUtensorMap*>(p.f.shared_w ? m.ws_down : m.w_down);
  // the 16-byte-box maps exist for the e2m1 store only; the other formats pass the weight maps again (never used)
  const CUtensorMap* c1 = QF == 2 ? reinterpret_cast<const CUtensorMap*>(m.sc_gateup) : w1;
  const CUtensorMap* cs1 = QF == 2 ? reinterpret_cast<const CUtensorMap*>(p.f.shared_w ? m.ssc_gateup : m.sc_gateup) : w1;
  const CUtensorMap* c2 = QF == 2 ? reinterpret_cast<const CUtensorMap*>(m.sc_down) : w2;
  const CUtensorMap* cs2 = QF == 2 ? reinterpret_cast<const CUtensorMap*>(p.f.shared_w ? m.ssc_down : m.sc_down) : w2;
  const CUtensorMap* xg = reinterpret_cast<const CUtensorMap*>(m.xg);
  cfg.blockDim = dim3(tc_threads(QF), 1, 1);
  // Each CTA allocates all 512 TMEM columns, so two CTAs must never share an SM (the second would sit in
  // tcgen05.alloc until the first has finished): ask for more than half an SM's shared memory in any case.
  const size_t one_per_sm = 120 * 1024;
  cfg.dynamicSmemBytes = ring1 + p.nstage1 * st1 + 1024 > one_per_sm ? ring1 + p.nstage1 * st1 + 1024 : one_per_sm;
  cudaError_t e = cudaLaunchKernelEx(&cfg, ffn_tc_gemm_kernel<1, QF>, *w1, *ws1, *c1, *cs1, *xg, *xg, p);
  if (e != cudaSuccess) return e;
  cfg.dynamicSmemBytes = ring2 + p.nstage2 * st2 + 1024 > one_per_sm ? ring2 + p.nstage2 * st2 + 1024 : one_per_sm;
  return cudaLaunchKernelEx(&cfg, ffn_tc_gemm_kernel<2, QF>, *w2, *ws2, *c2, *cs2, *reinterpret_cast<const CUtensorMap*>(m.act),
                            *reinterpret_cast<const CUtensorMap*>(m.act_lo), p);
}
template <int QF>
cudaError_t configure_tc(int budget) {
  cudaError_t e = cudaFuncSetAttribute(ffn_tc_gemm_kernel<1, QF>, cudaFuncAttributeMaxDynamicSharedMemorySize, budget);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(ffn_tc_gemm_kernel<2, QF>, cudaFuncAttributeMaxDynamicSharedMemorySize, budget);
}
}  // namespace

cudaError_t launch_ffn_tc(const TcParams& p_in, const TcMaps& m, int n_sm, cudaStream_t s) {
  static bool configured[kMaxDevices] = {};  // the attribute is per device
  const size_t budget = 196 * 1024;  // ring bytes per CTA
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev < 0 || dev >= kMaxDevices || !configured[dev]) {
    cudaError_t e = configure_tc<0>((int)budget + 1024);
    if (e == cudaSuccess) e = configure_tc<1>((int)budget + 1024);
    if (e == cudaSuccess) e = configure_tc<2>((int)budget + 1024);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < kMaxDevices) configured[dev] = true;
  }
  TcParams p = p_in;
  const int qf = p.f.fmt;
  const int b32 = (p.f.B + 31) & ~31;
  p.nmax1 = b32 < 128 ? b32 : 128;
  p.nmax2 = b32 < 64 ? b32 : 64;
  const size_t ring1 = 0, ring2 = 0;
  const size_t st1 = 2 * 128 * 128 + (size_t)p.nmax1 * 128 + tc_raw_bytes(1, qf);
  const size_t st2 = tc_tiles_per_stage(2, qf) * (2 * 64 * 128 + 2 * (size_t)p.nmax2 * 128) + tc_raw_bytes(2, qf);
  p.nstage1 = (int)(budget / st1) < 4 ? (int)(budget / st1) : 4;
  p.nstage2 = (int)(budget / st2) < 4 ? (int)(budget / st2) : 4;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;  // prologues overlap the preceding kernel's tail
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.stream = s;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cfg.gridDim = dim3(n_sm * 2, 1, 1);
  cfg.blockDim = dim3(256, 1, 1);
  cfg.dynamicSmemBytes = 0;
  cudaError_t e = cudaLaunchKernelEx(&cfg, ffn_tc_gather_kernel, p);
  if (e != cudaSuccess) return e;
  cfg.gridDim = dim3(n_sm, 1, 1);
  return qf == 1 ? launch_tc_gemms<1>(p, m, cfg, ring1, ring2, st1, st2)
                 : qf == 2 ? launch_tc_gemms<2>(p, m, cfg, ring1, ring2, st1, st2) : launch_tc_gemms<0>(p, m, cfg, ring1, ring2, st1, st2);
}

}  // namespace apex

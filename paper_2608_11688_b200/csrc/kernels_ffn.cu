// Expert FFN over the HBM slot cache: y = sum_{e in K~} g_e W_down,e ( silu(W_gate,e h') * (W_up,e h') )
// (Sec. III-A weighted sum of expert outputs; Sec. IV-E execution modes; Algorithm 1).
//
// The step is bandwidth-bound at decode batch sizes: every weight byte is used once per token.
// Layout: a slot holds [I][3][d] bf16 -- for intermediate index i the three d-vectors gate_i, up_i,
// downT_i are contiguous (downT is W_down transposed) -- so one pass suffices and every CTA reads one
// contiguous byte range:  a_i = g_e * silu(gate_i . h') * (up_i . h'),  y += a_i * downT_i.
//
// Kernel: persistent, one CTA per SM.  The (pair, i) row space -- a pair is (token, expert) -- is
// cut into equal contiguous ranges, one per CTA.  Each of the eight warps streams its own rows
// (row q of the CTA belongs to warp q mod 8) into its stages of a shared-memory ring with one bulk
// asynchronous copy per row (TMA, mbarrier completion; issuing from eight threads instead of one
// matters: one thread sustains only about one bulk copy per 570 cycles), does the two dot products
// with warp-shuffle reductions and accumulates the down projection in registers (fp32).  Partial y
// vectors are reduced across the warps of the CTA in shared memory and added to y with vector
// atomics.  Launched with programmatic stream serialization: the prologue overlaps the tail of the
// gate kernel.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "apex_internal.hpp"
#include "ptx.cuh"
#include "timeline.cuh"
#include "ffn_rows.cuh"
#include "token_plan.cuh"

namespace apex {

// Debug builds (-DAPEX_TIMELINE) record per-CTA time stamps of the streaming kernel.
#ifdef APEX_TIMELINE
__device__ unsigned long long g_timeline[1024 * 16];
#define TL(slot)                                                                      \
  do {                                                                                \
    g_timeline[blockIdx.x * 16 + (slot)] = (slot) == 0 ? globaltimer_ns_raw() : (unsigned long long)clock64(); \
  } while (0)
#define TLG(slot) do { g_timeline[blockIdx.x * 16 + (slot)] = globaltimer_ns_raw(); } while (0)
#else
#define TL(slot) do { } while (0)
#define TLG(slot) do { } while (0)
#endif

#ifndef APEX_FFN_WARPS
#define APEX_FFN_WARPS 8
#endif
#ifndef APEX_FFN_CTAS_PER_SM
#define APEX_FFN_CTAS_PER_SM 1
#endif
constexpr int kConsumerWarps = APEX_FFN_WARPS;
constexpr int kCtasPerSm = APEX_FFN_CTAS_PER_SM;
constexpr int kFfnThreads = kConsumerWarps * 32;
constexpr int kMaxStages = 64;
// ring bytes; static tables fit in what is left of the 227 KB per-CTA limit (of half an SM's 228 KB with two CTAs per SM)
constexpr int kSmemBudget = kCtasPerSm == 1 ? 224 * 1024 : 110 * 1024;

__host__ __device__ constexpr int ring_stages(uint32_t entry_bytes) {
  int n = kSmemBudget / (int)entry_bytes;
  if (n > kMaxStages) n = kMaxStages;
  return n / kConsumerWarps * kConsumerWarps;
}

// ---------------------------------------------------------------- the streaming FFN kernel
// Row space: pair p (a (token, expert) pair; routed pairs first, then the shared-expert pairs) owns
// I (or I_shared) consecutive rows; row r of pair p is intermediate index i = r - offset(p).
struct RowMap {
  int n_routed;          // routed pairs
  int n_pairs;           // all pairs
  int routed_rows;       // n_routed * I (the host refuses shapes whose row count does not fit 31 bits)
  int total_rows;
};


template <int NCH, bool H_REGS, int FMT>
__global__ void __launch_bounds__(kFfnThreads, kCtasPerSm) moe_ffn_stream_kernel(const FfnParams p) {
  extern __shared__ __align__(128) uint8_t smem[];
  __shared__ uint64_t s_full[kMaxStages];
  __shared__ float s_gate[kMaxStages];
  __shared__ int s_tok[kMaxStages];
  __shared__ int s_exp[kMaxStages];
  __shared__ int s_pos[kConsumerWarps][APEX_MAX_TOPK];  // B == 1: expert at each position of the row space (a copy per warp)
  __shared__ int s_abort;

  constexpr int d = NCH * 256;
  constexpr uint32_t row_bytes = fmt_vec_bytes(FMT, d);      // one of the three vectors of a row
  constexpr uint32_t entry_bytes = fmt_entry_bytes(FMT, d);  // the three vectors and, for the quantised formats, their scales
  // Each warp streams its own rows: it owns the ring stages {w, w+8, ...} and keeps NSW of its rows
  // in flight, so a stage is produced and consumed by the same warp (no "empty" barriers, and a
  // parity wait can never be a phase ahead).
  constexpr int NS = ring_stages(entry_bytes);
  constexpr int NSW = NS / kConsumerWarps;
  static_assert(NS >= kConsumerWarps && NS % kConsumerWarps == 0, "ring depth must be a multiple of the warp count");
  static_assert(NS * entry_bytes >= kConsumerWarps * d * 4, "ring must also hold the cross-warp reduction buffer");

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int N = p.N, k = p.k, I = p.I, B = p.B;
  const int G = gridDim.x, cta = blockIdx.x;

  // ---- work that does not depend on the preceding kernel
  SPAN_BEGIN();
  if (tid == 0) {
    TL(0);
    TL(1);
    s_abort = 0;
    if (cta == 0) *p.ticket_reset = 0u;  // the counter of a launch far in the future (nobody uses it now)
  }
  if (tid < NS) mbar_init(&s_full[tid], 1);
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  __syncthreads();  // barriers initialised
  float hreg[H_REGS ? NCH * 8 : 1];
  int cur_tok = -1;
  if (H_REGS && B == 1) {  // h' is an input of the gate kernel as well: complete long before this kernel
    cur_tok = 0;
#pragma unroll
    for (int c = 0; c < NCH; ++c) {
      const float4 a = __ldg(reinterpret_cast<const float4*>(p.hpost) + (c * 32 + lane) * 2);
      const float4 b2 = __ldg(reinterpret_cast<const float4*>(p.hpost) + (c * 32 + lane) * 2 + 1);
      hreg[c * 8 + 0] = a.x; hreg[c * 8 + 1] = a.y; hreg[c * 8 + 2] = a.z; hreg[c * 8 + 3] = a.w;
      hreg[c * 8 + 4] = b2.x; hreg[c * 8 + 5] = b2.y; hreg[c * 8 + 6] = b2.z; hreg[c * 8 + 7] = b2.w;
    }
  }
  // y is zeroed by all CTAs together (a slice each) and the slice is published through a counter.
  // Before the dependency wait when the host knows that the preceding kernel does not touch y (the
  // usual case: the gate kernel), after it otherwise.
  auto zero_slice = [&]() {
    if (p.accumulate) return;
    const size_t n4 = (size_t)B * d / 4;
    const size_t per = (n4 + G - 1) / G;
    const size_t lo = per * cta, hi = lo + per < n4 ? lo + per : n4;
    float4* y4 = reinterpret_cast<float4*>(p.y);
    for (size_t i = lo + tid; i < hi; i += kFfnThreads) y4[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    __syncthreads();
    if (tid == 0) {
      __threadfence();
      atomicAdd(p.zero_counter, 1ull);
    }
  };
  if (p.zero_early) zero_slice();

  // Slot-ready flags: lanes own experts lane and lane+32.  The flag is written by the copy engine
  // after the expert's bytes; a relaxed load suffices here because the bulk copies that follow are
  // issued only after the value has been inspected (and they read through L2, like the flag).
  // Neither the flags nor the slot snapshot come from the preceding kernel.
  const int sl0 = lane < N ? p.snap.expert_slot[lane] : -1, sl1 = lane + 32 < N ? p.snap.expert_slot[lane + 32] : -1;
  const uint32_t f0 = sl0 >= 0 ? ld_relaxed_sys(p.slot_ready + sl0) : 0u;
  const uint32_t f1 = sl1 >= 0 ? ld_relaxed_sys(p.slot_ready + sl1) : 0u;
  unsigned long long ready_mask;
  {
    const bool r0 = sl0 >= 0 && (int32_t)(f0 - p.snap.need_gen[lane]) >= 0;
    const bool r1 = sl1 >= 0 && (int32_t)(f1 - p.snap.need_gen[(lane + 32) & 63]) >= 0;
    ready_mask = ((unsigned long long)__ballot_sync(0xffffffffu, r1) << 32) | __ballot_sync(0xffffffffu, r0);
  }

  // Row space and work split.  Short launches (fewer than two ring fills per CTA): equal contiguous
  // ranges, all known at launch, no shared counter (a ticket per row costs more than it balances
  // there: every warp would hit one counter within the same microsecond).  Long launches: every CTA
  // owns NS (the ring depth) consecutive rows, so all its stages are filled at once, and the remaining
  // rows are handed out in tickets from a global counter to whichever warp has a free stage first.
  RowMap rm;
  bool dynamic = false;
  int S = 0, chunk = 1, n_static = 0;
  int static_base = 0, dyn_begin = 0, dyn_rows = 0;
  auto set_geometry = [&](int n_routed, int n_pairs) {
    rm.n_routed = n_routed;
    rm.n_pairs = n_pairs;
    rm.routed_rows = n_routed * I;
    rm.total_rows = rm.routed_rows + (n_pairs - n_routed) * p.I_shared;
    const int per_cta = rm.total_rows / G, extra = rm.total_rows - per_cta * G;  // the first `extra` CTAs take one row more
    dynamic = per_cta >= 2 * NS;
    const int range_lo = cta * per_cta + (cta < extra ? cta : extra), range_hi = range_lo + per_cta + (cta < extra ? 1 : 0);
    S = dynamic ? NS : (int)(range_hi - range_lo);  // rows this CTA knows about at launch
    static_base = dynamic ? cta * NS : range_lo;
    dyn_begin = dynamic ? G * NS : rm.total_rows;
    dyn_rows = rm.total_rows - dyn_begin;
    const int per_ticket = (dyn_rows + G * kConsumerWarps * 4 - 1) / (G * kConsumerWarps * 4);
    chunk = per_ticket > 1 ? (int)per_ticket : 1;   // rows per ticket: about four tickets per warp
    n_static = S > warp ? (S - warp + kConsumerWarps - 1) / kConsumerWarps : 0;  // static rows of this warp
  };
  // (position in the row space, index inside the expert) of row r
  auto locate = [&](int r, int* pidx, int* i) {
    if (r < rm.routed_rows) {
      *pidx = (int)(r / I);
      *i = r - *pidx * I;
    } else {
      *pidx = rm.n_routed + (int)((r - rm.routed_rows) / p.I_shared);
      *i = r - rm.routed_rows - (*pidx - rm.n_routed) * p.I_shared;
    }
  };

  // ---- speculative first fill (B == 1).  The prefetch router ranked this step's experts long ago;
  // its first k are the best guess of the routed set.  Their rows are requested now, while the gate
  // kernel is still running; after the dependency wait each guess is either confirmed (the copy is
  // already in flight or has landed) or dropped and its stage refilled.  Positions of the row space
  // that hold a confirmed guess keep it, so confirmed rows stay with the CTA that requested them.
  bool spec_on = B == 1 && p.spec != nullptr;
  int spec_e = -1;
  bool spec_issued = false;  // this lane started a speculative copy into its stage (stage index = lane)
  if (spec_on) {
    spec_e = lane < k ? __ldg(p.spec + lane) : -1;
    const unsigned kmask = k >= 32 ? 0xffffffffu : ((1u << k) - 1u);
    const bool bad = lane < k && (spec_e < 0 || spec_e >= N);
    const unsigned same = __match_any_sync(0xffffffffu, spec_e);
    const bool dup = lane < k && (same & kmask) != (1u << lane);
    spec_on = !__any_sync(0xffffffffu, bad || dup);
  }
  if (spec_on) {
    if (lane < k) s_pos[warp][lane] = spec_e;
    __syncwarp();
    if (p.spec_delay_ns > 0) {
      // When the preceding kernel is the (latency-bound) gate, flooding the memory system at once delays the
      // gate's own few loads by as much as the speculation saves: hold the copies back for a moment.
      const unsigned long long t0 = globaltimer_ns();
      while ((long long)(globaltimer_ns() - t0) < p.spec_delay_ns) __nanosleep(200);
    }
    set_geometry(k, k + (p.run_shared ? 1 : 0));
    const int fill = n_static < NSW ? n_static : NSW;
    if (lane < fill) {
      int pidx;
      int i;
      locate(static_base + warp + kConsumerWarps * lane, &pidx, &i);
      const int e = pidx < k ? s_pos[warp][pidx] : N;
      const uint8_t* base = nullptr;
      if (e >= N) {
        base = p.shared_w;
      } else if ((ready_mask >> e) & 1) {
        base = p.cache + (size_t)p.snap.expert_slot[e] * p.slot_stride;
      }
      if (base) {
        const int s = warp + kConsumerWarps * lane;
        s_gate[s] = 0.f;
        s_tok[s] = 0;
        s_exp[s] = e;
        mbar_expect_tx(&s_full[s], entry_bytes);
        bulk_g2s(smem + (size_t)s * entry_bytes, base + (size_t)i * entry_bytes, entry_bytes, &s_full[s]);
        spec_issued = true;
      }
    }
  }

  pdl_wait();               // the gate's outputs (K_r, alpha, z_r) are complete from here on
  pdl_launch_dependents();  // the next kernel may start its own prologue
  if (tid == 0) TL(4);
  if (tid == 0) TLG(11);
  if (!p.zero_early) zero_slice();  // a preceding launch of this library may still be adding to the same y

  // ---- every global load of the prologue is issued before the first use, so the latencies overlap.
  TokenLoads tl1;
  if (B == 1) tl1 = load_token(p.idx, p.z_r, p.alpha, N, k, p.mode, lane);
  if (tid == 0) TL(10);

  // ---- plan: B == 1 every warp derives the execution set itself; B > 1 the plan kernel wrote it
  unsigned long long run = 0;
  float g0 = 0.f, g1 = 0.f;
  TokenPlan tp1;
  tp1.exec_mask = tp1.kr_mask = 0ull;
  tp1.g0 = tp1.g1 = 0.f;
  bool spec_geometry = false;  // the speculative row space is the final one
  if (B == 1) {
    const TokenPlan tp = plan_token(tl1, p.mode, p.norm_topk, p.snap.resident_mask, lane);
    g0 = tp.g0;
    g1 = tp.g1;
    tp1 = tp;
    run = tp.exec_mask & p.run_mask;
    const int n_routed = __popcll(run);
    spec_geometry = spec_on && n_routed == k;
    int pos_e = -1;
    if (spec_geometry) {
      // a confirmed guess keeps its position; the other executed experts fill the gaps in ascending order
      const bool keep = lane < k && ((run >> spec_e) & 1ull);
      const unsigned keep_lanes = __ballot_sync(0xffffffffu, keep);
      const unsigned lo = __reduce_or_sync(0xffffffffu, keep && spec_e < 32 ? (1u << spec_e) : 0u);
      const unsigned hi = __reduce_or_sync(0xffffffffu, keep && spec_e >= 32 ? (1u << (spec_e - 32)) : 0u);
      const unsigned long long rest = run & ~(((unsigned long long)hi << 32) | lo);
      const unsigned gaps = ~keep_lanes & (k >= 32 ? 0xffffffffu : ((1u << k) - 1u));
      if (lane < k) pos_e = keep ? spec_e : nth_set_bit64(rest, __popc(gaps & ((1u << lane) - 1u)));
    } else {
      if (lane < n_routed) pos_e = nth_set_bit64(run, lane);
      set_geometry(n_routed, n_routed + (p.run_shared ? 1 : 0));
    }
    if (lane < APEX_MAX_TOPK) s_pos[warp][lane] = pos_e;
    __syncwarp();
  } else {
    const int n_pairs = p.n_pairs[0];
    set_geometry(n_pairs - (p.run_shared ? B : 0), n_pairs);
  }
  if (tid == 0) TL(2);  // plan done

  float acc[NCH * 8];
#pragma unroll
  for (int i = 0; i < NCH * 8; ++i) acc[i] = 0.f;
  const float* hrow = p.hpost;
  bool zero_seen = p.accumulate != 0;
  bool ok = true;
  unsigned long long waited = 0;
  int dm_e = -1, dm_slot = -1;  // last expert this lane had to wait for on demand

  auto poll_zeroed = [&](bool spin) {  // y must be all zero before anybody adds to it
    if (zero_seen) return;
    if (ld_acquire_gpu_u64(p.zero_counter) >= p.zero_target) {
      zero_seen = true;
      return;
    }
    if (!spin) return;
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

  // Starts the copy of row r as this warp's n-th row, into stage (n mod NSW) of the warp.
  auto issue = [&](int r, int n) {
    int pidx, e, tok, i;
    float gate = 0.f;
    locate(r, &pidx, &i);
    if (B == 1) {
      e = pidx < rm.n_routed ? s_pos[warp][pidx] : N;
      tok = 0;
    } else {
      e = p.pair_expert[pidx];
      tok = p.pair_tok[pidx];
      gate = p.pair_gate[pidx];
    }
    const uint8_t* base;
    if (e < N) {
      int slot = p.snap.expert_slot[e];
      if (slot < 0) {
        // not resident when the kernel was launched: the host fetches it on demand and publishes
        // (tag, slot) after the copy -- asynchronous miss correction inside one launch
        if (!p.demand_in_kernel) {  // refuse rather than read out of range
          ok = false;
          return;
        }
        if (e == dm_e) {
          slot = dm_slot;
        } else {
          const uint32_t* w = p.demand + e;
          uint32_t v = ld_acquire_sys(w);
          if ((v >> 8) != p.demand_tag) {
            const unsigned long long t0 = globaltimer_ns();
            while (((v = ld_acquire_sys(w)) >> 8) != p.demand_tag) {
              if ((long long)(globaltimer_ns() - t0) > p.wait_limit_ns) {
                ok = false;
                break;
              }
              __nanosleep(128);
            }
            waited += globaltimer_ns() - t0;
            if (!ok) return;
          }
          slot = (int)(v & 0xffu);
          if (slot >= p.C) {  // a published slot outside the cache: refuse rather than read out of range
            ok = false;
            return;
          }
          dm_e = e;
          dm_slot = slot;
          asm volatile("fence.proxy.async;" ::: "memory");
        }
      } else if (!((ready_mask >> e) & 1)) {
        const uint32_t need = p.snap.need_gen[e];
        const uint32_t* flag = p.slot_ready + slot;
        const unsigned long long t0 = globaltimer_ns();
        while ((int32_t)(ld_acquire_sys(flag) - need) < 0) {
          if ((long long)(globaltimer_ns() - t0) > p.wait_limit_ns) {
            ok = false;
            break;
          }
          __nanosleep(64);
        }
        waited += globaltimer_ns() - t0;
        if (!ok) return;
        ready_mask |= 1ull << e;
        asm volatile("fence.proxy.async;" ::: "memory");
      }
      base = p.cache + (size_t)slot * p.slot_stride;
    } else {
      base = p.shared_w;
    }
    const int s = warp + kConsumerWarps * (n % NSW);
    s_gate[s] = gate;
    s_tok[s] = tok;
    s_exp[s] = e;
    mbar_expect_tx(&s_full[s], entry_bytes);
    bulk_g2s(smem + (size_t)s * entry_bytes, base + (size_t)i * entry_bytes, entry_bytes, &s_full[s]);
  };

  auto post_plan = [&]() {
    // The routed and the execution set go to the caller's buffers and, as masks, to the host mailbox: each in ONE
    // aligned 16-byte store that carries its own sequence number, so no system-scope fence (a round trip over the
    // host link) sits in this warp's way -- it has rows to stream like every other warp.
    store_token_plan(tp1, lane, k, p.exec_idx, p.exec_gate, nullptr);
    if (lane == 0) {
      if (p.stats) {
        const int ns = __popcll(tp1.exec_mask & ~tp1.kr_mask);
        if (ns) atomicAdd(&p.stats->substitutions, (unsigned long long)ns);
        atomicAdd(&p.stats->hits_R, (unsigned long long)__popcll(tp1.kr_mask & p.snap.resident_mask));
      }
      asm volatile("st.global.v4.u32 [%0], {%1, %2, %3, %4};" ::"l"(p.mbox_rec), "r"((uint32_t)tp1.kr_mask),
                   "r"((uint32_t)(tp1.kr_mask >> 32)), "r"(p.seq_value), "r"(0u)
                   : "memory");
      asm volatile("st.global.v4.u32 [%0], {%1, %2, %3, %4};" ::"l"(p.mbox_rec + 4), "r"((uint32_t)tp1.exec_mask),
                   "r"((uint32_t)(tp1.exec_mask >> 32)), "r"(p.seq_value), "r"(0u)
                   : "memory");
    }
  };
  const bool poster = B == 1 && cta == 0 && warp == 0 && p.post_exec;
  // If an expert of this launch still has to be fetched, the host cannot start before it has seen
  // K_r: post first.  Otherwise post while the first rows are in flight.
  const bool will_wait_for_host = p.demand_in_kernel && (run & ~p.snap.resident_mask) != 0ull;
  if (poster && will_wait_for_host) post_plan();
  // ---- row supply of this warp (state lives in lane 0; the other lanes learn the outcome by shuffle)
  int next_static = 0;                 // static rows of this warp already started
  int dyn_cur = 0, dyn_end = 0;  // rows of the current ticket
  bool dyn_done = dyn_rows <= 0;
  auto next_row = [&]() -> int {  // lane 0 only
    if (next_static < n_static) return static_base + warp + kConsumerWarps * next_static++;
    if (dyn_cur < dyn_end) return dyn_cur++;
    if (dyn_done) return -1;
    // Tickets are taken on demand, never ahead: the rows must go to the warps that are free first
    // (all stages of all SMs are requested at once at the start, and which SM is served first is a
    // matter of queueing; an SM whose first rows land late should not also hold extra rows).
    const unsigned int ticket = atomicAdd(p.ticket, 1u);
    // (the host bounds the row count well below 2^31, and at most a few hundred tickets overshoot the end)
    const long long first64 = (long long)dyn_begin + (long long)ticket * chunk;
    if (first64 >= rm.total_rows) {
      dyn_done = true;
      return -1;
    }
    const int first = (int)first64;
    dyn_cur = first;
    dyn_end = first + chunk < rm.total_rows ? first + chunk : rm.total_rows;
    return dyn_cur++;
  };
  // first fill: the static rows go out from NSW lanes in one instruction.  A speculative copy that
  // was confirmed is this lane's first row already; one that was not has to land (nothing cancels
  // a bulk copy) before its stage is filled again, and from then on that stage's barrier runs one
  // phase ahead of the row count.
  const int first_fill = n_static < NSW ? n_static : NSW;
  bool dropped = false;
  if (spec_issued) {
    bool confirmed = false;
    if (spec_geometry && lane < first_fill) {
      int pidx;
      int i;
      locate(static_base + warp + kConsumerWarps * lane, &pidx, &i);
      confirmed = s_exp[warp + kConsumerWarps * lane] == (pidx < rm.n_routed ? s_pos[warp][pidx] : N);
    }
    if (!confirmed) {
      dropped = true;
      spec_issued = false;
      if (!mbar_wait(&s_full[warp + kConsumerWarps * lane], 0u, nullptr, p.wait_limit_ns)) ok = false;
    }
  }
  const unsigned phase_ahead = __ballot_sync(0xffffffffu, dropped);  // bit n: stage n of this warp
  if (lane < first_fill && !spec_issued && ok) {
    if (lane == 0 && warp == 0) TL(3);
    issue(static_base + warp + kConsumerWarps * lane, lane);
  }
  if (!ok) atomicExch(&s_abort, 1);
  __syncwarp();
  int tail = first_fill;  // rows of this warp whose copy has been started (uniform across the warp)
  next_static = first_fill;
  if (poster && !will_wait_for_host) post_plan();
  // a warp with fewer static rows than stages tops up from the dynamic part
  while (tail < NSW) {
    int more = 0;
    if (lane == 0 && ok) {
      const int r = next_row();
      if (r >= 0) {
        issue(r, tail);
        if (!ok) atomicExch(&s_abort, 1);
        more = ok ? 1 : 0;
      }
    }
    more = __shfl_sync(0xffffffffu, more, 0);
    if (!more) break;
    ++tail;
  }
  bool polled = false;
  float sgate = -1.f;  // B == 1: value of the shared expert's gate, once computed
  for (int head = 0; head < tail; ++head) {
    if (__any_sync(0xffffffffu, *(volatile int*)&s_abort != 0)) break;
    const int s = warp + kConsumerWarps * (head % NSW);
    const uint32_t parity = (uint32_t)((head / NSW + ((phase_ahead >> (head % NSW)) & 1u)) & 1);
    if (!__all_sync(0xffffffffu, mbar_wait(&s_full[s], parity, &s_abort, p.wait_limit_ns))) {
      atomicExch(&s_abort, 1);
      break;
    }
    if (lane == 0 && warp == 0 && head == 0) TL(5);
    if (lane == 0 && warp == 0) TL(6);
    const int e = s_exp[s];
    const int tok = s_tok[s];
    float gate;
    if (B == 1) {
      gate = __shfl_sync(0xffffffffu, e < 32 ? g0 : g1, e & 31);
      if (e >= N) {  // the shared expert: weight 1, or its gate's value (computed when the warp meets its first shared row)
        if (p.shared_gate && sgate < 0.f) sgate = shared_gate_weight(p.shared_gate, p.hpost, d, lane);
        gate = p.shared_gate ? sgate : 1.f;
      }
    } else {
      gate = s_gate[s];
    }
    if (tok != cur_tok) {
      if (cur_tok >= 0) {
        // batched case: this warp moves to another token, flush its partial sums
        if (lane == 0) poll_zeroed(true);
        __syncwarp();
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
      cur_tok = tok;
      hrow = p.hpost + (size_t)tok * d;
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
    const uint8_t* gs = smem + (size_t)s * entry_bytes;
    const uint8_t* us = gs + row_bytes;
    const uint8_t* ds = us + row_bytes;
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
        const float4 a = __ldg(reinterpret_cast<const float4*>(hrow) + (c * 32 + lane) * 2);
        const float4 b2 = __ldg(reinterpret_cast<const float4*>(hrow) + (c * 32 + lane) * 2 + 1);
        hh[0] = a.x; hh[1] = a.y; hh[2] = a.z; hh[3] = a.w; hh[4] = b2.x; hh[5] = b2.y; hh[6] = b2.z; hh[7] = b2.w;
      }
      if (FMT == kFmtMxfp4) {  // the lane's eight elements share one block scale
        float pg = 0.f, pu = 0.f;
#pragma unroll
        for (int m = 0; m < 8; ++m) pg = fmaf(gw[m], hh[m], pg);
#pragma unroll
        for (int m = 0; m < 8; ++m) pu = fmaf(uw[m], hh[m], pu);
        const uint8_t* sc = ds + row_bytes;  // gate | up | downT block scales, d/32 bytes each
        g = fmaf(block_scale(sc, c * 32 + lane), pg, g);
        u = fmaf(block_scale(sc + d / 32, c * 32 + lane), pu, u);
      } else {
#pragma unroll
        for (int m = 0; m < 8; ++m) g = fmaf(gw[m], hh[m], g);
#pragma unroll
        for (int m = 0; m < 8; ++m) u = fmaf(uw[m], hh[m], u);
      }
    }
    g = warp_sum(g);
    u = warp_sum(u);
    float down_scale = 1.f;
    if (FMT == kFmtE4m3) {  // per-row scales of the e4m3 store: value = scale * code
      const float* sc = reinterpret_cast<const float*>(ds + row_bytes);
      g *= sc[0];
      u *= sc[1];
      down_scale = sc[2];
    }
    const float a = gate * (g / (1.f + expf(-g))) * u * down_scale;
#pragma unroll
    for (int c = 0; c < NCH; ++c) {
      float dw[8];
      load8<FMT>(ds, c * 32 + lane, dw);
      const float ac = FMT == kFmtMxfp4 ? a * block_scale(ds + row_bytes + 2 * (d / 32), c * 32 + lane) : a;
#pragma unroll
      for (int m = 0; m < 8; ++m) acc[c * 8 + m] = fmaf(ac, dw[m], acc[c * 8 + m]);
    }
    __syncwarp();  // every lane has read stage s: it may be refilled
    {
      int more = 0;
      if (lane == 0 && ok) {
        const int r = next_row();
        if (r >= 0) {
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
          issue(r, tail);
          if (!ok) atomicExch(&s_abort, 1);
          more = ok ? 1 : 0;
        } else if (!polled) {
          polled = true;
          poll_zeroed(false);  // no more rows to fetch: the latency hides behind the rows still in flight
        }
      }
      tail += __shfl_sync(0xffffffffu, more, 0);
    }
  }
  waited = warp_max_u64(waited);
  ok = __all_sync(0xffffffffu, ok);
  if (lane == 0) {
    if (waited && p.stats) atomicAdd(&p.stats->stall_ns, waited);
    if (!ok) {
      if (p.stats) atomicAdd(&p.stats->timeouts, 1ull);
      *p.mbox_status = 1u;
      __threadfence_system();
    }
  }
  const bool aborted = *(volatile int*)&s_abort != 0;
  if (aborted) {
    // leave only after every copy this warp started has landed (bounded), so that no copy is in
    // flight into the shared memory of an exited CTA
    for (int jj = 0; jj < tail; ++jj) {
      const int s = warp + kConsumerWarps * (jj % NSW);
      if (jj + NSW >= tail)
        mbar_wait(&s_full[s], (uint32_t)((jj / NSW + ((phase_ahead >> (jj % NSW)) & 1u)) & 1), nullptr, p.wait_limit_ns);
    }
  }

  if (B > 1) {
    if (cur_tok >= 0 && !aborted) {
      if (lane == 0) poll_zeroed(true);
      __syncwarp();
      float4* y4 = reinterpret_cast<float4*>(p.y + (size_t)cur_tok * d);
#pragma unroll
      for (int c = 0; c < NCH; ++c) {
        const int col4 = (c * 32 + lane) * 2;
        atomicAdd(y4 + col4, make_float4(acc[c * 8 + 0], acc[c * 8 + 1], acc[c * 8 + 2], acc[c * 8 + 3]));
        atomicAdd(y4 + col4 + 1, make_float4(acc[c * 8 + 4], acc[c * 8 + 5], acc[c * 8 + 6], acc[c * 8 + 7]));
      }
    }
    return;
  }

  // ---- B == 1: reduce the eight partial vectors in shared memory, then one vector atomic per float4
  __syncthreads();  // every ring entry has been consumed; the ring is free
  if (tid == 0) TL(7);
  float* red = reinterpret_cast<float*>(smem);
  {
    float4* dst = reinterpret_cast<float4*>(red + (size_t)warp * d);
#pragma unroll
    for (int c = 0; c < NCH; ++c) {
      const int col4 = (c * 32 + lane) * 2;
      dst[col4] = make_float4(acc[c * 8 + 0], acc[c * 8 + 1], acc[c * 8 + 2], acc[c * 8 + 3]);
      dst[col4 + 1] = make_float4(acc[c * 8 + 4], acc[c * 8 + 5], acc[c * 8 + 6], acc[c * 8 + 7]);
    }
  }
  // one thread makes sure that every CTA has zeroed its slice of y (normally seen long ago)
  if (!__syncthreads_or((lane == 0 && zero_seen) ? 1 : 0)) {
    if (tid == 0) poll_zeroed(true);
    __syncthreads();
  }
  if (tid == 0) TL(8);
  if (!aborted) {  // (a CTA that took no row adds zeros)
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
  if (tid == 0) TLG(12);
  SPAN_END(5);
}

#ifdef APEX_TIMELINE
__device__ SpanLog g_spans;
extern "C" int apex_debug_read_timeline(unsigned long long* host, int n) {
  return (int)cudaMemcpyFromSymbol(host, g_timeline, sizeof(unsigned long long) * n);
}
extern "C" int apex_debug_read_spans(unsigned long long* host) {
  return (int)cudaMemcpyFromSymbol(host, g_spans, sizeof(SpanLog));
}
extern "C" int apex_debug_reset_spans() {
  SpanLog* z = new SpanLog();
  int r = (int)cudaMemcpyToSymbol(g_spans, z, sizeof(SpanLog));
  delete z;
  return r;
}
#endif

template <int NCH, int FMT>
static cudaError_t launch_ffn_t(const FfnParams& p, int n_ctas, cudaStream_t s) {
  constexpr bool HR = NCH <= 8;
  constexpr uint32_t entry = fmt_entry_bytes(FMT, NCH * 256);
  constexpr int NS = ring_stages(entry);
  const size_t smem = (size_t)NS * entry;
  static bool configured[kMaxDevices] = {};  // the attribute is per device
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev < 0 || dev >= kMaxDevices || !configured[dev]) {
    cudaError_t e = cudaFuncSetAttribute(moe_ffn_stream_kernel<NCH, HR, FMT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < kMaxDevices) configured[dev] = true;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(n_ctas, 1, 1);
  cfg.blockDim = dim3(kFfnThreads, 1, 1);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;  // prologue overlaps the gate kernel's tail
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, moe_ffn_stream_kernel<NCH, HR, FMT>, p);
}

bool ffn_shape_supported(int d) {
  switch (d) {
    case 256: case 512: case 768: case 1024: case 1536: case 2048: case 3072: case 4096:
      return true;
  }
  return false;
}

int ffn_grid_ctas(int n_sm) { return n_sm * kCtasPerSm; }

cudaError_t launch_ffn(const FfnParams& p, int n_ctas, cudaStream_t s) {
  if (p.fmt == kFmtE4m3 || p.fmt == kFmtMxfp4) {  // quantised stores: the widths of the paper-sized configs
#define APEX_FFN_CASE(NCH_) \
  case NCH_ * 256: return p.fmt == kFmtE4m3 ? launch_ffn_t<NCH_, kFmtE4m3>(p, n_ctas, s) : launch_ffn_t<NCH_, kFmtMxfp4>(p, n_ctas, s);
    switch (p.d) {
      APEX_FFN_CASE(2)
      APEX_FFN_CASE(4)
      APEX_FFN_CASE(6)
      APEX_FFN_CASE(8)
      APEX_FFN_CASE(16)
    }
#undef APEX_FFN_CASE
    return cudaErrorInvalidValue;
  }
  switch (p.d) {
    case 256: return launch_ffn_t<1, kFmtBf16>(p, n_ctas, s);
    case 512: return launch_ffn_t<2, kFmtBf16>(p, n_ctas, s);
    case 768: return launch_ffn_t<3, kFmtBf16>(p, n_ctas, s);
    case 1024: return launch_ffn_t<4, kFmtBf16>(p, n_ctas, s);
    case 1536: return launch_ffn_t<6, kFmtBf16>(p, n_ctas, s);
    case 2048: return launch_ffn_t<8, kFmtBf16>(p, n_ctas, s);
    case 3072: return launch_ffn_t<12, kFmtBf16>(p, n_ctas, s);
    case 4096: return launch_ffn_t<16, kFmtBf16>(p, n_ctas, s);
  }
  return cudaErrorInvalidValue;
}

bool ffn_quantised_shape_supported(int d) { return d == 512 || d == 1024 || d == 1536 || d == 2048 || d == 4096; }

size_t ffn_row_bytes(int fmt, int d) { return fmt_entry_bytes(fmt, d); }

}  // namespace apex

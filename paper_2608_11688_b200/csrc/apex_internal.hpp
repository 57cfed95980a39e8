// Internal declarations shared by the translation units of libapex.so.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdint>
#include <string>
#include <vector>

#include "../../include/apex.h"
#include "slot_table.hpp"

namespace apex {

// Debug builds (-DAPEX_TIMELINE): every kernel logs (id, start, end) of its block 0 in device memory.
#ifdef APEX_TIMELINE
struct SpanLog {
  unsigned long long n;
  unsigned long long rec[4096][3];
};
extern __device__ SpanLog g_spans;
__device__ __forceinline__ unsigned long long span_now() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
#define SPAN_BEGIN() const unsigned long long _span_t0 = span_now()
#define SPAN_END(id)                                                                     \
  do {                                                                                   \
    if (blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0) {                         \
      const unsigned long long _i = atomicAdd(&apex::g_spans.n, 1ull) & 4095ull;         \
      apex::g_spans.rec[_i][0] = (id);                                                   \
      apex::g_spans.rec[_i][1] = _span_t0;                                               \
      apex::g_spans.rec[_i][2] = span_now();                                             \
    }                                                                                    \
  } while (0)
#else
#define SPAN_BEGIN() do { } while (0)
#define SPAN_END(id) do { } while (0)
#endif

// ---- mapped host mailbox: the kernels post small decision records here so that the host can
// plan copies without a stream synchronisation.  One per context; sequence numbers only grow.
struct MailboxHeader {
  volatile uint32_t sel_seq;  // written by the candidate-selection kernel, after the lists
  volatile uint32_t status;   // sticky device status (0 ok, 1 a bounded wait ran out)
  uint32_t pad[2];
};

// Byte offsets inside the mailbox.  Per layer: route_seq[l] is written by the gate kernel after
// K_r of that layer, exec_seq[l] by the FFN's plan step after the execution sets.
struct MailboxLayout {
  size_t off_exec_seq, off_sel_rec, off_exec_rec, off_ncand, off_cand, off_kr, off_exec, kr_stride, bytes;
};

// Device-side counters of one layer (S9), accumulated with 64-bit atomics.
struct DevStats {
  unsigned long long tokens, sum_delta_hat, sum_delta_star, sum_ncand, capped, routed, hits_P, hits_R, covered,
      substitutions, stall_ns, timeouts, near_full;
};

// Small tables handed to kernels by value at launch: a snapshot of the layer's slot table.
struct SlotSnapshot {
  int8_t expert_slot[APEX_MAX_EXPERTS];   // -1 = not resident
  uint32_t need_gen[APEX_MAX_EXPERTS];    // slot-ready value to wait for
  unsigned long long resident_mask;
};

struct SelectParams {
  const float* q;       // [B][N]
  const int32_t* pi;    // [B][N]
  const float* w;       // [N]
  const float* theta;   // [N-k+1]
  int32_t* cand_out;    // [B][C] device, caller's
  int32_t* ncand_out;   // [B]
  int32_t* ncand_keep;  // [B] context-owned copy for the metrics
  int32_t* mbox_cand;   // mapped host [B][C]
  int32_t* mbox_ncand;  // mapped host [B]
  volatile uint32_t* mbox_seq;
  uint32_t* mbox_rec;   // mapped host, 16-byte aligned: {mask lo, mask hi, ncand, seq} for B == 1
  uint32_t seq_value;
  unsigned long long* done_counter;
  unsigned long long done_target;
  DevStats* stats;
  float t_tau;
  int force;  // 0: threshold test, 1: delta_hat = 0, 2: delta_hat = N-k
  int N, k, C, B;
};

struct RouterParams {
  const float* W;     // [N][d]
  const float* bias;  // [N] or null
  const float* x;     // [B][d]
  float* z_out;       // [B][N]
  float* q_out;       // [B][N] softmax
  int32_t* pi_out;    // [B][N] ranking, or null
  int32_t* topk_out;  // [B][k] or null
  int N, d, B, k;
  int warps_per_cta;
  int tok_per_group;  // batched kernel: tokens a cluster handles per pass (set by the launcher)
  // gate-kernel epilogue (S9 metrics + mailbox); all null/0 for the prefetch router
  const int32_t* pi_pred;     // [B][N] ranking of the prefetch router for this step, or null
  const int32_t* ncand_pred;  // [B]
  DevStats* stats;
  int C;
  int fuse_select;   // 1: the leader warp also runs the budget selection (sel) for its token
  SelectParams sel;
};


struct FfnParams {
  const float* hpost;       // [B][d]
  float* y;                 // [B][d]
  const int32_t* idx;       // [B][k] K_r
  const float* alpha;       // [B][N]
  const float* z_r;         // [B][N]
  int32_t* exec_idx;        // [B][k] out or null
  float* exec_gate;         // [B][k] out or null
  const uint8_t* cache;     // slot 0 of this layer
  const uint8_t* shared_w;  // or null
  const float* shared_gate; // [d] gate vector of the shared expert, or null: weight 1
  const uint32_t* slot_ready;  // [C]
  // batched plan (B > 1), context-owned
  int32_t* plan_exec_idx;   // [B][k]
  float* plan_exec_gate;    // [B][k]
  int32_t* pair_tok;        // [B*k + B]
  float* pair_gate;         // [B*k + B]
  int32_t* pair_expert;     // [B*k + B]   (N = shared expert)
  int32_t* n_pairs;         // [1]
  int32_t* grp;             // [4 + 3*(N+1)]: routed groups, all groups, 0, 0, then (expert, pair offset, tokens) per group
  int32_t* mbox_exec;       // mapped host [B][k]
  int32_t* mbox_kr;         // mapped host [B][k]: the routed sets, posted with the execution sets
  uint32_t* mbox_rec;       // mapped host, B = 1: two 16-byte records {mask lo, mask hi, sequence number, 0}: routed set, execution set
  volatile uint32_t* mbox_seq;
  volatile uint32_t* mbox_status;
  uint32_t seq_value;
  DevStats* stats;
  unsigned long long* zero_counter;
  unsigned long long zero_target;
  unsigned int* ticket;        // row-ticket counter of this launch (zero at launch)
  unsigned int* ticket_reset;  // counter of the launch 32 launches ahead, reset by this one
  unsigned long long run_mask;  // experts this launch executes
  const uint32_t* demand;       // [N] per layer: (tag << 8 | slot), published by the host after a demand copy
  uint32_t demand_tag;          // tag of this launch
  int demand_in_kernel;         // 1: a routed expert without a slot is waited for inside the kernel
  int fmt;                      // storage format of the slots: 0 bf16, 1 e4m3 with per-row scales, 2 e2m1 with block scales
  int zero_early;               // 1: y may be zeroed before the dependency wait (the preceding kernel does not touch y)
  long long spec_delay_ns;      // the speculative first fill starts this long after the CTA does
  const int32_t* spec;          // [k] predicted top-k of this layer-step (complete before the preceding kernel began), or null
  SlotSnapshot snap;
  size_t slot_stride;
  long long wait_limit_ns;
  int d, N, k, I, I_shared, B, C, mode, norm_topk, accumulate, run_shared, post_exec;
};

constexpr int kMaxDevices = 64;  // per-device launch attributes are remembered for this many devices

// Batched tensor-core path (kernels_ffn_tc.cu)
constexpr int kTcMinBatch = 2;  // from this many tokens per step the tensor-core grouped GEMM runs (it beats the per-pair kernel at every B > 1)
struct TcParams {
  FfnParams f;
  const int32_t* grp;
  __nv_bfloat16* xg;    // [pairs][d] gathered activations, bf16
  __nv_bfloat16* act;   // two planes [2][rows][act_stride]: bf16(a) and bf16(a - bf16(a))
  size_t act_plane;     // elements per plane
  int act_stride;
  int layer_slot0;      // index of this layer's slot 0 in the all-layers weight tensor map
  int nmax1, nmax2;     // tokens per unit of the gate/up and of the down kernel (set by the launcher)
  int nstage1, nstage2; // pipeline depths
};
struct TcMaps {          // opaque 128-byte CUtensorMap objects
  alignas(64) unsigned char w_gateup[128], w_down[128], ws_gateup[128], ws_down[128], xg[128], act[128], act_lo[128];
  // e2m1 stores only: the same bytes as w_* / ws_* with 16-byte boxes, for the block-scale bytes
  alignas(64) unsigned char sc_gateup[128], sc_down[128], ssc_gateup[128], ssc_down[128];
};

// Persistent decode kernel (kernels_decode.cu): all layers of one token in one cooperative launch.
constexpr int kDecWarps = 8;
constexpr int kDecThreads = kDecWarps * 32;
constexpr int kDecCluster = 8;  // CTAs per cluster: CTA r owns the router rows of experts 8r .. 8r+7, so N <= 64
// A layer's new slot table, published by the host in mapped memory after it has issued the prefetch copies of the step.
struct DecodeHostSnap {
  SlotSnapshot tab;
  uint32_t seq;  // sequence number of the token the snapshot belongs to; written last
  uint32_t pad[3];
};
// Records of one layer-step for the host, in mapped memory; each record is one aligned 16-byte store that carries the
// token's sequence number.
struct DecodeMbox {
  uint32_t sel_rec[4];   // candidate set: mask lo, mask hi, k + delta_hat, sequence number
  uint32_t kr_rec[4];    // routed set: mask lo, mask hi, sequence number, 0
  uint32_t exec_rec[4];  // execution set: the same
  uint32_t pad[4];
  int32_t cand[APEX_MAX_EXPERTS];  // candidates in rank order (advisory: the order in which the copies are issued)
};
struct DecodeParams {
  const float* h;       // [L][d] pre-attention states
  const float* hpost;   // [L][d] post-attention states
  float* y;             // [L][d], zero at launch
  const float *W_p, *b_p, *W_r, *b_r;  // [L][N][d], [L][N] (zeros where a layer has no bias)
  const float *w, *theta;               // [L][N], [L][N-k+1]
  const uint8_t* cache;                 // [L][C][slot_stride]
  const uint8_t* const* shared_w;       // [L] pointers (device array), or null
  const float* const* shared_gate;      // [L] pointers to the shared expert's gate vectors [d] (null entries: weight 1)
  const uint32_t* slot_ready;           // [L][C]
  const uint32_t* demand;               // [L][N]
  const SlotSnapshot* tab;              // [L] slot tables as they stand at launch (device memory)
  const uint8_t* opt;                   // [L] 1: the host expects this layer's table to stay as it is in this step
  const DecodeHostSnap* snap;           // [L] mapped host memory
  DecodeHostSnap* snap_dev;             // [L] device memory: the same, passed on by the one warp that reads the host's
  DecodeMbox* mbox;                     // [L] mapped host memory
  volatile uint32_t* mbox_status;
  DevStats* stats;                      // [L]
  float *zp_out, *qp_out;               // [N] of the layer processed last
  int32_t* pi_out;                      // [N]
  float *zr_out, *alpha_out;            // [L] rows of zr_stride floats
  int32_t* idx_out;                     // [L] rows of idx_stride ints
  int32_t *ncand_keep, *cand_dev, *ncand_dev;  // context scratch of the selection
  unsigned long long* cand_rec;         // [L][2] device: candidate mask of the layer-step, then the token's sequence number
  unsigned long long* bar;              // [L][2] device counters: CTAs done with the expert FFN / with the stand-in
  unsigned long long bar_target;        // value both counters reach when every CTA of this launch has counted itself in
  unsigned int* abort_flag;             // device word: somebody gave up
  const uint8_t* attn;
  size_t attn_bytes;
  int attn_layers, run_attn;
  int standin_ahead;                    // 1: the stand-in's chunks are requested ahead of the previous layer's completion
  int fmt;                              // storage format of the expert rows (FfnParams::fmt)
  uint32_t seq;                         // this token's sequence number
  uint32_t demand_tag;
  float t_tau;
  int force, prefetching;
  size_t slot_stride, zr_stride, idx_stride;
  long long wait_limit_ns;
  int d, N, k, I, I_shared, C, L, mode, norm_topk, cache_reuse, n_sm;
};

struct AttnParams {
  const uint4* buf;
  size_t n_vec;  // 16-byte vectors
  float* sink;
  int wait_first;       // 1: wait for the preceding kernel before streaming; 0: stream beside it, wait before exiting
};

// launchers (kernels_*.cu).  Each returns the cudaError_t of the launch.
cudaError_t launch_router(const RouterParams& p, cudaStream_t s);
cudaError_t launch_select(const SelectParams& p, cudaStream_t s);
cudaError_t launch_attention(const AttnParams& p, int n_sm, cudaStream_t s);
cudaError_t launch_ffn_plan(const FfnParams& p, cudaStream_t s);
cudaError_t launch_ffn(const FfnParams& p, int n_ctas, cudaStream_t s);  // n_ctas: grid size, at most ffn_grid_ctas(SM count)
int ffn_grid_ctas(int n_sm);  // CTAs of one streaming-kernel launch (each adds one to the zero counter)
cudaError_t launch_ffn_tc(const TcParams& p, const TcMaps& m, int n_sm, cudaStream_t s);
bool tc_make_weight_map(void* out, const void* base, int d, int I, size_t n_slots, size_t slot_bytes, int box_rows);
bool tc_make_rows_map(void* out, const void* base, int cols, size_t rows, size_t stride_elems);
bool tc_make_store_maps(int fmt, void* gateup, void* down, void* sc_gateup, void* sc_down, const void* base, int d, int I, size_t n_slots,
                        size_t slot_bytes);   // weight maps of one store in storage format fmt
bool tc_shape_supported(int d, int I, int I_shared, int fmt);
bool ffn_shape_supported(int d);
bool ffn_quantised_shape_supported(int d);   // widths the e4m3 / e2m1 kernels were built for
size_t ffn_row_bytes(int fmt, int d);        // bytes of one intermediate index (three vectors and their scales)
int decode_max_clusters(int d, int fmt);     // clusters of kDecCluster CTAs the current device holds at once (0: not supported)
cudaError_t launch_decode(const DecodeParams& p, int n_clusters, cudaStream_t s);

}  // namespace apex

// ---- the context ----------------------------------------------------------------------------
struct apex_ctx {
  apex_config cfg;
  std::string err;
  int device = 0;
  int n_sm = 0;
  int fmt = 0;  // storage format of stores and slots (see FfnParams::fmt)
  size_t expert_bytes = 0;   // 3*I*d*2
  size_t shared_bytes = 0;

  // device memory
  float* d_Wr = nullptr;  // [L][N][d]
  float* d_br = nullptr;  // [L][N]
  float* d_Wp = nullptr;
  float* d_bp = nullptr;
  float* d_w = nullptr;      // [L][N]
  float* d_theta = nullptr;  // [L][N-k+1]
  std::vector<uint8_t> has_br, has_bp, has_cdf;
  uint8_t* d_cache = nullptr;     // [L][C][expert_bytes]
  uint32_t* d_slot_ready = nullptr;  // [L][C]
  float *d_zp = nullptr, *d_qp = nullptr;  // [maxB][N]
  float* d_zr = nullptr;                   // [L][maxB][N]
  uint32_t* d_demand = nullptr;            // [L][N]
  int32_t *d_pi = nullptr, *d_ncand = nullptr;              // [maxB][N], [maxB]
  apex::DevStats* d_stats = nullptr;                        // [L]
  unsigned long long* d_counters = nullptr;                 // [2]: select done, zero
  int32_t *d_plan_exec_idx = nullptr, *d_pair_tok = nullptr, *d_pair_expert = nullptr, *d_n_pairs = nullptr;
  float *d_plan_exec_gate = nullptr, *d_pair_gate = nullptr;
  // batched tensor-core path
  bool tc_ok = false;
  int32_t* d_grp = nullptr;
  __nv_bfloat16 *d_xg = nullptr, *d_act = nullptr;
  int act_stride = 0;
  size_t act_plane = 0;
  apex::TcMaps tc_maps{};
  std::vector<apex::TcMaps> tc_shared_maps;  // per layer: ws_gateup / ws_down filled
  uint8_t* d_attn = nullptr;
  size_t attn_bytes = 0, attn_layers = 1;
  float* d_attn_sink = nullptr;
  // scratch for apex_decode_token
  int32_t *d_cand = nullptr, *d_cand_ncand = nullptr, *d_exec_idx = nullptr;
  float* d_exec_gate = nullptr;
  int32_t* d_idx = nullptr;  // [L][maxB][k]
  float* d_alpha = nullptr;  // [L][maxB][N]
  float *d_h_stage = nullptr, *d_hp_stage = nullptr, *d_y_stage = nullptr;  // [L][maxB][d] for the host variant

  // mapped host mailbox
  uint8_t* mbox = nullptr;
  apex::MailboxLayout ml{};
  uint32_t sel_seq = 0;
  std::vector<uint32_t> exec_seq;                 // per layer, last value asked for
  unsigned long long sel_done = 0, zero_done = 0;
  unsigned int* d_tickets = nullptr;  // [64] ring of row-ticket counters
  int32_t* d_spec = nullptr;          // [L][APEX_MAX_TOPK]: top-k of the prefetch router (B = 1), the FFN's speculative first fill
  uint32_t ffn_launch_id = 0;
  // what this context queued last, and where: an expert-FFN launch may still be adding to its y when
  // the next kernel's prologue runs (programmatic dependent launch)
  bool last_was_ffn = false;
  cudaStream_t last_stream = nullptr;
  uint32_t launch_tag = 0;
  uint32_t* gen_src = nullptr;  // pinned ring of flag values for the ready-flag copies
  size_t gen_src_pos = 0, gen_src_len = 0;

  // host state per layer
  std::vector<apex::SlotTable> tables;
  std::vector<const uint8_t*> store_base;
  std::vector<size_t> store_stride;
  std::vector<const uint8_t*> shared_dev;
  std::vector<float*> shared_gate_dev;        // [L] library-owned gate vectors of the shared expert, or null
  std::vector<char> shared_gate_on;           // [L] 1: the layer's shared expert is gated
  std::vector<std::vector<uint32_t>> slot_gen;  // [L][C] install count
  std::vector<std::vector<int32_t>> phys_expert;  // [L][C] whose bytes the slot holds (or is receiving)
  // emulated link (cfg.link_gbs > 0): padding copies over the host link stretch every expert copy
  uint8_t* pad_src = nullptr;    // pinned host scratch
  uint8_t* pad_dst = nullptr;    // device scratch
  size_t pad_bytes = 0;
  bool link_calibrated = false;
  double real_copy_us = 0.0;     // measured duration of one expert copy from the registered store
  double pad_lat_us = 0.0, pad_us_per_byte = 0.0;  // measured: padding copy time = pad_lat_us + bytes * pad_us_per_byte
  uint32_t* withheld_flag = nullptr;  // test hook: a ready flag that was not written
  uint32_t withheld_gen = 0;
  cudaStream_t withheld_stream = nullptr;
  std::vector<std::vector<apex::SlotCopy>> last_copies;
  std::vector<apex_step_stats> host_stats;
  struct StepState {
    int B = 0;
    bool predicted = false, selected = false, prefetched = false, routed = false;
    cudaStream_t route_stream = nullptr;   // stream of this step's gate kernel
    const int32_t* idx_dev = nullptr;
    const float* alpha_dev = nullptr;
    // an FFN launch whose host-side completion (LRU touch, demand copies) is still due
    bool pending = false;
    int pend_mode = 0;
    uint32_t pend_tag = 0;
    cudaStream_t pend_stream = nullptr;
  };
  std::vector<StepState> step;
  std::vector<apex::FfnParams> ffn_params;  // [L] parameters of the last FFN launch of each layer

  // Copies of a slot always travel on the same stream (slot index modulo the stream count), so two
  // installs into one slot stay ordered; two streams hide the gap between consecutive copies (+6 % on
  // the host link; a third and a fourth add nothing: measured).
  static constexpr int kMaxCopyStreams = 4;
  int n_copy_streams = 2;
  cudaStream_t copy_streams[kMaxCopyStreams] = {};      // own
  cudaStream_t cur_copy_streams[kMaxCopyStreams] = {};  // in use: own, or the caller's (then all the same)
  cudaStream_t stream_of_slot(int slot) const { return cur_copy_streams[slot % n_copy_streams]; }
  cudaStream_t pred_stream = nullptr;   // stream of the last apex_predict
  uintptr_t last_ffn_y_lo = 0, last_ffn_y_hi = 0;  // output range of the last streaming-kernel launch
  int last_pred_layer = -1;             // layer whose prefetch stage (router, budget selection) was the last launch, else -1
  cudaEvent_t ev_wave = nullptr, ev_in = nullptr;
  // persistent decode kernel (B = 1): device copies of the slot tables, mapped snapshots and records, counters
  int dec_clusters = 0;                       // clusters per launch; 0: the persistent path is not available
  apex::SlotSnapshot* d_dec_tab = nullptr;    // [L]
  uint8_t* d_dec_opt = nullptr;               // [L]
  uint8_t* dec_opt_stage = nullptr;           // pinned [2][L]
  std::vector<uint8_t> dec_opt_host, dec_opt_last;  // expectation per layer: now / as uploaded
  apex::SlotSnapshot* dec_tab_stage = nullptr;  // pinned [2][L]: staging of the table upload
  std::vector<apex::SlotSnapshot> dec_tab_last;  // what the device holds
  bool dec_tab_valid = false;
  int dec_stage_sel = 0;
  apex::DecodeHostSnap* dec_snap = nullptr;   // mapped [L]
  apex::DecodeHostSnap* d_dec_snap = nullptr; // device [L]
  apex::DecodeMbox* dec_mbox = nullptr;       // mapped [L]
  unsigned long long* d_dec_bar = nullptr;    // [L][2]
  unsigned long long* d_dec_cand = nullptr;   // [L][2]
  unsigned int* d_dec_abort = nullptr;
  const uint8_t** d_shared_ptrs = nullptr;    // [L]
  const float** d_shared_gate_ptrs = nullptr; // [L]
  unsigned long long dec_epoch = 0;           // persistent launches since the counters were last cleared
  uint32_t dec_seq = 0;
  bool dec_dirty = false;                     // a launch gave up: counters and abort flag must be cleared before the next
  int inject = 0;
  bool host_waves = false;  // B = 1 exact mode: misses are corrected by further launches, not by a wait inside the kernel
  int64_t launches = 0;
  void* fn_write_value32 = nullptr;  // cuStreamWriteValue32 when the driver offers it
};

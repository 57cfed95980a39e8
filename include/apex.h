/*
 * apex.h -- C ABI of the B200-native MoE decode step with adaptive expert prefetch.
 *
 * One layer-step of decoding, as the paper sequences it (the two stages of Sec. IV-A, the run-time
 * sequence of Sec. IV-D):
 *
 *   apex_predict            prefetch router on the pre-attention state h       (Sec. IV-D)
 *   apex_select_candidates  confidence-driven budget delta_hat and K_p         (Eq. (8), (9), (1))
 *   apex_prefetch           asynchronous copy of K_p into HBM cache slots      (Sec. IV-A stage 1)
 *   apex_attention_standin  the window that hides the copies                   (Eq. (12))
 *   apex_route_topk         exact top-k gate on the post-attention state h'    (Sec. III-A)
 *   apex_moe_ffn            expert FFNs + weighted sum, in one of two modes    (Sec. IV-E, Alg. 1)
 *
 * Conventions
 *   - Every function returns an int: APEX_OK (0) or a negative error code.  Nothing throws or
 *     aborts across this boundary.  apex_last_error() gives a text owned by the context.
 *   - "dev" pointers are device (HBM) addresses, "host" pointers host addresses.  All buffers
 *     are owned by the caller and only borrowed for the duration stated at each call.
 *   - Streams are cudaStream_t handles passed as void*; NULL is the legacy default stream.
 *   - Row-major everywhere.  Expert indices, slots and counts are int32, probabilities and
 *     hidden states fp32, expert weights bf16 (fp32 accumulation inside the kernels).
 *   - All orderings are "value descending, then lower expert index".
 *   - Limits of this build: N <= 64 experts per layer, k <= 16, d a multiple of 256 and
 *     d <= 4096, 1 <= B <= max_batch <= 256, k <= C <= N.
 *   - A context is not thread-safe; use one host thread per context.
 *
 * Expert store layout (host, pinned): expert e of a layer starts at base + e*stride and holds
 *   [I][3][d] bf16:  for each intermediate index i the three rows gate_i, up_i, downT_i,
 * where downT_i[j] = W_down[j][i] (the down projection transposed), so that index i owns one
 * contiguous block of 3*d values.  apex_pack_expert() converts from the usual
 * gate[I][d], up[I][d], down[d][I].
 * With APEX_FLAG_FP8_EXPERTS (the expert-weight precision study of Sec. V-G: smaller experts, smaller
 * copies) a row is 3*d e4m3 codes followed by three fp32 scales and 4 bytes of padding,
 *   [I][ gate_i (d bytes) | up_i (d bytes) | downT_i (d bytes) | s_gate, s_up, s_down, 0 ],
 * weight = scale * code; 3*d + 16 bytes per row.
 * With APEX_FLAG_FP4_EXPERTS a row is 3*d e2m1 codes (two per byte, the even element in the low nibble),
 * then one scale byte per 32 elements of each vector (a biased exponent: scale = 2^(byte - 127)), padded
 * to a multiple of 16 bytes,
 *   [I][ gate_i (d/2 bytes) | up_i (d/2) | downT_i (d/2) | gate scales (d/32) | up scales | downT scales | pad ],
 * weight = scale of its block * code.
 * Both need d in {512, 1024, 1536, 2048, 4096} and exclude each other; batched steps then run the
 * streaming kernel per (token, expert) pair (no tensor-core path for these formats yet).
 */
#ifndef APEX_H
#define APEX_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define APEX_OK 0
#define APEX_EINVAL (-1)   /* bad argument or unsupported shape */
#define APEX_ENOMEM (-2)   /* host or device allocation failed */
#define APEX_ECUDA (-3)    /* a CUDA runtime call failed; see apex_last_error */
#define APEX_ETIMEOUT (-4) /* a bounded wait (host or device side) ran out */
#define APEX_ESTATE (-5)   /* calls out of order, or no evictable slot */
#define APEX_ENOTIMPL (-6)

#define APEX_MODE_EXACT 0      /* correctness-preserving: follow K_r, fetch what is missing */
#define APEX_MODE_STALL_FREE 1 /* Algorithm 1: resident experts only, gates renormalised */

#define APEX_FLAG_FP8_EXPERTS 1 /* apex_config.flags: expert stores and slots hold e4m3 rows (see below) */
#define APEX_FLAG_FP4_EXPERTS 4 /* apex_config.flags: expert stores and slots hold block-scaled e2m1 rows (see below) */
#define APEX_FLAG_SPECULATE 2 /* apex_config.flags: at B = 1 the expert FFN starts streaming the k experts the prefetch router
                                 ranked first before the gate's decision is visible, and drops the guesses the gate does not
                                 confirm (results are identical either way).  Pays when FFN launches follow one another
                                 directly, costs inside the decode loop, where the early copies delay the gate kernel; off by
                                 default */

#define APEX_FLAG_HOST_WAVES 8 /* apex_config.flags: at B = 1 in exact mode a missing expert is NOT waited for inside the
                                 running kernel; the first launch executes the resident routed experts and one further launch
                                 per demand wave adds the rest (the scheme B > 1 always uses).  Needed wherever a kernel
                                 launch does not return before the kernel has finished -- see apex_moe_ffn.  Set
                                 automatically when the process runs with CUDA_LAUNCH_BLOCKING=1 or under a CUDA
                                 injection tool (a profiler that serialises kernels), and after the first in-kernel wait
                                 for a demand copy that ran out on this context.  APEX_ASYNC_LAUNCHES=1 in the environment
                                 switches the detection off (for profiling a run in which nothing can miss) */

#define APEX_FLAG_LAYER_LAUNCHES 16 /* apex_config.flags: apex_decode_token always runs its per-layer kernel sequence.  Without it
                                       a batch-1 token over bf16 stores runs as ONE persistent kernel over all layers (the
                                       same steps, the same results; no launch and no host round trip between layers on the
                                       hit path), unless launches may block (see APEX_FLAG_HOST_WAVES) */
#define APEX_FLAG_SKIP_STANDIN 32   /* apex_config.flags: apex_decode_token leaves the stand-in attention out (the hiding
                                       window of Eq. (12) is then empty: for measuring the method's own bytes) */

#define APEX_FLAG_STANDIN_AHEAD 64  /* apex_config.flags: the persistent token kernel requests a layer's stand-in attention bytes
                                       while the previous layer is still finishing (they are parameters and old KV entries),
                                       instead of when that layer's output is complete.  Faster, but the hiding window of
                                       Eq. (12) then overlaps the previous layer's tail, so it is off by default */

#define APEX_MAX_EXPERTS 64
#define APEX_MAX_TOPK 16
#define APEX_MAX_BATCH 256
#define APEX_STATIC_MAX_BATCH 64 /* largest B of apex_route_topk_static */

typedef struct apex_ctx apex_ctx;

typedef struct apex_config {
  int32_t d;             /* hidden size */
  int32_t N;             /* experts per layer */
  int32_t k;             /* routed experts per token */
  int32_t I;             /* expert intermediate size */
  int32_t I_shared;      /* always-on shared SwiGLU FFN intermediate size, 0 = none */
  int32_t C;             /* HBM cache slots per layer */
  int32_t L;             /* layers */
  int32_t max_batch;     /* largest B that will be passed */
  int32_t norm_topk;     /* 1: g_e = alpha_e / sum over the executed set; 0: g_e = alpha_e */
  int32_t cache_reuse;   /* 1: slots persist across steps; 0: load-use-evict per layer-step */
  int32_t ctx_len;       /* context length that sizes the stand-in attention kernel */
  int32_t flags;         /* APEX_FLAG_* bits */
  int64_t wait_limit_ns; /* bound of every host- and device-side wait; 0 = 2 s */
  double link_gbs;       /* 0: expert copies run at the speed of the link they cross.  > 0: every expert copy is
                            stretched to expert bytes / link_gbs (GB/s) by a padding copy over the host link behind it,
                            on one copy stream -- a stand-in for a slower far tier than this machine's host link
                            (Sec. V-G bandwidth study) */
} apex_config;

/* Counters of one layer, accumulated over layer-steps since the last reset. */
typedef struct apex_step_stats {
  int64_t layer_steps;
  int64_t tokens;
  int64_t sum_delta_hat;   /* selected extra budget (after the cap) */
  int64_t sum_delta_star;  /* oracle budget, Eq. (3) */
  int64_t sum_ncand;       /* k + delta_hat */
  int64_t capped;          /* tokens whose budget hit the buffer cap C - k */
  int64_t routed;          /* tokens * k */
  int64_t hits_P;          /* routed experts inside the token's candidate set K_p */
  int64_t hits_R;          /* routed experts resident after the prefetch plan */
  int64_t covered;         /* tokens with K_r subset of K_p, Eq. (2) */
  int64_t substitutions;   /* stall-free replacements */
  int64_t prefetch_copies;
  int64_t demand_copies;
  int64_t bytes_copied;
  int64_t extra_waves;     /* FFN launches beyond the first, exact mode */
  int64_t stall_ns;        /* device time spent waiting for slot-ready flags or demand copies, mean over the SMs */
  int64_t timeouts;
  int64_t near_full_prefetch; /* tokens with k + delta_hat > N/2 */
} apex_step_stats;

/* ---- life cycle ------------------------------------------------------------------------ */

/* Allocates the context: router tables, the L*C slot cache in HBM, flags, mailboxes.
 * Returns APEX_EINVAL for shapes outside the limits above, APEX_ENOMEM / APEX_ECUDA otherwise. */
int apex_create(const apex_config* cfg, apex_ctx** out);
int apex_destroy(apex_ctx* ctx);
/* Text of the last error on this context.  With ctx == NULL: the reason the last apex_create on the calling
 * thread failed (the context it was building no longer exists). */
const char* apex_last_error(const apex_ctx* ctx);

/* ---- parameters (host pointers, copied into library-owned device memory) ---------------- */

/* Original router of a layer (Sec. III-A): W_r [N][d], b_r [N] or NULL. */
int apex_set_router(apex_ctx* ctx, int layer, const float* W_r_host, const float* b_r_host);
/* Prefetch router (Sec. IV-D: mirrors the original router): W_p [N][d], b_p [N] or NULL. */
int apex_set_prefetch_router(apex_ctx* ctx, int layer, const float* W_p_host, const float* b_p_host);
/* Ordinal-logistic confidence model (Eq. (8)): w [N], theta [N-k+1].  theta must be
 * non-decreasing (Table I), else APEX_EINVAL. */
int apex_set_cdf(apex_ctx* ctx, int layer, const float* w_host, const float* theta_host);
/* Off-chip expert store of a layer (Sec. III-A: expert weights live off-package): pinned host
 * memory in the store layout described above.  Borrowed until apex_destroy. */
int apex_register_experts(apex_ctx* ctx, int layer, const void* pinned_base, size_t expert_stride_bytes);
/* Always-on shared expert (Sec. V-A: shared experts are outside the routing and the budget):
 * device pointer to [I_shared][3][d] bf16 in the store layout.  Borrowed. */
int apex_set_shared_expert(apex_ctx* ctx, int layer, const void* dev_weights);
/* Gate on the shared expert, for model families that scale their shared FFN per token (the paper's configurations
 * run theirs with weight 1, Sec. V-A; this variant has no counterpart in the paper):
 *   y = sum_e g_e FFN_e(h') + sigmoid(w_sg . h') FFN_shared(h').
 * w_sg [d] fp32 (host or device pointer) is copied into library-owned device memory; NULL removes the gate again
 * (weight 1).  APEX_EINVAL without a shared expert (I_shared = 0).  Must not be called while a step of the layer is
 * in flight. */
int apex_set_shared_gate(apex_ctx* ctx, int layer, const float* w_sg);
/* Host helper: gate[I][d], up[I][d], down[d][I] -> store layout.  dst holds 3*I*d bf16. */
int apex_pack_expert(const void* gate, const void* up, const void* down, int d, int I, void* dst);

/* ---- the layer-step ---------------------------------------------------------------------- */

/* S1+S2 (Sec. IV-D): z_p = W_p h + b_p, q_p = softmax(z_p), ranking E of Sec. IV-B.  h_dev is
 * [B][d].  Results stay in the context for apex_select_candidates.  Starts a new layer-step
 * for this layer (advances its slot-table clock). */
int apex_predict(apex_ctx* ctx, int layer, const float* h_dev, int B, void* stream);
/* S3 (Eq. (9), (1)): x = q_p sorted descending, delta_hat = min{delta: theta_delta - w.x >=
 * ln(tau/(1-tau))}, capped to C-k; cand_dev [B][C] receives e_1..e_{k+delta_hat} in rank order,
 * padded with -1; ncand_dev [B] receives k+delta_hat.  tau<=0 gives delta_hat=0, tau>=1 gives
 * the cap. */
int apex_select_candidates(apex_ctx* ctx, int layer, int B, float tau, int32_t* cand_dev,
                           int32_t* ncand_dev, void* stream);
/* S5 (Sec. IV-A stage 1): waits (host side, bounded) for the candidate lists, plans slots and
 * issues one cudaMemcpyAsync per non-resident candidate on copy_stream (NULL: the context's
 * own copy stream), each followed by a slot-ready flag.  Returns without waiting for the
 * copies. */
int apex_prefetch(apex_ctx* ctx, int layer, int B, void* copy_stream);
/* Streams the bytes of an attention block (4 d^2 + 2 ctx_len d bf16 values): the hiding window
 * of Eq. (12).  It does not produce h'.  An attention block reads the layer's input, not the prefetch
 * stage's output: when apex_predict / apex_select_candidates of this layer are the calls just before it on
 * the same stream, the kernel runs beside them and only waits for them before it exits (everything launched
 * after it still finds all earlier work complete); behind anything else it waits first. */
int apex_attention_standin(apex_ctx* ctx, int layer, void* stream);
/* S4 (Sec. III-A; Alg. 1 line 3): z_r = W_r h' + b_r, idx_dev [B][k] = K_r in rank order,
 * alpha_dev [B][N] = softmax(z_r).  Both buffers must stay valid until apex_moe_ffn of the
 * same layer-step has been called. */
int apex_route_topk(apex_ctx* ctx, int layer, const float* hpost_dev, int B, int32_t* idx_dev,
                    float* alpha_dev, void* stream);
/* S6-S8 (Sec. IV-E): y_dev [B][d] = sum over the execution set of g_e FFN_e(h') (+ shared FFN).
 * APEX_MODE_EXACT executes K_r: resident experts first, missing ones are copied on demand while
 * those run (asynchronous miss correction) -- at B = 1 the one kernel waits (bounded) for each
 * missing expert and then executes it, at B > 1 further launches follow.  APEX_MODE_STALL_FREE executes
 * Algorithm 1 with K_p := the resident set.  exec_idx_dev [B][k] (ascending expert index) and
 * exec_gate_dev [B][k] may be NULL.  Device-side waits on slot-ready flags are bounded; when one
 * runs out the call (or the next call on this context) returns APEX_ETIMEOUT.
 * Asynchronous launches are assumed at B = 1 in exact mode: the kernel waits for demand copies that this same
 * call issues only after the launch has returned.  Where a launch blocks until the kernel is done
 * (CUDA_LAUNCH_BLOCKING=1, a profiler or debugger that serialises kernels) that wait could only run out, so
 * the context then uses APEX_FLAG_HOST_WAVES (detected at apex_create from the environment; it can also be
 * set by hand): same results, one more launch per step that misses. */
int apex_moe_ffn(apex_ctx* ctx, int layer, int mode, const float* hpost_dev, int B, float* y_dev,
                 int32_t* exec_idx_dev, float* exec_gate_dev, void* stream);

/* The same in two halves, for callers that pipeline layers themselves (Sec. IV-E "asynchronous miss
 * correction": the expert computation starts while the host is still arranging the copies).
 * apex_moe_ffn_begin queues the expert FFN of the layer-step and returns at once.  apex_moe_ffn_end
 * does the host part that needs the gate's decision -- recency stamps, demand copies for missing
 * experts (B = 1: the queued kernel is already waiting for them; B > 1: further launches) -- and must
 * be called before the next apex_predict / apex_route_topk of the same layer (APEX_ESTATE otherwise).
 * apex_moe_ffn is begin followed by end. */
int apex_moe_ffn_begin(apex_ctx* ctx, int layer, int mode, const float* hpost_dev, int B, float* y_dev,
                       int32_t* exec_idx_dev, float* exec_gate_dev, void* stream);
int apex_moe_ffn_end(apex_ctx* ctx, int layer);

/* All L layers of one decode step, in the order above.  h_dev, hpost_dev, y_dev are [L][B][d].
 * At B = 1 the whole token is one cooperative kernel launch that loops over the layers (bf16 stores: d = 256 ... 4096 in the
 * supported widths; e4m3 / e2m1 stores: d = 512, 1024, 1536, 2048, 4096)
 * (prefetch router, stand-in attention, gate, expert FFN as roles inside it; layers handed over through bounded
 * device-side counters); the host thread only plans and issues copies from the records the kernel posts and, on the
 * hit path, is never waited for.  Otherwise, and with APEX_FLAG_LAYER_LAUNCHES, one kernel sequence per layer.
 * tau < 0 skips the prefetch stage altogether: the "No Prefetch" baseline of Sec. V-A, where every
 * non-resident routed expert is loaded on the critical path (static over-fetch baselines are a
 * confidence model with w = 0 and a step in theta). */
int apex_decode_token(apex_ctx* ctx, const float* h_dev, const float* hpost_dev, int B, float tau,
                      int mode, float* y_dev, void* stream);
/* Same with host buffers (pinned for full speed): inputs are copied to the device and y back
 * inside the call, which returns after y_host is complete. */
int apex_decode_token_host(apex_ctx* ctx, const float* h_host, const float* hpost_host, int B,
                           float tau, int mode, float* y_host, void* stream);

/* ---- observation, checkpoint, test hooks --------------------------------------------------- */

int apex_get_stats(apex_ctx* ctx, int layer, apex_step_stats* out); /* layer -1: sum over layers */
int apex_reset_stats(apex_ctx* ctx);
/* Results of the last apex_predict (synchronises the stream it ran on): z_p, q_p [B][N], pi [B][N]. */
int apex_read_prediction(apex_ctx* ctx, int B, float* z_p_host, float* q_p_host, int32_t* pi_host);
/* Copies issued by the last layer-step of `layer`: first the prefetch copies, then the demand
 * copies, as (expert, slot) pairs; arrays hold up to 2*N entries. */
int apex_get_last_copies(apex_ctx* ctx, int layer, int32_t* expert, int32_t* slot, int32_t* n_prefetch,
                         int32_t* n_demand);
/* Slot table of a layer: expert_slot [N] (-1 = not resident), slot_stamp [C], clock.  Setting a
 * table marks the named slots as holding valid data only if they already do (checkpoint/resume
 * within one context); other residents are dropped. */
int apex_get_slot_table(apex_ctx* ctx, int layer, int32_t* expert_slot, int64_t* slot_stamp, int64_t* clock);
int apex_set_slot_table(apex_ctx* ctx, int layer, const int32_t* expert_slot, const int64_t* slot_stamp,
                        int64_t clock);
/* Makes every expert of every layer resident (needs C == N) and waits for the copies. */
int apex_warm_all(apex_ctx* ctx);
/* Host-side fault hooks for tests: what = 1 the next copy issue fails (APEX_ECUDA path);
 * what = 2 the next slot-ready flag is withheld (device wait runs out); 0 clears. */
int apex_test_inject(apex_ctx* ctx, int what);
/* Number of kernels this library has launched on the context so far. */
int64_t apex_launch_count(const apex_ctx* ctx);

/* ---- allocation-free gate ----------------------------------------------------------------- */

/* (No counterpart in the paper: an addition for deployment.)
 * The exact top-k gate of apex_route_topk for callers that cannot allocate device memory -- for
 * example a serving process whose HBM is owned by a fixed pool, where a stray cudaMalloc would
 * both escape the pool's accounting and stall the device.  No context is needed and nothing is
 * allocated or freed, here or in any library it calls.
 *   W_r_dev [N][d], b_r_dev [N] or NULL, hpost_dev [B][d]: device inputs, borrowed for the launch.
 *   W_r_dev and b_r_dev must be complete in memory before the call is made, not merely ordered before it
 *   on the stream: the kernel starts reading the weights while the kernel ahead of it on the stream may still
 *   be finishing (hpost_dev, like every other input of this library, only needs stream order).
 *   idx_dev [B][k] (K_r in rank order) and alpha_dev [B][N] (softmax of the logits): device outputs.
 *   Limits: B <= APEX_STATIC_MAX_BATCH (64), N <= APEX_MAX_EXPERTS (64), k <= min(N, 16),
 *   d a multiple of 4 and d <= 4096.  Larger sizes are refused with APEX_EINVAL and a message.
 * The kernel's only scratch, the raw logits, lives in a 16 KiB array built into the library; every
 * GPU that loads the library holds it until the process ends.  The first call on a device looks
 * up the array's address on that device (make that first call outside any stream capture).  All
 * calls on a device share the array and it keeps the previous call's logits; the kernel overwrites
 * what it uses, so nothing has to be cleared, but two calls that overlap on the GPU (different
 * streams) race on it: serialise them.  First calls from several host threads are serialised inside.
 * err (optional, err_len bytes, caller-owned) receives a text on failure.  Returns APEX_OK,
 * APEX_EINVAL or APEX_ECUDA. */
int apex_route_topk_static(const float* W_r_dev, const float* b_r_dev, const float* hpost_dev, int N, int d, int k,
                           int B, int32_t* idx_dev, float* alpha_dev, void* stream, char* err, size_t err_len);

/* ---- fitting the confidence model on the GPU (Sec. IV-C, Eq. (8) and Eq. (11)) ---------------
 * Fits p_delta(x) = sigmoid(theta_delta - w.x) to a calibration set by minimising the cumulative binary
 * cross-entropy  -(1/T) sum_t sum_delta [ y log p + (1-y) log(1-p) ],  y = [delta >= delta*_t],
 * with theta kept non-decreasing (theta_delta = t0 + sum_{i<=delta} softplus(u_i)).  Full-batch Adam
 * (0.9 / 0.999 / 1e-8) in fp64, `iters` steps of size lr, from w = 0 and the logit of the empirical
 * distribution of delta* (clipped to [1e-3, 1-1e-3], increments at least 1e-3); all sums run in a fixed
 * order, so the result is reproducible bit for bit.
 *   X_dev [T][N] fp64 (device): x of each calibration token (its prefetch probabilities sorted in
 *   descending order); dstar_dev [T] int32 (device): its oracle budget delta* (Eq. (3)), 0 <= delta* <= N-k.
 *   w_host [N], theta_host [N-k+1] (host, fp32): the fitted parameters, theta made monotone again after
 *   the rounding to fp32 -- ready for apex_set_cdf.
 * Context-free; allocates and frees its own scratch; synchronises `stream` before it returns.
 * N <= APEX_MAX_EXPERTS.  err (optional) receives a text on failure.  Returns APEX_OK, APEX_EINVAL,
 * APEX_ENOMEM or APEX_ECUDA. */
int apex_fit_cdf(const double* X_dev, const int32_t* dstar_dev, int T, int N, int k, int iters, double lr,
                 float* w_host, float* theta_host, void* stream, char* err, size_t err_len);

/* Distils the prefetch router from the frozen router (Sec. IV-C, Eq. (10)): minimises the mean over the
 * calibration tokens of KL(q_r || q_p), q_p = softmax(W_p h + b_p), by `iters` steps of full-batch Adam
 * (0.9 / 0.999 / 1e-8, step lr) in fp64; sums in a fixed order (bit-reproducible).
 *   H_dev [T][d] fp32 (device): the hidden states the prefetch router will see (before attention);
 *   Qr_dev [T][N] fp32 (device): the router's distribution for the same tokens (after attention), e.g. the
 *   alpha output of apex_route_topk.
 *   W_host [N][d], b_host [N] (host, fp32): in: the starting point; out: the trained parameters, ready for
 *   apex_set_prefetch_router.
 * Context-free; allocates and frees its own scratch; synchronises `stream` before it returns.
 * N <= APEX_MAX_EXPERTS.  Returns APEX_OK, APEX_EINVAL, APEX_ENOMEM or APEX_ECUDA. */
int apex_distill_router(const float* H_dev, const float* Qr_dev, int T, int N, int d, int iters, double lr,
                        float* W_host, float* b_host, void* stream, char* err, size_t err_len);

/* ---- host-only slot planner (the state machine behind apex_prefetch / apex_moe_ffn) -------- */

typedef struct apex_slots apex_slots;
apex_slots* apex_slots_create(int N, int C, int cache_reuse);
void apex_slots_destroy(apex_slots* s);
int apex_slots_begin_step(apex_slots* s);
/* cand [B][stride], ncand [B]: plans the union (most wanted first, truncated to C).  Outputs:
 * copy_expert/copy_slot (up to C entries), *n_copies. */
int apex_slots_prefetch(apex_slots* s, const int32_t* cand, const int32_t* ncand, int B, int stride,
                        int32_t* copy_expert, int32_t* copy_slot, int32_t* n_copies);
/* K_r [B][k]: touches resident routed experts and installs the missing ones in chunks of C.
 * Outputs: copy_expert/copy_slot (up to N entries), wave_of_copy (1-based wave), *n_copies. */
int apex_slots_demand(apex_slots* s, const int32_t* K_r, int B, int k, int32_t* copy_expert,
                      int32_t* copy_slot, int32_t* wave_of_copy, int32_t* n_copies);
int apex_slots_touch(apex_slots* s, const int32_t* experts, int n);
int apex_slots_get(const apex_slots* s, int32_t* expert_slot, int64_t* slot_stamp, int64_t* clock);
int apex_slots_set(apex_slots* s, const int32_t* expert_slot, const int64_t* slot_stamp, int64_t clock);

#ifdef __cplusplus
}
#endif
#endif /* APEX_H */

// Host-side helpers shared by the translation units that implement the C ABI: error recording, argument checks,
// the mapped mailbox, stream-ordered flag writes, bounded host waits.
#ifndef APEX_HOST_HPP
#define APEX_HOST_HPP

#include <chrono>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <string>
#include <thread>
#include <vector>

#include "apex_internal.hpp"

namespace apex {

typedef int (*WriteValue32Fn)(cudaStream_t, unsigned long long, uint32_t, unsigned int);

inline int fail(apex_ctx* ctx, int code, const char* what, cudaError_t e = cudaSuccess) {
  if (ctx) {
    char buf[512];
    if (e != cudaSuccess)
      snprintf(buf, sizeof buf, "%s: %s", what, cudaGetErrorString(e));
    else
      snprintf(buf, sizeof buf, "%s", what);
    ctx->err = buf;
  }
  return code;
}

#define CU_TRY(ctx, expr)                                              \
  do {                                                                 \
    cudaError_t _e = (expr);                                           \
    if (_e != cudaSuccess) return fail(ctx, APEX_ECUDA, #expr, _e);    \
  } while (0)

#define CHECK_CTX(ctx) \
  if (!(ctx)) return APEX_EINVAL
#define CHECK_LAYER(ctx, layer) \
  if ((layer) < 0 || (layer) >= (ctx)->cfg.L) return fail(ctx, APEX_EINVAL, "layer out of range")

template <typename T>
inline cudaError_t dev_alloc(T** p, size_t n) {
  return cudaMalloc(reinterpret_cast<void**>(p), n * sizeof(T) > 0 ? n * sizeof(T) : 16);
}

inline MailboxHeader* mhdr(apex_ctx* ctx) { return reinterpret_cast<MailboxHeader*>(ctx->mbox); }
inline int32_t* mbox_i32(apex_ctx* ctx, size_t off) { return reinterpret_cast<int32_t*>(ctx->mbox + off); }
inline volatile uint32_t* mbox_sel_rec(apex_ctx* ctx) { return reinterpret_cast<volatile uint32_t*>(ctx->mbox + ctx->ml.off_sel_rec); }
inline volatile uint32_t* mbox_exec_seq(apex_ctx* ctx, int l) {
  return reinterpret_cast<volatile uint32_t*>(ctx->mbox + ctx->ml.off_exec_seq) + l;
}
inline volatile uint32_t* mbox_exec_rec(apex_ctx* ctx, int l) {
  return reinterpret_cast<volatile uint32_t*>(ctx->mbox + ctx->ml.off_exec_rec) + 8 * l;
}
inline int32_t* mbox_kr(apex_ctx* ctx, int l) { return mbox_i32(ctx, ctx->ml.off_kr + (size_t)l * ctx->ml.kr_stride); }
inline int32_t* mbox_exec(apex_ctx* ctx, int l) { return mbox_i32(ctx, ctx->ml.off_exec + (size_t)l * ctx->ml.kr_stride); }

// A 32-bit word written in stream order (after everything queued before it on that stream).
inline int stream_write32(apex_ctx* ctx, cudaStream_t cs, uint32_t* dev, uint32_t value) {
  if (ctx->fn_write_value32) {
    int r = reinterpret_cast<WriteValue32Fn>(ctx->fn_write_value32)(cs, (unsigned long long)(uintptr_t)dev, value, 0);
    if (r != 0) return fail(ctx, APEX_ECUDA, "cuStreamWriteValue32 failed");
    return APEX_OK;
  }
  uint32_t* srcv = ctx->gen_src + (ctx->gen_src_pos++ % ctx->gen_src_len);
  *srcv = value;
  CU_TRY(ctx, cudaMemcpyAsync(dev, srcv, sizeof(uint32_t), cudaMemcpyHostToDevice, cs));
  return APEX_OK;
}

// Bounded host wait for a mailbox sequence number.  Records of the hit path arrive within microseconds and a batched
// layer-step lasts a few hundred, so the first millisecond is a plain spin (a sleep, however short it is asked to be,
// returns after the timer slack of about 50 us: with a 50 us spin phase the batched decode loop lost 28 us per
// layer-step to it).  After that the core is given up between polls -- yields up to 5 ms, then sleeps growing to
// 32 us nominal -- so a wait behind a long copy or a stalled device does not burn a core until its limit.
inline bool host_wait_seq(apex_ctx* ctx, volatile uint32_t* p, uint32_t want) {
  if ((int32_t)(*p - want) >= 0) return true;
  const auto t0 = std::chrono::steady_clock::now();
  const int64_t limit = ctx->cfg.wait_limit_ns * 2 + 1000000000ll;  // the device side gives up first
  int64_t sleep_us = 1;
  bool slow = false;
  for (uint32_t it = 0;; ++it) {
    if ((int32_t)(*p - want) >= 0) return true;
    if (!slow && (it & 255u) != 255u) {
#if defined(__x86_64__)
      __builtin_ia32_pause();
#endif
      continue;
    }
    const int64_t ns = std::chrono::duration_cast<std::chrono::nanoseconds>(std::chrono::steady_clock::now() - t0).count();
    if (ns > limit) return false;
    if (ns < 50000) continue;
    if (mhdr(ctx)->status != 0) return false;  // a kernel gave up: what it was going to post will not come
    if (ns < 1000000) continue;
    slow = true;
    if (ns < 5000000) {
      std::this_thread::yield();
    } else {
      std::this_thread::sleep_for(std::chrono::microseconds(sleep_us));
      sleep_us = sleep_us < 32 ? sleep_us * 2 : 32;
    }
  }
}

// Why the last apex_create on this thread failed (the context it was building is gone by then).
inline std::string& create_error() {
  static thread_local std::string s;
  return s;
}

// Copy machinery and device status (apex_step.cu)
int issue_copy(apex_ctx* ctx, int layer, int e, int slot, cudaStream_t cs);
int release_withheld(apex_ctx* ctx);
SlotSnapshot make_snapshot(apex_ctx* ctx, int layer);
int check_device_status(apex_ctx* ctx);

// Persistent decode path (apex_decode.cu)
int decode_setup(apex_ctx* ctx);
void decode_teardown(apex_ctx* ctx);
bool decode_persistent_usable(const apex_ctx* ctx, int B);
int decode_token_persistent(apex_ctx* ctx, const float* h_dev, const float* hpost_dev, float tau, int mode, float* y_dev,
                            cudaStream_t cs);

}  // namespace apex

#endif  // APEX_HOST_HPP

// apex_route_topk_static: the exact top-k gate for callers that must not allocate.
//
// Some users of this library run where a device allocation is not an option: a serving loop whose
// memory is owned entirely by a pool that was sized at start-up (any cudaMalloc outside the pool
// would break its accounting, and cudaMalloc synchronises the whole device), or code that runs
// after the process has handed every remaining byte of HBM to the model.  The context API
// (apex_create) allocates; this entry point does not.  It runs the same gate kernel as
// apex_route_topk and keeps the one buffer the kernel needs beyond its inputs and outputs -- the
// raw logits z_r -- in a fixed array that is part of the library image.
#include <cstdio>
#include <mutex>

#include "apex_internal.hpp"

namespace {

// Scratch of the gate kernel: logits [B][N] for B <= APEX_STATIC_MAX_BATCH, N <= APEX_MAX_EXPERTS.
// 16 KiB, resident on every GPU that loads the library, until the process exits.
static __device__ __align__(256) float g_gate_logits[APEX_STATIC_MAX_BATCH * APEX_MAX_EXPERTS];

constexpr int kMaxDevices = 64;
float* g_logits_addr[kMaxDevices];  // device address of g_gate_logits on each device, 0 = not looked up yet
std::mutex g_setup_mutex;

void say(char* err, size_t err_len, const char* msg) {
  if (err && err_len) snprintf(err, err_len, "%s", msg);
}

}  // namespace

extern "C" int apex_route_topk_static(const float* W_r_dev, const float* b_r_dev, const float* hpost_dev, int N, int d,
                                      int k, int B, int32_t* idx_dev, float* alpha_dev, void* stream, char* err,
                                      size_t err_len) {
  say(err, err_len, "");
  if (!W_r_dev || !hpost_dev || !idx_dev || !alpha_dev) {
    say(err, err_len, "apex_route_topk_static: W_r, h', idx and alpha must not be null");
    return APEX_EINVAL;
  }
  if (B < 1 || B > APEX_STATIC_MAX_BATCH || N < 1 || N > APEX_MAX_EXPERTS) {
    if (err && err_len)
      snprintf(err, err_len, "apex_route_topk_static: B=%d N=%d exceed the built-in scratch (B <= %d, N <= %d)", B, N,
               APEX_STATIC_MAX_BATCH, APEX_MAX_EXPERTS);
    return APEX_EINVAL;
  }
  if (k < 1 || k > N || k > APEX_MAX_TOPK || d < 4 || d > 4096 || (d & 3)) {
    say(err, err_len, "apex_route_topk_static: need 1 <= k <= min(N, 16) and d a multiple of 4, d <= 4096");
    return APEX_EINVAL;
  }
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
    say(err, err_len, e != cudaSuccess ? cudaGetErrorString(e) : "apex_route_topk_static: device index out of range");
    return APEX_ECUDA;
  }
  // First call on this device: look up where the array lives on it.  The name of a __device__
  // array is only a handle in host code; the kernel needs the address cudaGetSymbolAddress returns
  // for the current device.
  float* logits = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_logits_addr[dev]) {
      void* p = nullptr;
      e = cudaGetSymbolAddress(&p, g_gate_logits);
      if (e != cudaSuccess || !p) {
        say(err, err_len, e != cudaSuccess ? cudaGetErrorString(e) : "cudaGetSymbolAddress returned null");
        return APEX_ECUDA;
      }
      g_logits_addr[dev] = static_cast<float*>(p);
    }
    logits = g_logits_addr[dev];
  }
  apex::RouterParams p{};
  p.W = W_r_dev;
  p.bias = b_r_dev;
  p.x = hpost_dev;
  p.z_out = logits;     // scratch: every entry the kernel reads is written by this launch first
  p.q_out = alpha_dev;
  p.pi_out = nullptr;
  p.topk_out = idx_dev;
  p.N = N;
  p.d = d;
  p.B = B;
  p.k = k;
  p.C = N;
  e = apex::launch_router(p, (cudaStream_t)stream);
  if (e != cudaSuccess) {
    say(err, err_len, cudaGetErrorString(e));
    return APEX_ECUDA;
  }
  return APEX_OK;
}

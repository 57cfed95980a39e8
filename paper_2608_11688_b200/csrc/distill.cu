// apex_distill_router: trains the prefetch router q_p = softmax(W_p h + b_p) to match the frozen router's
// distribution q_r on a calibration set (Sec. IV-C, Eq. (10)): minimise the mean over tokens of
// KL(q_r || q_p) by full-batch Adam (0.9 / 0.999 / 1e-8) in fp64 with a fixed iteration count.
//
// Three kernels per iteration, captured once into a CUDA graph and replayed:
//   distill_fwd_kernel   a warp per token: the N logits (lanes stride over d, xor-tree reduction), softmax,
//                        G[t][e] = (q_p - q_r) / T                                   (d loss / d logits)
//   distill_bwd_kernel   d loss / d W[e][j] = sum_t G[t][e] * h[t][j] (j = d is the bias: h = 1); a thread per
//                        column j and tile of eight experts, the tokens cut into kSeg segments whose partial
//                        sums are written separately
//   distill_step_kernel  a thread per parameter: adds the segments' partials in order, Adam update
// Every sum runs in a fixed order, so the result is reproducible bit for bit.
#include <cmath>
#include <cstdio>
#include <vector>

#include "apex_internal.hpp"

namespace {

constexpr int kSeg = 8;      // token segments of the backward pass
constexpr int kTileE = 8;    // experts per thread in the backward pass

struct DistillParams {
  const float* H;    // [T][d]
  const float* Qr;   // [T][N]
  double* Wb;        // [N][d + 1]: W | b
  double* m;         // Adam moments, same shape
  double* v;
  double* G;         // [T][N]
  double* partial;   // [kSeg][N][d + 1]
  int* iter;
  int T, N, d;
  double lr;
};

__device__ __forceinline__ double warp_sum_tree(double x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
  return x;
}
__device__ __forceinline__ double warp_max_tree(double x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x = fmax(x, __shfl_xor_sync(0xffffffffu, x, o));
  return x;
}

__global__ void __launch_bounds__(256) distill_fwd_kernel(const DistillParams p) {
  __shared__ double s_z[8][APEX_MAX_EXPERTS];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int t = blockIdx.x * 8 + warp;
  if (t >= p.T) return;
  const int N = p.N, d = p.d, ld = d + 1;
  const float* h = p.H + (size_t)t * d;
  for (int e = 0; e < N; ++e) {
    const double* w = p.Wb + (size_t)e * ld;
    double a = 0.0;
    for (int j = lane; j < d; j += 32) a = fma((double)h[j], w[j], a);
    a = warp_sum_tree(a);
    if (lane == 0) s_z[warp][e] = a + w[d];
  }
  __syncwarp();
  const int e0 = lane, e1 = lane + 32;
  const double z0 = e0 < N ? s_z[warp][e0] : -INFINITY, z1 = e1 < N ? s_z[warp][e1] : -INFINITY;
  const double mx = warp_max_tree(fmax(z0, z1));
  const double x0 = e0 < N ? exp(z0 - mx) : 0.0, x1 = e1 < N ? exp(z1 - mx) : 0.0;
  const double sum = warp_sum_tree(x0 + x1);
  const double inv_T = 1.0 / (double)p.T;
  if (e0 < N) p.G[(size_t)t * N + e0] = (x0 / sum - (double)p.Qr[(size_t)t * N + e0]) * inv_T;
  if (e1 < N) p.G[(size_t)t * N + e1] = (x1 / sum - (double)p.Qr[(size_t)t * N + e1]) * inv_T;
}

// grid: (ceil((d + 1) / 128), ceil(N / kTileE), kSeg)
__global__ void __launch_bounds__(128) distill_bwd_kernel(const DistillParams p) {
  const int j = blockIdx.x * 128 + threadIdx.x;
  const int e_base = blockIdx.y * kTileE;
  const int seg = blockIdx.z;
  const int N = p.N, d = p.d, ld = d + 1;
  if (j >= ld) return;
  const int per = (p.T + kSeg - 1) / kSeg;
  const int t_lo = seg * per, t_hi = t_lo + per < p.T ? t_lo + per : p.T;
  double acc[kTileE];
#pragma unroll
  for (int q = 0; q < kTileE; ++q) acc[q] = 0.0;
  for (int t = t_lo; t < t_hi; ++t) {
    const double hj = j < d ? (double)p.H[(size_t)t * d + j] : 1.0;
    const double* g = p.G + (size_t)t * N + e_base;
#pragma unroll
    for (int q = 0; q < kTileE; ++q)
      if (e_base + q < N) acc[q] = fma(g[q], hj, acc[q]);
  }
#pragma unroll
  for (int q = 0; q < kTileE; ++q)
    if (e_base + q < N) p.partial[((size_t)seg * N + e_base + q) * ld + j] = acc[q];
}

__global__ void __launch_bounds__(256) distill_step_kernel(const DistillParams p) {
  const size_t n = (size_t)p.N * (p.d + 1);
  const size_t i = (size_t)blockIdx.x * 256 + threadIdx.x;
  const int it = *p.iter + 1;
  if (i < n) {
    double g = 0.0;
#pragma unroll
    for (int s = 0; s < kSeg; ++s) g += p.partial[(size_t)s * n + i];
    const double m = 0.9 * p.m[i] + 0.1 * g;
    const double v = 0.999 * p.v[i] + 0.001 * g * g;
    p.m[i] = m;
    p.v[i] = v;
    const double mh = m / (1.0 - pow(0.9, (double)it)), vh = v / (1.0 - pow(0.999, (double)it));
    p.Wb[i] = p.Wb[i] - p.lr * mh / (sqrt(vh) + 1e-8);
  }
}

// every CTA of the step kernel reads the counter, so it is advanced by a kernel of its own
__global__ void distill_tick_kernel(int* iter) { *iter += 1; }

void say(char* err, size_t err_len, const char* msg) {
  if (err && err_len) snprintf(err, err_len, "%s", msg);
}

}  // namespace

extern "C" int apex_distill_router(const float* H_dev, const float* Qr_dev, int T, int N, int d, int iters, double lr,
                                   float* W_host, float* b_host, void* stream, char* err, size_t err_len) {
  say(err, err_len, "");
  if (!H_dev || !Qr_dev || !W_host || !b_host || T < 1 || N < 1 || N > APEX_MAX_EXPERTS || d < 1 || iters < 1 || !(lr > 0.0)) {
    say(err, err_len, "apex_distill_router: bad argument (N <= 64, T, d, iters >= 1, lr > 0, no null pointer)");
    return APEX_EINVAL;
  }
  cudaStream_t cs = (cudaStream_t)stream;
  const int ld = d + 1;
  const size_t n = (size_t)N * ld;
  std::vector<double> init(n);
  for (int e = 0; e < N; ++e) {
    for (int j = 0; j < d; ++j) init[(size_t)e * ld + j] = (double)W_host[(size_t)e * d + j];
    init[(size_t)e * ld + d] = (double)b_host[e];
  }
  DistillParams p{};
  p.H = H_dev; p.Qr = Qr_dev; p.T = T; p.N = N; p.d = d; p.lr = lr;
  double* buf = nullptr;
  const size_t n_dbl = 3 * n + (size_t)T * N + (size_t)kSeg * n;
  cudaGraph_t graph = nullptr;
  cudaGraphExec_t exec = nullptr;
  int rc = APEX_OK;
  cudaError_t e = cudaSuccess;
  auto fail = [&](cudaError_t ce) {
    say(err, err_len, cudaGetErrorString(ce));
    rc = ce == cudaErrorMemoryAllocation ? APEX_ENOMEM : APEX_ECUDA;
  };
  do {
    if ((e = cudaMalloc(&buf, n_dbl * sizeof(double) + sizeof(int))) != cudaSuccess) { fail(e); break; }
    p.Wb = buf; p.m = buf + n; p.v = buf + 2 * n; p.G = buf + 3 * n; p.partial = buf + 3 * n + (size_t)T * N;
    p.iter = reinterpret_cast<int*>(buf + n_dbl);
    if ((e = cudaMemsetAsync(buf, 0, n_dbl * sizeof(double) + sizeof(int), cs)) != cudaSuccess) { fail(e); break; }
    if ((e = cudaMemcpyAsync(p.Wb, init.data(), sizeof(double) * n, cudaMemcpyHostToDevice, cs)) != cudaSuccess) { fail(e); break; }
    cudaStream_t cap = nullptr;
    if ((e = cudaStreamCreateWithFlags(&cap, cudaStreamNonBlocking)) != cudaSuccess) { fail(e); break; }
    e = cudaStreamBeginCapture(cap, cudaStreamCaptureModeThreadLocal);
    if (e == cudaSuccess) {
      distill_fwd_kernel<<<(T + 7) / 8, 256, 0, cap>>>(p);
      distill_bwd_kernel<<<dim3((ld + 127) / 128, (N + kTileE - 1) / kTileE, kSeg), 128, 0, cap>>>(p);
      distill_step_kernel<<<(unsigned)((n + 255) / 256), 256, 0, cap>>>(p);
      distill_tick_kernel<<<1, 1, 0, cap>>>(p.iter);
      e = cudaStreamEndCapture(cap, &graph);
    }
    cudaStreamDestroy(cap);
    if (e != cudaSuccess) { fail(e); break; }
    if ((e = cudaGraphInstantiate(&exec, graph, 0)) != cudaSuccess) { fail(e); break; }
    for (int it = 0; it < iters && e == cudaSuccess; ++it) e = cudaGraphLaunch(exec, cs);
    if (e != cudaSuccess) { fail(e); break; }
    std::vector<double> out(n);
    if ((e = cudaMemcpyAsync(out.data(), p.Wb, sizeof(double) * n, cudaMemcpyDeviceToHost, cs)) != cudaSuccess) { fail(e); break; }
    if ((e = cudaStreamSynchronize(cs)) != cudaSuccess) { fail(e); break; }
    for (int ex = 0; ex < N; ++ex) {
      for (int j = 0; j < d; ++j) W_host[(size_t)ex * d + j] = (float)out[(size_t)ex * ld + j];
      b_host[ex] = (float)out[(size_t)ex * ld + d];
    }
  } while (false);
  if (exec) cudaGraphExecDestroy(exec);
  if (graph) cudaGraphDestroy(graph);
  if (buf) cudaFree(buf);
  return rc;
}

// apex_fit_cdf: fits the ordinal-logistic confidence model p_delta(x) = sigmoid(theta_delta - w.x)
// (Eq. (8)) on a calibration set by the cumulative binary cross-entropy of Eq. (11), on the GPU.
//
//   loss(w, theta) = -(1/T) sum_t sum_delta [ y log p + (1 - y) log(1 - p) ],  y = [delta >= delta*_t]
//
// theta is kept non-decreasing by the parametrisation theta_delta = t0 + sum_{i <= delta} softplus(u_i).
// Full-batch Adam (beta 0.9 / 0.999, eps 1e-8) in fp64 with a fixed iteration count, started from
// w = 0 and the logit of the empirical distribution of delta*; every reduction runs in a fixed order,
// so two runs give the same bits.
//
// Two kernels per iteration: `cdf_grad_kernel` (a thread per calibration token: s = w.x and the nth
// sigmoids; then a thread per parameter adds the tokens' contributions in ascending token order and
// writes one partial vector per CTA), `cdf_step_kernel` (one CTA: sums the
// partials in CTA order, chain rule through the softplus parametrisation, Adam update, new theta).
// The iterations are captured once into a CUDA graph and replayed.
#include <cmath>
#include <cstdio>
#include <vector>

#include "apex_internal.hpp"

namespace {

constexpr int kFitThreads = 64;
constexpr int kMaxTheta = APEX_MAX_EXPERTS + 1;          // N - k + 1 <= N
constexpr int kMaxParams = APEX_MAX_EXPERTS + kMaxTheta;  // w, then t0 and u_1..u_{nth-1}

struct FitParams {
  const double* X;       // [T][N]
  const int32_t* dstar;  // [T]
  double* params;        // [N + nth]: w | t0 | u
  double* theta;         // [nth]
  double* m;             // Adam moments
  double* v;
  double* partial;       // [grid][N + nth]: per-CTA sums of d loss/d w (N) and d loss/d theta (nth)
  int* iter;             // Adam step counter (device)
  int T, N, nth, grid;
  double lr;
};

// Per-CTA partial gradient.  The CTA walks its tokens in chunks of kFitThreads: a thread per token
// computes that token's d loss / d z for every threshold into shared memory; then a thread per
// parameter adds the chunk's contributions in ascending token order (a fixed order, no atomics).
__global__ void __launch_bounds__(kFitThreads) cdf_grad_kernel(const FitParams p) {
  __shared__ double s_w[APEX_MAX_EXPERTS];
  __shared__ double s_theta[kMaxTheta];
  __shared__ double s_g[kFitThreads][kMaxTheta];  // d loss / d z of the chunk's tokens
  __shared__ double s_gsum[kFitThreads];
  const int tid = threadIdx.x;
  const int N = p.N, nth = p.nth, P = N + nth;
  for (int i = tid; i < N; i += kFitThreads) s_w[i] = p.params[i];
  for (int i = tid; i < nth; i += kFitThreads) s_theta[i] = p.theta[i];
  __syncthreads();
  double acc[(kMaxParams + kFitThreads - 1) / kFitThreads];  // parameters tid, tid + kFitThreads, ...
#pragma unroll
  for (int q = 0; q < (kMaxParams + kFitThreads - 1) / kFitThreads; ++q) acc[q] = 0.0;
  const double inv_T = 1.0 / (double)p.T;
  for (int base = blockIdx.x * kFitThreads; base < p.T; base += gridDim.x * kFitThreads) {
    const int t = base + tid;
    const int n_tok = p.T - base < kFitThreads ? p.T - base : kFitThreads;
    if (t < p.T) {
      const double* x = p.X + (size_t)t * N;
      double s = 0.0;
      for (int j = 0; j < N; ++j) s = fma(x[j], s_w[j], s);
      const int ds = p.dstar[t];
      double gsum = 0.0;
      for (int dl = 0; dl < nth; ++dl) {
        const double z = s_theta[dl] - s;
        const double pr = 1.0 / (1.0 + exp(-z));
        const double g = (pr - (dl >= ds ? 1.0 : 0.0)) * inv_T;  // d loss / d z
        s_g[tid][dl] = g;
        gsum += g;
      }
      s_gsum[tid] = gsum;
    }
    __syncthreads();
#pragma unroll
    for (int q = 0; q < (kMaxParams + kFitThreads - 1) / kFitThreads; ++q) {
      const int i = tid + q * kFitThreads;
      if (i < N) {  // z = theta - w.x: d z / d w_i = -x_i
        double a = acc[q];
        for (int u = 0; u < n_tok; ++u) a = fma(-s_gsum[u], p.X[(size_t)(base + u) * N + i], a);
        acc[q] = a;
      } else if (i < P) {
        double a = acc[q];
        for (int u = 0; u < n_tok; ++u) a += s_g[u][i - N];
        acc[q] = a;
      }
    }
    __syncthreads();
  }
#pragma unroll
  for (int q = 0; q < (kMaxParams + kFitThreads - 1) / kFitThreads; ++q) {
    const int i = tid + q * kFitThreads;
    if (i < P) p.partial[(size_t)blockIdx.x * P + i] = acc[q];
  }
}

// One Adam step.  One CTA: thread i sums partial gradient i over the CTAs in ascending order; thread 0
// then walks the short sequential parts (suffix sums for the softplus chain rule, new theta).
__global__ void __launch_bounds__(kFitThreads * 2) cdf_step_kernel(const FitParams p) {
  __shared__ double s_g[kMaxParams];      // d loss / d w | d loss / d theta
  __shared__ double s_grad[kMaxParams];   // gradient in parameter space: w | t0 | u
  const int tid = threadIdx.x;
  const int N = p.N, nth = p.nth, P = N + nth;
  for (int i = tid; i < P; i += blockDim.x) {
    double a = 0.0;
    for (int c = 0; c < p.grid; ++c) a += p.partial[(size_t)c * P + i];
    s_g[i] = a;
  }
  __syncthreads();
  if (tid == 0) {
    // theta_j = t0 + sum_{i <= j} softplus(u_i):  d/d t0 = sum_j g_theta[j],  d/d u_i = sigmoid(u_i) * sum_{j >= i} g_theta[j]
    double tail = 0.0;
    for (int j = nth - 1; j >= 1; --j) {
      tail += s_g[N + j];
      const double u = p.params[N + j];
      s_grad[N + j] = tail / (1.0 + exp(-u));
    }
    s_grad[N] = tail + s_g[N];
  }
  if (tid < N) s_grad[tid] = s_g[tid];
  __syncthreads();
  const int it = *p.iter + 1;
  if (tid < P) {
    const double g = s_grad[tid];
    const double m = 0.9 * p.m[tid] + 0.1 * g;
    const double v = 0.999 * p.v[tid] + 0.001 * g * g;
    p.m[tid] = m;
    p.v[tid] = v;
    const double mh = m / (1.0 - pow(0.9, (double)it)), vh = v / (1.0 - pow(0.999, (double)it));
    p.params[tid] = p.params[tid] - p.lr * mh / (sqrt(vh) + 1e-8);
  }
  __syncthreads();
  if (tid == 0) {
    *p.iter = it;
    const double t0 = p.params[N];
    p.theta[0] = t0;
    double c = 0.0;
    for (int j = 1; j < nth; ++j) {
      const double u = p.params[N + j];
      c += fmax(u, 0.0) + log1p(exp(-fabs(u)));  // softplus
      p.theta[j] = t0 + c;
    }
  }
}

void say(char* err, size_t err_len, const char* msg) {
  if (err && err_len) snprintf(err, err_len, "%s", msg);
}

}  // namespace

extern "C" int apex_fit_cdf(const double* X_dev, const int32_t* dstar_dev, int T, int N, int k, int iters, double lr,
                            float* w_host, float* theta_host, void* stream, char* err, size_t err_len) {
  say(err, err_len, "");
  if (!X_dev || !dstar_dev || !w_host || !theta_host || T < 1 || N < 1 || N > APEX_MAX_EXPERTS || k < 1 || k > N || iters < 1 ||
      !(lr > 0.0)) {
    say(err, err_len, "apex_fit_cdf: bad argument (N <= 64, 1 <= k <= N, T >= 1, iters >= 1, lr > 0)");
    return APEX_EINVAL;
  }
  cudaStream_t cs = (cudaStream_t)stream;
  const int nth = N - k + 1, P = N + nth;
  // start: w = 0, theta = logit of the empirical distribution of delta*, increments at least 1e-3
  std::vector<int32_t> ds(T);
  cudaError_t e = cudaMemcpyAsync(ds.data(), dstar_dev, sizeof(int32_t) * T, cudaMemcpyDeviceToHost, cs);
  if (e == cudaSuccess) e = cudaStreamSynchronize(cs);
  if (e != cudaSuccess) {
    say(err, err_len, cudaGetErrorString(e));
    return APEX_ECUDA;
  }
  std::vector<double> init(P, 0.0), th0(nth);
  for (int j = 0; j < nth; ++j) {
    long long c = 0;
    for (int t = 0; t < T; ++t) c += (j >= ds[t]) ? 1 : 0;
    double f = (double)c / (double)T;
    f = f < 1e-3 ? 1e-3 : (f > 1.0 - 1e-3 ? 1.0 - 1e-3 : f);
    th0[j] = std::log(f / (1.0 - f));
  }
  init[N] = th0[0];
  for (int j = 1; j < nth; ++j) {
    const double inc = th0[j] - th0[j - 1] > 1e-3 ? th0[j] - th0[j - 1] : 1e-3;
    init[N + j] = std::log(std::expm1(inc));  // inverse softplus
  }
  std::vector<double> theta_init(nth);
  theta_init[0] = init[N];
  double csum = 0.0;
  for (int j = 1; j < nth; ++j) {
    const double u = init[N + j];
    csum += std::fmax(u, 0.0) + std::log1p(std::exp(-std::fabs(u)));
    theta_init[j] = init[N] + csum;
  }

  int n_sm = 0, dev = 0;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev);
  FitParams p{};
  p.T = T; p.N = N; p.nth = nth; p.lr = lr;
  p.grid = (T + kFitThreads - 1) / kFitThreads;
  if (p.grid > 2 * n_sm) p.grid = 2 * n_sm;
  double* buf = nullptr;
  const size_t n_dbl = (size_t)P * 3 + nth + (size_t)p.grid * P;
  cudaGraph_t graph = nullptr;
  cudaGraphExec_t exec = nullptr;
  int rc = APEX_OK;
  auto fail = [&](cudaError_t ce) {
    say(err, err_len, cudaGetErrorString(ce));
    rc = ce == cudaErrorMemoryAllocation ? APEX_ENOMEM : APEX_ECUDA;
  };
  do {
    if ((e = cudaMalloc(&buf, n_dbl * sizeof(double) + sizeof(int))) != cudaSuccess) { fail(e); break; }
    p.X = X_dev; p.dstar = dstar_dev;
    p.params = buf; p.m = buf + P; p.v = buf + 2 * P; p.theta = buf + 3 * P; p.partial = buf + 3 * P + nth;
    p.iter = reinterpret_cast<int*>(buf + n_dbl);
    if ((e = cudaMemsetAsync(buf, 0, n_dbl * sizeof(double) + sizeof(int), cs)) != cudaSuccess) { fail(e); break; }
    if ((e = cudaMemcpyAsync(p.params, init.data(), sizeof(double) * P, cudaMemcpyHostToDevice, cs)) != cudaSuccess) { fail(e); break; }
    if ((e = cudaMemcpyAsync(p.theta, theta_init.data(), sizeof(double) * nth, cudaMemcpyHostToDevice, cs)) != cudaSuccess) { fail(e); break; }
    // one iteration as a graph, replayed `iters` times
    cudaStream_t cap = nullptr;
    if ((e = cudaStreamCreateWithFlags(&cap, cudaStreamNonBlocking)) != cudaSuccess) { fail(e); break; }
    e = cudaStreamBeginCapture(cap, cudaStreamCaptureModeThreadLocal);
    if (e == cudaSuccess) {
      cdf_grad_kernel<<<p.grid, kFitThreads, 0, cap>>>(p);
      cdf_step_kernel<<<1, kFitThreads * 2, 0, cap>>>(p);
      e = cudaStreamEndCapture(cap, &graph);
    }
    cudaStreamDestroy(cap);
    if (e != cudaSuccess) { fail(e); break; }
    if ((e = cudaGraphInstantiate(&exec, graph, 0)) != cudaSuccess) { fail(e); break; }
    for (int it = 0; it < iters && e == cudaSuccess; ++it) e = cudaGraphLaunch(exec, cs);
    if (e != cudaSuccess) { fail(e); break; }
    std::vector<double> out(P + nth);
    if ((e = cudaMemcpyAsync(out.data(), p.params, sizeof(double) * N, cudaMemcpyDeviceToHost, cs)) != cudaSuccess) { fail(e); break; }
    if ((e = cudaMemcpyAsync(out.data() + P, p.theta, sizeof(double) * nth, cudaMemcpyDeviceToHost, cs)) != cudaSuccess) { fail(e); break; }
    if ((e = cudaStreamSynchronize(cs)) != cudaSuccess) { fail(e); break; }
    for (int j = 0; j < N; ++j) w_host[j] = (float)out[j];
    float run = -INFINITY;
    for (int j = 0; j < nth; ++j) {  // fp32 rounding must not break the order
      const float t = (float)out[P + j];
      run = t > run ? t : run;
      theta_host[j] = run;
    }
  } while (false);
  if (exec) cudaGraphExecDestroy(exec);
  if (graph) cudaGraphDestroy(graph);
  if (buf) cudaFree(buf);
  return rc;
}

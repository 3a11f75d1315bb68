// AdamW for the parameters outside the Muon set (Algorithm 1 line 11 of the
// paper: biases, normalisation scales and everything outside the transformer
// blocks keep the baseline's AdamW).  One multi-tensor kernel: up to
// kAdamwTensors tensors per launch, pointers passed by value, so no workspace
// and no allocation is needed.  Bandwidth-bound and, for the small tensors of
// this group, launch-bound; fp32 arithmetic, moments in fp32.
//
//   p <- p*(1 - lr*wd)
//   m <- beta1*m + (1-beta1)*g,   v <- beta2*v + (1-beta2)*g^2
//   p <- p - lr * (m/(1-beta1^t)) / (sqrt(v/(1-beta2^t)) + eps)
#include <math.h>

#include "common.cuh"

namespace {

using namespace prm;

constexpr int kAdamwTensors = 48;
constexpr int kAdamwThreads = 256;
constexpr int kAdamwPerBlock = kAdamwThreads * 8 * 4;   // elements per CTA

struct AdamwBatch {
  void* p[kAdamwTensors];
  const void* g[kAdamwTensors];
  float* m[kAdamwTensors];
  float* v[kAdamwTensors];
  long long n[kAdamwTensors];
};

struct AdamwScalars {
  float decay;      // 1 - lr*wd
  float beta1, omb1, beta2, omb2;
  float step_size;  // lr / (1 - beta1^t)
  float inv_bc2;    // 1 / sqrt(1 - beta2^t)
  float eps;
};

__device__ __forceinline__ float adamw_one(float p, float g, float& m, float& v, const AdamwScalars& s) {
  m = s.beta1 * m + s.omb1 * g;
  v = s.beta2 * v + s.omb2 * g * g;
  const float denom = sqrtf(v) * s.inv_bc2 + s.eps;
  return p * s.decay - s.step_size * (m / denom);
}

template <typename IO>
__global__ void __launch_bounds__(kAdamwThreads)
adamw_kernel(AdamwBatch b, AdamwScalars s) {
  const int t = blockIdx.y;
  const long long n = b.n[t];
  const long long base = (long long)blockIdx.x * kAdamwPerBlock;
  if (base >= n) return;
  IO* __restrict__ p = reinterpret_cast<IO*>(b.p[t]);
  const IO* __restrict__ g = reinterpret_cast<const IO*>(b.g[t]);
  float* __restrict__ m = b.m[t];
  float* __restrict__ v = b.v[t];
  const long long end = min(n, base + (long long)kAdamwPerBlock);
  const long long vec_end = base + ((end - base) & ~7LL);
  for (long long i = base + 8LL * threadIdx.x; i < vec_end; i += 8LL * kAdamwThreads) {
    float pv[8], gv[8], mv[8], vv[8];
    load8(p + i, pv);
    load8_stream(g + i, gv);
    load8(m + i, mv);
    load8(v + i, vv);
#pragma unroll
    for (int e = 0; e < 8; ++e) pv[e] = adamw_one(pv[e], gv[e], mv[e], vv[e], s);
    store8(m + i, mv);
    store8(v + i, vv);
    store8(p + i, pv);
  }
  for (long long i = vec_end + threadIdx.x; i < end; i += kAdamwThreads) {
    float mm = m[i], vv = v[i];
    const float pn = adamw_one(to_f32(p[i]), to_f32(g[i]), mm, vv, s);
    m[i] = mm;
    v[i] = vv;
    from_f32(p + i, pn);
  }
}

}  // namespace

extern "C" int prm_adamw_step(int n_tensors, void* const* params, const void* const* grads,
                              float* const* exp_avg, float* const* exp_avg_sq, const int64_t* numel,
                              int io_fp32, float lr, float beta1, float beta2, float eps, float wd,
                              int64_t step, void* cuda_stream) {
  if (n_tensors < 0 || step < 1) return PRM_ERR_ARG;
  if (n_tensors == 0) return PRM_OK;
  if (!params || !grads || !exp_avg || !exp_avg_sq || !numel) return PRM_ERR_ARG;
  if (!(beta1 >= 0.f && beta1 < 1.f) || !(beta2 >= 0.f && beta2 < 1.f) || eps < 0.f) return PRM_ERR_ARG;
  for (int i = 0; i < n_tensors; ++i) {
    if (numel[i] < 0) return PRM_ERR_SHAPE;
    if (numel[i] == 0) continue;
    if (!params[i] || !grads[i] || !exp_avg[i] || !exp_avg_sq[i]) return PRM_ERR_ARG;
    if ((((uintptr_t)params[i] | (uintptr_t)grads[i] | (uintptr_t)exp_avg[i] | (uintptr_t)exp_avg_sq[i]) & 15) != 0)
      return PRM_ERR_ALIGN;
  }
  AdamwScalars s;
  s.decay = 1.f - lr * wd;
  s.beta1 = beta1; s.omb1 = 1.f - beta1;
  s.beta2 = beta2; s.omb2 = 1.f - beta2;
  s.step_size = (float)((double)lr / (1.0 - pow((double)beta1, (double)step)));
  s.inv_bc2 = (float)(1.0 / sqrt(1.0 - pow((double)beta2, (double)step)));
  s.eps = eps;
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  for (int first = 0; first < n_tensors; first += kAdamwTensors) {
    AdamwBatch b;
    const int cnt = n_tensors - first < kAdamwTensors ? n_tensors - first : kAdamwTensors;
    long long max_n = 0;
    for (int k = 0; k < kAdamwTensors; ++k) {
      const bool live = k < cnt;
      b.p[k] = live ? params[first + k] : nullptr;
      b.g[k] = live ? grads[first + k] : nullptr;
      b.m[k] = live ? exp_avg[first + k] : nullptr;
      b.v[k] = live ? exp_avg_sq[first + k] : nullptr;
      b.n[k] = live ? (long long)numel[first + k] : 0;
      if (b.n[k] > max_n) max_n = b.n[k];
    }
    if (max_n == 0) continue;
    const long long blocks = (max_n + kAdamwPerBlock - 1) / kAdamwPerBlock;
    if (blocks > 0x7fffffffLL) return PRM_ERR_SHAPE;
    dim3 grid((unsigned)blocks, (unsigned)cnt, 1);
    if (io_fp32) adamw_kernel<float><<<grid, kAdamwThreads, 0, stream>>>(b, s);
    else adamw_kernel<__nv_bfloat16><<<grid, kAdamwThreads, 0, stream>>>(b, s);
    if (cudaGetLastError() != cudaSuccess) return PRM_ERR_CUDA;
  }
  return PRM_OK;
}

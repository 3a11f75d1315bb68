// Row step of ONE tall matrix for callers that cannot allocate device memory.
//
// The regular path (prm_step) keeps the column partial sums and column norms
// of tall matrices in a workspace that the caller allocates.  Some callers
// have no way to do that: a plug-in running inside a host process whose
// memory pool has already claimed the device's memory, or a control loop that
// must never hit the device-wide synchronisation hidden in cudaMalloc and
// cudaFree.  For them this file keeps the scratch in a fixed array that is
// part of the library image: every GPU that loads the library holds
// kNoAllocFloats * 4 bytes (4 MiB) of it until the process exits.
//
// The array is shared by every call.  It keeps whatever the last call left;
// nothing in it has to start at zero, because each call overwrites every
// entry it later reads (one partial per row block and column, one norm per
// column).  Two calls that overlap on the GPU (different streams, no ordering
// between them) race on the array and give wrong results.
#include <mutex>

#include <stdio.h>

#include "tall_kernels.cuh"

namespace {

using namespace prm;

constexpr size_t kNoAllocFloats = (size_t)1 << 20;
constexpr int kNaMaxDevices = 64;

// In host code this name is only a handle for cudaGetSymbolAddress: it is not
// a device address and must never be passed to a kernel as one.
static __device__ __align__(256) float g_noalloc_scratch[kNoAllocFloats];

std::mutex g_na_mutex;
float* g_na_addr[kNaMaxDevices] = {};   // device address of the array, per device

template <typename IO>
__global__ void __launch_bounds__(kTallThreads)
na_pass1_kernel(const IO* __restrict__ g, float* __restrict__ m, int rows, int cols, float beta,
                float omb, int nesterov, float* __restrict__ partial /*[row blocks][cols]*/) {
  const int row0 = blockIdx.y * kTallRows;
  tall_pass1_block<IO>(g, m, cols, row0, min(rows, row0 + kTallRows), blockIdx.x, beta, omb, nesterov,
                       partial + (int64_t)blockIdx.y * cols);
}

__global__ void __launch_bounds__(kTallThreads)
na_colnorm_kernel(const float* __restrict__ partial, float* __restrict__ nu, int nblk, int cols,
                  float eps) {
  const int col = blockIdx.x * kTallThreads + threadIdx.x;
  if (col >= cols) return;
  nu[col] = fmaxf(sqrtf(tall_column_sum(partial, nblk, cols, col)), eps);
}

template <typename IO>
__global__ void __launch_bounds__(kTallThreads)
na_pass2_kernel(IO* __restrict__ p, const IO* __restrict__ g, const float* __restrict__ m, int rows,
                int cols, float beta, float omb, int nesterov, float decay, float lr_s_gamma,
                const float* __restrict__ nu) {
  const int row0 = blockIdx.y * kTallRows;
  tall_pass2_block<IO>(p, g, m, cols, row0, min(rows, row0 + kTallRows), blockIdx.x, beta, omb, nesterov, decay,
                       [&](int col) { return lr_s_gamma / nu[col]; });
}

int na_fail(char* errbuf, size_t len, int code, const char* msg) {
  if (errbuf && len) snprintf(errbuf, len, "%s", msg);
  return code;
}

template <typename IO>
cudaError_t na_launch(void* param, const void* grad, float* momentum, int rows, int cols, float beta,
                      int nesterov, float decay, float lr_s_gamma, float eps, float* scratch,
                      cudaStream_t stream) {
  const int nblk = (rows + kTallRows - 1) / kTallRows;
  float* partial = scratch;
  float* nu = scratch + (size_t)nblk * cols;
  dim3 grid((cols + 255) / 256, nblk, 1);
  na_pass1_kernel<IO><<<grid, kTallThreads, 0, stream>>>((const IO*)grad, momentum, rows, cols, beta,
                                                       1.f - beta, nesterov, partial);
  na_colnorm_kernel<<<(cols + kTallThreads - 1) / kTallThreads, kTallThreads, 0, stream>>>(partial, nu, nblk, cols, eps);
  na_pass2_kernel<IO><<<grid, kTallThreads, 0, stream>>>((IO*)param, (const IO*)grad, momentum, rows, cols,
                                                       beta, 1.f - beta, nesterov, decay, lr_s_gamma, nu);
  return cudaGetLastError();
}

}  // namespace

extern "C" int prm_rowstep_tall_noalloc(void* param, const void* grad, float* momentum, int64_t rows,
                                        int64_t cols, int io_fp32, float beta, int nesterov, float lr,
                                        float wd, float gamma, float eps_row, float scale,
                                        void* cuda_stream, char* errbuf, size_t errbuf_len) {
  if (errbuf && errbuf_len) errbuf[0] = 0;
  if (!param || !grad || !momentum) return na_fail(errbuf, errbuf_len, PRM_ERR_ARG, "NULL matrix pointer");
  if ((((uintptr_t)param | (uintptr_t)grad | (uintptr_t)momentum) & 15) != 0)
    return na_fail(errbuf, errbuf_len, PRM_ERR_ALIGN, "matrix pointer not 16-byte aligned");
  if (rows < 1 || cols < 1 || rows <= cols)
    return na_fail(errbuf, errbuf_len, PRM_ERR_SHAPE, "only tall matrices (rows > cols) need scratch; use prm_step for the rest");
  if (cols % 8 != 0) return na_fail(errbuf, errbuf_len, PRM_ERR_SHAPE, "cols must be a multiple of 8");
  const int64_t nblk = (rows + kTallRows - 1) / kTallRows;
  if (nblk > 65535 || rows > 0x7fffffffLL)
    return na_fail(errbuf, errbuf_len, PRM_ERR_SHAPE, "too many rows");
  const size_t need = (size_t)(nblk + 1) * (size_t)cols;
  if (need > kNoAllocFloats) {
    char msg[200];
    snprintf(msg, sizeof msg,
             "matrix needs %zu floats of scratch ((ceil(rows/128)+1)*cols), the built-in array holds %zu",
             need, kNoAllocFloats);
    return na_fail(errbuf, errbuf_len, PRM_ERR_WORKSPACE, msg);
  }
  int dev = -1;
  cudaError_t ce = cudaGetDevice(&dev);
  if (ce != cudaSuccess) return na_fail(errbuf, errbuf_len, PRM_ERR_CUDA, cudaGetErrorString(ce));
  if (dev < 0 || dev >= kNaMaxDevices) return na_fail(errbuf, errbuf_len, PRM_ERR_CUDA, "device index out of range");
  float* scratch = nullptr;
  {
    // Set-up, once per device, with that device current: resolve the device
    // address of the built-in array.
    std::lock_guard<std::mutex> lock(g_na_mutex);
    if (!g_na_addr[dev]) {
      float* ptr = nullptr;
      ce = cudaGetSymbolAddress((void**)&ptr, g_noalloc_scratch);
      if (ce != cudaSuccess || !ptr)
        return na_fail(errbuf, errbuf_len, PRM_ERR_CUDA,
                       ce != cudaSuccess ? cudaGetErrorString(ce) : "cudaGetSymbolAddress returned NULL");
      g_na_addr[dev] = ptr;
    }
    scratch = g_na_addr[dev];
  }
  const float decay = 1.f - lr * wd;
  const float lr_s_gamma = lr * scale * gamma;
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  ce = io_fp32 ? na_launch<float>(param, grad, momentum, (int)rows, (int)cols, beta, nesterov ? 1 : 0,
                                  decay, lr_s_gamma, eps_row, scratch, stream)
               : na_launch<__nv_bfloat16>(param, grad, momentum, (int)rows, (int)cols, beta,
                                          nesterov ? 1 : 0, decay, lr_s_gamma, eps_row, scratch, stream);
  if (ce != cudaSuccess) return na_fail(errbuf, errbuf_len, PRM_ERR_CUDA, cudaGetErrorString(ce));
  return PRM_OK;
}

// Sharded tall RowNorm: the row step of a tall matrix whose rows are split
// over ranks (paper, Section 3.3, Eq. sharded-tall-rownorm; Algorithm 2 lines
// 9-13; correctness: the sharded-RowNorm proposition of the appendix).
//
// For m > n the oriented rows are stored columns, so each one spans all
// ranks.  Rank q first updates its momentum rows and reduces its local column
// sums of squares  q_j^(q) = sum_{i in S_q} U_ij^2  (prm_tall_shard_stats);
// the caller sum-all-reduces those n numbers per matrix (a packed buffer for
// all tall matrices; NCCL or any other transport, overlapped with the wide
// matrices' row steps); then every rank finishes its rows with the global
// norms  nu_j = max(sqrt(sum_q q_j^(q)), eps)  (prm_tall_shard_apply).
// The square root and the clamp come after the sum, as the algorithm states.
//
// Reductions run in a fixed order; only the all-reduce may reorder the sum
// over ranks, which is the paper's own caveat.
#include "common.cuh"

namespace {

using namespace prm;

constexpr int kShThreads = 256;

template <typename IO>
__global__ void __launch_bounds__(kShThreads)
shard_pass1_kernel(const IO* __restrict__ g, float* __restrict__ m, int rows, int cols, float beta, float omb,
                   int nesterov, float* __restrict__ partial /*[row blocks][cols]*/) {
  __shared__ float red[kShThreads / 32][32 * 8 + 1];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int col0 = (blockIdx.x * 32 + lane) * 8;
  const int row0 = blockIdx.y * kTallRows;
  const int row1 = min(rows, row0 + kTallRows);
  float cs[8];
#pragma unroll
  for (int e = 0; e < 8; ++e) cs[e] = 0.f;
  if (col0 < cols) {
#pragma unroll 4
    for (int row = row0 + warp; row < row1; row += kShThreads / 32) {
      const int64_t off = (int64_t)row * cols + col0;
      float gv[8], mv[8];
      load8_stream(g + off, gv);
      load8(m + off, mv);
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const float mn = blend(beta, mv[e], omb, gv[e]);
        mv[e] = mn;
        const float uu = nesterov ? blend(beta, mn, omb, gv[e]) : mn;
        cs[e] += uu * uu;
      }
      store8(m + off, mv);
    }
  }
#pragma unroll
  for (int e = 0; e < 8; ++e) red[warp][lane * 8 + e] = cs[e];
  __syncthreads();
  const int col = blockIdx.x * 256 + threadIdx.x;
  if (col < cols) {
    float tot = 0.f;
#pragma unroll
    for (int w = 0; w < kShThreads / 32; ++w) tot += red[w][threadIdx.x];
    partial[(int64_t)blockIdx.y * cols + col] = tot;
  }
}

// Local column sums of squares: sum over this rank's row blocks, no root.
__global__ void __launch_bounds__(kShThreads)
shard_colsum_kernel(const float* __restrict__ partial, float* __restrict__ colsumsq, int nblk, int cols) {
  const int col = blockIdx.x * kShThreads + threadIdx.x;
  if (col >= cols) return;
  float tot = 0.f;
  for (int b = 0; b < nblk; ++b) tot += partial[(int64_t)b * cols + col];
  colsumsq[col] = tot;
}

template <typename IO>
__global__ void __launch_bounds__(kShThreads)
shard_pass2_kernel(IO* __restrict__ p, const IO* __restrict__ g, const float* __restrict__ m, int rows, int cols,
                   float beta, float omb, int nesterov, float decay, float lr_s_gamma, float eps,
                   const float* __restrict__ colsumsq /*[cols], summed over all ranks*/) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int col0 = (blockIdx.x * 32 + lane) * 8;
  if (col0 >= cols) return;
  const int row0 = blockIdx.y * kTallRows;
  const int row1 = min(rows, row0 + kTallRows);
  float coef[8];
#pragma unroll
  for (int e = 0; e < 8; ++e) coef[e] = lr_s_gamma / fmaxf(sqrtf(colsumsq[col0 + e]), eps);   // sqrt, then clamp
#pragma unroll 4
  for (int row = row0 + warp; row < row1; row += kShThreads / 32) {
    const int64_t off = (int64_t)row * cols + col0;
    float mv[8], pv[8];
    load8_stream(m + off, mv);
    load8_stream(p + off, pv);
    if (nesterov) {
      float gv[8];
      load8_stream(g + off, gv);
#pragma unroll
      for (int e = 0; e < 8; ++e) mv[e] = blend(beta, mv[e], omb, gv[e]);
    }
#pragma unroll
    for (int e = 0; e < 8; ++e) pv[e] = decay * pv[e] - coef[e] * mv[e];
    store8(p + off, pv);
  }
}

int shard_check(const void* a, const void* b, const void* c, int64_t rows, int64_t cols) {
  if (!a || !b || !c) return PRM_ERR_ARG;
  if ((((uintptr_t)a | (uintptr_t)b | (uintptr_t)c) & 15) != 0) return PRM_ERR_ALIGN;
  if (rows < 1 || cols < 1 || rows > 0x7fffffffLL || cols > 0x7fffffffLL || cols % 8 != 0) return PRM_ERR_SHAPE;
  if ((rows + kTallRows - 1) / kTallRows > 65535) return PRM_ERR_SHAPE;
  return PRM_OK;
}

}  // namespace

extern "C" size_t prm_tall_shard_scratch_bytes(int64_t rows_local, int64_t cols) {
  if (rows_local < 1 || cols < 1) return 0;
  return (size_t)((rows_local + kTallRows - 1) / kTallRows) * (size_t)cols * sizeof(float);
}

extern "C" int prm_tall_shard_stats(const void* grad_shard, float* momentum_shard, int64_t rows_local,
                                    int64_t cols, int io_fp32, float beta, int nesterov,
                                    float* colsumsq_out, float* scratch, size_t scratch_bytes,
                                    void* cuda_stream) {
  int rc = shard_check(grad_shard, momentum_shard, colsumsq_out, rows_local, cols);
  if (rc != PRM_OK) return rc;
  if (!scratch || ((uintptr_t)scratch & 15) != 0) return PRM_ERR_ARG;
  if (scratch_bytes < prm_tall_shard_scratch_bytes(rows_local, cols)) return PRM_ERR_WORKSPACE;
  const int rows = (int)rows_local, n = (int)cols;
  const int nblk = (rows + kTallRows - 1) / kTallRows;
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  dim3 grid((n + 255) / 256, nblk, 1);
  if (io_fp32)
    shard_pass1_kernel<float><<<grid, kShThreads, 0, stream>>>((const float*)grad_shard, momentum_shard, rows, n,
                                                               beta, 1.f - beta, nesterov ? 1 : 0, scratch);
  else
    shard_pass1_kernel<__nv_bfloat16><<<grid, kShThreads, 0, stream>>>((const __nv_bfloat16*)grad_shard,
                                                                       momentum_shard, rows, n, beta, 1.f - beta,
                                                                       nesterov ? 1 : 0, scratch);
  shard_colsum_kernel<<<(n + kShThreads - 1) / kShThreads, kShThreads, 0, stream>>>(scratch, colsumsq_out, nblk, n);
  return cudaGetLastError() == cudaSuccess ? PRM_OK : PRM_ERR_CUDA;
}

extern "C" int prm_tall_shard_apply(void* param_shard, const void* grad_shard, const float* momentum_shard,
                                    int64_t rows_local, int64_t cols, int io_fp32, float beta, int nesterov,
                                    float lr, float wd, float gamma, float eps_row, float scale,
                                    const float* colsumsq, void* cuda_stream) {
  int rc = shard_check(param_shard, grad_shard, momentum_shard, rows_local, cols);
  if (rc != PRM_OK) return rc;
  if (!colsumsq) return PRM_ERR_ARG;
  const int rows = (int)rows_local, n = (int)cols;
  const int nblk = (rows + kTallRows - 1) / kTallRows;
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  dim3 grid((n + 255) / 256, nblk, 1);
  const float decay = 1.f - lr * wd, k = lr * scale * gamma;
  if (io_fp32)
    shard_pass2_kernel<float><<<grid, kShThreads, 0, stream>>>((float*)param_shard, (const float*)grad_shard,
                                                               momentum_shard, rows, n, beta, 1.f - beta,
                                                               nesterov ? 1 : 0, decay, k, eps_row, colsumsq);
  else
    shard_pass2_kernel<__nv_bfloat16><<<grid, kShThreads, 0, stream>>>(
        (__nv_bfloat16*)param_shard, (const __nv_bfloat16*)grad_shard, momentum_shard, rows, n, beta, 1.f - beta,
        nesterov ? 1 : 0, decay, k, eps_row, colsumsq);
  return cudaGetLastError() == cudaSuccess ? PRM_OK : PRM_ERR_CUDA;
}

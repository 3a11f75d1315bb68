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
#include "tall_kernels.cuh"

namespace {

using namespace prm;


template <typename IO>
__global__ void __launch_bounds__(kTallThreads)
shard_pass1_kernel(const IO* __restrict__ g, float* __restrict__ m, int rows, int cols, float beta, float omb,
                   int nesterov, float* __restrict__ partial /*[row blocks][cols]*/) {
  const int row0 = blockIdx.y * kTallRows;
  tall_pass1_block<IO>(g, m, cols, row0, min(rows, row0 + kTallRows), blockIdx.x, beta, omb, nesterov,
                       partial + (int64_t)blockIdx.y * cols);
}

// Local column sums of squares: sum over this rank's row blocks, no root.
__global__ void __launch_bounds__(kTallThreads)
shard_colsum_kernel(const float* __restrict__ partial, float* __restrict__ colsumsq, int nblk, int cols) {
  const int col = blockIdx.x * kTallThreads + threadIdx.x;
  if (col >= cols) return;
  colsumsq[col] = tall_column_sum(partial, nblk, cols, col);
}

template <typename IO>
__global__ void __launch_bounds__(kTallThreads)
shard_pass2_kernel(IO* __restrict__ p, const IO* __restrict__ g, const float* __restrict__ m, int rows, int cols,
                   float beta, float omb, int nesterov, float decay, float lr_s_gamma, float eps,
                   const float* __restrict__ colsumsq /*[cols], summed over all ranks*/) {
  const int row0 = blockIdx.y * kTallRows;
  tall_pass2_block<IO>(p, g, m, cols, row0, min(rows, row0 + kTallRows), blockIdx.x, beta, omb, nesterov, decay,
                       [&](int col) { return lr_s_gamma / fmaxf(sqrtf(colsumsq[col]), eps); });   // sqrt, then clamp
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
    shard_pass1_kernel<float><<<grid, kTallThreads, 0, stream>>>((const float*)grad_shard, momentum_shard, rows, n,
                                                               beta, 1.f - beta, nesterov ? 1 : 0, scratch);
  else
    shard_pass1_kernel<__nv_bfloat16><<<grid, kTallThreads, 0, stream>>>((const __nv_bfloat16*)grad_shard,
                                                                       momentum_shard, rows, n, beta, 1.f - beta,
                                                                       nesterov ? 1 : 0, scratch);
  shard_colsum_kernel<<<(n + kTallThreads - 1) / kTallThreads, kTallThreads, 0, stream>>>(scratch, colsumsq_out, nblk, n);
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
    shard_pass2_kernel<float><<<grid, kTallThreads, 0, stream>>>((float*)param_shard, (const float*)grad_shard,
                                                               momentum_shard, rows, n, beta, 1.f - beta,
                                                               nesterov ? 1 : 0, decay, k, eps_row, colsumsq);
  else
    shard_pass2_kernel<__nv_bfloat16><<<grid, kTallThreads, 0, stream>>>(
        (__nv_bfloat16*)param_shard, (const __nv_bfloat16*)grad_shard, momentum_shard, rows, n, beta, 1.f - beta,
        nesterov ? 1 : 0, decay, k, eps_row, colsumsq);
  return cudaGetLastError() == cudaSuccess ? PRM_OK : PRM_ERR_CUDA;
}

// The two passes of the tall-matrix row step (RowNorm on stored columns, Eq.
// rownorm with the orientation of Section 3.1), as device functions shared by
// every kernel that runs them: the batched kernels behind prm_step, the
// allocation-free single-matrix entry point, and the row-sharded entry points
// of Algorithm 2 lines 9-13.  One CTA of kTallThreads threads handles a block
// of kTallRows rows x 256 columns; a lane owns 8 consecutive columns, the 8
// warps take interleaved rows and are combined in a fixed order.
#pragma once

#include "common.cuh"

namespace prm {

constexpr int kTallThreads = 256;

// Pass 1 on rows [row0, row1) and the 256 columns of column block `cblock`:
// momentum update in place and the block's column sums of squares of the
// direction input, written to partial_row[col] (one entry per column of the
// matrix; this row block's row of the partial-sum array).
template <typename IO>
__device__ __forceinline__ void tall_pass1_block(const IO* __restrict__ g, float* __restrict__ m, int cols,
                                                 int row0, int row1, int cblock, float beta, float omb,
                                                 int nesterov, float* __restrict__ partial_row) {
  __shared__ float red[kTallThreads / 32][32 * 8 + 1];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int col0 = (cblock * 32 + lane) * 8;
  float cs[8];
#pragma unroll
  for (int e = 0; e < 8; ++e) cs[e] = 0.f;
  if (col0 < cols) {
#pragma unroll 4
    for (int row = row0 + warp; row < row1; row += kTallThreads / 32) {
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
  const int col = cblock * 256 + threadIdx.x;
  if (col < cols) {
    float tot = 0.f;
#pragma unroll
    for (int w = 0; w < kTallThreads / 32; ++w) tot += red[w][threadIdx.x];
    partial_row[col] = tot;
  }
}

// Pass 2 on the same block: W <- decay*W - coef_j * U with coef_j = lr*s*gamma/nu_j
// taken from coef_of(col) for each of the lane's 8 columns.
template <typename IO, typename CoefFn>
__device__ __forceinline__ void tall_pass2_block(IO* __restrict__ p, const IO* __restrict__ g,
                                                 const float* __restrict__ m, int cols, int row0, int row1,
                                                 int cblock, float beta, float omb, int nesterov, float decay,
                                                 CoefFn coef_of) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int col0 = (cblock * 32 + lane) * 8;
  if (col0 >= cols) return;
  float coef[8];
#pragma unroll
  for (int e = 0; e < 8; ++e) coef[e] = coef_of(col0 + e);
#pragma unroll 4
  for (int row = row0 + warp; row < row1; row += kTallThreads / 32) {
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

// Sum of one column over nblk row blocks of partial sums, fixed order.
__device__ __forceinline__ float tall_column_sum(const float* __restrict__ partial, int nblk, int cols, int col) {
  float tot = 0.f;
  for (int b = 0; b < nblk; ++b) tot += partial[(int64_t)b * cols + col];
  return tot;
}

}  // namespace prm

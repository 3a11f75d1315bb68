// NS5 pre-pass: the refresh step's only read of gradients and momentum.
//
// For every matrix of a sub-batch it updates the momentum in place
// (Algorithm 1 line 2), forms the direction input U, and writes U - unscaled -
// into the NS5 workspace as the oriented matrix X (r x c) of Section 3.1: as
// stored for wide matrices, transposed through a shared-memory tile for tall
// ones.  The Frobenius norm of U is reduced alongside (per-CTA partials, then
// one fixed-order sum per matrix) and enters the recurrence as
// alpha = 1/(||U||_F + eps_ns) in the first iteration's epilogues, so the
// normalisation costs no extra pass.
//
// The workspace copies are zero-padded to multiples of kPad; zero rows and
// columns stay zero under X -> aX + (bA + cA^2)X.
#include "launch.cuh"

namespace prm {

constexpr int kPreTile = 64;
constexpr int kPreThreads = 256;

// Split input (lo_off != 0, bf16 workspace): X is written as two planes, H = bf16(U) at the
// usual place and L = bf16(U - H) lo_off elements further, so that H + L carries 16 mantissa
// bits of U into the two NS5 products that read X_0.
__device__ __forceinline__ float through_storage(float v, const __nv_bfloat16*) {
  return __bfloat162float(__float2bfloat16_rn(v));
}
__device__ __forceinline__ float through_storage(float v, const float*) { return v; }
template <typename XT_>
__device__ __forceinline__ void store8_planes(XT_* p, int64_t lo_off, const float (&u)[8]) {
  store8(p, u);
  if (lo_off) {
    float l[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) l[e] = u[e] - through_storage(u[e], p);
    store8(p + lo_off, l);
  }
}

template <typename IO, typename XT_, bool VEC>
__global__ void __launch_bounds__(kPreThreads)
ns_prepass_kernel(PtrTables t, int first, int rows, int cols, StepScalars s,
                  XT_* __restrict__ straight, int64_t ld_s, int64_t bs_s,
                  XT_* __restrict__ transposed, int64_t ld_t, int64_t bs_t, int64_t lo_off,
                  float* __restrict__ fro_partial) {
  __shared__ float tile[kPreTile][kPreTile + 1];
  __shared__ float warp_part[kPreThreads / 32];
  const int b = blockIdx.z;
  const IO* __restrict__ g = reinterpret_cast<const IO*>(t.grads[first + b]);
  float* __restrict__ m = t.momentum[first + b];
  XT_* __restrict__ ds = straight ? straight + (int64_t)b * bs_s : nullptr;
  XT_* __restrict__ dt = transposed ? transposed + (int64_t)b * bs_t : nullptr;
  const int r0 = blockIdx.y * kPreTile, c0 = blockIdx.x * kPreTile;
  const int tx = threadIdx.x & 7, ty = threadIdx.x >> 3;   // 8 column vectors x 32 rows
  float acc = 0.f;
#pragma unroll
  for (int half = 0; half < 2; ++half) {
    const int lr = ty + 32 * half;
    const int row = r0 + lr, col = c0 + tx * 8;
    float u[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) u[e] = 0.f;
    if (row < rows) {
      const int64_t off = (int64_t)row * cols + col;
      if (VEC) {
        if (col < cols) {
          float gv[8], mv[8];
          load8_stream(g + off, gv);
          load8_stream(m + off, mv);
#pragma unroll
          for (int e = 0; e < 8; ++e) {
            const float mn = blend(s.beta, mv[e], s.omb, gv[e]);
            mv[e] = mn;
            u[e] = s.nesterov ? blend(s.beta, mn, s.omb, gv[e]) : mn;
          }
          store8(m + off, mv);
        }
      } else {
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          if (col + e < cols) {
            const float gv = to_f32(g[off + e]);
            const float mn = blend(s.beta, m[off + e], s.omb, gv);
            m[off + e] = mn;
            u[e] = s.nesterov ? blend(s.beta, mn, s.omb, gv) : mn;
          }
        }
      }
    }
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      acc += u[e] * u[e];
      tile[lr][tx * 8 + e] = u[e];
    }
    if (straight != nullptr) store8_planes(ds + (int64_t)row * ld_s + col, lo_off, u);   // padded extent: always in range
  }
  acc = warp_sum(acc);
  if ((threadIdx.x & 31) == 0) warp_part[threadIdx.x >> 5] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    float tot = 0.f;
#pragma unroll
    for (int w = 0; w < kPreThreads / 32; ++w) tot += warp_part[w];
    fro_partial[((int64_t)b * gridDim.y + blockIdx.y) * gridDim.x + blockIdx.x] = tot;
  }
  if (transposed == nullptr) return;
#pragma unroll
  for (int half = 0; half < 2; ++half) {
    const int lc = ty + 32 * half;            // column of the tile = row of the transposed copy
    float u[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) u[e] = tile[tx * 8 + e][lc];
    store8_planes(dt + (int64_t)(c0 + lc) * ld_t + r0 + tx * 8, lo_off, u);
  }
}

// Wide matrices need no transposition, so no shared-memory tile: a CTA streams
// kWideRows rows x kWideCols columns, every thread holding one 8-element vector
// of each row, all loads issued before the first use (12 outstanding 16-byte
// loads per thread with bf16 gradients).  Rows and columns of the padded
// workspace extent that lie outside the matrix are written as zeros.
constexpr int kWideRows = 4;
constexpr int kWideCols = kPreThreads * 8;

template <typename IO, typename XT_>
__global__ void __launch_bounds__(kPreThreads)
ns_prepass_wide_kernel(PtrTables t, int first, int rows, int cols, StepScalars s,
                       XT_* __restrict__ X, int64_t ld_x, int64_t bs_x, int prow, int64_t lo_off,
                       float* __restrict__ fro_partial) {
  __shared__ float warp_part[kPreThreads / 32];
  const int b = blockIdx.z;
  const IO* __restrict__ g = reinterpret_cast<const IO*>(t.grads[first + b]);
  float* __restrict__ m = t.momentum[first + b];
  XT_* __restrict__ x = X + (int64_t)b * bs_x;
  const int col = blockIdx.x * kWideCols + threadIdx.x * 8;
  const int row0 = blockIdx.y * kWideRows;
  const bool col_in = col < cols;             // cols % 8 == 0: the whole vector is inside or outside
  float gv[kWideRows][8], mv[kWideRows][8];
#pragma unroll
  for (int k = 0; k < kWideRows; ++k) {
    if (col_in && row0 + k < rows) {
      const int64_t off = (int64_t)(row0 + k) * cols + col;
      load8_stream(g + off, gv[k]);
      load8_stream(m + off, mv[k]);
    }
  }
  float acc = 0.f;
#pragma unroll
  for (int k = 0; k < kWideRows; ++k) {
    const int row = row0 + k;
    float u[8];
    if (col_in && row < rows) {
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const float mn = blend(s.beta, mv[k][e], s.omb, gv[k][e]);
        mv[k][e] = mn;
        u[e] = s.nesterov ? blend(s.beta, mn, s.omb, gv[k][e]) : mn;
        acc += u[e] * u[e];
      }
      store8(m + (int64_t)row * cols + col, mv[k]);
    } else {
#pragma unroll
      for (int e = 0; e < 8; ++e) u[e] = 0.f;
    }
    if (col < ld_x && row < prow) store8_planes(x + (int64_t)row * ld_x + col, lo_off, u);
  }
  acc = warp_sum(acc);
  if ((threadIdx.x & 31) == 0) warp_part[threadIdx.x >> 5] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    float tot = 0.f;
#pragma unroll
    for (int w = 0; w < kPreThreads / 32; ++w) tot += warp_part[w];
    fro_partial[((int64_t)b * gridDim.y + blockIdx.y) * gridDim.x + blockIdx.x] = tot;
  }
}

// alpha[b] = 1/(sqrt(sum of partials) + eps_ns); one CTA per matrix, fixed
// summation order.
__global__ void __launch_bounds__(kPreThreads)
ns_alpha_kernel(const float* __restrict__ fro_partial, int nparts, float eps_ns,
                float* __restrict__ alpha) {
  __shared__ float part[kPreThreads];
  const float* src = fro_partial + (int64_t)blockIdx.x * nparts;
  float acc = 0.f;
  for (int i = threadIdx.x; i < nparts; i += kPreThreads) acc += src[i];
  part[threadIdx.x] = acc;
  __syncthreads();
  for (int w = kPreThreads / 2; w > 0; w >>= 1) {
    if (threadIdx.x < w) part[threadIdx.x] += part[threadIdx.x + w];
    __syncthreads();
  }
  if (threadIdx.x == 0) alpha[blockIdx.x] = 1.f / (sqrtf(part[0]) + eps_ns);
}

void launch_ns_alpha(const float* fro_partial, int nparts, float eps_ns, float* alpha, int batch,
                     cudaStream_t stream) {
  ns_alpha_kernel<<<batch, kPreThreads, 0, stream>>>(fro_partial, nparts, eps_ns, alpha);
}

template <typename IO, typename XT_>
static cudaError_t prepass_inst(const PtrTables& t, const Group& g, int first, int batch,
                                const StepScalars& s, XT_* X, int split, float* fro_partial, float* alpha,
                                cudaStream_t stream) {
  // Stored extent padded: wide -> (rp, cp), tall -> (cp, rp).
  const int64_t prow = g.tall ? g.cp : g.rp, pcol = g.tall ? g.rp : g.cp;
  XT_* straight = g.tall ? nullptr : X;
  XT_* transposed = g.tall ? X : nullptr;
  const int64_t lo_off = split ? g.rp * g.cp : 0;      // the L plane of a matrix follows its H plane
  const int64_t bs = (split ? 2 : 1) * g.rp * g.cp;
  const bool vec = (g.cols % 8 == 0);
  if (!g.tall && vec) {
    dim3 gw((unsigned)((pcol + kWideCols - 1) / kWideCols), (unsigned)(prow / kWideRows), (unsigned)batch);
    if (gw.y <= 65535 && gw.z <= 65535) {
      ns_prepass_wide_kernel<IO, XT_><<<gw, kPreThreads, 0, stream>>>(t, first, (int)g.rows, (int)g.cols, s, X, pcol, bs,
                                                                        (int)prow, lo_off, fro_partial);
      ns_alpha_kernel<<<batch, kPreThreads, 0, stream>>>(fro_partial, (int)(gw.x * gw.y), s.eps_ns, alpha);
      return cudaGetLastError();
    }
  }
  dim3 grid((unsigned)(pcol / kPreTile), (unsigned)(prow / kPreTile), (unsigned)batch);
  if (grid.y > 65535 || grid.z > 65535) return cudaErrorInvalidValue;
  if (vec)
    ns_prepass_kernel<IO, XT_, true><<<grid, kPreThreads, 0, stream>>>(
        t, first, (int)g.rows, (int)g.cols, s, straight, pcol, bs, transposed, prow, bs, lo_off, fro_partial);
  else
    ns_prepass_kernel<IO, XT_, false><<<grid, kPreThreads, 0, stream>>>(
        t, first, (int)g.rows, (int)g.cols, s, straight, pcol, bs, transposed, prow, bs, lo_off, fro_partial);
  ns_alpha_kernel<<<batch, kPreThreads, 0, stream>>>(fro_partial, (int)(grid.x * grid.y), s.eps_ns, alpha);
  return cudaGetLastError();
}

cudaError_t launch_ns_prepass(const PtrTables& t, const Group& g, int first, int batch,
                              const StepScalars& s, int io_fp32, int x_fp32, int split, void* X,
                              float* fro_partial, float* alpha, cudaStream_t stream,
                              int64_t* launches) {
  *launches += 2;
  if (split && x_fp32) return cudaErrorInvalidValue;
  if (io_fp32) {
    if (x_fp32) return prepass_inst<float, float>(t, g, first, batch, s, (float*)X, 0, fro_partial, alpha, stream);
    return prepass_inst<float, __nv_bfloat16>(t, g, first, batch, s, (__nv_bfloat16*)X, split, fro_partial, alpha, stream);
  }
  if (x_fp32) return prepass_inst<__nv_bfloat16, float>(t, g, first, batch, s, (float*)X, 0, fro_partial, alpha, stream);
  return prepass_inst<__nv_bfloat16, __nv_bfloat16>(t, g, first, batch, s, (__nv_bfloat16*)X, split, fro_partial, alpha, stream);
}

}  // namespace prm

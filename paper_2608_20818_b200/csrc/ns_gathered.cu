// Refresh branch over dim-0 row shards (paper, Section 3.3 "Distributed
// Execution"; Algorithm 2 lines 1-7): device work around the all-gather.
//
//   prm_shard_momentum_pack   every rank: momentum update of its row shard
//                             (Algorithm 1 line 2) and the direction input U
//                             written as bf16 into its segment of the bucket's
//                             send buffer
//   (all-gather by the caller: every rank then holds all segments, rank-major;
//    or no copy at all: the segments stay where they were written and are
//    read through peer-mapped pointers)
//   ns_gather_prepass_kernel  the full-matrix rebuild (line 5): reads the rows of a
//                             matrix from the segments they arrived in (or
//                             straight from the owning GPUs' memory) and
//                             writes the oriented, zero-padded NS5 input X with
//                             its Frobenius partial sums; the reconstruction is
//                             index arithmetic, no full matrix is assembled
//                             outside the NS5 workspace
//   (NS5 products as on one GPU)
//   ns_slice_update_kernel    each rank keeps its own rows of the result (also line 5):
//                             W_shard <- (1 - eta lambda) W_shard - eta s X_5
//                             on this rank's rows only
//
// A matrix of `rows` stored rows is split as torch.chunk does: rank q owns
// rows [q*chunk, min(rows, (q+1)*chunk)), chunk = ceil(rows / world).  Every
// rank's segment reserves chunk*cols elements for the matrix (rounded up to 8
// elements), so that all segments have the same size; unused rows are zero.
#include <algorithm>

#include "launch.cuh"

namespace prm {

namespace {

constexpr int kTile = 64;
constexpr int kThreads = 256;

template <typename IO>
__global__ void __launch_bounds__(kThreads)
shard_pack_kernel(const IO* __restrict__ g, float* __restrict__ m, int64_t n_local, int64_t n_reserved,
                  float beta, float omb, int nesterov, __nv_bfloat16* __restrict__ u_out) {
  // 8 elements per thread; n_local and n_reserved are multiples of 8 here.
  const int64_t stride = (int64_t)gridDim.x * blockDim.x * 8;
  for (int64_t i = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * 8; i < n_reserved; i += stride) {
    float u[8];
    if (i < n_local) {
      float gv[8], mv[8];
      load8_stream(g + i, gv);
      load8_stream(m + i, mv);
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const float mn = blend(beta, mv[e], omb, gv[e]);
        mv[e] = mn;
        u[e] = nesterov ? blend(beta, mn, omb, gv[e]) : mn;
      }
      store8(m + i, mv);
    } else {
#pragma unroll
      for (int e = 0; e < 8; ++e) u[e] = 0.f;
    }
    store8(u_out + i, u);
  }
}

template <typename IO>
__global__ void __launch_bounds__(kThreads)
shard_pack_scalar_kernel(const IO* __restrict__ g, float* __restrict__ m, int64_t n_local, int64_t n_reserved,
                         float beta, float omb, int nesterov, __nv_bfloat16* __restrict__ u_out) {
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_reserved; i += stride) {
    float u = 0.f;
    if (i < n_local) {
      const float gv = to_f32(g[i]);
      const float mn = blend(beta, m[i], omb, gv);
      m[i] = mn;
      u = nesterov ? blend(beta, mn, omb, gv) : mn;
    }
    u_out[i] = __float2bfloat16_rn(u);
  }
}

template <typename XT_, bool VEC>
__global__ void __launch_bounds__(kThreads)
ns_gather_prepass_kernel(SegmentPtrs segs, int chunk_rows, GatherBatch src, int rows, int cols,
                         XT_* __restrict__ straight, int64_t ld_s, int64_t bs_s,
                         XT_* __restrict__ transposed, int64_t ld_t, int64_t bs_t,
                         float* __restrict__ fro_partial) {
  __shared__ float tile[kTile][kTile + 1];
  __shared__ float warp_part[kThreads / 32];
  const int b = blockIdx.z;
  const int64_t off_b = src.off[b];
  XT_* __restrict__ ds = straight ? straight + (int64_t)b * bs_s : nullptr;
  XT_* __restrict__ dt = transposed ? transposed + (int64_t)b * bs_t : nullptr;
  const int r0 = blockIdx.y * kTile, c0 = blockIdx.x * kTile;
  const int tx = threadIdx.x & 7, ty = threadIdx.x >> 3;
  float acc = 0.f;
#pragma unroll
  for (int half = 0; half < 2; ++half) {
    const int lr = ty + 32 * half;
    const int row = r0 + lr, col = c0 + tx * 8;
    float u[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) u[e] = 0.f;
    if (row < rows) {
      const int q = row / chunk_rows;                       // rank that sent this row
      // plain loads: the segment may live in this GPU's memory or in a peer's
      const __nv_bfloat16* p = reinterpret_cast<const __nv_bfloat16*>(segs.seg[q]) + off_b +
                               (int64_t)(row - q * chunk_rows) * cols + col;
      if (VEC) {
        if (col < cols) load8_stream(p, u);
      } else {
#pragma unroll
        for (int e = 0; e < 8; ++e)
          if (col + e < cols) u[e] = __bfloat162float(p[e]);
      }
    }
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      acc += u[e] * u[e];
      tile[lr][tx * 8 + e] = u[e];
    }
    if (straight != nullptr) store8(ds + (int64_t)row * ld_s + col, u);
  }
  acc = warp_sum(acc);
  if ((threadIdx.x & 31) == 0) warp_part[threadIdx.x >> 5] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    float tot = 0.f;
#pragma unroll
    for (int w = 0; w < kThreads / 32; ++w) tot += warp_part[w];
    fro_partial[((int64_t)b * gridDim.y + blockIdx.y) * gridDim.x + blockIdx.x] = tot;
  }
  if (transposed == nullptr) return;
#pragma unroll
  for (int half = 0; half < 2; ++half) {
    const int lc = ty + 32 * half;
    float u[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) u[e] = tile[tx * 8 + e][lc];
    store8(dt + (int64_t)(c0 + lc) * ld_t + r0 + tx * 8, u);
  }
}

// One 64x64 tile of this rank's rows of one matrix.  x5 is the oriented NS5
// result (r_p x c_p): element (row, col) of a wide matrix, (col, row) of a
// tall one.  VEC: 8-element accesses (cols % 8 == 0 and, for tall matrices,
// row_start % 8 == 0); otherwise element-wise.
template <typename IO, typename XT_, bool VEC>
__global__ void __launch_bounds__(kThreads)
ns_slice_update_kernel(SliceBatch dst, const XT_* __restrict__ x5, int64_t ld_x, int64_t bs_x, int tall,
                       int row_start, int rows_local, int cols, float decay, float lr_s) {
  __shared__ float tile[kTile][kTile + 1];
  const int b = blockIdx.z;
  IO* __restrict__ w = reinterpret_cast<IO*>(dst.param[b]);
  const XT_* __restrict__ x = x5 + (int64_t)b * bs_x;
  const int r0 = blockIdx.y * kTile, c0 = blockIdx.x * kTile;   // shard-local row, column
  const int tx = threadIdx.x & 7, ty = threadIdx.x >> 3;
  if (tall) {
    // x tile: rows = columns c0.., columns = stored rows row_start + r0..
#pragma unroll
    for (int half = 0; half < 2; ++half) {
      const int xc = c0 + ty + 32 * half;            // oriented row = stored column
      const int xr = row_start + r0 + tx * 8;        // oriented column = stored row
      float u[8];
      if (VEC) {
        // row_start % 8 == 0: a group of 8 that starts below rows_local ends inside the padded row
        if (r0 + tx * 8 < rows_local) load8(x + (int64_t)xc * ld_x + xr, u);
        else {
#pragma unroll
          for (int e = 0; e < 8; ++e) u[e] = 0.f;
        }
      } else {
#pragma unroll
        for (int e = 0; e < 8; ++e) u[e] = (r0 + tx * 8 + e < rows_local) ? to_f32(x[(int64_t)xc * ld_x + xr + e]) : 0.f;
      }
#pragma unroll
      for (int e = 0; e < 8; ++e) tile[tx * 8 + e][ty + 32 * half] = u[e];   // tile[stored row][stored col]
    }
    __syncthreads();
  }
#pragma unroll
  for (int half = 0; half < 2; ++half) {
    const int lr = ty + 32 * half;
    const int row = r0 + lr, col = c0 + tx * 8;
    if (row >= rows_local || col >= cols) continue;
    float d[8];
    if (tall) {
#pragma unroll
      for (int e = 0; e < 8; ++e) d[e] = tile[lr][tx * 8 + e];
    } else if (VEC) {
      load8(x + (int64_t)(row_start + row) * ld_x + col, d);
    } else {
#pragma unroll
      for (int e = 0; e < 8; ++e) d[e] = to_f32(x[(int64_t)(row_start + row) * ld_x + col + e]);   // padded extent
    }
    IO* p = w + (int64_t)row * cols + col;
    if (VEC) {
      float wv[8];
      load8(p, wv);
#pragma unroll
      for (int e = 0; e < 8; ++e) wv[e] = decay * wv[e] - lr_s * d[e];
      store8(p, wv);
    } else {
#pragma unroll
      for (int e = 0; e < 8; ++e)
        if (col + e < cols) from_f32(p + e, decay * to_f32(p[e]) - lr_s * d[e]);
    }
  }
}

template <typename XT_>
cudaError_t gather_prepass_inst(const SegmentPtrs& segs, bool vec_ok, int64_t chunk_rows,
                                const int64_t* offs, const Group& g, int batch, float eps_ns, XT_* X,
                                float* fro_partial, float* alpha, cudaStream_t stream, int64_t* launches) {
  const int64_t prow = g.tall ? g.cp : g.rp, pcol = g.tall ? g.rp : g.cp;
  const int64_t bs = g.rp * g.cp;
  const unsigned gx = (unsigned)(pcol / kTile), gy = (unsigned)(prow / kTile);
  if (gy > 65535) return cudaErrorInvalidValue;
  const bool vec = (g.cols % 8 == 0) && vec_ok;
  for (int done = 0; done < batch; done += kGatherMax) {
    const int nb = std::min(kGatherMax, batch - done);
    GatherBatch src;
    for (int k = 0; k < nb; ++k) {
      src.off[k] = offs[done + k];
      if (vec && (src.off[k] % 8) != 0) return cudaErrorInvalidValue;
    }
    XT_* Xb = X + (int64_t)done * bs;
    XT_* straight = g.tall ? nullptr : Xb;
    XT_* transposed = g.tall ? Xb : nullptr;
    float* fp = fro_partial + (int64_t)done * gx * gy;
    dim3 grid(gx, gy, (unsigned)nb);
    if (vec)
      ns_gather_prepass_kernel<XT_, true><<<grid, kThreads, 0, stream>>>(
          segs, (int)chunk_rows, src, (int)g.rows, (int)g.cols, straight, pcol, bs, transposed, prow, bs, fp);
    else
      ns_gather_prepass_kernel<XT_, false><<<grid, kThreads, 0, stream>>>(
          segs, (int)chunk_rows, src, (int)g.rows, (int)g.cols, straight, pcol, bs, transposed, prow, bs, fp);
    *launches += 1;
  }
  launch_ns_alpha(fro_partial, (int)(gx * gy), eps_ns, alpha, batch, stream);
  *launches += 1;
  return cudaGetLastError();
}

template <typename IO, typename XT_>
cudaError_t slice_update_inst(const XT_* X5, const Group& g, int batch, void* const* param_shards,
                              int64_t row_start, int64_t rows_local, float decay, float lr_s,
                              cudaStream_t stream, int64_t* launches) {
  if (rows_local <= 0) return cudaSuccess;            // this rank owns no row of these matrices
  const int64_t bs = g.rp * g.cp;
  const unsigned gx = (unsigned)((g.cols + kTile - 1) / kTile), gy = (unsigned)((rows_local + kTile - 1) / kTile);
  if (gy > 65535) return cudaErrorInvalidValue;
  bool vec = (g.cols % 8 == 0) && (!g.tall || row_start % 8 == 0);
  for (int k = 0; k < batch && vec; ++k) vec = ((uintptr_t)param_shards[k] & 15) == 0;
  for (int done = 0; done < batch; done += kGatherMax) {
    const int nb = std::min(kGatherMax, batch - done);
    SliceBatch dst;
    for (int k = 0; k < nb; ++k) dst.param[k] = param_shards[done + k];
    dim3 grid(gx, gy, (unsigned)nb);
    const XT_* xb = X5 + (int64_t)done * bs;
    if (vec)
      ns_slice_update_kernel<IO, XT_, true><<<grid, kThreads, 0, stream>>>(
          dst, xb, g.cp, bs, g.tall ? 1 : 0, (int)row_start, (int)rows_local, (int)g.cols, decay, lr_s);
    else
      ns_slice_update_kernel<IO, XT_, false><<<grid, kThreads, 0, stream>>>(
          dst, xb, g.cp, bs, g.tall ? 1 : 0, (int)row_start, (int)rows_local, (int)g.cols, decay, lr_s);
    *launches += 1;
  }
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_ns_gather_prepass(const SegmentPtrs& segs, bool vec_ok, int64_t chunk_rows,
                                     const int64_t* offs, const Group& g, int batch, float eps_ns, int x_fp32,
                                     void* X, float* fro_partial, float* alpha, cudaStream_t stream,
                                     int64_t* launches) {
  if (x_fp32)
    return gather_prepass_inst<float>(segs, vec_ok, chunk_rows, offs, g, batch, eps_ns, (float*)X, fro_partial, alpha,
                                      stream, launches);
  return gather_prepass_inst<__nv_bfloat16>(segs, vec_ok, chunk_rows, offs, g, batch, eps_ns, (__nv_bfloat16*)X,
                                            fro_partial, alpha, stream, launches);
}

cudaError_t launch_ns_slice_update(const void* X5, int x_fp32, const Group& g, int batch,
                                   void* const* param_shards, int64_t row_start, int64_t rows_local, int io_fp32,
                                   float decay, float lr_s, cudaStream_t stream, int64_t* launches) {
  if (io_fp32) {
    if (x_fp32)
      return slice_update_inst<float, float>((const float*)X5, g, batch, param_shards, row_start, rows_local, decay,
                                             lr_s, stream, launches);
    return slice_update_inst<float, __nv_bfloat16>((const __nv_bfloat16*)X5, g, batch, param_shards, row_start,
                                                   rows_local, decay, lr_s, stream, launches);
  }
  if (x_fp32)
    return slice_update_inst<__nv_bfloat16, float>((const float*)X5, g, batch, param_shards, row_start, rows_local,
                                                   decay, lr_s, stream, launches);
  return slice_update_inst<__nv_bfloat16, __nv_bfloat16>((const __nv_bfloat16*)X5, g, batch, param_shards, row_start,
                                                         rows_local, decay, lr_s, stream, launches);
}

}  // namespace prm

using namespace prm;

extern "C" int prm_shard_momentum_pack(const void* grad_shard, float* momentum_shard, int64_t rows_local,
                                       int64_t cols, int64_t reserved_elems, int io_fp32, float beta, int nesterov,
                                       void* u_out, void* cuda_stream) {
  if (rows_local < 0 || cols < 1 || reserved_elems < rows_local * cols) return PRM_ERR_SHAPE;
  if (!u_out || ((uintptr_t)u_out & 15) != 0) return u_out ? PRM_ERR_ALIGN : PRM_ERR_ARG;
  if (reserved_elems == 0) return PRM_OK;
  const int64_t n_local = rows_local * cols;
  if (n_local > 0) {
    if (!grad_shard || !momentum_shard) return PRM_ERR_ARG;
    if ((((uintptr_t)grad_shard | (uintptr_t)momentum_shard) & 15) != 0) return PRM_ERR_ALIGN;
  }
  if (!(beta >= 0.f && beta < 1.f)) return PRM_ERR_ARG;
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  const bool vec = (n_local % 8 == 0) && (reserved_elems % 8 == 0);
  const int64_t work = vec ? reserved_elems / 8 : reserved_elems;
  const int blocks = (int)std::min<int64_t>((work + kThreads - 1) / kThreads, 148 * 16);
  __nv_bfloat16* out = (__nv_bfloat16*)u_out;
  const float omb = 1.f - beta;
  const int nes = nesterov ? 1 : 0;
  if (io_fp32) {
    if (vec) shard_pack_kernel<float><<<blocks, kThreads, 0, stream>>>((const float*)grad_shard, momentum_shard, n_local, reserved_elems, beta, omb, nes, out);
    else shard_pack_scalar_kernel<float><<<blocks, kThreads, 0, stream>>>((const float*)grad_shard, momentum_shard, n_local, reserved_elems, beta, omb, nes, out);
  } else {
    if (vec) shard_pack_kernel<__nv_bfloat16><<<blocks, kThreads, 0, stream>>>((const __nv_bfloat16*)grad_shard, momentum_shard, n_local, reserved_elems, beta, omb, nes, out);
    else shard_pack_scalar_kernel<__nv_bfloat16><<<blocks, kThreads, 0, stream>>>((const __nv_bfloat16*)grad_shard, momentum_shard, n_local, reserved_elems, beta, omb, nes, out);
  }
  return cudaGetLastError() == cudaSuccess ? PRM_OK : PRM_ERR_CUDA;
}

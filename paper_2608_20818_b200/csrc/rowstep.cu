// Row-step kernels: the rho_t = 0 branch of the paper's Algorithm 1 in one
// fused pass (wide matrices) or two passes plus a tiny column-norm kernel
// (tall matrices, where the oriented rows are stored columns).
//
//   M_t = beta*M_{t-1} + (1-beta)*G_t                      (Algorithm 1 line 2)
//   U   = M_t  or  beta*M_t + (1-beta)*G_t (Nesterov)
//   nu_i = max(sqrt(sum_j U~_ij^2), eps)                   (Eq. rownorm)
//   W   = (1 - lr*wd)*W - lr*s*gamma * U~_i / nu_i          (Eq. periodic-direction)
//
// All arithmetic is fp32; reductions have a fixed order (no atomics), so the
// result is bit-reproducible from run to run.
#include <cooperative_groups.h>

#include "launch.cuh"
#include "tall_kernels.cuh"

namespace cg = cooperative_groups;

namespace prm {

constexpr int kRowThreads = kTallThreads;

// ------------------------------------------------------------------ wide
// One row per CTA of THREADS threads (or per cluster of CLUSTER CTAs for very
// long rows); each thread keeps VPT vectors of 8 elements of U in registers
// between the reduction and the update, so every byte crosses HBM once:
// 14 B/element with bf16 I/O.  PREP loads the parameters before the
// reduction (more registers, fewer resident CTAs); MINB is the number of CTAs
// per SM the register allocation must allow.
template <typename IO, int VPT, int CLUSTER, int THREADS, bool PREP = true, int MINB = 1>
__global__ void __launch_bounds__(THREADS, MINB)
rowstep_wide_kernel(PtrTables t, int first, int rows, int cols, StepScalars s) {
  __shared__ float warp_part[THREADS / 32];
  __shared__ float cta_part;

  const int rank = CLUSTER > 1 ? (int)cg::this_cluster().block_rank() : 0;
  const int64_t row_global = blockIdx.x / CLUSTER;
  const int mat = (int)(row_global / rows);
  const int row = (int)(row_global % rows);
  const int64_t off = (int64_t)row * cols;
  const IO* __restrict__ g = reinterpret_cast<const IO*>(t.grads[first + mat]) + off;
  float* __restrict__ m = t.momentum[first + mat] + off;
  IO* __restrict__ p = reinterpret_cast<IO*>(t.params[first + mat]) + off;

  const int nvec = cols >> 3;
  const int part = (nvec + CLUSTER - 1) / CLUSTER;
  const int v_begin = rank * part;
  const int v_end = min(nvec, v_begin + part);

  float u[VPT][8];
  Raw8<IO> pv[VPT];
  float acc = 0.f;
#pragma unroll
  for (int k = 0; k < VPT; ++k) {
    const int v = v_begin + threadIdx.x + k * (int)blockDim.x;
    if (v < v_end) {
      float gv[8], mv[8];
      load8_stream(g + 8 * v, gv);
      load8_stream(m + 8 * v, mv);
      if (PREP) pv[k].load_stream(p + 8 * v);
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const float mn = blend(s.beta, mv[e], s.omb, gv[e]);
        mv[e] = mn;
        const float uu = s.nesterov ? blend(s.beta, mn, s.omb, gv[e]) : mn;
        u[k][e] = uu;
        acc += uu * uu;
      }
      store8(m + 8 * v, mv);
    }
  }
  acc = warp_sum(acc);
  if ((threadIdx.x & 31) == 0) warp_part[threadIdx.x >> 5] = acc;
  __syncthreads();
  float total = 0.f;
#pragma unroll
  for (int w = 0; w < THREADS / 32; ++w) total += (w < (int)(blockDim.x >> 5)) ? warp_part[w] : 0.f;
  if constexpr (CLUSTER > 1) {
    cg::cluster_group cluster = cg::this_cluster();
    if (threadIdx.x == 0) cta_part = total;
    cluster.sync();
    total = 0.f;
#pragma unroll
    for (int r = 0; r < CLUSTER; ++r) total += *cluster.map_shared_rank(&cta_part, r);
    cluster.sync();   // peers may not exit while their shared memory is read
  }
  const float nu = fmaxf(sqrtf(total), s.eps_row);
  const float coef = s.lr_s * s.gamma / nu;
  if (!PREP) {
#pragma unroll
    for (int k = 0; k < VPT; ++k) {
      const int v = v_begin + threadIdx.x + k * (int)blockDim.x;
      if (v < v_end) pv[k].load_stream(p + 8 * v);
    }
  }
#pragma unroll
  for (int k = 0; k < VPT; ++k) {
    const int v = v_begin + threadIdx.x + k * (int)blockDim.x;
    if (v < v_end) {
      float pf[8];
      pv[k].get(pf);
#pragma unroll
      for (int e = 0; e < 8; ++e) pf[e] = s.decay * pf[e] - coef * u[k][e];
      store8(p + 8 * v, pf);
    }
  }
}

// Any row length, any alignment: one CTA per row, two sweeps.  The first sweep
// only reduces; the second recomputes the blend from the untouched inputs.
template <typename IO>
__global__ void __launch_bounds__(kRowThreads)
rowstep_wide_generic_kernel(PtrTables t, int first, int rows, int cols, StepScalars s) {
  __shared__ float warp_part[kRowThreads / 32];
  const int mat = blockIdx.x / rows;
  const int row = blockIdx.x % rows;
  const int64_t off = (int64_t)row * cols;
  const IO* __restrict__ g = reinterpret_cast<const IO*>(t.grads[first + mat]) + off;
  float* __restrict__ m = t.momentum[first + mat] + off;
  IO* __restrict__ p = reinterpret_cast<IO*>(t.params[first + mat]) + off;
  float acc = 0.f;
  for (int j = threadIdx.x; j < cols; j += kRowThreads) {
    const float gv = to_f32(g[j]);
    const float mn = blend(s.beta, m[j], s.omb, gv);
    const float uu = s.nesterov ? blend(s.beta, mn, s.omb, gv) : mn;
    acc += uu * uu;
  }
  acc = warp_sum(acc);
  if ((threadIdx.x & 31) == 0) warp_part[threadIdx.x >> 5] = acc;
  __syncthreads();
  float total = 0.f;
#pragma unroll
  for (int w = 0; w < kRowThreads / 32; ++w) total += warp_part[w];
  const float nu = fmaxf(sqrtf(total), s.eps_row);
  const float coef = s.lr_s * s.gamma / nu;
  for (int j = threadIdx.x; j < cols; j += kRowThreads) {
    const float gv = to_f32(g[j]);
    const float mn = blend(s.beta, m[j], s.omb, gv);
    const float uu = s.nesterov ? blend(s.beta, mn, s.omb, gv) : mn;
    m[j] = mn;
    from_f32(p + j, s.decay * to_f32(p[j]) - coef * uu);
  }
}

// ------------------------------------------------------------------ tall
// Pass 1: momentum update and per-column partial sums of squares over a block
// of kTallRows rows.  Matrices whose column count is a multiple of 8 run the
// shared vector bodies (tall_kernels.cuh); the rest a scalar version with one
// column per lane.
template <typename IO, int V>
__global__ void __launch_bounds__(kRowThreads)
rowstep_tall_pass1_kernel(PtrTables t, int first, int rows, int cols, StepScalars s,
                          float* __restrict__ partial /*[count][row blocks][cols]*/) {
  const int mat = blockIdx.z;
  const int row0 = blockIdx.y * kTallRows;
  const int row1 = min(rows, row0 + kTallRows);
  const IO* __restrict__ g = reinterpret_cast<const IO*>(t.grads[first + mat]);
  float* __restrict__ m = t.momentum[first + mat];
  float* prow = partial + ((int64_t)mat * gridDim.y + blockIdx.y) * cols;
  if constexpr (V == 8) {
    tall_pass1_block<IO>(g, m, cols, row0, row1, blockIdx.x, s.beta, s.omb, s.nesterov, prow);
  } else {
    __shared__ float red[kRowThreads / 32][33];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int col = blockIdx.x * 32 + lane;
    float cs = 0.f;
    if (col < cols) {
      for (int row = row0 + warp; row < row1; row += kRowThreads / 32) {
        const int64_t off = (int64_t)row * cols + col;
        const float gv = to_f32(g[off]);
        const float mn = blend(s.beta, m[off], s.omb, gv);
        m[off] = mn;
        const float uu = s.nesterov ? blend(s.beta, mn, s.omb, gv) : mn;
        cs += uu * uu;
      }
    }
    red[warp][lane] = cs;
    __syncthreads();
    if (threadIdx.x < 32 && col < cols) {
      float tot = 0.f;
#pragma unroll
      for (int w = 0; w < kRowThreads / 32; ++w) tot += red[w][threadIdx.x];
      prow[col] = tot;
    }
  }
}

// Column norms: nu_j = max(sqrt(sum over row blocks), eps), fixed order.
__global__ void __launch_bounds__(kRowThreads)
rowstep_tall_colnorm_kernel(const float* __restrict__ partial, float* __restrict__ nu,
                            int nblk, int cols, float eps) {
  const int mat = blockIdx.y;
  const int col = blockIdx.x * kRowThreads + threadIdx.x;
  if (col >= cols) return;
  nu[(int64_t)mat * cols + col] = fmaxf(sqrtf(tall_column_sum(partial + (int64_t)mat * nblk * cols, nblk, cols, col)), eps);
}

// Pass 2: scale by the column norms and update the parameters.
template <typename IO, int V>
__global__ void __launch_bounds__(kRowThreads)
rowstep_tall_pass2_kernel(PtrTables t, int first, int rows, int cols, StepScalars s,
                          const float* __restrict__ nu /*[count][cols]*/) {
  const int mat = blockIdx.z;
  const int row0 = blockIdx.y * kTallRows;
  const int row1 = min(rows, row0 + kTallRows);
  const IO* __restrict__ g = reinterpret_cast<const IO*>(t.grads[first + mat]);
  const float* __restrict__ m = t.momentum[first + mat];
  IO* __restrict__ p = reinterpret_cast<IO*>(t.params[first + mat]);
  const float* nu_m = nu + (int64_t)mat * cols;
  const float k = s.lr_s * s.gamma;
  if constexpr (V == 8) {
    tall_pass2_block<IO>(p, g, m, cols, row0, row1, blockIdx.x, s.beta, s.omb, s.nesterov, s.decay,
                         [&](int col) { return k / nu_m[col]; });
  } else {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int col = blockIdx.x * 32 + lane;
    if (col >= cols) return;
    const float coef = k / nu_m[col];
    for (int row = row0 + warp; row < row1; row += kRowThreads / 32) {
      const int64_t off = (int64_t)row * cols + col;
      float uu = m[off];
      if (s.nesterov) uu = blend(s.beta, uu, s.omb, to_f32(g[off]));
      from_f32(p + off, s.decay * to_f32(p[off]) - coef * uu);
    }
  }
}

// --------------------------------------------------------------- launchers
template <typename IO, int VPT, int CLUSTER, int THREADS = kRowThreads, bool PREP = true, int MINB = 1>
static cudaError_t launch_wide_inst(const PtrTables& t, const Group& g, const StepScalars& s,
                                    cudaStream_t stream) {
  const int64_t nrows = (int64_t)g.count * g.rows;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(nrows * CLUSTER), 1, 1);
  // Only as many threads as the row needs (whole warps): idle threads would
  // hold registers and lower the number of resident CTAs.
  const int part = (int)(((g.cols >> 3) + CLUSTER - 1) / CLUSTER);
  const int vpt = (part + THREADS - 1) / THREADS;          // vectors per thread actually used (<= VPT)
  const int need = ((part + vpt - 1) / vpt + 31) / 32 * 32;
  cfg.blockDim = dim3(need < THREADS ? need : THREADS, 1, 1);
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = CLUSTER;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, rowstep_wide_kernel<IO, VPT, CLUSTER, THREADS, PREP, MINB>, t, g.first, (int)g.rows,
                            (int)g.cols, s);
}

template <typename IO>
static cudaError_t launch_wide(const PtrTables& t, const Group& g, const StepScalars& s,
                               cudaStream_t stream, int64_t* launches) {
  const int64_t nrows = (int64_t)g.count * g.rows;
  *launches += 1;
  const int64_t cols = g.cols;
  if (cols % 8 != 0 || cols > 65536 || nrows * 8 > 0x7fffffffLL) {
    if (nrows > 0x7fffffffLL) return cudaErrorInvalidValue;
    rowstep_wide_generic_kernel<IO><<<(unsigned)nrows, kRowThreads, 0, stream>>>(
        t, g.first, (int)g.rows, (int)g.cols, s);
    return cudaGetLastError();
  }
  // Rows up to 32768 elements stay inside one CTA (wider CTAs for longer
  // rows): measured faster than splitting a row over a cluster, whose two
  // cluster barriers cost more than the lower occupancy.
  // Rows up to 32768 elements stay inside one CTA; the template arguments are
  // <IO, vectors per thread, cluster, threads, prefetch W, min CTAs per SM>.
  // Measured on B200: two or more resident CTAs per SM matter more than
  // prefetching the parameters before the reduction, and a row split over a
  // cluster pays two cluster barriers.
  if (cols <= 2048) return launch_wide_inst<IO, 1, 1, 256, false, 4>(t, g, s, stream);
  if (cols <= 4096) return launch_wide_inst<IO, 2, 1, 256, false, 4>(t, g, s, stream);
  if (cols <= 8192) return launch_wide_inst<IO, 2, 1, 512, false, 2>(t, g, s, stream);
  if (cols <= 16384) return launch_wide_inst<IO, 4, 1, 512, false, 2>(t, g, s, stream);
  if (cols <= 24576) return launch_wide_inst<IO, 3, 1, 1024, false, 1>(t, g, s, stream);
  if (cols <= 32768) return launch_wide_inst<IO, 4, 1, 1024, false, 1>(t, g, s, stream);
  return launch_wide_inst<IO, 4, 8>(t, g, s, stream);
}

template <typename IO>
static cudaError_t launch_tall(const PtrTables& t, const Group& g, const StepScalars& s,
                               float* partial, float* nu, cudaStream_t stream, int64_t* launches) {
  const int rows = (int)g.rows, cols = (int)g.cols;
  const int nblk = (rows + kTallRows - 1) / kTallRows;
  const bool vec = (cols % 8 == 0);
  const int cpb = vec ? kTallCols : 32;
  dim3 grid((cols + cpb - 1) / cpb, nblk, g.count);
  if (grid.y > 65535 || grid.z > 65535) return cudaErrorInvalidValue;
  *launches += 3;
  if (vec)
    rowstep_tall_pass1_kernel<IO, 8><<<grid, kRowThreads, 0, stream>>>(t, g.first, rows, cols, s, partial);
  else
    rowstep_tall_pass1_kernel<IO, 1><<<grid, kRowThreads, 0, stream>>>(t, g.first, rows, cols, s, partial);
  dim3 grid_n((cols + kRowThreads - 1) / kRowThreads, g.count, 1);
  rowstep_tall_colnorm_kernel<<<grid_n, kRowThreads, 0, stream>>>(partial, nu, nblk, cols, s.eps_row);
  if (vec)
    rowstep_tall_pass2_kernel<IO, 8><<<grid, kRowThreads, 0, stream>>>(t, g.first, rows, cols, s, nu);
  else
    rowstep_tall_pass2_kernel<IO, 1><<<grid, kRowThreads, 0, stream>>>(t, g.first, rows, cols, s, nu);
  return cudaGetLastError();
}

cudaError_t launch_rowstep(const PtrTables& t, const Group& g, const StepScalars& s, int io_fp32,
                           float* tall_partial, float* tall_nu, cudaStream_t stream,
                           int64_t* launches) {
  if (!g.tall) {
    return io_fp32 ? launch_wide<float>(t, g, s, stream, launches)
                   : launch_wide<__nv_bfloat16>(t, g, s, stream, launches);
  }
  return io_fp32 ? launch_tall<float>(t, g, s, tall_partial, tall_nu, stream, launches)
                 : launch_tall<__nv_bfloat16>(t, g, s, tall_partial, tall_nu, stream, launches);
}

}  // namespace prm

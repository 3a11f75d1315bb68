// Row step of wide matrices (rows <= cols) as a persistent, bulk-copy-fed kernel:
// bf16 parameters and gradients, fp32 momentum, cols % 8 == 0, up to 24576 columns.
//
// Same arithmetic as rowstep_wide_kernel (Algorithm 1 line 2, Eq. rownorm,
// Eq. periodic-direction) and the same 14 bytes per element.  What differs is
// who waits for memory: one CTA per SM walks over the rows of the group (row
// cta, cta + #CTAs, ...); a producer warp fetches each row with bulk
// asynchronous copies - gradient and momentum in chunks of 4096 elements
// through a ring, the parameter row whole into one of two buffers - and runs
// ahead of the 16 consumer warps, so the loads of the next rows are in flight
// while a row is being reduced and updated.  A consumer thread keeps the
// direction input of its elements in registers between the reduction and the
// update, as in the one-row-per-CTA kernel.  Reductions have a fixed order.
// Every mbarrier wait is bounded: on expiry the CTA raises the status word,
// stops taking rows, drains the copies in flight and returns.
#include "async_copy.cuh"
#include "launch.cuh"

namespace prm {

namespace {

constexpr int kConsWarps = 16;
constexpr int kConsThreads = 32 * kConsWarps;
constexpr int kThreads = kConsThreads + 32;          // warp 0 produces
constexpr int kChunkElems = kConsThreads * 8;        // 4096 elements: eight per consumer thread
constexpr int kStages = 4;                           // ring of gradient/momentum chunks
constexpr uint32_t kGBytes = kChunkElems * 2, kMBytes = kChunkElems * 4;
constexpr int kMaxVpt = 6;                           // rows of up to 24576 elements

__device__ __forceinline__ void bulk_load(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}
__device__ __forceinline__ void cons_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kConsThreads) : "memory"); }
__device__ __forceinline__ float2 bf16x2_f32(uint32_t w) {
  return make_float2(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u));
}
__device__ __forceinline__ uint32_t pack2(float a, float b) {
  __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&h);
}

struct WideArgs {
  PtrTables t;
  int first, rows, cols;
  int64_t total_rows;      // rows of all matrices of the group
  StepScalars s;
  int* status;
};

// Shared memory: [kStages][gradient chunk | momentum chunk], two parameter rows of VPT chunks, barriers.
template <int VPT>
constexpr size_t wide_smem_bytes() {
  return 1024 + (size_t)kStages * (kGBytes + kMBytes) + 2 * (size_t)VPT * kGBytes + 256;
}

template <int VPT, bool NESTEROV>
__global__ void __launch_bounds__(kThreads, 1) rowstep_wide_stream_kernel(const WideArgs a) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  uint8_t* gm = smem;                                              // [kStages][kGBytes + kMBytes]
  uint8_t* pb = gm + (size_t)kStages * (kGBytes + kMBytes);        // [2][VPT * kGBytes]
  uint64_t* bars = reinterpret_cast<uint64_t*>(pb + 2 * (size_t)VPT * kGBytes);
  uint64_t* full = bars;                 // [kStages]
  uint64_t* empty = full + kStages;      // [kStages]
  uint64_t* pfull = empty + kStages;     // [2]
  uint64_t* pempty = pfull + 2;          // [2]
  float* warp_part = reinterpret_cast<float*>(pempty + 2);         // [2][kConsWarps]
  volatile int* flags = reinterpret_cast<volatile int*>(warp_part + 2 * kConsWarps);
  volatile int* abort_flag = flags;      // set by whoever ran out of time
  volatile int* s_go = flags + 1;        // [2] consumers: carry on after this row (by row parity, one writer)

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int cols = a.cols;
  const uint32_t row_g = (uint32_t)cols * 2;

  if (threadIdx.x == 0) {
    for (int k = 0; k < kStages; ++k) { mbar_init(&full[k], 1); mbar_init(&empty[k], kConsWarps); }
    for (int k = 0; k < 2; ++k) { mbar_init(&pfull[k], 1); mbar_init(&pempty[k], kConsWarps); }
    flags[0] = 0; flags[1] = 1; flags[2] = 1;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncthreads();

  if (warp == 0) {
    // ------------------------------------------------------------ producer
    if (lane == 0) {
      uint32_t it = 0, nrow = 0;
      int issued_gm = 0, issued_p = 0;
      bool ok = true;
      int cur = -1;                          // the matrices' base pointers sit in global memory: fetched once per matrix
      const uint8_t *gb = nullptr, *mb = nullptr, *pbase = nullptr;
      for (int64_t rg = blockIdx.x; rg < a.total_rows && ok; rg += gridDim.x, ++nrow) {
        const int mat = (int)(rg / a.rows);
        const int64_t off = (rg - (int64_t)mat * a.rows) * cols;
        if (mat != cur) {
          gb = reinterpret_cast<const uint8_t*>(a.t.grads[a.first + mat]);
          mb = reinterpret_cast<const uint8_t*>(a.t.momentum[a.first + mat]);
          pbase = reinterpret_cast<const uint8_t*>(a.t.params[a.first + mat]);
          cur = mat;
        }
        const uint8_t* g = gb + off * 2;
        const uint8_t* m = mb + off * 4;
        const uint8_t* p = pbase + off * 2;
#pragma unroll 1
        for (int k = 0; k < VPT; ++k, ++it) {
          const int e0 = k * kChunkElems;
          if (e0 >= cols) break;
          const uint32_t n = (uint32_t)min(kChunkElems, cols - e0);
          const int s = it % kStages;
          if (!mbar_wait_quiet(&empty[s], ((it / kStages) & 1) ^ 1, abort_flag, a.status)) { ok = false; break; }
          uint8_t* dst = gm + (size_t)s * (kGBytes + kMBytes);
          mbar_expect_tx(&full[s], n * 6);
          bulk_load(dst, g + (size_t)e0 * 2, n * 2, &full[s]);
          bulk_load(dst + kGBytes, m + (size_t)e0 * 4, n * 4, &full[s]);
          ++issued_gm;
        }
        if (!ok) break;
        // it counts only the chunks issued; rows of fewer than VPT chunks leave no hole in the ring
        const int b = nrow & 1;
        if (!mbar_wait_quiet(&pempty[b], ((nrow >> 1) & 1) ^ 1, abort_flag, a.status)) break;
        mbar_expect_tx(&pfull[b], row_g);
        bulk_load(pb + (size_t)b * VPT * kGBytes, p, row_g, &pfull[b]);
        ++issued_p;
      }
      // Every copy issued must have landed before this CTA gives up its shared memory.
      for (int k = (issued_gm > kStages ? issued_gm - kStages : 0); k < issued_gm; ++k) {
        const uint64_t t0 = global_ns();
        while (!mbar_try_wait(&full[k % kStages], (k / kStages) & 1)) {
          if (global_ns() - t0 > 1000000ull) break;
        }
      }
      for (int k = (issued_p > 2 ? issued_p - 2 : 0); k < issued_p; ++k) {
        const uint64_t t0 = global_ns();
        while (!mbar_try_wait(&pfull[k & 1], (k >> 1) & 1)) {
          if (global_ns() - t0 > 1000000ull) break;
        }
      }
    }
    return;
  }

  // -------------------------------------------------------------- consumers
  // Thread t owns, in every chunk, the elements 4t .. 4t+3 and 2048+4t .. 2048+4t+3: 8- and
  // 16-byte shared-memory accesses without bank conflicts, 512-byte global stores per warp.
  const int tid = threadIdx.x - 32, cw = warp - 1;
  const float k_dir = a.s.lr_s * a.s.gamma;
  uint32_t it = 0, nrow = 0;
  int cur = -1;
  float* m_base = nullptr;
  __nv_bfloat16* p_base = nullptr;
  for (int64_t rg = blockIdx.x; rg < a.total_rows; rg += gridDim.x, ++nrow) {
    const int mat = (int)(rg / a.rows);
    const int64_t off = (rg - (int64_t)mat * a.rows) * cols;
    if (mat != cur) {
      m_base = a.t.momentum[a.first + mat];
      p_base = reinterpret_cast<__nv_bfloat16*>(a.t.params[a.first + mat]);
      cur = mat;
    }
    float* __restrict__ m_row = m_base + off;
    __nv_bfloat16* __restrict__ p_row = p_base + off;
    float u[VPT][8];
    float acc = 0.f;
    bool ok = true;
#pragma unroll
    for (int k = 0; k < VPT; ++k) {
      const int e0 = k * kChunkElems;
      if (e0 < cols) {
        const int s = it % kStages;
        if (ok && !mbar_wait_quiet(&full[s], (it / kStages) & 1, abort_flag, a.status)) ok = false;
        ++it;
        if (ok) {
          const uint8_t* gs = gm + (size_t)s * (kGBytes + kMBytes);
          const uint8_t* ms = gs + kGBytes;
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            const int e = e0 + h * (kChunkElems / 2) + 4 * tid;
            float* uu = &u[k][4 * h];
            if (e < cols) {
              const uint2 graw = *reinterpret_cast<const uint2*>(gs + h * (kGBytes / 2) + 8 * tid);
              const float4 mv = *reinterpret_cast<const float4*>(ms + h * (kMBytes / 2) + 16 * tid);
              const float2 g01 = bf16x2_f32(graw.x), g23 = bf16x2_f32(graw.y);
              const float gv[4] = {g01.x, g01.y, g23.x, g23.y};
              const float mo[4] = {mv.x, mv.y, mv.z, mv.w};
              float mn[4];
#pragma unroll
              for (int q = 0; q < 4; ++q) {
                mn[q] = blend(a.s.beta, mo[q], a.s.omb, gv[q]);
                uu[q] = NESTEROV ? blend(a.s.beta, mn[q], a.s.omb, gv[q]) : mn[q];
                acc += uu[q] * uu[q];
              }
              *reinterpret_cast<float4*>(m_row + e) = make_float4(mn[0], mn[1], mn[2], mn[3]);
            } else {
#pragma unroll
              for (int q = 0; q < 4; ++q) uu[q] = 0.f;
            }
          }
          __syncwarp();
          if (lane == 0) mbar_arrive(&empty[s]);
        }
      }
    }
    acc = warp_sum(acc);
    const int par = nrow & 1;
    if (lane == 0) warp_part[par * kConsWarps + cw] = acc;
    if (tid == 0) s_go[par] = (*abort_flag == 0) ? 1 : 0;
    cons_sync();
    // s_go is the same for everyone.  A thread whose own wait failed has set the abort flag and
    // keeps arriving at this barrier until everyone leaves, at the next row at the latest.
    if (!s_go[par]) break;
    float total = 0.f;
#pragma unroll
    for (int w = 0; w < kConsWarps; ++w) total += warp_part[par * kConsWarps + w];
    const float nu = fmaxf(sqrtf(total), a.s.eps_row);
    const float coef = k_dir / nu;
    const int b = nrow & 1;
    if (ok && !mbar_wait_quiet(&pfull[b], (nrow >> 1) & 1, abort_flag, a.status)) ok = false;
    if (ok) {
      const uint8_t* ps = pb + (size_t)b * VPT * kGBytes;
#pragma unroll
      for (int k = 0; k < VPT; ++k) {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const int e = k * kChunkElems + h * (kChunkElems / 2) + 4 * tid;
          if (e < cols) {
            const uint2 praw = *reinterpret_cast<const uint2*>(ps + (size_t)e * 2);
            const float2 p01 = bf16x2_f32(praw.x), p23 = bf16x2_f32(praw.y);
            const float* uu = &u[k][4 * h];
            const float q0 = a.s.decay * p01.x - coef * uu[0], q1 = a.s.decay * p01.y - coef * uu[1];
            const float q2 = a.s.decay * p23.x - coef * uu[2], q3 = a.s.decay * p23.y - coef * uu[3];
            *reinterpret_cast<uint2*>(p_row + e) = make_uint2(pack2(q0, q1), pack2(q2, q3));
          }
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&pempty[b]);
    }
  }
}

template <int VPT>
cudaError_t launch_inst(const WideArgs& a, int n_cta, cudaStream_t stream) {
  static PerDeviceOnce ready[2];
  const int nest = a.s.nesterov ? 1 : 0;
  const size_t smem = wide_smem_bytes<VPT>();
  cudaError_t ce;
  int dev;
  if (ready[nest].need(&dev)) {
    ce = nest ? cudaFuncSetAttribute(rowstep_wide_stream_kernel<VPT, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)
              : cudaFuncSetAttribute(rowstep_wide_stream_kernel<VPT, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (ce != cudaSuccess) return ce;
    ready[nest].mark(dev);
  }
  const int grid = (int)std::min<int64_t>(n_cta, a.total_rows);
  if (nest) rowstep_wide_stream_kernel<VPT, true><<<grid, kThreads, smem, stream>>>(a);
  else rowstep_wide_stream_kernel<VPT, false><<<grid, kThreads, smem, stream>>>(a);
  return cudaGetLastError();
}

}  // namespace

bool wide_stream_takes(const Group& g, int io_fp32) {
  return !g.tall && !io_fp32 && g.cols % 8 == 0 && g.cols >= 8 && g.cols <= (int64_t)kMaxVpt * kChunkElems;
}

cudaError_t launch_rowstep_wide_stream(const PtrTables& t, const Group& g, const StepScalars& s, int n_cta, int* status,
                                       cudaStream_t stream, int64_t* launches) {
  if (!wide_stream_takes(g, 0) || n_cta < 1) return cudaErrorInvalidValue;
  WideArgs a;
  a.t = t; a.first = g.first; a.rows = (int)g.rows; a.cols = (int)g.cols;
  a.total_rows = (int64_t)g.count * g.rows;
  a.s = s; a.status = status;
  *launches += 1;
  const int vpt = (int)((g.cols + kChunkElems - 1) / kChunkElems);
  switch (vpt) {
    case 1: return launch_inst<1>(a, n_cta, stream);
    case 2: return launch_inst<2>(a, n_cta, stream);
    case 3: return launch_inst<3>(a, n_cta, stream);
    case 4: return launch_inst<4>(a, n_cta, stream);
    case 5: return launch_inst<5>(a, n_cta, stream);
    default: return launch_inst<6>(a, n_cta, stream);
  }
}

}  // namespace prm

// NS5 pre-pass of wide matrices (stored rows = oriented rows) as a persistent,
// bulk-copy-fed kernel: bf16 gradients, fp32 momentum, bf16 workspace,
// cols % 8 == 0.  Same work as ns_prepass_wide_kernel - momentum update
// (Algorithm 1 line 2), direction input U written unscaled and zero-padded into
// the NS5 workspace as X_0, sums of squares for the Frobenius scale - and the
// same 12 bytes per element.  One CTA per SM walks over the padded rows of the
// sub-batch (row cta, cta + #CTAs, ...); a producer warp fetches gradient and
// momentum in chunks of 4096 elements with bulk asynchronous copies into a ring
// and runs ahead of the 16 consumer warps, which hold no loads in registers.
// A CTA adds its squares per matrix (fixed order) and leaves one partial per
// matrix and CTA, zeros included, for ns_alpha_kernel.  Every mbarrier wait is
// bounded: on expiry the CTA raises the status word, drains the copies in
// flight and returns.
#include "async_copy.cuh"
#include "launch.cuh"

namespace prm {

namespace {

constexpr int kConsWarps = 16;
constexpr int kConsThreads = 32 * kConsWarps;
constexpr int kThreads = kConsThreads + 32;          // warp 0 produces
constexpr int kChunkElems = kConsThreads * 8;        // 4096 elements: eight per consumer thread
constexpr int kStages = 6;
constexpr uint32_t kGBytes = kChunkElems * 2, kMBytes = kChunkElems * 4;
constexpr size_t kSmemBytes = 1024 + (size_t)kStages * (kGBytes + kMBytes) + 512;

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
__device__ __forceinline__ float through_bf16(float v) { return __bfloat162float(__float2bfloat16_rn(v)); }

struct PreArgs {
  PtrTables t;
  int first, batch, rows, cols;
  int prow, pcol;            // padded extent of X
  int64_t bs_x, lo_off;      // batch stride of X in elements; offset of the second plane (0: one plane)
  __nv_bfloat16* X;
  float* fro_partial;        // [batch][#CTAs]
  StepScalars s;
  int* status;
};

__global__ void __launch_bounds__(kThreads, 1) ns_prepass_wide_stream_kernel(const PreArgs a) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  uint8_t* gm = smem;                                              // [kStages][kGBytes + kMBytes]
  uint64_t* bars = reinterpret_cast<uint64_t*>(gm + (size_t)kStages * (kGBytes + kMBytes));
  uint64_t* full = bars;                 // [kStages]
  uint64_t* empty = full + kStages;      // [kStages]
  float* warp_part = reinterpret_cast<float*>(empty + kStages);    // [kConsWarps]
  volatile int* abort_flag = reinterpret_cast<volatile int*>(warp_part + kConsWarps);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int cols = a.cols;
  const int64_t total = (int64_t)a.batch * a.prow;     // padded rows of the sub-batch

  if (threadIdx.x == 0) {
    for (int k = 0; k < kStages; ++k) { mbar_init(&full[k], 1); mbar_init(&empty[k], kConsWarps); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncthreads();

  if (warp == 0) {
    // ------------------------------------------------------------ producer
    if (lane == 0) {
      uint32_t it = 0;
      int issued = 0, cur = -1;
      const uint8_t *gb = nullptr, *mb = nullptr;
      bool ok = true;
      for (int64_t rg = blockIdx.x; rg < total && ok; rg += gridDim.x) {
        const int b = (int)(rg / a.prow);
        const int row = (int)(rg - (int64_t)b * a.prow);
        if (row >= a.rows) continue;               // a padding row: nothing to fetch
        if (b != cur) {                            // base pointers sit in global memory: fetched once per matrix
          gb = reinterpret_cast<const uint8_t*>(a.t.grads[a.first + b]);
          mb = reinterpret_cast<const uint8_t*>(a.t.momentum[a.first + b]);
          cur = b;
        }
        const int64_t off = (int64_t)row * cols;
        for (int e0 = 0; e0 < cols; e0 += kChunkElems, ++it) {
          const uint32_t n = (uint32_t)min(kChunkElems, cols - e0);
          const int s = it % kStages;
          if (!mbar_wait_quiet(&empty[s], ((it / kStages) & 1) ^ 1, abort_flag, a.status)) { ok = false; break; }
          uint8_t* dst = gm + (size_t)s * (kGBytes + kMBytes);
          mbar_expect_tx(&full[s], n * 6);
          bulk_load(dst, gb + (off + e0) * 2, n * 2, &full[s]);
          bulk_load(dst + kGBytes, mb + (off + e0) * 4, n * 4, &full[s]);
          ++issued;
        }
      }
      // Every copy issued must have landed before this CTA gives up its shared memory.
      for (int k = (issued > kStages ? issued - kStages : 0); k < issued; ++k) {
        const uint64_t t0 = global_ns();
        while (!mbar_try_wait(&full[k % kStages], (k / kStages) & 1)) {
          if (global_ns() - t0 > 1000000ull) break;
        }
      }
    }
    return;
  }

  // -------------------------------------------------------------- consumers
  // Thread t owns, in every chunk, the elements 4t .. 4t+3 and 2048+4t .. 2048+4t+3.  No thread
  // leaves the row loop early: the per-matrix reductions below are barriers of all consumers, so
  // after a failed wait a thread only stops touching memory and barriers of the ring.
  const int tid = threadIdx.x - 32, cw = warp - 1;
  uint32_t it = 0;
  int cur = 0, cur_ptr = -1;
  float acc = 0.f;
  float* m_base = nullptr;
  bool ok = true;
  auto flush = [&](int b) {
    acc = warp_sum(acc);
    if (lane == 0) warp_part[cw] = acc;
    cons_sync();
    if (tid == 0) {
      float tot = 0.f;
#pragma unroll
      for (int w = 0; w < kConsWarps; ++w) tot += warp_part[w];
      a.fro_partial[(int64_t)b * gridDim.x + blockIdx.x] = tot;
    }
    cons_sync();
    acc = 0.f;
  };
  for (int64_t rg = blockIdx.x; rg < total; rg += gridDim.x) {
    const int b = (int)(rg / a.prow);
    const int row = (int)(rg - (int64_t)b * a.prow);
    while (cur < b) { flush(cur); ++cur; }
    const bool row_valid = row < a.rows;
    if (row_valid && b != cur_ptr) { m_base = a.t.momentum[a.first + b]; cur_ptr = b; }
    float* __restrict__ m_row = m_base + (int64_t)row * cols;
    __nv_bfloat16* __restrict__ x_row = a.X + (int64_t)b * a.bs_x + (int64_t)row * a.pcol;
    for (int e0 = 0; e0 < a.pcol; e0 += kChunkElems) {
      const bool has_load = row_valid && e0 < cols;
      int s = 0;
      if (has_load) {
        s = it % kStages;
        if (ok && !mbar_wait_quiet(&full[s], (it / kStages) & 1, abort_flag, a.status)) ok = false;
        ++it;
      }
      const uint8_t* gs = gm + (size_t)s * (kGBytes + kMBytes);
      const uint8_t* ms = gs + kGBytes;
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const int e = e0 + h * (kChunkElems / 2) + 4 * tid;
        if (e >= a.pcol) continue;
        float uu[4] = {0.f, 0.f, 0.f, 0.f};
        if (has_load && ok && e < cols) {
          const uint2 graw = *reinterpret_cast<const uint2*>(gs + h * (kGBytes / 2) + 8 * tid);
          const float4 mv = *reinterpret_cast<const float4*>(ms + h * (kMBytes / 2) + 16 * tid);
          const float2 g01 = bf16x2_f32(graw.x), g23 = bf16x2_f32(graw.y);
          const float gv[4] = {g01.x, g01.y, g23.x, g23.y};
          const float mo[4] = {mv.x, mv.y, mv.z, mv.w};
          float mn[4];
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            mn[q] = blend(a.s.beta, mo[q], a.s.omb, gv[q]);
            uu[q] = a.s.nesterov ? blend(a.s.beta, mn[q], a.s.omb, gv[q]) : mn[q];
            acc += uu[q] * uu[q];
          }
          *reinterpret_cast<float4*>(m_row + e) = make_float4(mn[0], mn[1], mn[2], mn[3]);
        }
        if (ok) {
          *reinterpret_cast<uint2*>(x_row + e) = make_uint2(pack2(uu[0], uu[1]), pack2(uu[2], uu[3]));
          if (a.lo_off) {          // second plane: what the bf16 rounding of the first one left
            *reinterpret_cast<uint2*>(x_row + a.lo_off + e) =
                make_uint2(pack2(uu[0] - through_bf16(uu[0]), uu[1] - through_bf16(uu[1])),
                           pack2(uu[2] - through_bf16(uu[2]), uu[3] - through_bf16(uu[3])));
          }
        }
      }
      if (has_load && ok) {
        __syncwarp();
        if (lane == 0) mbar_arrive(&empty[s]);
      }
    }
  }
  while (cur < a.batch) { flush(cur); ++cur; }
}

PerDeviceOnce g_ready;

}  // namespace

bool prepass_stream_takes(const Group& g, int io_fp32, int x_fp32) {
  return !g.tall && !io_fp32 && !x_fp32 && g.cols % 8 == 0 && g.cols >= 8;
}

// Partials per matrix: one per CTA.
int prepass_stream_parts(int n_cta, int64_t prow, int batch) { return (int)std::min<int64_t>(n_cta, prow * batch); }

cudaError_t launch_ns_prepass_stream(const PtrTables& t, const Group& g, int first, int batch, const StepScalars& s,
                                     int split, void* X, float* fro_partial, int n_cta, int* status, cudaStream_t stream) {
  if (!prepass_stream_takes(g, 0, 0) || n_cta < 1) return cudaErrorInvalidValue;
  cudaError_t ce;
  int dev;
  if (g_ready.need(&dev)) {
    ce = cudaFuncSetAttribute(ns_prepass_wide_stream_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
    if (ce != cudaSuccess) return ce;
    g_ready.mark(dev);
  }
  PreArgs a;
  a.t = t; a.first = first; a.batch = batch; a.rows = (int)g.rows; a.cols = (int)g.cols;
  a.prow = (int)g.rp; a.pcol = (int)g.cp;
  a.lo_off = split ? g.rp * g.cp : 0;
  a.bs_x = (split ? 2 : 1) * g.rp * g.cp;
  a.X = reinterpret_cast<__nv_bfloat16*>(X);
  a.fro_partial = fro_partial; a.s = s; a.status = status;
  const int grid = prepass_stream_parts(n_cta, g.rp, batch);
  ns_prepass_wide_stream_kernel<<<grid, kThreads, kSmemBytes, stream>>>(a);
  return cudaGetLastError();
}

}  // namespace prm

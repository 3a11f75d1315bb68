// Row step of tall matrices in ONE pass over HBM (bf16 parameters and
// gradients, fp32 momentum: 14 bytes per element).
//
// For a tall matrix (rows > cols) the oriented rows of Section 3.1 are stored
// columns, so RowNorm (Eq. rownorm) needs the norm of every stored column
// before any parameter of that column can be updated: the sharded-RowNorm
// proposition of the appendix, with the SMs of one GPU in the role of the
// ranks.  The two-pass kernels (rowstep.cu) park the data in HBM between the
// passes and read gradient and momentum twice: 20 bytes per element.  Here the
// data waits in shared memory instead.
//
// The matrices are cut into waves of 64 columns x all rows.  One persistent
// CTA per SM (cooperative launch: all CTAs are resident) owns the same slab of
// R = ceil(rows / #CTAs) consecutive rows in every wave.  Per wave and CTA:
//   phase 1  the slab's gradient and momentum tiles arrive by TMA; the
//            momentum is updated and written back, the direction input U
//            replaces it in shared memory, and the slab's column sums of
//            squares go to a small ring in global memory.  The CTA that
//            arrives last on the wave's counter adds the slabs' sums in CTA
//            order (fixed order: bit-reproducible), writes the column norms
//            nu_j = max(sqrt(sum), eps) and raises the wave's flag;
//   phase 2  `lag` waves later - by then the flag is normally up - the CTA
//            scales its U tile, still in shared memory, by gamma/nu_j and
//            updates the parameter tile, which has arrived by TMA meanwhile.
// A producer warp keeps `depth` waves of gradient/momentum tiles and of
// parameter tiles in flight ahead of the eight consumer warps; nothing is read
// twice and no thread holds loads in registers.  Every wait (mbarrier or flag)
// is bounded: on expiry the CTA raises the status word and a global abort
// flag, all CTAs leave, and loads in flight are drained before shared memory
// is released.
#include "async_copy.cuh"
#include "launch.cuh"

namespace prm {

namespace {

constexpr int kPanel = 64;               // columns per wave
constexpr int kConsWarps = 8;
constexpr int kConsThreads = 32 * kConsWarps;
constexpr int kStreamThreads = 32 + kConsThreads;   // warp 0 produces
constexpr int kRowsPerPass = 2 * kConsWarps;        // a warp covers two rows of 64 columns at a time
constexpr int kMaxLag = 6;
constexpr int kMaxDepth = 3;
constexpr int kSlots = 8;                // ring of per-wave partial sums; must exceed kMaxLag
constexpr int kMaxCtas = 256;
constexpr size_t kSmemLimit = 227 * 1024;
constexpr size_t kSmemFixed = 1024 /*alignment*/ + 512 /*barriers, flags*/ + kConsWarps * kPanel * 4 /*reduction*/;

struct StreamArgs {
  const CUtensorMap* maps;   // [count][3]: gradient, momentum, parameters of each matrix (global memory)
  PtrTables t;
  int first, count, rows, cols;
  int R, lag, depth;
  StepScalars s;
  float* partial;            // [kSlots][#CTAs][kPanel]
  float* nu;                 // [count][cols]
  int* sync;                 // [0] abort, [1 .. W] arrival counters, [1+W .. 2W] norms-ready flags
  int* status;
};

__device__ __forceinline__ void cons_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kConsThreads) : "memory"); }
__device__ __forceinline__ int ld_acquire_gpu(const int* p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_release_gpu(int* p, int v) {
  asm volatile("st.release.gpu.global.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
// Bounded wait for a flag another CTA raises.  False if this or another CTA gave up.
__device__ __forceinline__ bool wait_flag(const int* flag, int* abort_g, int* status) {
  if (ld_acquire_gpu(flag)) return true;
  uint64_t t0 = 0;
  for (uint32_t n = 1;; ++n) {
    if (ld_acquire_gpu(flag)) return true;
    __nanosleep(32);
    if ((n & 15u) == 0) {
      if (ld_acquire_gpu(abort_g)) return false;
      const uint64_t now = global_ns();
      if (t0 == 0) {
        t0 = now;
      } else if (now - t0 > kWaitLimitNs) {
        atomicOr(status, kStatusTimeout);
        atomicExch(abort_g, 1);
        return false;
      }
    }
  }
}
__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }
__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
  __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&v);
}

__global__ void __launch_bounds__(kStreamThreads, 1) rowstep_tall_stream_kernel(const StreamArgs a) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  const int R = a.R, lag = a.lag, D = a.depth;
  const int SG = D, SM = lag + D, SP = D;
  const uint32_t gB = (uint32_t)R * kPanel * 2, mB = (uint32_t)R * kPanel * 4, pB = gB;
  uint8_t* gbuf = smem;
  uint8_t* mbuf = gbuf + (size_t)SG * gB;
  uint8_t* pbuf = mbuf + (size_t)SM * mB;
  float* red = reinterpret_cast<float*>(pbuf + (size_t)SP * pB);             // [kConsWarps][kPanel]
  uint64_t* bars = reinterpret_cast<uint64_t*>(red + kConsWarps * kPanel);
  uint64_t* gfull = bars;                      // [kMaxDepth]
  uint64_t* gempty = gfull + kMaxDepth;        // [kMaxDepth]
  uint64_t* pfull = gempty + kMaxDepth;        // [kMaxDepth]
  uint64_t* pempty = pfull + kMaxDepth;        // [kMaxDepth]
  uint64_t* mfull = pempty + kMaxDepth;        // [kMaxLag + kMaxDepth]
  uint64_t* mempty = mfull + (kMaxLag + kMaxDepth);
  volatile int* flags = reinterpret_cast<volatile int*>(mempty + (kMaxLag + kMaxDepth));
  volatile int* abort_flag = flags;            // set by any role of this CTA whose wait ran out
  volatile int* s_go = flags + 1;              // consumers: carry on with this phase (written by one thread)
  volatile int* s_last = flags + 2;            // consumers: this CTA arrived last on the wave

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int cta = blockIdx.x, n_cta = gridDim.x;
  const int npanel = (a.cols + kPanel - 1) / kPanel;
  const int W = a.count * npanel;
  int* abort_g = a.sync;
  int* counter = a.sync + 1;
  int* ready = a.sync + 1 + W;

  if (threadIdx.x == 0) {
    for (int k = 0; k < kMaxDepth; ++k) {
      mbar_init(&gfull[k], 1); mbar_init(&gempty[k], kConsWarps);
      mbar_init(&pfull[k], 1); mbar_init(&pempty[k], kConsWarps);
    }
    for (int k = 0; k < kMaxLag + kMaxDepth; ++k) { mbar_init(&mfull[k], 1); mbar_init(&mempty[k], kConsWarps); }
    flags[0] = 0; flags[1] = 1; flags[2] = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncthreads();

  if (warp == 0) {
    // ------------------------------------------------------------ producer
    if (lane == 0) {
      int n_gm = 0, n_p = 0;                 // tiles issued so far
      int fenced_gm = -1, fenced_p = -1;     // matrices whose tensor maps have been acquired
      const int y0 = cta * R;
      bool ok = true;
      for (int i = 0; i < W + lag && ok; ++i) {
        if (i < W) {
          const int mat = i / npanel, x0 = (i - mat * npanel) * kPanel;
          const CUtensorMap* mg = a.maps + 3 * mat;
          if (mat != fenced_gm) { tensormap_acquire(mg); tensormap_acquire(mg + 1); fenced_gm = mat; }
          const int sg = i % SG, sm = i % SM;
          if (!mbar_wait(&gempty[sg], ((i / SG) & 1) ^ 1, abort_flag, a.status)) { ok = false; break; }
          if (!mbar_wait(&mempty[sm], ((i / SM) & 1) ^ 1, abort_flag, a.status)) { ok = false; break; }
          mbar_expect_tx(&gfull[sg], gB);
          tma_load_2d(gbuf + (size_t)sg * gB, mg, &gfull[sg], x0, y0);
          mbar_expect_tx(&mfull[sm], mB);
          tma_load_2d(mbuf + (size_t)sm * mB, mg + 1, &mfull[sm], x0, y0);
          ++n_gm;
        }
        const int j = i - lag;
        if (j >= 0) {
          const int mat = j / npanel, x0 = (j - mat * npanel) * kPanel;
          const CUtensorMap* mp = a.maps + 3 * mat + 2;
          if (mat != fenced_p) { tensormap_acquire(mp); fenced_p = mat; }
          const int sp = j % SP;
          if (!mbar_wait(&pempty[sp], ((j / SP) & 1) ^ 1, abort_flag, a.status)) { ok = false; break; }
          mbar_expect_tx(&pfull[sp], pB);
          tma_load_2d(pbuf + (size_t)sp * pB, mp, &pfull[sp], x0, y0);
          ++n_p;
        }
      }
      // Every load issued must have landed before this CTA gives up its shared memory.  After a
      // complete run this returns at once; after an abort it waits at most 1 ms per tile.
      auto drain = [&](uint64_t* full, int stages, int issued) {
        for (int k = (issued > stages ? issued - stages : 0); k < issued; ++k) {
          const uint64_t t0 = global_ns();
          while (!mbar_try_wait(&full[k % stages], (k / stages) & 1)) {
            if (global_ns() - t0 > 1000000ull) break;
          }
        }
      };
      drain(gfull, SG, n_gm);
      drain(mfull, SM, n_gm);
      drain(pfull, SP, n_p);
    }
  } else {
    // ------------------------------------------------------------ consumers
    const int cw = warp - 1, tid = threadIdx.x - 32;
    const int half = lane >> 4, l16 = lane & 15;
    const float beta = a.s.beta, omb = a.s.omb;
    const bool nesterov = a.s.nesterov != 0;
    const float k_dir = a.s.lr_s * a.s.gamma, decay = a.s.decay;
    for (int i = 0; i < W + lag; ++i) {
      if (i < W) {
        // -------- phase 1 of wave i
        const int mat = i / npanel, panel = i - mat * npanel;
        const int sg = i % SG, sm = i % SM;
        mbar_wait(&gfull[sg], (i / SG) & 1, abort_flag, a.status);
        mbar_wait(&mfull[sm], (i / SM) & 1, abort_flag, a.status);
        if (tid == 0) *s_go = (*abort_flag == 0) ? 1 : 0;
        cons_sync();
        if (!*s_go) break;
        const uint8_t* gs = gbuf + (size_t)sg * gB;
        uint8_t* ms = mbuf + (size_t)sm * mB;
        const int col0 = panel * kPanel + l16 * 4;
        const bool col_ok = col0 < a.cols;
        float* __restrict__ m_glob = a.t.momentum[a.first + mat];
        float cs0 = 0.f, cs1 = 0.f, cs2 = 0.f, cs3 = 0.f;
#pragma unroll 2
        for (int r = cw * 2 + half; r < R; r += kRowsPerPass) {
          const uint2 graw = *reinterpret_cast<const uint2*>(gs + (size_t)r * (kPanel * 2) + l16 * 8);
          float4* mptr = reinterpret_cast<float4*>(ms + (size_t)r * (kPanel * 4) + l16 * 16);
          const float4 mv = *mptr;
          const float g0 = bf16_lo(graw.x), g1 = bf16_hi(graw.x), g2 = bf16_lo(graw.y), g3 = bf16_hi(graw.y);
          float4 mn, u;
          mn.x = blend(beta, mv.x, omb, g0); mn.y = blend(beta, mv.y, omb, g1);
          mn.z = blend(beta, mv.z, omb, g2); mn.w = blend(beta, mv.w, omb, g3);
          u.x = nesterov ? blend(beta, mn.x, omb, g0) : mn.x;
          u.y = nesterov ? blend(beta, mn.y, omb, g1) : mn.y;
          u.z = nesterov ? blend(beta, mn.z, omb, g2) : mn.z;
          u.w = nesterov ? blend(beta, mn.w, omb, g3) : mn.w;
          cs0 += u.x * u.x; cs1 += u.y * u.y; cs2 += u.z * u.z; cs3 += u.w * u.w;
          *mptr = u;                                   // the direction input waits here for phase 2
          const int row = cta * R + r;
          if (row < a.rows && col_ok) *reinterpret_cast<float4*>(m_glob + (int64_t)row * a.cols + col0) = mn;
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&gempty[sg]);       // the gradient tile is done with
        cs0 += __shfl_xor_sync(0xffffffffu, cs0, 16); cs1 += __shfl_xor_sync(0xffffffffu, cs1, 16);
        cs2 += __shfl_xor_sync(0xffffffffu, cs2, 16); cs3 += __shfl_xor_sync(0xffffffffu, cs3, 16);
        if (half == 0) *reinterpret_cast<float4*>(red + cw * kPanel + l16 * 4) = make_float4(cs0, cs1, cs2, cs3);
        cons_sync();
        const int slot = i % kSlots;
        if (tid < kPanel) {
          float tot = 0.f;
#pragma unroll
          for (int w8 = 0; w8 < kConsWarps; ++w8) tot += red[w8 * kPanel + tid];
          a.partial[((size_t)slot * n_cta + cta) * kPanel + tid] = tot;
          __threadfence();
        }
        cons_sync();
        if (tid == 0) *s_last = (atomicAdd(&counter[i], 1) == n_cta - 1) ? 1 : 0;
        cons_sync();
        if (*s_last) {
          // Last slab of the wave: column norms, slabs added in CTA order.
          __threadfence();
          const int col = panel * kPanel + tid;
          if (tid < kPanel && col < a.cols) {
            const float* src = a.partial + (size_t)slot * n_cta * kPanel + tid;
            float tot = 0.f;
#pragma unroll 4
            for (int q = 0; q < n_cta; ++q) tot += __ldcg(src + (size_t)q * kPanel);
            a.nu[(int64_t)mat * a.cols + col] = fmaxf(sqrtf(tot), a.s.eps_row);
            __threadfence();
          }
          cons_sync();
          if (tid == 0) st_release_gpu(&ready[i], 1);
        }
      }
      const int j = i - lag;
      if (j >= 0) {
        // -------- phase 2 of wave j
        const int mat = j / npanel, panel = j - mat * npanel;
        const int sm = j % SM, sp = j % SP;
        mbar_wait(&pfull[sp], (j / SP) & 1, abort_flag, a.status);
        if (tid == 0) {
          const bool up = wait_flag(&ready[j], abort_g, a.status);
          *s_go = (up && *abort_flag == 0) ? 1 : 0;
        }
        cons_sync();
        if (!*s_go) break;
        const int col0 = panel * kPanel + l16 * 4;
        const bool col_ok = col0 < a.cols;
        float4 nu4 = make_float4(1.f, 1.f, 1.f, 1.f);
        if (col_ok) nu4 = __ldcg(reinterpret_cast<const float4*>(a.nu + (int64_t)mat * a.cols + col0));
        const float c0 = k_dir / nu4.x, c1 = k_dir / nu4.y, c2 = k_dir / nu4.z, c3 = k_dir / nu4.w;
        const uint8_t* ms = mbuf + (size_t)sm * mB;
        const uint8_t* ps = pbuf + (size_t)sp * pB;
        __nv_bfloat16* __restrict__ p_glob = reinterpret_cast<__nv_bfloat16*>(a.t.params[a.first + mat]);
#pragma unroll 2
        for (int r = cw * 2 + half; r < R; r += kRowsPerPass) {
          const float4 u = *reinterpret_cast<const float4*>(ms + (size_t)r * (kPanel * 4) + l16 * 16);
          const uint2 praw = *reinterpret_cast<const uint2*>(ps + (size_t)r * (kPanel * 2) + l16 * 8);
          const float p0 = decay * bf16_lo(praw.x) - c0 * u.x;
          const float p1 = decay * bf16_hi(praw.x) - c1 * u.y;
          const float p2 = decay * bf16_lo(praw.y) - c2 * u.z;
          const float p3 = decay * bf16_hi(praw.y) - c3 * u.w;
          const int row = cta * R + r;
          if (row < a.rows && col_ok)
            *reinterpret_cast<uint2*>(p_glob + (int64_t)row * a.cols + col0) = make_uint2(pack_bf16(p0, p1), pack_bf16(p2, p3));
        }
        // the tiles go back to the producer, whose next TMA load overwrites what this thread wrote
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (lane == 0) { mbar_arrive(&mempty[sm]); mbar_arrive(&pempty[sp]); }
      }
    }
    if (*abort_flag) atomicExch(abort_g, 1);   // let the other CTAs leave their flag waits at once
  }
  __syncthreads();
}

bool g_stream_ready = false;

}  // namespace

TallStreamPlan tall_stream_plan(int64_t rows, int64_t cols, int io_fp32, int n_cta) {
  TallStreamPlan p;
  if (io_fp32 || cols % 8 != 0 || rows <= cols || n_cta < 1 || n_cta > kMaxCtas) return p;
  if (rows > 0x7fffffffLL / 2 || cols > 0x7fffffffLL / 2) return p;
  const int64_t R = (rows + n_cta - 1) / n_cta;
  if (R < 1 || R > 256) return p;                       // one TMA box holds a slab
  const size_t unit = (size_t)R * kPanel * 2;           // a gradient or parameter tile; a momentum tile is two
  const size_t budget = kSmemLimit - kSmemFixed;
  for (int lag = kMaxLag; lag >= 1 && !p.ok; --lag) {
    for (int depth = kMaxDepth; depth >= 2; --depth) {
      if (unit * (size_t)(4 * depth + 2 * lag) <= budget) {
        p.ok = 1; p.R = (int)R; p.lag = lag; p.depth = depth;
        p.smem = kSmemFixed + unit * (size_t)(4 * depth + 2 * lag);
        break;
      }
    }
  }
  return p;
}

size_t tall_stream_partial_bytes() { return (size_t)kSlots * kMaxCtas * kPanel * sizeof(float); }
size_t tall_stream_sync_ints(int64_t cols, int count) { return 2 * (size_t)count * (size_t)((cols + kPanel - 1) / kPanel) + 1; }
int tall_stream_panel() { return kPanel; }

cudaError_t launch_rowstep_tall_stream(const PtrTables& t, const Group& g, const StepScalars& s,
                                       const TallStreamPlan& plan, const void* maps_dev, float* partial, float* nu,
                                       int* sync, int* status, int n_cta, cudaStream_t stream, int64_t* launches) {
  if (!plan.ok) return cudaErrorInvalidValue;
  cudaError_t ce;
  if (!g_stream_ready) {
    ce = cudaFuncSetAttribute(rowstep_tall_stream_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemLimit);
    if (ce != cudaSuccess) return ce;
    g_stream_ready = true;
  }
  ce = cudaMemsetAsync(sync, 0, tall_stream_sync_ints(g.cols, g.count) * sizeof(int), stream);
  if (ce != cudaSuccess) return ce;
  StreamArgs a;
  a.maps = reinterpret_cast<const CUtensorMap*>(maps_dev);
  a.t = t; a.first = g.first; a.count = g.count; a.rows = (int)g.rows; a.cols = (int)g.cols;
  a.R = plan.R; a.lag = plan.lag; a.depth = plan.depth;
  a.s = s; a.partial = partial; a.nu = nu; a.sync = sync; a.status = status;
  void* args[] = {&a};
  *launches += 1;
  // Cooperative: the CTAs wait on one another's flags, so all of them must be resident.
  return cudaLaunchCooperativeKernel((const void*)rowstep_tall_stream_kernel, dim3(n_cta), dim3(kStreamThreads), args,
                                     plan.smem, stream);
}

}  // namespace prm

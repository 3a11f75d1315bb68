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
//            squares are handed to the arrival warps;
//   arrival  the sums go to a small ring in global memory (L2) and the CTA
//            counts itself in on the wave;
//   norms    once all CTAs have arrived, every CTA adds the slabs' sums itself,
//            in the same fixed order (bit-reproducible, and bit-identical in
//            all CTAs), and keeps the column norms nu_j = max(sqrt(sum), eps)
//            in shared memory: a few KB per CTA and wave from L2, and no CTA
//            waits for another one's arithmetic;
//   phase 2  `lag` waves after phase 1 - by then the norms are normally there -
//            the CTA scales its U tile, still in shared memory, by gamma/nu_j
//            and updates the parameter tile, which has arrived by TMA meanwhile.
// Warp roles: one producer (TMA loads, `depth` waves of gradient/momentum tiles
// and of parameter tiles in flight), fourteen consumers (both phases; they
// touch global memory only to store results), one arrival warp, one warp that
// polls the waves' arrival counters, and eight warps that add the slabs' sums
// (everything that waits on L2 or on other CTAs).  Nothing is read twice from
// HBM and no thread holds tile loads in registers.  Every wait (mbarrier or
// counter) is bounded: on expiry the CTA raises the status word and a global
// abort flag, all CTAs leave, and loads in flight are drained before shared
// memory is released.
//
// What it costs: a global hand-shake per 64 columns.  Measured on a B200
// (16384 x 4096 matrices, 148 CTAs): 0.92 GB of DRAM traffic per matrix against
// 1.34 GB for the two passes, and 7.8 ms for 42 matrices at full SM clock
// against 8.5 ms; but the kernel is bound by the SM's instruction issue, not
// by HBM, so at the ~1.3 GHz that row steps see right after a power-capped
// refresh it falls behind the two-pass kernels (9.0-9.4 ms against 8.7 ms).
#include "async_copy.cuh"
#include "launch.cuh"

namespace prm {

namespace {

constexpr int kPanel = 64;               // columns per wave
constexpr int kConsWarps = 14;           // 28 rows per pass: slabs of 56, 84, 111, 139 rows take 2, 3, 4, 5 passes
constexpr int kConsThreads = 32 * kConsWarps;
constexpr int kArrWarp = 1 + kConsWarps;
constexpr int kPollWarp = kArrWarp + 1;
constexpr int kFirstNormWarp = kPollWarp + 1;
constexpr int kNormWarps = 8;
constexpr int kNormThreads = 32 * kNormWarps;
constexpr int kNormParts = kNormThreads / (kPanel / 4);   // a norm thread adds every kNormParts-th CTA, four columns at a time
constexpr int kNormChunk = 10;           // 16-byte loads a norm thread has in flight (148 CTAs / 16 parts: one round)
constexpr int kStreamThreads = 32 * (kFirstNormWarp + kNormWarps);   // warp 0 produces
constexpr int kRowsPerPass = 2 * kConsWarps;        // a warp covers two rows of 64 columns at a time
constexpr int kMaxLag = 6;
constexpr int kMaxDepth = 3;
constexpr int kSlots = 16;               // global ring of per-wave partial sums; at least kMaxLag + kMaxDepth
constexpr int kRing = 4;                 // shared-memory rings between the consumers and the other roles
constexpr int kMaxCtas = 256;
constexpr size_t kSmemLimit = 227 * 1024;
constexpr size_t kSmemFixed = 1024 /*alignment*/ + 1024 /*barriers, flags*/ +
                              (kConsWarps + 2 * kRing + kNormParts) * kPanel * 4 /*reduction, column sums, norms, parts*/;

struct StreamArgs {
  const CUtensorMap* maps;   // [count][3]: gradient, momentum, parameters of each matrix (global memory)
  PtrTables t;
  int first, count, rows, cols;
  int R, lag, depth;
  StepScalars s;
  float* partial;            // [kSlots][#CTAs][kPanel]
  int* sync;                 // [0] abort, [1 .. W] arrival counters
  int* status;
};

__device__ __forceinline__ void cons_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kConsThreads) : "memory"); }
__device__ __forceinline__ void norm_sync() { asm volatile("bar.sync 2, %0;" ::"n"(kNormThreads) : "memory"); }
__device__ __forceinline__ int ld_acquire_gpu(const int* p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void red_add_release_gpu(int* p, int v) {
  asm volatile("red.release.gpu.global.add.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
// Bounded wait until a counter that the other CTAs add to reaches `want`.  False if this or
// another CTA gave up.
__device__ __forceinline__ bool wait_count(const int* ctr, int want, int* abort_g, volatile int* abort_flag,
                                           int* status) {
  if (ld_acquire_gpu(ctr) >= want) return true;
  uint64_t t0 = 0;
  for (uint32_t n = 1;; ++n) {
    if (ld_acquire_gpu(ctr) >= want) return true;
    __nanosleep(20);
    if ((n & 15u) == 0) {
      if (*abort_flag || ld_acquire_gpu(abort_g)) { *abort_flag = 1; return false; }
      const uint64_t now = global_ns();
      if (t0 == 0) {
        t0 = now;
      } else if (now - t0 > kWaitLimitNs) {
        *abort_flag = 1;
        atomicOr(status, kStatusTimeout);
        atomicExch(abort_g, 1);
        return false;
      }
    }
  }
}
__device__ __forceinline__ float2 bf16x2_to_f32x2(uint32_t w) {
  return make_float2(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u));
}
__device__ __forceinline__ uint32_t pack_bf16(float2 v) {
  __nv_bfloat162 h = __floats2bfloat162_rn(v.x, v.y);
  return *reinterpret_cast<uint32_t*>(&h);
}
// beta*x + omb*y on two lanes at once (packed fp32 arithmetic of sm_100): bit for bit what
// blend() gives per element, in half the instructions.
__device__ __forceinline__ float2 blend2(float2 beta, float2 x, float2 omb_y) { return __ffma2_rn(beta, x, omb_y); }

// Position in a ring of n stages: stage index and the parity of its current use.  Kept by
// increments: a division per wave and ring in every warp costs more than the tile arithmetic.
struct Ring {
  int idx = 0, n;
  uint32_t phase = 0;
  __device__ __forceinline__ explicit Ring(int size) : n(size) {}
  __device__ __forceinline__ void next() {
    if (++idx == n) { idx = 0; phase ^= 1u; }
  }
};
// Wave number -> (matrix, column panel), also by increments.
struct Wave {
  int mat = 0, panel = 0, npanel;
  __device__ __forceinline__ explicit Wave(int panels) : npanel(panels) {}
  __device__ __forceinline__ void next() {
    if (++panel == npanel) { panel = 0; ++mat; }
  }
  __device__ __forceinline__ void skip(int k) {
    for (int q = 0; q < k; ++q) next();
  }
};

template <bool NESTEROV>
__global__ void __launch_bounds__(kStreamThreads, 1) rowstep_tall_stream_kernel(const StreamArgs a) {
  extern __shared__ uint8_t smem_raw[];
  // Aligned by pointer arithmetic (not through an integer) so that the compiler keeps treating
  // every tile access as a shared-memory access.
  uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  const int R = a.R, lag = a.lag, D = a.depth;
  const int SG = D, SM = lag + D, SP = D;
  const uint32_t gB = (uint32_t)R * kPanel * 2, mB = (uint32_t)R * kPanel * 4, pB = gB;
  uint8_t* gbuf = smem;
  uint8_t* mbuf = gbuf + (size_t)SG * gB;
  uint8_t* pbuf = mbuf + (size_t)SM * mB;
  float* red = reinterpret_cast<float*>(pbuf + (size_t)SP * pB);             // [kConsWarps][kPanel]
  float* csum = red + kConsWarps * kPanel;     // [kRing][kPanel] this slab's column sums, consumers -> arrival warp
  float* nus = csum + kRing * kPanel;          // [kRing][kPanel] column norms, norm warps -> consumers
  float* comb = nus + kRing * kPanel;          // [kNormParts][kPanel] the parts of a wave's sum
  uint64_t* bars = reinterpret_cast<uint64_t*>(comb + kNormParts * kPanel);
  uint64_t* gfull = bars;                      // [kMaxDepth]
  uint64_t* gempty = gfull + kMaxDepth;        // [kMaxDepth]
  uint64_t* pfull = gempty + kMaxDepth;        // [kMaxDepth]
  uint64_t* pempty = pfull + kMaxDepth;        // [kMaxDepth]
  uint64_t* mfull = pempty + kMaxDepth;        // [kMaxLag + kMaxDepth]
  uint64_t* mempty = mfull + (kMaxLag + kMaxDepth);
  uint64_t* cfull = mempty + (kMaxLag + kMaxDepth);   // [kRing]
  uint64_t* cempty = cfull + kRing;
  uint64_t* nfull = cempty + kRing;
  uint64_t* nempty = nfull + kRing;
  uint64_t* rfull = nempty + kRing;            // [kRing] poll warp -> norm warps: every CTA has arrived on the wave
  uint64_t* rempty = rfull + kRing;
  volatile int* flags = reinterpret_cast<volatile int*>(rempty + kRing);
  volatile int* abort_flag = flags;            // set by any role of this CTA whose wait ran out
  volatile int* s_go = flags + 1;              // consumers: carry on with this phase (written by one thread)
  volatile int* s_ngo = flags + 2;             // norm warps: carry on

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int cta = blockIdx.x, n_cta = gridDim.x;
  const int npanel = (a.cols + kPanel - 1) / kPanel;
  const int W = a.count * npanel;
  int* abort_g = a.sync;
  int* counter = a.sync + 1;

  if (threadIdx.x == 0) {
    for (int k = 0; k < kMaxDepth; ++k) {
      mbar_init(&gfull[k], 1); mbar_init(&gempty[k], kConsWarps);
      mbar_init(&pfull[k], 1); mbar_init(&pempty[k], kConsWarps);
    }
    for (int k = 0; k < kMaxLag + kMaxDepth; ++k) { mbar_init(&mfull[k], 1); mbar_init(&mempty[k], kConsWarps); }
    for (int k = 0; k < kRing; ++k) {
      mbar_init(&cfull[k], kPanel); mbar_init(&cempty[k], 1);
      mbar_init(&nfull[k], 1); mbar_init(&nempty[k], kConsWarps);
      mbar_init(&rfull[k], 1); mbar_init(&rempty[k], 1);
    }
    flags[0] = 0; flags[1] = 1; flags[2] = 1; flags[3] = 1;
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
      Ring rg(SG), rm(SM), rp(SP);
      Wave w1(npanel), w2(npanel);
      for (int i = 0; i < W + lag; ++i) {
        if (i < W) {
          const CUtensorMap* mg = a.maps + 3 * w1.mat;
          if (w1.mat != fenced_gm) { tensormap_acquire(mg); tensormap_acquire(mg + 1); fenced_gm = w1.mat; }
          if (!mbar_wait_quiet(&gempty[rg.idx], rg.phase ^ 1, abort_flag, a.status)) break;
          if (!mbar_wait_quiet(&mempty[rm.idx], rm.phase ^ 1, abort_flag, a.status)) break;
          mbar_expect_tx(&gfull[rg.idx], gB);
          tma_load_2d(gbuf + (size_t)rg.idx * gB, mg, &gfull[rg.idx], w1.panel * kPanel, y0);
          mbar_expect_tx(&mfull[rm.idx], mB);
          tma_load_2d(mbuf + (size_t)rm.idx * mB, mg + 1, &mfull[rm.idx], w1.panel * kPanel, y0);
          ++n_gm; rg.next(); rm.next(); w1.next();
        }
        if (i >= lag) {
          const CUtensorMap* mp = a.maps + 3 * w2.mat + 2;
          if (w2.mat != fenced_p) { tensormap_acquire(mp); fenced_p = w2.mat; }
          if (!mbar_wait_quiet(&pempty[rp.idx], rp.phase ^ 1, abort_flag, a.status)) break;
          mbar_expect_tx(&pfull[rp.idx], pB);
          tma_load_2d(pbuf + (size_t)rp.idx * pB, mp, &pfull[rp.idx], w2.panel * kPanel, y0);
          ++n_p; rp.next(); w2.next();
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
  } else if (warp < kArrWarp) {
    // ------------------------------------------------------------ consumers
    const int cw = warp - 1, tid = threadIdx.x - 32;
    const int half = lane >> 4, l16 = lane & 15;
    const float2 beta2 = make_float2(a.s.beta, a.s.beta), omb2 = make_float2(a.s.omb, a.s.omb);
    const float k_dir = a.s.lr_s * a.s.gamma;
    const float2 decay2 = make_float2(a.s.decay, a.s.decay);
    const int r_end = min(R, a.rows - cta * R);          // rows of this slab inside the matrix (may be <= 0)
    const int r0 = cw * 2 + half;                        // this thread's first row of a tile
    const int64_t gstep = (int64_t)kRowsPerPass * a.cols;
    // The matrices' base pointers sit in global memory: fetched once per matrix, not once per wave
    // (a dependent L2 access on the consumers' path costs more than the whole tile arithmetic).
    int mat1 = -1, mat2 = -1;
    float* m_base = nullptr;
    __nv_bfloat16* p_base = nullptr;
    Ring rg(SG), rm1(SM), rm2(SM), rp(SP);
    Wave w1(npanel), w2(npanel);
    for (int i = 0; i < W + lag; ++i) {
      if (i < W) {
        // -------- phase 1 of wave i
        mbar_wait_quiet(&gfull[rg.idx], rg.phase, abort_flag, a.status);
        mbar_wait_quiet(&mfull[rm1.idx], rm1.phase, abort_flag, a.status);
        if (tid == 0) *s_go = (*abort_flag == 0) ? 1 : 0;
        cons_sync();
        if (!*s_go) break;
        const int col0 = w1.panel * kPanel + l16 * 4;
        const bool col_ok = col0 < a.cols;
        if (w1.mat != mat1) { m_base = a.t.momentum[a.first + w1.mat] + ((int64_t)cta * R + r0) * a.cols; mat1 = w1.mat; }
        const uint8_t* gs = gbuf + (size_t)rg.idx * gB + (size_t)r0 * (kPanel * 2) + l16 * 8;
        uint8_t* ms = mbuf + (size_t)rm1.idx * mB + (size_t)r0 * (kPanel * 4) + l16 * 16;
        float* __restrict__ m_glob = m_base + col0;
        float2 cs01 = make_float2(0.f, 0.f), cs23 = cs01;
        // rows beyond the matrix arrive as zeros and add nothing
#pragma unroll 4
        for (int r = r0; r < R; r += kRowsPerPass) {
          const uint2 graw = *reinterpret_cast<const uint2*>(gs);
          float4* mptr = reinterpret_cast<float4*>(ms);
          const float4 mv = *mptr;
          const float2 og01 = __fmul2_rn(omb2, bf16x2_to_f32x2(graw.x)), og23 = __fmul2_rn(omb2, bf16x2_to_f32x2(graw.y));
          const float2 mn01 = blend2(beta2, make_float2(mv.x, mv.y), og01);
          const float2 mn23 = blend2(beta2, make_float2(mv.z, mv.w), og23);
          const float2 u01 = NESTEROV ? blend2(beta2, mn01, og01) : mn01;
          const float2 u23 = NESTEROV ? blend2(beta2, mn23, og23) : mn23;
          cs01 = __ffma2_rn(u01, u01, cs01);
          cs23 = __ffma2_rn(u23, u23, cs23);
          *mptr = make_float4(u01.x, u01.y, u23.x, u23.y);   // the direction input waits here for phase 2
          if (r < r_end && col_ok) *reinterpret_cast<float4*>(m_glob) = make_float4(mn01.x, mn01.y, mn23.x, mn23.y);
          gs += kRowsPerPass * kPanel * 2;
          ms += kRowsPerPass * kPanel * 4;
          m_glob += gstep;
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&gempty[rg.idx]);   // the gradient tile is done with
        float cs0 = cs01.x, cs1 = cs01.y, cs2 = cs23.x, cs3 = cs23.y;
        cs0 += __shfl_xor_sync(0xffffffffu, cs0, 16); cs1 += __shfl_xor_sync(0xffffffffu, cs1, 16);
        cs2 += __shfl_xor_sync(0xffffffffu, cs2, 16); cs3 += __shfl_xor_sync(0xffffffffu, cs3, 16);
        if (half == 0) *reinterpret_cast<float4*>(red + cw * kPanel + l16 * 4) = make_float4(cs0, cs1, cs2, cs3);
        cons_sync();
        if (tid < kPanel) {
          const int cr = i & (kRing - 1);
          mbar_wait_quiet(&cempty[cr], ((i / kRing) & 1) ^ 1, abort_flag, a.status);
          float tot = 0.f;
#pragma unroll
          for (int w8 = 0; w8 < kConsWarps; ++w8) tot += red[w8 * kPanel + tid];
          csum[cr * kPanel + tid] = tot;
          mbar_arrive(&cfull[cr]);
        }
        rg.next(); rm1.next(); w1.next();
      }
      if (i >= lag) {
        // -------- phase 2 of wave j = i - lag
        const int j = i - lag, nr = j & (kRing - 1);
        mbar_wait_quiet(&pfull[rp.idx], rp.phase, abort_flag, a.status);
        mbar_wait_quiet(&nfull[nr], (j / kRing) & 1, abort_flag, a.status);
        if (tid == 0) *s_go = (*abort_flag == 0) ? 1 : 0;
        cons_sync();
        if (!*s_go) break;
        const int col0 = w2.panel * kPanel + l16 * 4;
        const bool col_ok = col0 < a.cols;
        const float4 nu4 = *reinterpret_cast<const float4*>(nus + nr * kPanel + l16 * 4);
        __syncwarp();
        if (lane == 0) mbar_arrive(&nempty[nr]);
        const float2 nc01 = make_float2(-__fdividef(k_dir, nu4.x), -__fdividef(k_dir, nu4.y));
        const float2 nc23 = make_float2(-__fdividef(k_dir, nu4.z), -__fdividef(k_dir, nu4.w));
        if (w2.mat != mat2) {
          p_base = reinterpret_cast<__nv_bfloat16*>(a.t.params[a.first + w2.mat]) + ((int64_t)cta * R + r0) * a.cols;
          mat2 = w2.mat;
        }
        const uint8_t* ms = mbuf + (size_t)rm2.idx * mB + (size_t)r0 * (kPanel * 4) + l16 * 16;
        const uint8_t* ps = pbuf + (size_t)rp.idx * pB + (size_t)r0 * (kPanel * 2) + l16 * 8;
        __nv_bfloat16* __restrict__ p_glob = p_base + col0;
#pragma unroll 4
        for (int r = r0; r < R; r += kRowsPerPass) {
          const float4 u = *reinterpret_cast<const float4*>(ms);
          const uint2 praw = *reinterpret_cast<const uint2*>(ps);
          // W <- decay*W - lr*s*gamma*U/nu
          const float2 p01 = __ffma2_rn(nc01, make_float2(u.x, u.y), __fmul2_rn(decay2, bf16x2_to_f32x2(praw.x)));
          const float2 p23 = __ffma2_rn(nc23, make_float2(u.z, u.w), __fmul2_rn(decay2, bf16x2_to_f32x2(praw.y)));
          if (r < r_end && col_ok) *reinterpret_cast<uint2*>(p_glob) = make_uint2(pack_bf16(p01), pack_bf16(p23));
          ms += kRowsPerPass * kPanel * 4;
          ps += kRowsPerPass * kPanel * 2;
          p_glob += gstep;
        }
        // the tiles go back to the producer, whose next TMA load overwrites what this thread wrote
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (lane == 0) { mbar_arrive(&mempty[rm2.idx]); mbar_arrive(&pempty[rp.idx]); }
        rm2.next(); rp.next(); w2.next();
      }
    }
  } else if (warp == kArrWarp) {
    // ------------------------------------------------------------ arrival
    // The slab's column sums go to global memory and the CTA counts itself in on the wave.  The
    // release on the counter waits for the stores, which is why this is not the consumers' job.
    int slot = 0;
    for (int i = 0; i < W; ++i) {
      const int cr = i & (kRing - 1);
      if (!mbar_wait_quiet(&cfull[cr], (i / kRing) & 1, abort_flag, a.status)) break;
      const float2 v = *reinterpret_cast<const float2*>(csum + cr * kPanel + lane * 2);
      *reinterpret_cast<float2*>(a.partial + ((size_t)slot * n_cta + cta) * kPanel + lane * 2) = v;
      __syncwarp();                                          // orders the lanes' stores before the release below
      if (lane == 0) {
        mbar_arrive(&cempty[cr]);
        red_add_release_gpu(&counter[i], 1);
      }
      slot = (slot + 1) & (kSlots - 1);
    }
  } else if (warp == kPollWarp) {
    // ------------------------------------------------------------ poll
    // Watches the waves' arrival counters one after the other, so that the norm warps never
    // spend an L2 round trip on a counter.
    if (lane == 0) {
      for (int j = 0; j < W; ++j) {
        const int rr = j & (kRing - 1);
        if (!mbar_wait_quiet(&rempty[rr], ((j / kRing) & 1) ^ 1, abort_flag, a.status)) break;
        if (!wait_count(&counter[j], n_cta, abort_g, abort_flag, a.status)) break;
        mbar_arrive(&rfull[rr]);
      }
    }
  } else {
    // ------------------------------------------------------------ norms
    // Once every CTA has arrived on wave j, add the slabs' sums - each thread every 16th CTA in
    // ascending order, then the 16 parts in order: the same fixed order in every CTA - and leave
    // the column norms in shared memory.  One round of 16-byte loads: the sum is bound by L2
    // latency and by the instructions it takes, not by bandwidth.
    const int nt = threadIdx.x - 32 * kFirstNormWarp;
    const int c4 = nt & (kPanel / 4 - 1), part = nt / (kPanel / 4);   // four columns of the panel, CTAs part, part + 16, ...
    for (int j = 0; j < W; ++j) {
      const int nr = j & (kRing - 1), slot = j & (kSlots - 1);
      if (nt == 0) {
        const bool ok = mbar_wait_quiet(&nempty[nr], ((j / kRing) & 1) ^ 1, abort_flag, a.status) &&
                        mbar_wait_quiet(&rfull[nr], (j / kRing) & 1, abort_flag, a.status);
        *s_ngo = (ok && *abort_flag == 0) ? 1 : 0;
      }
      norm_sync();
      if (!*s_ngo) break;
      const float4* src = reinterpret_cast<const float4*>(a.partial + (size_t)slot * n_cta * kPanel) + c4;
      float4 tot = make_float4(0.f, 0.f, 0.f, 0.f);
      for (int q0 = part; q0 < n_cta; q0 += kNormParts * kNormChunk) {
        float4 v[kNormChunk];
#pragma unroll
        for (int k = 0; k < kNormChunk; ++k) {
          const int q = q0 + k * kNormParts;
          v[k] = (q < n_cta) ? __ldcg(src + (size_t)q * (kPanel / 4)) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int k = 0; k < kNormChunk; ++k) { tot.x += v[k].x; tot.y += v[k].y; tot.z += v[k].z; tot.w += v[k].w; }
      }
      *reinterpret_cast<float4*>(comb + part * kPanel + c4 * 4) = tot;
      norm_sync();
      if (nt < kPanel) {
        float sum = comb[nt];
#pragma unroll
        for (int q = 1; q < kNormParts; ++q) sum += comb[q * kPanel + nt];
        nus[nr * kPanel + nt] = fmaxf(sqrtf(sum), a.s.eps_row);
      }
      norm_sync();                                           // also keeps comb from being rewritten too early
      if (nt == 0) { mbar_arrive(&nfull[nr]); mbar_arrive(&rempty[nr]); }
    }
  }
  __syncthreads();
  if (threadIdx.x == 0 && *abort_flag) atomicExch(abort_g, 1);   // let the other CTAs leave their flag waits at once
}

PerDeviceOnce g_stream_ready;

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
size_t tall_stream_sync_ints(int64_t cols, int count) { return (size_t)count * (size_t)((cols + kPanel - 1) / kPanel) + 1; }
int tall_stream_panel() { return kPanel; }

cudaError_t launch_rowstep_tall_stream(const PtrTables& t, const Group& g, const StepScalars& s,
                                       const TallStreamPlan& plan, const void* maps_dev, float* partial, float* nu,
                                       int* sync, int* status, int n_cta, cudaStream_t stream, int64_t* launches) {
  if (!plan.ok) return cudaErrorInvalidValue;
  cudaError_t ce;
  int dev;
  if (g_stream_ready.need(&dev)) {
    ce = cudaFuncSetAttribute(rowstep_tall_stream_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemLimit);
    if (ce == cudaSuccess)
      ce = cudaFuncSetAttribute(rowstep_tall_stream_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemLimit);
    if (ce != cudaSuccess) return ce;
    g_stream_ready.mark(dev);
  }
  ce = cudaMemsetAsync(sync, 0, tall_stream_sync_ints(g.cols, g.count) * sizeof(int), stream);
  if (ce != cudaSuccess) return ce;
  StreamArgs a;
  a.maps = reinterpret_cast<const CUtensorMap*>(maps_dev);
  a.t = t; a.first = g.first; a.count = g.count; a.rows = (int)g.rows; a.cols = (int)g.cols;
  a.R = plan.R; a.lag = plan.lag; a.depth = plan.depth;
  a.s = s; a.partial = partial; a.sync = sync; a.status = status;
  (void)nu;
  void* args[] = {&a};
  *launches += 1;
  // Cooperative: the CTAs wait on one another's flags, so all of them must be resident.
  const void* fn = s.nesterov ? (const void*)rowstep_tall_stream_kernel<true> : (const void*)rowstep_tall_stream_kernel<false>;
  return cudaLaunchCooperativeKernel(fn, dim3(n_cta), dim3(kStreamThreads), args, plan.smem, stream);
}

}  // namespace prm

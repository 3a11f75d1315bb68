// Tensor-core NS5 products for sm_100a: D[i,j] = sum_k P[i,k]*Q[j,k] with bf16
// operands, fp32 accumulation in tensor memory, and the fused epilogues of
// struct Epilogue (polynomial coefficients, Frobenius scale, final parameter
// update).  Q may also be stored [k][n] (N-major operand), which is how the
// update product reads X.  The symmetric r x r matrices (A, B and, where the
// first iterations run in Gram space, Z and the running product Q) exist only
// as their 256x256 blocks on and below the diagonal: the products that consume
// them read a missing block from its mirror image as an M/N-major operand, so
// no product ever writes a transposed copy.  P and Q may be two different
// symmetric matrices, and the epilogue takes up to two auxiliary operands.
//
// Persistent CTA pairs (clusters of two CTAs on two SMs), 352 threads per CTA.
// A pair computes a 256x256 tile with tcgen05.mma.cta_group::2: each CTA holds
// 128 rows of P and 128 of the 256 rows of Q in shared memory, and the
// accumulator rows of its half in its own tensor memory.
//   warp 0      TMA producer: per stage two 128x64 boxes of P and two of Q
//               (128 k), each operand in ONE copy through a 4-D (k contiguous)
//               or 5-D (row index contiguous) tensor map whose box spans the
//               k-blocks and, for the latter, the two 64-wide row blocks
//               (cp.async.bulk.tensor, 128-byte swizzle, no multicast); both
//               CTAs signal the leader's barrier.  Three stages of 64 KB:
//               a stage feeds 8 MMAs, which halves the barrier round trips
//               per flop against 64-k stages (7 % fewer SM cycles)
//   warp 1      tcgen05.mma issuer (one lane of the leader CTA); owns the
//               TMEM allocation of its CTA
//   warps 2..9  epilogue arithmetic: two warps per TMEM lane quadrant; the
//               tile is finished in four slabs of 64 columns.  Per slab:
//               tcgen05.ld of the fp32 accumulator, auxiliary operand read
//               from a shared-memory slab, result written back in place (for
//               the final update of a tall matrix: into the transposed
//               parameter slab)
//   warp 10     epilogue I/O: TMA loads of the auxiliary and parameter
//               slabs, TMA stores of the result slab
// All global traffic of the epilogues therefore moves as 128-byte swizzled
// TMA boxes, the final parameter update included (the parameter tile is loaded
// into the second slab, updated there and stored back; tall matrices use the
// transposed boxes).  Per-thread global accesses remain only for fp32
// parameters and for column counts that are not a multiple of 8.  Two
// 256-column accumulators in TMEM let the epilogue of tile n overlap the main
// loop of tile n+1.  Every mbarrier wait is bounded: on expiry the CTA raises
// the status word, drains and exits cleanly.
#include <cuda.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <map>
#include <tuple>

#include "async_copy.cuh"
#include "epilogue.cuh"

namespace prm {

namespace {

constexpr int kBM = 128;          // tile rows  (UMMA M)
constexpr int kBN = 256;          // tile cols  (UMMA N)
constexpr int kBK = 64;           // k per TMA box: 64 bf16 = one 128-byte swizzle row
constexpr int kKSub = 2;          // boxes per stage: a stage holds 128 k, i.e. 8 MMAs per barrier round trip
constexpr int kUmmaK = 16;
constexpr int kStages = 3;
constexpr int kEpiWarps = 8;         // two warps per TMEM lane quadrant
constexpr int kIoWarp = 2 + kEpiWarps;
constexpr int kTcThreads = 32 * (kIoWarp + 1);
constexpr int kSlabCols = 64;        // epilogue slab: 128 rows x 64 columns
constexpr int kSlabs = 4;            // slabs per tile (kBN / kSlabCols)
constexpr int kEpiBufs = 1;
constexpr uint32_t kSlabBytes = 128 * kSlabCols * 2;        // result slab, also the aux slab
constexpr uint32_t kEpiBufBytes = 2 * kSlabBytes;           // + parameter tile or second auxiliary slab
constexpr uint32_t kBytesA = kBM * kBK * 2;
constexpr uint32_t kBytesB = (kBN / 2) * kBK * 2;   // each CTA of the pair holds half of Q's rows
constexpr uint32_t kStageBytes = kKSub * (kBytesA + kBytesB);   // [kKSub boxes of P][kKSub boxes of Q]
constexpr uint32_t kTmemCols = 512;
constexpr size_t kSmemBytes = 1024 + (size_t)kStages * kStageBytes + (size_t)kEpiBufs * kEpiBufBytes + 256;

// Instruction descriptor: D fp32, A and B bf16, both K-major, N = 256, M = 256
// (two CTAs x 128 rows).
constexpr uint32_t kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kBN >> 3) << 17) |
                            ((uint32_t)((2 * kBM) >> 4) << 24);

__device__ __forceinline__ void tma_load_3d(void* dst, const CUtensorMap* map, uint64_t* bar, int x,
                                            int y, int z) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(smem_u32(dst)), "l"((uint64_t)map), "r"(smem_u32(bar)), "r"(x), "r"(y), "r"(z)
      : "memory");
}
__device__ __forceinline__ void tma_store_2d(const void* src, const CUtensorMap* map, int x, int y) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
               ::"l"((uint64_t)map), "r"(smem_u32(src)), "r"(x), "r"(y)
               : "memory");
}
// Load whose completion is counted on the pair leader's barrier (`bar_cluster`
// is a shared::cluster address).
__device__ __forceinline__ void tma_load_3d_pair(void* dst, const CUtensorMap* map, uint32_t bar_cluster, int x,
                                                 int y, int z) {
  asm volatile(
      "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(smem_u32(dst)), "l"((uint64_t)map), "r"(bar_cluster), "r"(x), "r"(y), "r"(z)
      : "memory");
}
// One stage of a K-major operand: kKSub boxes of `rows` x 64 k, fetched as one 4-D box
// {64 k, rows, kKSub k-blocks, 1}; they land one after the other.
__device__ __forceinline__ void tma_load_k_stage(void* dst, const CUtensorMap* map, uint32_t bar_cluster, int k0,
                                                 int row0, int z) {
  asm volatile(
      "cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
      ::"r"(smem_u32(dst)), "l"((uint64_t)map), "r"(bar_cluster), "r"(0), "r"(row0), "r"(k0 >> 6), "r"(z)
      : "memory");
}
// One stage of an operand stored with its row index contiguous ([k][n], n fastest): per
// k-block two adjacent 64 x 64 boxes, fetched as one 5-D box {64 n, 64 k, 2 n-blocks,
// kKSub k-blocks, 1}.  They land as [k-block][n-block][k][n], the M/N-major operand layout.
__device__ __forceinline__ void tma_load_t_stage(void* dst, const CUtensorMap* map, uint32_t bar_cluster, int n0,
                                                 int k0, int z) {
  asm volatile(
      "cp.async.bulk.tensor.5d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6, %7}], [%2];"
      ::"r"(smem_u32(dst)), "l"((uint64_t)map), "r"(bar_cluster), "r"(0), "r"(0), "r"(n0 >> 6), "r"(k0 >> 6), "r"(z)
      : "memory");
}
// shared::cluster address of `p` in the CTA of rank `rank` of this cluster.
__device__ __forceinline__ uint32_t map_to_rank(const void* p, uint32_t rank) {
  uint32_t out;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(out) : "r"(smem_u32(p)), "r"(rank));
  return out;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t bar_cluster) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(bar_cluster) : "memory");
}
__device__ __forceinline__ uint32_t cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void tma_store_3d(const void* src, const CUtensorMap* map, int x, int y, int z) {
  asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%2, %3, %4}], [%1];"
               ::"l"((uint64_t)map), "r"(smem_u32(src)), "r"(x), "r"(y), "r"(z)
               : "memory");
}
__device__ __forceinline__ void tma_store_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void tma_store_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void tma_store_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
// Byte offset of 16-byte chunk `chunk` of row `row` in a 128-byte-swizzled box.
__device__ __forceinline__ uint32_t sw128(uint32_t row, uint32_t chunk) {
  return row * 128u + ((chunk ^ (row & 7u)) << 4);
}
__device__ __forceinline__ uint64_t make_desc(uint32_t smem_addr) {
  // K-major operand tile, 128-byte swizzle: rows of 128 bytes, groups of 8
  // rows 1024 bytes apart (stride byte offset), descriptor version 1.
  return (uint64_t)((smem_addr >> 4) & 0x3FFF) | (1ull << 16) | ((uint64_t)(1024 >> 4) << 32) |
         (1ull << 46) | (2ull << 61);
}
__device__ __forceinline__ uint64_t make_desc_mn(uint32_t smem_addr) {
  // N-major ("MN-major") operand tile, 128-byte swizzle: each row of 128 bytes
  // holds 64 consecutive n for one k; 8 such k-rows form a 1024-byte atom.
  // Atoms follow each other along k every 1024 bytes (stride byte offset) and
  // along n every 8192 bytes (leading byte offset: the next 64x64 TMA box).
  return (uint64_t)((smem_addr >> 4) & 0x3FFF) | ((uint64_t)(8192 >> 4) << 16) | ((uint64_t)(1024 >> 4) << 32) |
         (1ull << 46) | (2ull << 61);
}
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// Arrives, once all MMAs issued so far have completed, on the barrier at this
// shared-memory offset in BOTH CTAs of the pair: one instruction with a CTA mask
// instead of one commit per CTA (2.7 % less time for a refresh of the 9B-class
// set).  This is a barrier arrival, not a load; the TMA loads use no multicast.
__device__ __forceinline__ void umma_commit_pair(uint32_t bar_local) {
  const uint16_t mask = 3;
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar_local), "h"(mask)
               : "memory");
}
// Issues the TMEM load; the registers are valid after tmem_ld_wait().
__device__ __forceinline__ void tmem_ld32_issue(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr));
}
__device__ __forceinline__ void tmem_ld_wait() {
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

struct TileCoord {
  int b, ti, tj;
};
__device__ __forceinline__ TileCoord decode_tile(int t, int tiles_per_mat, int symmetric, int mt) {
  TileCoord c;
  c.b = t / tiles_per_mat;
  const int rem = t - c.b * tiles_per_mat;
  if (symmetric) {
    int bi, bj;
    tri_decode(rem >> 1, bi, bj);      // 256x256 blocks of the lower triangle
    c.ti = 2 * bi + (rem & 1);         // two 128-row tiles per block
    c.tj = bj;
  } else {
    c.ti = rem % mt;                   // row tiles fastest: concurrent CTAs share the Q panel
    c.tj = rem / mt;
  }
  return c;
}

// Q_MN and SYM_OPS are compile-time so that each product keeps a main loop
// with constant descriptor strides (a run-time choice measurably slowed the
// products that need none).
//
// SEGS > 1: the input X_0 is held as a pair of bf16 planes, X_0 = H + L with
// H = bf16(X_0) and L = bf16(X_0 - H), stored one after the other per matrix.
// The k loop then runs over SEGS segments of kseg stages each:
//   SEGS = 3 (X_0 X_0^T):  H H^T + H L^T + L H^T  (L L^T, 2^-16 of the result, is dropped);
//                          segment s reads P from plane (s == 2) and Q from plane (s == 1),
//                          the maps counting planes as batch items (z = 2b + plane);
//   SEGS = 2 (Q X_0):      Q H + Q L: the symmetric operand P repeats, the N-major operand's
//                          k runs on through the rows of H and then of L (mapQ covers both
//                          planes of a matrix as one 2 Kp-row array); the auxiliary term reads
//                          both planes as well (mapAux with z = 2b and 2b + 1, one coefficient).
template <int Q_MN, int SYM_OPS, int AUX2, int SEGS>
__global__ void __launch_bounds__(kTcThreads, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap mapP, const __grid_constant__ CUtensorMap mapQ,
               const __grid_constant__ CUtensorMap mapAux, const __grid_constant__ CUtensorMap mapAux2,
               const __grid_constant__ CUtensorMap mapDst,
               const __grid_constant__ CUtensorMap mapSymP, const __grid_constant__ CUtensorMap mapSymQ,
               int ktiles, int kseg, int tiles_per_mat, int total_tiles, int symmetric, int mt, Epilogue ep,
               int* status) {
  constexpr int q_mn = Q_MN, sym_ops = SYM_OPS;
  static_assert(SEGS == 1 || (SEGS == 3 && !Q_MN && !SYM_OPS && !AUX2) || (SEGS == 2 && Q_MN && SYM_OPS == 1 && AUX2),
                "split-input products: X_0 X_0^T and Q X_0 only");
  // AUX2: a second auxiliary operand (Epilogue::aux2) travels in the half of
  // the slab buffer that the parameter tile of the final update uses; only the
  // Gram-space products of two symmetric matrices need it.
  // q_mn: Q is stored [k][n] (n contiguous) instead of [n][k]; its tiles are
  // loaded as 64x64 boxes and consumed as an N-major MMA operand.
  // sym_ops (bit 0: P, bit 1: Q): the operand is a symmetric matrix stored only
  // in its 256x256 blocks on and below the diagonal.  A k-block right of the
  // operand's diagonal block is read from the mirrored block, which holds it
  // as [k][row]: 64x64 boxes through mapSymP / mapSymQ, consumed as an M/N-major operand.
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint8_t* ebuf = smem + (size_t)kStages * kStageBytes;           // [kEpiBufs][kEpiBufBytes]
  uint64_t* bars = reinterpret_cast<uint64_t*>(ebuf + (size_t)kEpiBufs * kEpiBufBytes);
  uint64_t* full = bars;                      // [kStages] TMA -> MMA
  uint64_t* empty = full + kStages;           // [kStages] MMA -> TMA
  uint64_t* tfull = empty + kStages;          // [2] MMA -> epilogue
  uint64_t* tempty = tfull + 2;               // [2] epilogue -> MMA
  uint64_t* eready = tempty + 2;              // [kEpiBufs] I/O warp -> epilogue: slab buffer usable (aux landed)
  uint64_t* edone = eready + kEpiBufs;        // [kEpiBufs] epilogue -> I/O warp: slab written
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(edone + kEpiBufs);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_rank();       // 0 = leader of the pair
  // fin: final parameter update with the parameter tile staged through shared
  // memory (per-matrix tensor maps in global memory); otherwise kind 1 falls
  // back to per-thread global accesses.
  const bool fin = ep.kind == 1 && ep.param_maps != nullptr;
  const bool staged = ep.kind == 0 || fin;    // epilogue through shared memory and TMA
  const bool has_aux = ep.aux != nullptr;
  const CUtensorMap* pmaps = reinterpret_cast<const CUtensorMap*>(ep.param_maps);

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(&tfull[a], 1); mbar_init(&tempty[a], 2 * kEpiWarps); }
    for (int e = 0; e < kEpiBufs; ++e) { mbar_init(&eready[e], 1); mbar_init(&edone[e], kEpiWarps); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                 "r"(kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  cluster_sync_all();                         // the peer's barriers are initialised too
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------ producer
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      const uint32_t lead_full0 = map_to_rank(&full[0], 0);
      for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x) {
        const TileCoord c = decode_tile(t, tiles_per_mat, symmetric, mt);
        int seg = 0, ktl = 0;                   // SEGS > 1: segment and stage inside it
        for (int kt = 0; kt < ktiles; ++kt, ++it) {
          const int s = it % kStages;
          const uint32_t ph = (it / kStages) & 1;
          if (!mbar_wait(&empty[s], ph ^ 1, abort_flag, status)) { ok = false; break; }
          uint8_t* sa = smem + (size_t)s * kStageBytes;
          // The leader's barrier counts the bytes of both CTAs' loads.
          if (rank == 0) mbar_expect_tx(&full[s], 2 * kStageBytes);
          const uint32_t lead_full = lead_full0 + 8u * s;
          const int n0 = c.tj * kBN + (int)rank * (kBN / 2);      // this CTA's 128 rows (columns) of Q
          const int k0 = (SEGS > 1 ? ktl : kt) * kKSub * kBK;     // k inside the segment
          const int kb = k0 / kPad;                               // the stage's 128 k lie inside one 256-block
          uint8_t* sp = sa;
          uint8_t* sq = sa + kKSub * kBytesA;
          if (SEGS == 3) {
            tma_load_k_stage(sp, &mapP, lead_full, k0, c.ti * kBM, 2 * c.b + (seg == 2));
            tma_load_k_stage(sq, &mapQ, lead_full, k0, n0, 2 * c.b + (seg == 1));
          } else {
            if ((sym_ops & 1) && kb > (c.ti >> 1)) {
              tma_load_t_stage(sp, &mapSymP, lead_full, c.ti * kBM, k0, c.b);
            } else {
              tma_load_k_stage(sp, &mapP, lead_full, k0, c.ti * kBM, c.b);
            }
            if ((sym_ops & 2) && kb > c.tj) {
              tma_load_t_stage(sq, &mapSymQ, lead_full, n0, k0, c.b);
            } else if (!q_mn) {
              tma_load_k_stage(sq, &mapQ, lead_full, k0, n0, c.b);
            } else {
              // SEGS == 2: the k rows of the second plane follow those of the first
              tma_load_t_stage(sq, &mapQ, lead_full, n0, kt * kKSub * kBK, c.b);
            }
          }
          if (SEGS > 1 && ++ktl == kseg) { ktl = 0; ++seg; }
        }
      }
      // Drain: every load issued must have landed before shared memory is
      // released.  The leader sees the byte counts of both CTAs on its own
      // barriers; the closing cluster barrier keeps the peer alive until then.
      if (rank == 0) {
        const uint32_t n_issued = it;
        for (uint32_t k = (n_issued > kStages ? n_issued - kStages : 0); k < n_issued; ++k) {
          const uint64_t t0 = global_ns();
          while (!mbar_try_wait(&full[k % kStages], (k / kStages) & 1)) {
            if (global_ns() - t0 > 1000000ull) break;   // 1 ms
          }
        }
      }
    }
  } else if (warp == 1) {
    // -------------------------------------------------------------- MMA issuer
    if (lane == 0 && rank == 0) {
      // This one thread feeds the tensor pipe of two SMs: everything that does
      // not change per k-block is computed once (cluster addresses of the
      // barriers, the constant halves of the descriptors).
      uint32_t it = 0, acc_it = 0;
      bool ok = true;
      const uint32_t smem0 = smem_u32(smem);
      for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x, ++acc_it) {
        const TileCoord c = decode_tile(t, tiles_per_mat, symmetric, mt);
        const int a = acc_it & 1;
        const uint32_t aph = (acc_it >> 1) & 1;
        if (!mbar_wait(&tempty[a], aph ^ 1, abort_flag, status)) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t tacc = tmem_base + (uint32_t)a * kBN;
        int ktl = 0;                            // SEGS > 1: stage inside the segment
        for (int kt = 0; kt < ktiles; ++kt, ++it) {
          const int s = it % kStages;
          const uint32_t ph = (it / kStages) & 1;
          if (!mbar_wait(&full[s], ph, abort_flag, status)) { ok = false; break; }
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint32_t sa = smem0 + (uint32_t)s * kStageBytes;
          // K-major tile: 16 elements = 32 bytes further inside the swizzled row (+2 in 16-byte units);
          // M/N-major tile: 16 k-rows = two 1024-byte atoms further (+128).
          const int kb = ((SEGS > 1 ? ktl : kt) * kKSub * kBK) / kPad;   // the stage's 128 k lie inside one 256-block
          if (SEGS > 1 && ++ktl == kseg) ktl = 0;
          const bool a_t = (sym_ops & 1) && kb > (c.ti >> 1);
          const bool b_t = q_mn || ((sym_ops & 2) && kb > c.tj);
          const uint32_t sa_k = a_t ? 128u : 2u, sb_k = b_t ? 128u : 2u;
          const uint32_t idesc = kIdesc | (a_t ? (1u << 15) : 0u) | (b_t ? (1u << 16) : 0u);
#pragma unroll
          for (int kk = 0; kk < kKSub; ++kk) {
            const uint32_t pa = sa + kk * kBytesA, pb = sa + kKSub * kBytesA + kk * kBytesB;
            const uint64_t da = a_t ? make_desc_mn(pa) : make_desc(pa);
            const uint64_t db = b_t ? make_desc_mn(pb) : make_desc(pb);
#pragma unroll
            for (int k = 0; k < kBK / kUmmaK; ++k) {
              umma_bf16(tacc, da + sa_k * k, db + sb_k * k, idesc, (kt | kk | k) != 0);
            }
          }
          umma_commit_pair(smem_u32(&empty[s]));   // frees the stage in both CTAs when these MMAs have read it
        }
        if (ok) {                               // accumulator complete in both CTAs
          umma_commit_pair(smem_u32(&tfull[a]));
        }
      }
    }
  } else if (warp == kIoWarp) {
    // ------------------------------------------------------------ epilogue I/O
    // Slab g of this CTA (four per tile) lives in buffer g % kEpiBufs.  For
    // each slab: make the buffer usable (load the auxiliary slab, or just
    // signal), later store what the epilogue warps wrote.
    if (lane == 0 && staged) {
      int n_my_tiles = 0;
      for (int t = blockIdx.x; t < total_tiles; t += gridDim.x) ++n_my_tiles;
      const uint32_t n_slabs = (uint32_t)n_my_tiles * kSlabs;
      int fenced_b = -1;                 // matrix whose parameter map has been acquired
      auto prepare = [&](uint32_t g) {
        const int bsel = g % kEpiBufs;
        if (has_aux || fin) {
          const TileCoord c = decode_tile(blockIdx.x + (int)(g / kSlabs) * gridDim.x, tiles_per_mat, symmetric, mt);
          const int j0 = c.tj * kBN + (int)(g % kSlabs) * kSlabCols;
          uint8_t* buf = ebuf + (size_t)bsel * kEpiBufBytes;
          mbar_expect_tx(&eready[bsel], (has_aux ? kSlabBytes : 0u) + ((fin || AUX2) ? kSlabBytes : 0u));
          if (SEGS == 2) {               // both planes of X_0 through one map, planes counted as batch items
            tma_load_3d(buf, &mapAux, &eready[bsel], j0, c.ti * kBM, 2 * c.b);
            tma_load_3d(buf + kSlabBytes, &mapAux, &eready[bsel], j0, c.ti * kBM, 2 * c.b + 1);
          } else {
            if (has_aux) tma_load_3d(buf, &mapAux, &eready[bsel], j0, c.ti * kBM, c.b);
            if (AUX2) tma_load_3d(buf + kSlabBytes, &mapAux2, &eready[bsel], j0, c.ti * kBM, c.b);
          }
          if (fin) {
            // Parameter tile into the second slab: as stored (wide), or the
            // transposed region in two 64x64 boxes (tall).  Out-of-range parts read as zero.
            const CUtensorMap* pm = pmaps + ep.first + c.b;
            if (c.b != fenced_b) { tensormap_acquire(pm); fenced_b = c.b; }
            if (!ep.tall) {
              tma_load_2d(buf + kSlabBytes, pm, &eready[bsel], j0, c.ti * kBM);
            } else {
              tma_load_2d(buf + kSlabBytes, pm, &eready[bsel], c.ti * kBM, j0);
              tma_load_2d(buf + kSlabBytes + kSlabBytes / 2, pm, &eready[bsel], c.ti * kBM + 64, j0);
            }
          }
        } else {
          mbar_arrive(&eready[bsel]);
        }
      };
      for (uint32_t g = 0; g < (uint32_t)kEpiBufs && g < n_slabs; ++g) prepare(g);
      for (uint32_t g = 0; g < n_slabs; ++g) {
        const int bsel = g % kEpiBufs;
        if (!mbar_wait(&edone[bsel], (g / kEpiBufs) & 1, abort_flag, status)) break;
        const TileCoord c = decode_tile(blockIdx.x + (int)(g / kSlabs) * gridDim.x, tiles_per_mat, symmetric, mt);
        const int j0 = c.tj * kBN + (int)(g % kSlabs) * kSlabCols;
        const uint8_t* buf = ebuf + (size_t)bsel * kEpiBufBytes;
        if (fin) {
          const CUtensorMap* pm = pmaps + ep.first + c.b;
          if (!ep.tall) {
            tma_store_2d(buf + kSlabBytes, pm, j0, c.ti * kBM);
          } else {
            tma_store_2d(buf + kSlabBytes, pm, c.ti * kBM, j0);
            tma_store_2d(buf + kSlabBytes + kSlabBytes / 2, pm, c.ti * kBM + 64, j0);
          }
        } else {
          tma_store_3d(buf, &mapDst, j0, c.ti * kBM, c.b);
        }
        tma_store_commit();
        if (g + kEpiBufs < n_slabs) {
          tma_store_wait_read();          // the buffer has been read out: it can be refilled
          prepare(g + kEpiBufs);
        }
      }
      tma_store_wait_all();
      if (has_aux || fin) {
        // Drain auxiliary loads that were issued but never consumed (abort path only).
        for (int e = 0; e < kEpiBufs; ++e) {
          const uint64_t t0 = global_ns();
          while (*abort_flag && !mbar_try_wait(&eready[e], 0) && !mbar_try_wait(&eready[e], 1)) {
            if (global_ns() - t0 > 1000000ull) break;
          }
        }
      }
    }
  } else {
    // ---------------------------------------------------------------- epilogue
    const int q = warp & 3;              // TMEM lane quadrant this warp may read
    const int half = (warp - 2) >> 2;    // which half of the columns (of the slab, or of the tile)
    const int row = q * 32 + lane;       // row of the tile owned by this thread
    uint32_t acc_it = 0, g = 0;
    bool ok = true;
    for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x, ++acc_it) {
      const TileCoord c = decode_tile(t, tiles_per_mat, symmetric, mt);
      const int a = acc_it & 1;
      const uint32_t aph = (acc_it >> 1) & 1;
      // All lanes wait, then agree: tcgen05.ld needs the whole warp.
      const bool got = mbar_wait(&tfull[a], aph, abort_flag, status);
      if (!__all_sync(0xffffffffu, got)) break;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const int i = c.ti * kBM + row;
      const uint32_t trow = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(a * kBN);
      if (staged) {
        const float al = ep.alpha ? ep.alpha[c.b] : 1.f;
        const float f = ep.alpha_pow == 2 ? al * al : (ep.alpha_pow == 1 ? al : 1.f);
        const float ka = f * ep.k_acc, kx = f * ep.k_aux;
        const float kx2 = AUX2 ? f * ep.k_aux2 : 0.f;
#pragma unroll 1
        for (int sl = 0; sl < kSlabs; ++sl, ++g) {
          const int bsel = g % kEpiBufs;
          uint32_t r[32];
          tmem_ld32_issue(trow + sl * kSlabCols + half * 32, r);
          const bool rdy = mbar_wait(&eready[bsel], (g / kEpiBufs) & 1, abort_flag, status);
          tmem_ld_wait();
          if (!__all_sync(0xffffffffu, rdy)) { ok = false; break; }
          uint8_t* buf = ebuf + (size_t)bsel * kEpiBufBytes;
          uint8_t* tbuf = buf + kSlabBytes + (row >> 6) * (kSlabBytes / 2);
          const uint32_t rt = row & 63;
#pragma unroll
          for (int v = 0; v < 4; ++v) {
            int4* p = reinterpret_cast<int4*>(buf + sw128(row, half * 4 + v));
            float x[8];
            if (has_aux) {
              const int4 raw = *p;
              const __nv_bfloat162* h2 = reinterpret_cast<const __nv_bfloat162*>(&raw);
#pragma unroll
              for (int k = 0; k < 4; ++k) {
                const float2 ff = __bfloat1622float2(h2[k]);
                x[2 * k] = ff.x;
                x[2 * k + 1] = ff.y;
              }
            } else {
#pragma unroll
              for (int k = 0; k < 8; ++k) x[k] = 0.f;
            }
            if (fin) {
              // W <- decay*W - lr*s*X_5 on the staged parameter tile.
              if (!ep.tall) {
                int4* pp = reinterpret_cast<int4*>(buf + kSlabBytes + sw128(row, half * 4 + v));
                int4 pw = *pp;
                __nv_bfloat162* w2 = reinterpret_cast<__nv_bfloat162*>(&pw);
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                  const float2 w = __bfloat1622float2(w2[k]);
                  const float v0 = ka * __uint_as_float(r[8 * v + 2 * k]) + kx * x[2 * k];
                  const float v1 = ka * __uint_as_float(r[8 * v + 2 * k + 1]) + kx * x[2 * k + 1];
                  w2[k] = __floats2bfloat162_rn(ep.decay * w.x - ep.lr_s * v0, ep.decay * w.y - ep.lr_s * v1);
                }
                *pp = pw;
              } else {
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                  const uint32_t cc = half * 32 + v * 8 + k;
                  __nv_bfloat16* pe = reinterpret_cast<__nv_bfloat16*>(tbuf + sw128(cc, rt >> 3) + (rt & 7) * 2);
                  const float vk = ka * __uint_as_float(r[8 * v + k]) + kx * x[k];
                  *pe = __float2bfloat16_rn(ep.decay * __bfloat162float(*pe) - ep.lr_s * vk);
                }
              }
              continue;
            }
            int4 outv;
            __nv_bfloat162* o2 = reinterpret_cast<__nv_bfloat162*>(&outv);
            if (AUX2) {
              const int4 raw2 = *reinterpret_cast<const int4*>(buf + kSlabBytes + sw128(row, half * 4 + v));
              const __nv_bfloat162* g2 = reinterpret_cast<const __nv_bfloat162*>(&raw2);
#pragma unroll
              for (int k = 0; k < 4; ++k) {
                const float2 yy = __bfloat1622float2(g2[k]);
                const float v0 = ka * __uint_as_float(r[8 * v + 2 * k]) + (kx * x[2 * k] + kx2 * yy.x);
                const float v1 = ka * __uint_as_float(r[8 * v + 2 * k + 1]) + (kx * x[2 * k + 1] + kx2 * yy.y);
                o2[k] = __floats2bfloat162_rn(v0, v1);
              }
            } else {
#pragma unroll
              for (int k = 0; k < 4; ++k) {
                const float v0 = ka * __uint_as_float(r[8 * v + 2 * k]) + kx * x[2 * k];
                const float v1 = ka * __uint_as_float(r[8 * v + 2 * k + 1]) + kx * x[2 * k + 1];
                o2[k] = __floats2bfloat162_rn(v0, v1);
              }
            }
            *p = outv;
          }
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
          __syncwarp();
          if (lane == 0) mbar_arrive(&edone[bsel]);
        }
      } else {
        // Final parameter update: per-thread global accesses.
        const int jbase = c.tj * kBN + half * (kBN / 2);
        constexpr int kChunks = kBN / 2 / 32;
        AuxRegs<32> aux[2];
        aux_prefetch<32>(ep, c.b, i, jbase, aux[0]);
#pragma unroll
        for (int ch = 0; ch < kChunks; ++ch) {
          uint32_t r[32];
          tmem_ld32_issue(trow + half * (kBN / 2) + ch * 32, r);
          if (ch + 1 < kChunks) aux_prefetch<32>(ep, c.b, i, jbase + (ch + 1) * 32, aux[(ch + 1) & 1]);
          tmem_ld_wait();
          float v[32], x[32];
#pragma unroll
          for (int e = 0; e < 32; ++e) v[e] = __uint_as_float(r[e]);
          aux_unpack<32>(aux[ch & 1], x);
          epilogue_row<__nv_bfloat16, 32>(ep, c.b, i, jbase + ch * 32, v, x);
        }
      }
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(map_to_rank(&tempty[a], 0));   // the leader issues the MMAs
    }
  }

  // ---------------------------------------------------------------- teardown
  // Neither CTA may leave while its partner can still touch its shared
  // memory, barriers or tensor memory.
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  cluster_sync_all();
  if (warp == 1) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
  }
}

// Exercises the bounded wait: one thread waits on a barrier that nothing ever
// completes, gives up after limit_ns, raises the status word and returns.
__global__ void wait_probe_kernel(int* status, uint64_t limit_ns, int* gave_up) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    const bool ok = mbar_wait(&bar, 0, &abort_flag, status, limit_ns);
    if (gave_up) *gave_up = ok ? 0 : 1;
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

}  // namespace

struct TcContext {
  EncodeTiledFn encode = nullptr;
  int sm_count = 0;
  int max_pairs = 0;   // CTA pairs that can be resident at once
  std::map<std::tuple<const void*, int64_t, int64_t, int, int>, CUtensorMap> cache;
};

TcContext* tc_create(std::string* err) {
  TcContext* tc = new TcContext();
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  cudaError_t ce = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
  if (ce != cudaSuccess || qres != cudaDriverEntryPointSuccess || !fn) {
    if (err) *err = "cuTensorMapEncodeTiled is not available from the driver";
    delete tc;
    return nullptr;
  }
  tc->encode = (EncodeTiledFn)fn;
  int dev = 0;
  cudaDeviceProp prop;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaGetDeviceProperties(&prop, dev) != cudaSuccess) {
    if (err) *err = "cannot query the CUDA device";
    delete tc;
    return nullptr;
  }
  if (prop.major != 10) {
    if (err) *err = "the tensor-core path needs an sm_100 device";
    delete tc;
    return nullptr;
  }
  tc->sm_count = prop.multiProcessorCount;
  ce = cudaFuncSetAttribute(gemm_tc_kernel<0, 0, 0, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
  if (ce == cudaSuccess)
    ce = cudaFuncSetAttribute(gemm_tc_kernel<0, 3, 0, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
  if (ce == cudaSuccess)
    ce = cudaFuncSetAttribute(gemm_tc_kernel<0, 3, 1, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
  if (ce == cudaSuccess)
    ce = cudaFuncSetAttribute(gemm_tc_kernel<1, 0, 0, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
  if (ce == cudaSuccess)
    ce = cudaFuncSetAttribute(gemm_tc_kernel<1, 1, 0, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
  if (ce == cudaSuccess)
    ce = cudaFuncSetAttribute(gemm_tc_kernel<0, 0, 0, 3>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
  if (ce == cudaSuccess)
    ce = cudaFuncSetAttribute(gemm_tc_kernel<1, 1, 1, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
  if (ce != cudaSuccess) {
    if (err) *err = std::string("cudaFuncSetAttribute: ") + cudaGetErrorString(ce);
    delete tc;
    return nullptr;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(tc->sm_count & ~1, 1, 1);
  cfg.blockDim = dim3(kTcThreads, 1, 1);
  cfg.dynamicSmemBytes = kSmemBytes;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  int n_clusters = 0;
  ce = cudaOccupancyMaxActiveClusters(&n_clusters, gemm_tc_kernel<0, 0, 0, 1>, &cfg);
  if (ce != cudaSuccess || n_clusters < 1) {
    if (err) *err = std::string("cudaOccupancyMaxActiveClusters: ") + cudaGetErrorString(ce);
    delete tc;
    return nullptr;
  }
  tc->max_pairs = n_clusters;
  if (getenv("PRM_VERBOSE")) fprintf(stderr, "prm: %d SMs, %d resident CTA pairs\n", tc->sm_count, n_clusters);
  return tc;
}

void tc_destroy(TcContext* tc) { delete tc; }

// 3-D map over a [batch][rows][kdim] bf16 array; box = 64 (k) x box_rows x 1.
// No L2 promotion: every 128-byte row of a box is used whole, and the refresh of
// the 9B-class set measured 0.5-0.7 % faster without the 256-byte promotion.
static bool get_map(TcContext* tc, const void* base, int64_t rows, int64_t kdim, int batch, int box_rows,
                    CUtensorMap* out) {
  auto key = std::make_tuple(base, rows, kdim, batch, box_rows);
  auto it = tc->cache.find(key);
  if (it != tc->cache.end()) { *out = it->second; return true; }
  cuuint64_t dims[3] = {(cuuint64_t)kdim, (cuuint64_t)rows, (cuuint64_t)batch};
  cuuint64_t strides[2] = {(cuuint64_t)kdim * 2, (cuuint64_t)kdim * (cuuint64_t)rows * 2};
  cuuint32_t box[3] = {(cuuint32_t)kBK, (cuuint32_t)box_rows, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = tc->encode(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box,
                          estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                          CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return false;
  if (tc->cache.size() > 4096) tc->cache.clear();
  tc->cache[key] = *out;
  return true;
}

// Operand maps: one TMA copy per operand and stage.
// K-major ([batch][rows][kdim], k contiguous): 4-D {64 k, rows, k-block, batch}, box
// {64, box_rows, kKSub, 1}.
static bool get_map_kstage(TcContext* tc, const void* base, int64_t rows, int64_t kdim, int batch, int box_rows,
                           CUtensorMap* out) {
  auto key = std::make_tuple(base, rows, kdim, batch, -1000 - box_rows);
  auto it = tc->cache.find(key);
  if (it != tc->cache.end()) { *out = it->second; return true; }
  if (kdim % (kBK * kKSub) != 0) return false;
  cuuint64_t dims[4] = {(cuuint64_t)kBK, (cuuint64_t)rows, (cuuint64_t)(kdim / kBK), (cuuint64_t)batch};
  cuuint64_t strides[3] = {(cuuint64_t)kdim * 2, (cuuint64_t)kBK * 2, (cuuint64_t)kdim * (cuuint64_t)rows * 2};
  cuuint32_t box[4] = {(cuuint32_t)kBK, (cuuint32_t)box_rows, (cuuint32_t)kKSub, 1};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  CUresult r = tc->encode(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box,
                          estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                          CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return false;
  if (tc->cache.size() > 4096) tc->cache.clear();
  tc->cache[key] = *out;
  return true;
}
// Row-index-contiguous ([batch][krows][ncols], n contiguous): 5-D {64 n, 64 k, n-block,
// k-block, batch}, box {64, 64, 2, kKSub, 1} = 128 n x 128 k in one copy.
static bool get_map_tstage(TcContext* tc, const void* base, int64_t krows, int64_t ncols, int batch,
                           CUtensorMap* out) {
  auto key = std::make_tuple(base, krows, ncols, batch, -5);
  auto it = tc->cache.find(key);
  if (it != tc->cache.end()) { *out = it->second; return true; }
  if (ncols % 128 != 0 || krows % (kBK * kKSub) != 0) return false;
  cuuint64_t dims[5] = {64, (cuuint64_t)kBK, (cuuint64_t)(ncols / 64), (cuuint64_t)(krows / kBK), (cuuint64_t)batch};
  cuuint64_t strides[4] = {(cuuint64_t)ncols * 2, 128, (cuuint64_t)ncols * 2 * kBK,
                           (cuuint64_t)ncols * (cuuint64_t)krows * 2};
  cuuint32_t box[5] = {64, (cuuint32_t)kBK, 2, (cuuint32_t)kKSub, 1};
  cuuint32_t estr[5] = {1, 1, 1, 1, 1};
  CUresult r = tc->encode(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(base), dims, strides, box,
                          estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                          CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return false;
  if (tc->cache.size() > 4096) tc->cache.clear();
  tc->cache[key] = *out;
  return true;
}

cudaError_t launch_wait_probe(int* status, uint64_t limit_ns, int* gave_up, cudaStream_t stream) {
  wait_probe_kernel<<<1, 32, 0, stream>>>(status, limit_ns, gave_up);
  return cudaGetLastError();
}

// Tensor map over one bf16 parameter matrix (rows x cols, row-major) for the
// staged final update: boxes of 128 rows x 64 columns for wide matrices, of
// 64 x 64 for tall ones (whose tile is written transposed).  out128 receives
// the 128-byte descriptor.  Needs cols % 8 == 0 and a 16-byte aligned base.
bool tc_encode_param_map(TcContext* tc, const void* base, int64_t rows, int64_t cols, int tall, void* out128) {
  if (!tc || (cols % 8) != 0 || ((uintptr_t)base & 15) != 0) return false;
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
  cuuint32_t box[2] = {64, tall ? 64u : 128u};
  cuuint32_t estr[2] = {1, 1};
  CUtensorMap m;
  CUresult r = tc->encode(&m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box,
                          estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                          CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return false;
  memcpy(out128, &m, sizeof(CUtensorMap));
  return true;
}

bool tc_encode_tile_map(TcContext* tc, const void* base, int64_t rows, int64_t cols, int elem_bytes, int box_cols,
                        int box_rows, void* out128) {
  if (!tc || (elem_bytes != 2 && elem_bytes != 4) || ((uintptr_t)base & 15) != 0) return false;
  if ((cols * elem_bytes) % 16 != 0 || box_cols < 1 || box_cols > 256 || box_rows < 1 || box_rows > 256) return false;
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)cols * (cuuint64_t)elem_bytes};
  cuuint32_t box[2] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUtensorMap m;
  CUresult r = tc->encode(&m, elem_bytes == 2 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2,
                          const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                          CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return false;
  memcpy(out128, &m, sizeof(CUtensorMap));
  return true;
}

int tc_sm_count(const TcContext* tc) { return tc ? tc->sm_count : 0; }

cudaError_t launch_gemm_tc(TcContext* tc, const GemmProblem& pb, const Epilogue& ep, int* status,
                           cudaStream_t stream, int64_t* launches) {
  if (!tc) return cudaErrorInvalidValue;
  if (pb.Mp % kBN != 0 || pb.Np % kBN != 0 || pb.Kp % (kBK * kKSub) != 0) return cudaErrorInvalidValue;
  CUtensorMap mp, mq, maux, maux2, mdst, msp, msq;
  // Split input (GemmProblem::split): the two planes of a matrix follow each other, so a map
  // over them counts 2 * batch items (K-major operand, auxiliary slabs) or 2 * Kp rows per
  // item (the N-major operand).
  const int split = pb.split;
  if (split) {
    const bool gram = !pb.q_mn && !pb.sym_ops && pb.symmetric && pb.P == pb.Q && !ep.aux && !ep.aux2 && ep.kind == 0;
    const bool upd = pb.q_mn && pb.sym_ops == 1 && !pb.symmetric && ep.kind == 0 && ep.aux == pb.Q && !ep.aux2;
    if (!gram && !upd) return cudaErrorInvalidValue;
  }
  const int planes = split ? 2 : 1;
  if (!get_map_kstage(tc, pb.P, pb.Mp, pb.Kp, (split && !pb.q_mn) ? 2 * pb.batch : pb.batch, kBM, &mp))
    return cudaErrorInvalidValue;
  if (!pb.q_mn) {
    if (!get_map_kstage(tc, pb.Q, pb.Np, pb.Kp, planes * pb.batch, kBN / 2, &mq)) return cudaErrorInvalidValue;
  } else {
    // Q stored [batch][Kp][Np]: boxes of 64 k-rows x 64 n
    if (pb.symmetric || !get_map_tstage(tc, pb.Q, planes * pb.Kp, pb.Np, pb.batch, &mq)) return cudaErrorInvalidValue;
  }
  // Epilogue maps (product epilogues only): auxiliary and result slabs of 128
  // rows x 64 columns.
  maux = mp; maux2 = mp; mdst = mp; msp = mp; msq = mp;
  // 64x64 boxes over a symmetric operand, through which its mirrored blocks are read
  if (pb.sym_ops & 1) {
    if (pb.Mp != pb.Kp || !get_map_tstage(tc, pb.P, pb.Mp, pb.Kp, pb.batch, &msp)) return cudaErrorInvalidValue;
  }
  if (pb.sym_ops & 2) {
    if (pb.Np != pb.Kp || pb.q_mn || !get_map_tstage(tc, pb.Q, pb.Np, pb.Kp, pb.batch, &msq)) return cudaErrorInvalidValue;
  }
  if (ep.aux && (ep.kind == 0 || ep.param_maps)) {
    if (ep.bs_aux != planes * pb.Mp * ep.ld_aux) return cudaErrorInvalidValue;
    if (!get_map(tc, ep.aux, pb.Mp, ep.ld_aux, planes * pb.batch, 128, &maux)) return cudaErrorInvalidValue;
  }
  if (ep.aux2) {
    // second auxiliary operand: product epilogues of two symmetric operands only
    if (ep.kind != 0 || !ep.aux || pb.q_mn || pb.sym_ops != 3) return cudaErrorInvalidValue;
    if (ep.bs_aux2 != pb.Mp * ep.ld_aux2) return cudaErrorInvalidValue;
    if (!get_map(tc, ep.aux2, pb.Mp, ep.ld_aux2, pb.batch, 128, &maux2)) return cudaErrorInvalidValue;
  }
  if (ep.kind == 0) {
    if (ep.bs_dst != pb.Mp * ep.ld_dst) return cudaErrorInvalidValue;
    if (!get_map(tc, ep.dst, pb.Mp, ep.ld_dst, pb.batch, 128, &mdst)) return cudaErrorInvalidValue;
  }
  const int64_t mt = pb.Mp / kBM, nt = pb.Np / kBN;
  int64_t per_mat;
  if (pb.symmetric) {
    const int64_t nb = pb.Mp / kBN;          // 256x256 blocks per side
    per_mat = nb * (nb + 1);                 // lower-triangle blocks x 2 row tiles
  } else {
    per_mat = mt * nt;
  }
  const int64_t total = per_mat * pb.batch;
  if (total > 0x7fffffffLL) return cudaErrorInvalidValue;
  // total is even: CTA 2p and 2p+1 (one cluster) take the two 128-row halves of a 256x256 tile.
  const int pairs = (int)std::min<int64_t>(total / 2, tc->max_pairs);
  *launches += 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2 * pairs, 1, 1);
  cfg.blockDim = dim3(kTcThreads, 1, 1);
  cfg.dynamicSmemBytes = kSmemBytes;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  const int kseg = (int)(pb.Kp / (kBK * kKSub));     // stages per pass over k
  const int segs = !split ? 1 : (pb.q_mn ? 2 : 3);
  const int kt = segs * kseg;
  Epilogue e2 = ep;
  if (segs == 2) e2.k_aux2 = ep.k_aux;               // both planes of X_0 carry the auxiliary coefficient
#define PRM_TC_LAUNCH(QMN, SYM, AX2, SG)                                                                          \
  return cudaLaunchKernelEx(&cfg, gemm_tc_kernel<QMN, SYM, AX2, SG>, mp, mq, maux, maux2, mdst, msp, msq, kt,      \
                            kseg, (int)per_mat, (int)total, pb.symmetric, (int)mt, e2, status)
  if (segs == 3) PRM_TC_LAUNCH(0, 0, 0, 3);
  if (segs == 2) PRM_TC_LAUNCH(1, 1, 1, 2);
  if (pb.q_mn && pb.sym_ops == 1) PRM_TC_LAUNCH(1, 1, 0, 1);
  if (pb.q_mn && !pb.sym_ops) PRM_TC_LAUNCH(1, 0, 0, 1);
  if (!pb.q_mn && pb.sym_ops == 3 && ep.aux2) PRM_TC_LAUNCH(0, 3, 1, 1);
  if (!pb.q_mn && pb.sym_ops == 3) PRM_TC_LAUNCH(0, 3, 0, 1);
  if (!pb.q_mn && !pb.sym_ops) PRM_TC_LAUNCH(0, 0, 0, 1);
#undef PRM_TC_LAUNCH
  return cudaErrorInvalidValue;   // no product of the recurrence needs another combination
}

}  // namespace prm

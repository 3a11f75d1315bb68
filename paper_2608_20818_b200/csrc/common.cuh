// Shared device helpers and host-side plan structures of the prm library.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <algorithm>
#include <string>
#include <vector>

#include "../../include/prm.h"

namespace prm {

// ---------------------------------------------------------------- constants
// Newton-Schulz coefficients and iteration count (paper, appendix "Optimizer
// and Training Hyperparameters").
constexpr float kNsA = 3.4445f;
constexpr float kNsB = -4.7750f;
constexpr float kNsC = 2.0315f;
constexpr int kNsIters = 5;
constexpr int kGramIters = 3;   // leading iterations that can run on the r x r Gram matrix alone

// NS5 operands live in the workspace padded to multiples of kPad in both
// dimensions; the padding is zero and stays zero through the recurrence.
constexpr int kPad = 256;

// Matrices with fewer oriented rows than this are refreshed in fp32 on CUDA
// cores even outside the check mode.  With so few rows the bf16 rounding of
// the r x r matrices does not average out: emulating bf16 storage with fp32
// accumulation on the CPU gives relative errors of the direction up to 6e-2
// at 5 rows and 2-3e-2 at 32 rows, against 1.2e-2 from 64 rows on.  The work
// is a single 256-row tile per product.
constexpr int kTinyRows = 64;

// Tall row-step: rows per column-partial block.
constexpr int kTallRows = 128;
// Tall row-step and pre-pass: columns per CTA.
constexpr int kTallCols = 256;

// Device status word values (bit flags).
constexpr int kStatusTimeout = 1;

// ------------------------------------------------------------- I/O helpers
struct alignas(16) bf16x8 {
  __nv_bfloat162 v[4];
};

// Load 8 consecutive elements as fp32.
__device__ __forceinline__ void load8(const __nv_bfloat16* p, float (&out)[8]) {
  bf16x8 raw = *reinterpret_cast<const bf16x8*>(p);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    float2 f = __bfloat1622float2(raw.v[i]);
    out[2 * i] = f.x;
    out[2 * i + 1] = f.y;
  }
}
__device__ __forceinline__ void load8(const float* p, float (&out)[8]) {
  float4 a = *reinterpret_cast<const float4*>(p);
  float4 b = *reinterpret_cast<const float4*>(p + 4);
  out[0] = a.x; out[1] = a.y; out[2] = a.z; out[3] = a.w;
  out[4] = b.x; out[5] = b.y; out[6] = b.z; out[7] = b.w;
}
// Streaming variants for data that is read exactly once.
__device__ __forceinline__ void load8_stream(const __nv_bfloat16* p, float (&out)[8]) {
  int4 r = __ldcs(reinterpret_cast<const int4*>(p));
  bf16x8 raw = *reinterpret_cast<bf16x8*>(&r);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    float2 f = __bfloat1622float2(raw.v[i]);
    out[2 * i] = f.x;
    out[2 * i + 1] = f.y;
  }
}
__device__ __forceinline__ void load8_stream(const float* p, float (&out)[8]) {
  float4 a = __ldcs(reinterpret_cast<const float4*>(p));
  float4 b = __ldcs(reinterpret_cast<const float4*>(p + 4));
  out[0] = a.x; out[1] = a.y; out[2] = a.z; out[3] = a.w;
  out[4] = b.x; out[5] = b.y; out[6] = b.z; out[7] = b.w;
}
// Eight elements kept in their storage format (registers), converted on use.
template <typename T> struct Raw8;
template <> struct Raw8<__nv_bfloat16> {
  int4 r;
  __device__ __forceinline__ void load_stream(const __nv_bfloat16* p) { r = __ldcs(reinterpret_cast<const int4*>(p)); }
  __device__ __forceinline__ void get(float (&out)[8]) const {
    const __nv_bfloat162* v = reinterpret_cast<const __nv_bfloat162*>(&r);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      float2 f = __bfloat1622float2(v[i]);
      out[2 * i] = f.x;
      out[2 * i + 1] = f.y;
    }
  }
};
template <> struct Raw8<float> {
  float4 a, b;
  __device__ __forceinline__ void load_stream(const float* p) {
    a = __ldcs(reinterpret_cast<const float4*>(p));
    b = __ldcs(reinterpret_cast<const float4*>(p + 4));
  }
  __device__ __forceinline__ void get(float (&out)[8]) const {
    out[0] = a.x; out[1] = a.y; out[2] = a.z; out[3] = a.w;
    out[4] = b.x; out[5] = b.y; out[6] = b.z; out[7] = b.w;
  }
};

// Store 8 consecutive elements (fp32 -> bf16 is round-to-nearest-even).
__device__ __forceinline__ void store8(__nv_bfloat16* p, const float (&in)[8]) {
  bf16x8 raw;
#pragma unroll
  for (int i = 0; i < 4; ++i) raw.v[i] = __floats2bfloat162_rn(in[2 * i], in[2 * i + 1]);
  *reinterpret_cast<bf16x8*>(p) = raw;
}
__device__ __forceinline__ void store8(float* p, const float (&in)[8]) {
  *reinterpret_cast<float4*>(p) = make_float4(in[0], in[1], in[2], in[3]);
  *reinterpret_cast<float4*>(p + 4) = make_float4(in[4], in[5], in[6], in[7]);
}
__device__ __forceinline__ float to_f32(__nv_bfloat16 x) { return __bfloat162float(x); }
__device__ __forceinline__ float to_f32(float x) { return x; }
__device__ __forceinline__ void from_f32(__nv_bfloat16* p, float x) { *p = __float2bfloat16_rn(x); }
__device__ __forceinline__ void from_f32(float* p, float x) { *p = x; }

// beta*x + omb*y in one fixed rounding order (a product, then a fused
// multiply-add), so that every kernel that updates the momentum or forms the
// direction input produces the same bits whatever else it does.
__device__ __forceinline__ float blend(float beta, float x, float omb, float y) {
  return __fmaf_rn(beta, x, __fmul_rn(omb, y));
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// ------------------------------------------------------------ host structs
// Per-step scalar hyper-parameters handed to kernels by value.
struct StepScalars {
  float beta;      // momentum coefficient
  float omb;       // 1 - beta
  int nesterov;
  float decay;     // 1 - lr*wd
  float lr_s;      // lr * s(W) for the group
  float gamma;
  float eps_row;
  float eps_ns;
};

// Device pointer tables, ordered by (group, order in group).
struct PtrTables {
  void** params;          // [n_mats]
  const void** grads;     // [n_mats]
  float** momentum;       // [n_mats]
};

// Launch geometry of the streaming (single-pass) row step of a tall group; ok = 0
// where the group does not qualify and the two-pass kernels run instead.
struct TallStreamPlan {
  int ok = 0;
  int R = 0;        // rows per CTA slab
  int lag = 0;      // waves between a slab's two phases
  int depth = 0;    // waves of tiles the producer keeps in flight
  size_t smem = 0;  // dynamic shared memory per CTA
};

struct Group {
  int64_t rows = 0, cols = 0;   // stored shape
  int count = 0;                // matrices in the group
  int first = 0;                // index of the group's first matrix in the grouped order
  bool tall = false;
  int64_t r = 0, c = 0;         // oriented shape, r <= c
  int64_t rp = 0, cp = 0;       // padded oriented shape (NS5 workspace)
  int ns_batch = 1;             // matrices refreshed per sub-batch
  int gram_iters = 0;           // leading NS5 iterations run in Gram space (0 or kGramIters)
  int last_gram_rec = 0;        // 1: the last iteration's Gram matrix comes from the previous one's
  int ns_fp32 = 0;              // 1: NS5 of this group runs in fp32 on CUDA cores (check mode, or a tiny matrix)
  int split = 0;                // 1: the NS5 input of this group is kept as two bf16 planes (PRM_OPT_NS_SPLIT_INPUT)
  size_t tall_scratch_off = 0;  // byte offset of column partials (tall groups)
  size_t tall_nu_off = 0;       // byte offset of column norms (tall groups)
  size_t tall_sync_off = 0;     // streaming row step: abort flag, per-wave counters and flags
  size_t tall_maps_off = 0;     // streaming row step: three tensor maps per matrix
  TallStreamPlan stream;        // filled when the workspace is attached (needs the SM count)
};

inline int64_t round_up(int64_t x, int64_t m) { return (x + m - 1) / m * m; }

// Which of the NS5 evaluation orders a matrix with oriented shape r x c takes under
// PRM_OPT_NS_GRAM_SPAN = span on the tensor-core path, and the flop it executes:
// X X^T products cost r^2 c (lower blocks only), r x c products 2 r^2 c, symmetric
// r x r products r^3.
struct Ns5Schedule {
  int gram_iters = 0;      // leading iterations on the Gram matrix (0 or kGramIters)
  int last_gram_rec = 0;   // the last Gram matrix comes from the one before it
  double flop = 0.0;
};
// split_input (tensor-core path only): X_0 is held as two bf16 planes; the matrix then takes the
// Gram-space order whatever its aspect ratio (X_0 must enter two products only and X_1, X_2 must
// never be rounded for the second plane to pay), and those two products run over both planes:
// + 4 r^2 c flop.  Below kGramMinRows padded rows the caller refreshes in fp32 instead
// (split_takes_fp32): there the Gram-space order costs benign inputs more than the planes gain.
constexpr int64_t kGramMinRows = 1024;
inline bool split_takes_fp32(int64_t r) { return round_up(r, kPad) < kGramMinRows; }
inline Ns5Schedule ns5_schedule(int64_t r, int64_t c, int span, bool fp32_path, bool split_input = false) {
  Ns5Schedule s;
  const int64_t rp = round_up(r, kPad), cp = round_up(c, kPad);
  const bool split = split_input && !fp32_path && rp >= kGramMinRows;
  // Gram-space iterations trade 6 r^2 (c - r) flop for six r^3 products: worth it from c = 1.5 r
  // on; below 1024 rows the time is noise and the bf16 rounding of the small r x r matrices
  // averages less well, so those stay on the printed recurrence.
  s.gram_iters = (!fp32_path && ((span && rp >= kGramMinRows && 2 * cp >= 3 * rp) || split)) ? kGramIters : 0;
  // Beyond c = 2r the Gram matrix of the last iteration is also cheaper from the one before it
  // (A_4 = P_3 A_3 P_3, two r^3 products) than from X_4 (one r^2 c product).
  s.last_gram_rec = (s.gram_iters && span >= 2 && cp > 2 * rp) ? 1 : 0;
  const double rd = (double)r, cd = (double)c;
  const double n_gram = s.gram_iters ? (s.last_gram_rec ? 2 : 3) : 5;
  const double n_rc = s.gram_iters ? 3 : 5;
  const double n_rr = s.gram_iters ? (s.last_gram_rec ? 13 : 11) : 5;
  s.flop = n_gram * rd * rd * cd + n_rc * 2.0 * rd * rd * cd + n_rr * rd * rd * rd;
  if (split) s.flop += 4.0 * rd * rd * cd;     // H L^T + L H^T (lower blocks) and Q L
  return s;
}

// dim-0 sharding as torch.chunk does it: rank q of `world` owns stored rows
// [start, start + count) with chunk = ceil(rows / world).
inline int64_t shard_chunk(int64_t rows, int world) { return (rows + world - 1) / world; }
inline void shard_rows(int64_t rows, int world, int rank, int64_t* start, int64_t* count) {
  const int64_t chunk = shard_chunk(rows, world);
  const int64_t lo = std::min(rows, (int64_t)rank * chunk);
  const int64_t hi = std::min(rows, lo + chunk);
  *start = lo;
  *count = hi - lo;
}

}  // namespace prm

// Host-side launch interfaces between the scheduler (api.cu) and the kernels.
#pragma once

#include "common.cuh"

namespace prm {

// cudaFuncSetAttribute holds per device: remembers, per kernel (one object per call site), on
// which devices the attribute has been set.
struct PerDeviceOnce {
  bool done[64] = {};
  // True if the caller still has to set the attribute on the current device.
  bool need(int* dev_out) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) { *dev_out = -1; return true; }
    *dev_out = dev;
    return !done[dev];
  }
  void mark(int dev) { if (dev >= 0) done[dev] = true; }
};

// Epilogue of every NS5 product D[i,j] = sum_k P[i,k]*Q[j,k].  With
// f = alpha[b]^alpha_pow (1 if alpha is null) and
// v = f*(k_acc*D[i,j] + k_aux*aux[i,j]):
// (plus f*k_aux2*aux2[i,j] where a second auxiliary operand is given: the
// Gram-space products of the tensor-core path)
//   kind 0: dst[i,j] = v.  The symmetric products store only the blocks they
//           compute (on and below the diagonal); their consumers read the
//           mirrored block instead of the missing one (GemmProblem::sym_ops).
//   kind 1: parameter update W = decay*W - lr_s*v at the stored position of
//           oriented element (i,j) (Eq. periodic-direction, rho_t = 1).
struct Epilogue {
  int kind = 0;
  float k_acc = 1.f, k_aux = 0.f;
  const float* alpha = nullptr;   // [batch] 1/(||U||_F + eps_ns)
  int alpha_pow = 0;
  const void* aux = nullptr;      // [batch][Mp][ld_aux]
  int64_t ld_aux = 0, bs_aux = 0;
  const void* aux2 = nullptr;     // [batch][Mp][ld_aux2], tensor-core path, kind 0 only
  float k_aux2 = 0.f;
  int64_t ld_aux2 = 0, bs_aux2 = 0;
  void* dst = nullptr;            // [batch][Mp][ld_dst]
  int64_t ld_dst = 0, bs_dst = 0;
  // kind 1
  PtrTables tables = {};
  int first = 0;                  // table index of the sub-batch's first matrix
  int rows = 0, cols = 0;         // stored shape
  int tall = 0;
  int io_fp32 = 0;
  float decay = 1.f, lr_s = 0.f;
  // Tensor-core path only: device array of 128-byte tensor maps over the
  // parameter matrices (table order); null selects per-thread accesses.
  const void* param_maps = nullptr;
};

// One batched product.  P: [batch][Mp][Kp], Q: [batch][Np][Kp]; Mp, Np, Kp
// are multiples of kPad.  symmetric != 0: the result is symmetric and only its
// 256x256 blocks on and below the diagonal are computed and stored.
struct GemmProblem {
  const void* P = nullptr;
  const void* Q = nullptr;
  int64_t Mp = 0, Np = 0, Kp = 0;
  int64_t bs_P = 0, bs_Q = 0;     // batch strides in elements
  int batch = 1;
  int symmetric = 0;
  int q_mn = 0;                   // Q is stored [batch][Kp][Np] (n contiguous) instead of [batch][Np][Kp]
  // Bit 0: P, bit 1: Q is a symmetric matrix of which only the 256x256 blocks on
  // and below the diagonal are stored; the rest is read from the mirrored block.
  // P and Q may be two different symmetric matrices (symmetric != 0 then
  // computes the lower blocks of P*Q, which is symmetric when they commute).
  int sym_ops = 0;
  // Tensor-core path: the input X_0 is a pair of bf16 planes H, L (X_0 = H + L), L directly
  // after H for every matrix (batch stride 2 * Mp * Kp resp. 2 * Kp * Np elements).  Two
  // products take it: P = Q = X_0, symmetric (computes H H^T + H L^T + L H^T), and the
  // N-major Q = X_0 under a symmetric P with aux = X_0 (computes P (H + L) and adds k_aux (H + L)).
  int split = 0;
};

cudaError_t launch_rowstep(const PtrTables& t, const Group& g, const StepScalars& s, int io_fp32,
                           float* tall_partial, float* tall_nu, cudaStream_t stream,
                           int64_t* launches);

// Persistent, bulk-copy-fed row step of a wide group (rowstep_wide_stream.cu): bf16 parameters and
// gradients, cols % 8 == 0, at most 24576 columns; n_cta CTAs, one per SM.
bool wide_stream_takes(const Group& g, int io_fp32);
cudaError_t launch_rowstep_wide_stream(const PtrTables& t, const Group& g, const StepScalars& s, int n_cta, int* status,
                                       cudaStream_t stream, int64_t* launches);

// Streaming row step of a tall group (rowstep_stream.cu): one pass over HBM,
// bf16 parameters and gradients with cols % 8 == 0.  maps_dev: three 128-byte
// tensor maps per matrix of the group (gradient, momentum, parameters; boxes of
// plan.R rows x tall_stream_panel() columns, no swizzle) in device memory.
// partial: tall_stream_partial_bytes(); sync: tall_stream_sync_ints() ints
// (zeroed by the launcher on the stream).  n_cta CTAs, one per SM, launched
// cooperatively.
TallStreamPlan tall_stream_plan(int64_t rows, int64_t cols, int io_fp32, int n_cta);
size_t tall_stream_partial_bytes();
size_t tall_stream_sync_ints(int64_t cols, int count);
int tall_stream_panel();
cudaError_t launch_rowstep_tall_stream(const PtrTables& t, const Group& g, const StepScalars& s,
                                       const TallStreamPlan& plan, const void* maps_dev, float* partial, float* nu,
                                       int* sync, int* status, int n_cta, cudaStream_t stream, int64_t* launches);

// Momentum update + direction input written to the NS5 workspace as the
// oriented matrix X (r_p x c_p, zero padded), with per-CTA partial sums of
// squares, then alpha per matrix.  x_fp32: workspace element type (1: fp32
// check mode, 0: bf16).  split (bf16 workspace only): X is written as the plane
// pair H = bf16(U), L = bf16(U - H), L directly after H for every matrix.
cudaError_t launch_ns_prepass(const PtrTables& t, const Group& g, int first, int batch,
                              const StepScalars& s, int io_fp32, int x_fp32, int split, void* X,
                              float* fro_partial, float* alpha, cudaStream_t stream,
                              int64_t* launches);

// The same pre-pass for wide groups with bf16 gradients and workspace and cols % 8 == 0, as a
// persistent bulk-copy-fed kernel (ns_prepass_stream.cu); n_cta CTAs, one per SM.  Leaves
// prepass_stream_parts() partials per matrix in fro_partial; the caller runs launch_ns_alpha.
bool prepass_stream_takes(const Group& g, int io_fp32, int x_fp32);
int prepass_stream_parts(int n_cta, int64_t prow, int batch);
cudaError_t launch_ns_prepass_stream(const PtrTables& t, const Group& g, int first, int batch, const StepScalars& s,
                                     int split, void* X, float* fro_partial, int n_cta, int* status, cudaStream_t stream);

// alpha[b] = 1/(sqrt(sum of nparts partials of matrix b) + eps_ns).
void launch_ns_alpha(const float* fro_partial, int nparts, float eps_ns, float* alpha, int batch,
                     cudaStream_t stream);

// Refresh over row shards (Algorithm 2 lines 1-7).  Matrices of one launch
// are described by value, kGatherMax at a time.
constexpr int kGatherMax = 32;
constexpr int kMaxWorld = 64;
struct GatherBatch { int64_t off[kGatherMax]; };   // element offset of the matrix inside every rank's segment
struct SliceBatch { void* param[kGatherMax]; };    // this rank's parameter rows
struct SegmentPtrs { const void* seg[kMaxWorld]; }; // start of every rank's segment (local or peer memory)
// The pre-pass on gathered rows: bf16 U of `batch` matrices of group g, read
// from `world` segments (rank q's at segs.seg[q]): row i of a matrix comes
// from segment i / chunk_rows, local row i % chunk_rows.  vec_ok: every
// segment start is 16-byte aligned.
cudaError_t launch_ns_gather_prepass(const SegmentPtrs& segs, bool vec_ok, int64_t chunk_rows,
                                     const int64_t* offs, const Group& g, int batch, float eps_ns, int x_fp32,
                                     void* X, float* fro_partial, float* alpha, cudaStream_t stream,
                                     int64_t* launches);
// W_shard <- decay*W_shard - lr_s*X5 on stored rows [row_start, row_start + rows_local).
cudaError_t launch_ns_slice_update(const void* X5, int x_fp32, const Group& g, int batch,
                                   void* const* param_shards, int64_t row_start, int64_t rows_local, int io_fp32,
                                   float decay, float lr_s, cudaStream_t stream, int64_t* launches);

// fp32 CUDA-core product (check mode).
cudaError_t launch_gemm_simt(const GemmProblem& pb, const Epilogue& ep, cudaStream_t stream,
                             int64_t* launches);

// bf16 tensor-core product (tcgen05, TMEM accumulators, TMA-fed tiles).
struct TcContext;
cudaError_t launch_gemm_tc(TcContext* tc, const GemmProblem& pb, const Epilogue& ep, int* status,
                           cudaStream_t stream, int64_t* launches);
bool tc_encode_param_map(TcContext* tc, const void* base, int64_t rows, int64_t cols, int tall, void* out128);
// Plain (unswizzled) 2-D map over a row-major rows x cols matrix of 2- or 4-byte elements,
// box = box_rows x box_cols; parts of a box outside the matrix read as zero.
bool tc_encode_tile_map(TcContext* tc, const void* base, int64_t rows, int64_t cols, int elem_bytes, int box_cols,
                        int box_rows, void* out128);
int tc_sm_count(const TcContext* tc);
TcContext* tc_create(std::string* err);
// One thread waits limit_ns on a barrier that never completes, then raises
// the status word (bit kStatusTimeout) and sets *gave_up (device int, may be null).
cudaError_t launch_wait_probe(int* status, uint64_t limit_ns, int* gave_up, cudaStream_t stream);
void tc_destroy(TcContext* tc);

}  // namespace prm

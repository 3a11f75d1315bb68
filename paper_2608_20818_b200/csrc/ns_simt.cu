// fp32 CUDA-core implementation of the NS5 products (check mode).  Same
// operands, schedule and epilogues as the tensor-core path, but fp32 storage
// and fp32 FMA arithmetic; the accumulation is folded every 256 terms so the
// rounding error does not grow with the contraction length.
#include "epilogue.cuh"

namespace prm {

constexpr int kSimtTile = 128;
constexpr int kSimtK = 8;
constexpr int kSimtThreads = 256;
constexpr int kSimtLd = kSimtTile + 4;
constexpr int kFoldSteps = 32;   // fold every 32 k-steps of 8

__global__ void __launch_bounds__(kSimtThreads)
gemm_simt_kernel(GemmProblem pb, Epilogue ep) {
  __shared__ __align__(16) float As[kSimtK][kSimtLd];
  __shared__ __align__(16) float Bs[kSimtK][kSimtLd];
  const int b = blockIdx.y;
  int ti, tj;
  if (pb.symmetric) {
    // every 128x128 tile of the 256x256 blocks on and below the diagonal
    int bi, bj;
    tri_decode(blockIdx.x >> 2, bi, bj);
    ti = 2 * bi + ((blockIdx.x >> 1) & 1);
    tj = 2 * bj + (blockIdx.x & 1);
  } else {
    const int nt = (int)(pb.Np / kSimtTile);
    ti = blockIdx.x / nt;
    tj = blockIdx.x % nt;
  }
  const float* __restrict__ P = reinterpret_cast<const float*>(pb.P) + (int64_t)b * pb.bs_P;
  const float* __restrict__ Q = reinterpret_cast<const float*>(pb.Q) + (int64_t)b * pb.bs_Q;
  const int qk = threadIdx.x >> 5, qj = (threadIdx.x & 31) * 4;   // transposed storage: one float4 of row k per thread
  const int lrow = threadIdx.x >> 1, lk = (threadIdx.x & 1) * 4;  // k-contiguous storage: four k of one row per thread
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  float acc[8][8], tot[8][8];
#pragma unroll
  for (int a = 0; a < 8; ++a)
#pragma unroll
    for (int c = 0; c < 8; ++c) { acc[a][c] = 0.f; tot[a][c] = 0.f; }

  // Where the 8 x 128 operand slice of k-step ks lives.  A symmetric operand
  // (sym_ops) is stored only in the 256x256 blocks on and below the diagonal:
  // right of its diagonal block the slice is read from the mirrored block,
  // which is stored [k][row].  Q with q_mn is stored [k][n] throughout.
  auto p_transposed = [&](int ks) { return (pb.sym_ops & 1) && (ks * kSimtK) / kPad > (ti * kSimtTile) / kPad; };
  auto q_transposed = [&](int ks) {
    return pb.q_mn || ((pb.sym_ops & 2) && (ks * kSimtK) / kPad > (tj * kSimtTile) / kPad);
  };
  auto fetch = [&](const float* base, int tile, int ks, bool tr, int64_t ld_t) -> float4 {
    return tr ? *reinterpret_cast<const float4*>(base + (int64_t)(ks * kSimtK + qk) * ld_t + tile * kSimtTile + qj)
              : *reinterpret_cast<const float4*>(base + (int64_t)(tile * kSimtTile + lrow) * pb.Kp + ks * kSimtK + lk);
  };
  const int64_t ldt_p = pb.Kp, ldt_q = pb.q_mn ? pb.Np : pb.Kp;
  const int ksteps = (int)(pb.Kp / kSimtK);
  float4 pa = fetch(P, ti, 0, p_transposed(0), ldt_p);
  float4 qa = fetch(Q, tj, 0, q_transposed(0), ldt_q);
  for (int ks = 0; ks < ksteps; ++ks) {
    if (p_transposed(ks)) {
      *reinterpret_cast<float4*>(&As[qk][qj]) = pa;
    } else {
      As[lk + 0][lrow] = pa.x; As[lk + 1][lrow] = pa.y; As[lk + 2][lrow] = pa.z; As[lk + 3][lrow] = pa.w;
    }
    if (q_transposed(ks)) {
      *reinterpret_cast<float4*>(&Bs[qk][qj]) = qa;
    } else {
      Bs[lk + 0][lrow] = qa.x; Bs[lk + 1][lrow] = qa.y; Bs[lk + 2][lrow] = qa.z; Bs[lk + 3][lrow] = qa.w;
    }
    __syncthreads();
    if (ks + 1 < ksteps) {
      pa = fetch(P, ti, ks + 1, p_transposed(ks + 1), ldt_p);
      qa = fetch(Q, tj, ks + 1, q_transposed(ks + 1), ldt_q);
    }
#pragma unroll
    for (int k = 0; k < kSimtK; ++k) {
      float av[8], bv[8];
      *reinterpret_cast<float4*>(&av[0]) = *reinterpret_cast<const float4*>(&As[k][ty * 8]);
      *reinterpret_cast<float4*>(&av[4]) = *reinterpret_cast<const float4*>(&As[k][ty * 8 + 4]);
      *reinterpret_cast<float4*>(&bv[0]) = *reinterpret_cast<const float4*>(&Bs[k][tx * 8]);
      *reinterpret_cast<float4*>(&bv[4]) = *reinterpret_cast<const float4*>(&Bs[k][tx * 8 + 4]);
#pragma unroll
      for (int a = 0; a < 8; ++a)
#pragma unroll
        for (int c = 0; c < 8; ++c) acc[a][c] = fmaf(av[a], bv[c], acc[a][c]);
    }
    __syncthreads();
    if ((ks + 1) % kFoldSteps == 0) {
#pragma unroll
      for (int a = 0; a < 8; ++a)
#pragma unroll
        for (int c = 0; c < 8; ++c) { tot[a][c] += acc[a][c]; acc[a][c] = 0.f; }
    }
  }
#pragma unroll
  for (int a = 0; a < 8; ++a)
#pragma unroll
    for (int c = 0; c < 8; ++c) tot[a][c] += acc[a][c];

#pragma unroll
  for (int a = 0; a < 8; ++a) {
    const int i = ti * kSimtTile + ty * 8 + a;
    const int j0 = tj * kSimtTile + tx * 8;
    epilogue_row<float, 8>(ep, b, i, j0, tot[a]);
  }
}

cudaError_t launch_gemm_simt(const GemmProblem& pb, const Epilogue& ep, cudaStream_t stream,
                             int64_t* launches) {
  const int64_t mt = pb.Mp / kSimtTile, nt = pb.Np / kSimtTile;
  const int64_t nb = pb.Mp / kPad;
  const int64_t tiles = pb.symmetric ? 4 * (nb * (nb + 1) / 2) : mt * nt;
  if (tiles > 0x7fffffffLL || pb.batch > 65535) return cudaErrorInvalidValue;
  *launches += 1;
  dim3 grid((unsigned)tiles, (unsigned)pb.batch, 1);
  gemm_simt_kernel<<<grid, kSimtThreads, 0, stream>>>(pb, ep);
  return cudaGetLastError();
}

}  // namespace prm

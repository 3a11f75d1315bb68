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
    tri_decode(blockIdx.x, ti, tj);
  } else {
    const int nt = (int)(pb.Np / kSimtTile);
    ti = blockIdx.x / nt;
    tj = blockIdx.x % nt;
  }
  const float* __restrict__ P = reinterpret_cast<const float*>(pb.P) + (int64_t)b * pb.bs_P +
                                (int64_t)ti * kSimtTile * pb.Kp;
  // Q is [Np][Kp] (k contiguous) or, with q_mn, [Kp][Np] (n contiguous).
  const float* __restrict__ Q = reinterpret_cast<const float*>(pb.Q) + (int64_t)b * pb.bs_Q +
                                (pb.q_mn ? (int64_t)tj * kSimtTile : (int64_t)tj * kSimtTile * pb.Kp);
  const int qk = threadIdx.x >> 5, qj = (threadIdx.x & 31) * 4;   // q_mn: one float4 of row k per thread
  const int lrow = threadIdx.x >> 1, lk = (threadIdx.x & 1) * 4;
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  float acc[8][8], tot[8][8];
#pragma unroll
  for (int a = 0; a < 8; ++a)
#pragma unroll
    for (int c = 0; c < 8; ++c) { acc[a][c] = 0.f; tot[a][c] = 0.f; }

  const int ksteps = (int)(pb.Kp / kSimtK);
  float4 pa = *reinterpret_cast<const float4*>(P + (int64_t)lrow * pb.Kp + lk);
  float4 qa = pb.q_mn ? *reinterpret_cast<const float4*>(Q + (int64_t)qk * pb.Np + qj)
                      : *reinterpret_cast<const float4*>(Q + (int64_t)lrow * pb.Kp + lk);
  for (int ks = 0; ks < ksteps; ++ks) {
    As[lk + 0][lrow] = pa.x; As[lk + 1][lrow] = pa.y; As[lk + 2][lrow] = pa.z; As[lk + 3][lrow] = pa.w;
    if (pb.q_mn) {
      *reinterpret_cast<float4*>(&Bs[qk][qj]) = qa;
    } else {
      Bs[lk + 0][lrow] = qa.x; Bs[lk + 1][lrow] = qa.y; Bs[lk + 2][lrow] = qa.z; Bs[lk + 3][lrow] = qa.w;
    }
    __syncthreads();
    if (ks + 1 < ksteps) {
      pa = *reinterpret_cast<const float4*>(P + (int64_t)lrow * pb.Kp + (ks + 1) * kSimtK + lk);
      qa = pb.q_mn ? *reinterpret_cast<const float4*>(Q + (int64_t)((ks + 1) * kSimtK + qk) * pb.Np + qj)
                   : *reinterpret_cast<const float4*>(Q + (int64_t)lrow * pb.Kp + (ks + 1) * kSimtK + lk);
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

  const bool mirror = pb.symmetric ? (ti != tj) : true;
#pragma unroll
  for (int a = 0; a < 8; ++a) {
    const int i = ti * kSimtTile + ty * 8 + a;
    const int j0 = tj * kSimtTile + tx * 8;
    epilogue_row<float, 8>(ep, b, i, j0, tot[a], mirror);
  }
}

cudaError_t launch_gemm_simt(const GemmProblem& pb, const Epilogue& ep, cudaStream_t stream,
                             int64_t* launches) {
  const int64_t mt = pb.Mp / kSimtTile, nt = pb.Np / kSimtTile;
  const int64_t tiles = pb.symmetric ? mt * (mt + 1) / 2 : mt * nt;
  if (tiles > 0x7fffffffLL || pb.batch > 65535) return cudaErrorInvalidValue;
  *launches += 1;
  dim3 grid((unsigned)tiles, (unsigned)pb.batch, 1);
  gemm_simt_kernel<<<grid, kSimtThreads, 0, stream>>>(pb, ep);
  return cudaGetLastError();
}

}  // namespace prm

// Device side of the NS5 product epilogue (see struct Epilogue): one call
// handles N consecutive columns j0..j0+N-1 of output row i of batch item b.
#pragma once

#include "launch.cuh"

namespace prm {

// XT_: element type of the workspace arrays (bf16 or float).  N multiple of 8.
// pre: optional N auxiliary values already fetched by the caller (see
// aux_prefetch); when null the auxiliary operand is loaded here.
template <typename XT_, int N>
__device__ __forceinline__ void epilogue_row(const Epilogue& ep, int b, int i, int j0,
                                             float (&acc)[N], const float* pre = nullptr) {
  const float al = ep.alpha ? ep.alpha[b] : 1.f;
  const float f = ep.alpha_pow == 2 ? al * al : (ep.alpha_pow == 1 ? al : 1.f);
  const float ka = f * ep.k_acc, kx = f * ep.k_aux;
  if (ep.aux != nullptr) {
    const XT_* aux = reinterpret_cast<const XT_*>(ep.aux) + (int64_t)b * ep.bs_aux +
                     (int64_t)i * ep.ld_aux + j0;
#pragma unroll
    for (int v = 0; v < N; v += 8) {
      float x[8];
      if (pre != nullptr) {
#pragma unroll
        for (int e = 0; e < 8; ++e) x[e] = pre[v + e];
      } else {
        load8(aux + v, x);
      }
#pragma unroll
      for (int e = 0; e < 8; ++e) acc[v + e] = ka * acc[v + e] + kx * x[e];
    }
  } else {
#pragma unroll
    for (int e = 0; e < N; ++e) acc[e] = ka * acc[e];
  }
  if (ep.kind == 0) {
    XT_* dst = reinterpret_cast<XT_*>(ep.dst) + (int64_t)b * ep.bs_dst + (int64_t)i * ep.ld_dst + j0;
#pragma unroll
    for (int v = 0; v < N; v += 8) {
      float x[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) x[e] = acc[v + e];
      store8(dst + v, x);
    }
  } else {
    // Parameter update at the stored position of oriented element (i, j).
    const int r = ep.tall ? ep.cols : ep.rows, c = ep.tall ? ep.rows : ep.cols;
    if (i >= r) return;
    void* pbase = ep.tables.params[ep.first + b];
    if (!ep.tall) {
      const int64_t off = (int64_t)i * ep.cols + j0;
      if (j0 + N <= c && (ep.cols & 7) == 0) {
#pragma unroll
        for (int v = 0; v < N; v += 8) {
          float x[8];
          if (ep.io_fp32) {
            float* p = reinterpret_cast<float*>(pbase) + off + v;
            load8(p, x);
#pragma unroll
            for (int e = 0; e < 8; ++e) x[e] = ep.decay * x[e] - ep.lr_s * acc[v + e];
            store8(p, x);
          } else {
            __nv_bfloat16* p = reinterpret_cast<__nv_bfloat16*>(pbase) + off + v;
            load8(p, x);
#pragma unroll
            for (int e = 0; e < 8; ++e) x[e] = ep.decay * x[e] - ep.lr_s * acc[v + e];
            store8(p, x);
          }
        }
      } else {
#pragma unroll
        for (int e = 0; e < N; ++e) {
          if (j0 + e < c) {
            if (ep.io_fp32) {
              float* p = reinterpret_cast<float*>(pbase) + off + e;
              *p = ep.decay * (*p) - ep.lr_s * acc[e];
            } else {
              __nv_bfloat16* p = reinterpret_cast<__nv_bfloat16*>(pbase) + off + e;
              *p = __float2bfloat16_rn(ep.decay * __bfloat162float(*p) - ep.lr_s * acc[e]);
            }
          }
        }
      }
    } else {
#pragma unroll
      for (int e = 0; e < N; ++e) {
        if (j0 + e < c) {
          const int64_t off = (int64_t)(j0 + e) * ep.cols + i;
          if (ep.io_fp32) {
            float* p = reinterpret_cast<float*>(pbase) + off;
            *p = ep.decay * (*p) - ep.lr_s * acc[e];
          } else {
            __nv_bfloat16* p = reinterpret_cast<__nv_bfloat16*>(pbase) + off;
            *p = __float2bfloat16_rn(ep.decay * __bfloat162float(*p) - ep.lr_s * acc[e]);
          }
        }
      }
    }
  }
}

// N bf16 auxiliary values of one output row, fetched ahead of use.
template <int N>
struct AuxRegs {
  int4 r[N / 8];
};
template <int N>
__device__ __forceinline__ void aux_prefetch(const Epilogue& ep, int b, int i, int j0, AuxRegs<N>& a) {
  if (ep.aux == nullptr) return;
  const int4* p = reinterpret_cast<const int4*>(reinterpret_cast<const __nv_bfloat16*>(ep.aux) +
                                                (int64_t)b * ep.bs_aux + (int64_t)i * ep.ld_aux + j0);
#pragma unroll
  for (int v = 0; v < N / 8; ++v) a.r[v] = p[v];
}
template <int N>
__device__ __forceinline__ void aux_unpack(const AuxRegs<N>& a, float (&x)[N]) {
#pragma unroll
  for (int v = 0; v < N / 8; ++v) {
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&a.r[v]);
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const float2 f = __bfloat1622float2(h[k]);
      x[8 * v + 2 * k] = f.x;
      x[8 * v + 2 * k + 1] = f.y;
    }
  }
}

// Lower-triangle tile index -> (ti, tj), ti >= tj, rows of the triangle in order.
__device__ __forceinline__ void tri_decode(int t, int& ti, int& tj) {
  int i = (int)((sqrtf(8.f * (float)t + 1.f) - 1.f) * 0.5f);
  while ((i + 1) * (i + 2) / 2 <= t) ++i;
  while (i * (i + 1) / 2 > t) --i;
  ti = i;
  tj = t - i * (i + 1) / 2;
}

}  // namespace prm

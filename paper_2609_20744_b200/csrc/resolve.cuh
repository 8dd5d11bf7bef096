// Resolve (Eq. 5, Alg. 1 step 4):  C_t = (I + A_t)^{-1} in fp32, one CTA per frame (b,h,t).
//
// I + A_t is symmetric positive definite with every eigenvalue >= 1 (A_t is a Gram matrix weighted
// by beta >= 0), so in-place Gauss-Jordan elimination needs no pivot search.  The matrix lives in
// registers, an R x R tile per thread on a 16 x 16 thread grid; for every pivot the owning threads
// publish the pivot row and column through (double-buffered) shared memory and everybody applies
// the rank-1 update: one barrier per pivot.
#pragma once
#include "common.cuh"

namespace vdn {

template <int D>
__global__ void __launch_bounds__(256) resolve_kernel(const float* __restrict__ stats,
                                                       float* __restrict__ inv, long long nframes) {
  constexpr int R = D / 16;
  __shared__ __align__(16) float rowbuf[2][D];
  __shared__ __align__(16) float colbuf[2][D];

  const long long n = blockIdx.x;
  if (n >= nframes) return;
  const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;
  const float* A = stats + (size_t)n * D * 2 * D;   // row stride 2D: [A | B^T]

  float m[R][R];
#pragma unroll
  for (int r = 0; r < R; ++r) {
    const int i = ty * R + r;
#pragma unroll
    for (int c = 0; c < R; c += 4) {
      float4 x = load4(A + (size_t)i * 2 * D + tx * R + c);
      m[r][c] = x.x; m[r][c + 1] = x.y; m[r][c + 2] = x.z; m[r][c + 3] = x.w;
    }
#pragma unroll
    for (int c = 0; c < R; ++c)
      if (i == tx * R + c) m[r][c] += 1.0f;
  }

  for (int p = 0; p < D; ++p) {
    const int par = p & 1;
    const int pb = p / R, pr = p % R;
    if (ty == pb) {
#pragma unroll
      for (int r = 0; r < R; ++r)
        if (r == pr) {
#pragma unroll
          for (int c = 0; c < R; ++c) rowbuf[par][tx * R + c] = m[r][c];
        }
    }
    if (tx == pb) {
#pragma unroll
      for (int c = 0; c < R; ++c)
        if (c == pr) {
#pragma unroll
          for (int r = 0; r < R; ++r) colbuf[par][ty * R + r] = m[r][c];
        }
    }
    __syncthreads();
    const float ipiv = 1.0f / rowbuf[par][p];
    float rowv[R], colv[R];
#pragma unroll
    for (int c = 0; c < R; c += 4) {
      float4 x = load4(&rowbuf[par][tx * R + c]);
      rowv[c] = x.x; rowv[c + 1] = x.y; rowv[c + 2] = x.z; rowv[c + 3] = x.w;
    }
#pragma unroll
    for (int r = 0; r < R; r += 4) {
      float4 x = load4(&colbuf[par][ty * R + r]);
      colv[r] = x.x; colv[r + 1] = x.y; colv[r + 2] = x.z; colv[r + 3] = x.w;
    }
#pragma unroll
    for (int r = 0; r < R; ++r) {
      const bool prow = (ty * R + r == p);
      const float f = colv[r] * ipiv;
#pragma unroll
      for (int c = 0; c < R; ++c) {
        const bool pcol = (tx * R + c == p);
        float upd = fmaf(-f, rowv[c], m[r][c]);       // ordinary entry
        if (prow) upd = rowv[c] * ipiv;               // pivot row
        if (pcol) upd = -f;                           // pivot column
        if (prow && pcol) upd = ipiv;                 // pivot itself
        m[r][c] = upd;
      }
    }
  }

  float* C = inv + (size_t)n * D * D;
#pragma unroll
  for (int r = 0; r < R; ++r)
#pragma unroll
    for (int c = 0; c < R; c += 4)
      store4(C + (size_t)(ty * R + r) * D + tx * R + c, make_float4(m[r][c], m[r][c + 1], m[r][c + 2], m[r][c + 3]));
}

}  // namespace vdn

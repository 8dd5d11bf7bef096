// Resolve (Eq. 5, Alg. 1 step 4):  C_t = (I + A_t)^{-1} in fp32, one CTA per frame (b,h,t).
//
// I + A_t is symmetric positive definite with every eigenvalue >= 1 (A_t is a Gram matrix weighted
// by beta >= 0), so in-place Gauss-Jordan elimination needs no pivot search.  The matrix lives in
// registers: thread (ty,tx) of a 16 x 16 grid owns rows ty+16r and columns tx+16c (cyclic), so the
// owner of pivot p = 16q+o is known from o alone and the register index q is a compile-time constant.
//
// Per pivot the owners publish the pivot row and column through double-buffered shared memory and
// then zero them in their registers; with the published column entry of the pivot row set to -1 and
// the published row entry of the pivot column set to 1/pivot, the uniform update
//        m[i][j] -= col[i] * row[j] / pivot
// also produces the pivot row (row/pivot), the pivot column (-col/pivot) and the pivot (1/pivot):
// one FMA per element, no predication, one barrier per pivot.
//
// When `split` is non-null the inverse is also written as three bf16 matrices C1 + C2 + C3 (each the
// truncation to bf16 of what the previous ones leave over, 24 mantissa bits in all) for the tensor-core scan.
#pragma once
#include <cuda_bf16.h>

#include "common.cuh"

namespace vdn {

// In-place inverse of the D x D matrix held as R x R cyclic tiles by a 16 x 16 thread grid.
// rowbuf / colbuf: 2 x D floats each in shared memory; sync(): a barrier over the 256 threads.
template <int D, typename Sync>
__device__ __forceinline__ void gauss_jordan_tiles(float (&m)[D / 16][D / 16], float* rowbuf, float* colbuf,
                                                   int tx, int ty, Sync sync) {
  constexpr int R = D / 16;
#pragma unroll
  for (int q = 0; q < R; ++q) {
#pragma unroll 2
    for (int o = 0; o < 16; ++o) {
      float* rb = rowbuf + (o & 1) * D;      // indexed [owner tx][c]
      float* cb = colbuf + (o & 1) * D;      // indexed [owner ty][r]
      if (ty == o) {                      // owners of the pivot row: publish it, then clear it
#pragma unroll
        for (int c = 0; c < R; c += 4) {
          store4(rb + tx * R + c, make_float4(m[q][c], m[q][c + 1], m[q][c + 2], m[q][c + 3]));
          m[q][c] = 0.f; m[q][c + 1] = 0.f; m[q][c + 2] = 0.f; m[q][c + 3] = 0.f;
        }
      }
      if (tx == o) {                      // owners of the pivot column
        float cv[R];
#pragma unroll
        for (int r = 0; r < R; ++r) { cv[r] = m[r][q]; m[r][q] = 0.f; }
        if (ty == o) cv[q] = -1.0f;       // (the pivot itself was already published with the row)
#pragma unroll
        for (int r = 0; r < R; r += 4) store4(cb + ty * R + r, make_float4(cv[r], cv[r + 1], cv[r + 2], cv[r + 3]));
      }
      sync();
      const float ipiv = __frcp_rn(rb[o * R + q]);
      float rv[R], cv[R];
#pragma unroll
      for (int c = 0; c < R; c += 4) {
        float4 x = load4(rb + tx * R + c);
        rv[c] = x.x * ipiv; rv[c + 1] = x.y * ipiv; rv[c + 2] = x.z * ipiv; rv[c + 3] = x.w * ipiv;
      }
      if (tx == o) rv[q] = ipiv;
#pragma unroll
      for (int r = 0; r < R; r += 4) {
        float4 x = load4(cb + ty * R + r);
        cv[r] = x.x; cv[r + 1] = x.y; cv[r + 2] = x.z; cv[r + 3] = x.w;
      }
#pragma unroll
      for (int r = 0; r < R; ++r)
#pragma unroll
        for (int c = 0; c < R; ++c) m[r][c] = fmaf(-cv[r], rv[c], m[r][c]);
    }
  }
}

// The tiles as three bf16 matrices S[0] + S[1] + S[2] (each D x D, row-major).
template <int D>
__device__ __forceinline__ void store_split_tiles(const float (&m)[D / 16][D / 16], __nv_bfloat16* S, int tx, int ty) {
  constexpr int R = D / 16;
#pragma unroll
  for (int r = 0; r < R; ++r)
#pragma unroll
    for (int c = 0; c < R; ++c) {
      const size_t e = (size_t)(ty + 16 * r) * D + tx + 16 * c;
      // truncating three-way split: x = p1 + p2 + p3 exactly
      const float x = m[r][c];
      const uint32_t u1 = __float_as_uint(x) & 0xFFFF0000u;
      const float r1 = x - __uint_as_float(u1);
      const uint32_t u2 = __float_as_uint(r1) & 0xFFFF0000u;
      const uint32_t u3 = __float_as_uint(r1 - __uint_as_float(u2)) & 0xFFFF0000u;
      S[e] = __ushort_as_bfloat16((unsigned short)(u1 >> 16));
      S[(size_t)D * D + e] = __ushort_as_bfloat16((unsigned short)(u2 >> 16));
      S[(size_t)2 * D * D + e] = __ushort_as_bfloat16((unsigned short)(u3 >> 16));
    }
}

// The transition of the additive baseline (Eq. 3c with the frame-size key scaling of Sec. 3.3): no inverse,
//     C_t = I - sym(A_t) / F          (fp32, and/or its three-way bf16 split for the tensor-core scan)
// taking the place of (I + A_t)^{-1} in the scan.  One CTA per frame.
template <int D>
__global__ void __launch_bounds__(256) additive_transition_kernel(const float* __restrict__ stats,
                                                                  float* __restrict__ inv,
                                                                  __nv_bfloat16* __restrict__ split,
                                                                  long long nframes, float inv_f, Shape shp) {
  const long long n = blockIdx.x;
  if (n >= nframes) return;
  if ((int)(n % shp.T) < shp.t0 || (int)(n % shp.T) >= shp.t0 + shp.Tn) return;   // an anchor frame: not scanned
  const float* A = stats + (size_t)n * 2 * D * D;
  for (int e = threadIdx.x; e < D * D; e += 256) {
    const int i = e / D, j = e % D;
    const float c = (i == j ? 1.0f : 0.0f) - 0.5f * (__ldg(A + e) + __ldg(A + (size_t)j * D + i)) * inv_f;
    if (inv != nullptr) inv[(size_t)n * D * D + e] = c;
    if (split != nullptr) {
      __nv_bfloat16* S = split + (size_t)n * 3 * D * D;
      const uint32_t u1 = __float_as_uint(c) & 0xFFFF0000u;
      const float r1 = c - __uint_as_float(u1);
      const uint32_t u2 = __float_as_uint(r1) & 0xFFFF0000u;
      const uint32_t u3 = __float_as_uint(r1 - __uint_as_float(u2)) & 0xFFFF0000u;
      S[e] = __ushort_as_bfloat16((unsigned short)(u1 >> 16));
      S[(size_t)D * D + e] = __ushort_as_bfloat16((unsigned short)(u2 >> 16));
      S[(size_t)2 * D * D + e] = __ushort_as_bfloat16((unsigned short)(u3 >> 16));
    }
  }
}

template <int D>
__global__ void __launch_bounds__(256, 2) resolve_kernel(const float* __restrict__ stats,
                                                          float* __restrict__ inv,
                                                          __nv_bfloat16* __restrict__ split, long long nframes,
                                                          Shape shp) {
  constexpr int R = D / 16;
  __shared__ __align__(16) float rowbuf[2 * D];
  __shared__ __align__(16) float colbuf[2 * D];

  const long long n = blockIdx.x;
  if (n >= nframes) return;
  if ((int)(n % shp.T) < shp.t0 || (int)(n % shp.T) >= shp.t0 + shp.Tn) return;   // an anchor frame: not scanned
  const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;
  const float* A = stats + (size_t)n * 2 * D * D;   // first d rows of the frame's [2d][d] block

  float m[R][R];
#pragma unroll
  for (int r = 0; r < R; ++r)
#pragma unroll
    for (int c = 0; c < R; ++c) {
      const int i = ty + 16 * r, j = tx + 16 * c;
      // the symmetric part: the tensor-core statistics are symmetric only up to the bf16 rounding of one factor
      // (the plain-fp32 ones to the last bit or two), and the symmetric part is what Eq. 3b means
      m[r][c] = 0.5f * (__ldg(A + (size_t)i * D + j) + __ldg(A + (size_t)j * D + i)) + (i == j ? 1.0f : 0.0f);
    }

  gauss_jordan_tiles<D>(m, rowbuf, colbuf, tx, ty, [] { __syncthreads(); });

  if (inv != nullptr) {
    float* C = inv + (size_t)n * D * D;
#pragma unroll
    for (int r = 0; r < R; ++r)
#pragma unroll
      for (int c = 0; c < R; ++c) C[(size_t)(ty + 16 * r) * D + tx + 16 * c] = m[r][c];
  }
  if (split != nullptr) store_split_tiles<D>(m, split + (size_t)n * 3 * D * D, tx, ty);
}

}  // namespace vdn

// Frame statistics (Eq. 3b) in plain fp32:  for frame n = (b,h,t)
//     stats[n][j][i]      = A_t[j][i] = sum_u beta_u k_u[j] k_u[i]      rows 0..d-1
//     stats[n][d + c][i]  = B_t[c][i] = sum_u beta_u v_u[c] k_u[i]      rows d..2d-1  (B_t is d_v x d_k)
// One CTA per (frame, 64-wide column block of [K | V]); tokens are streamed in tiles of TU and
// summed in token order, so the result is deterministic.  Used by f32 mode and as a second opinion
// for the tensor-core kernel.
#pragma once
#include "common.cuh"

namespace vdn {

template <typename Tio, int D>
__global__ void __launch_bounds__(256) gram_simt_kernel(const Tio* __restrict__ k, const Tio* __restrict__ v,
                                                         const float* __restrict__ beta,
                                                         float* __restrict__ stats, Shape s) {
  constexpr int TU = 32;        // tokens per tile
  constexpr int CB = 64;        // output columns per CTA
  constexpr int TI = D / 16;    // rows per thread
  __shared__ __align__(16) float Ks[TU][D];    // beta_u * k_u
  __shared__ __align__(16) float Ws[TU][CB];   // the CTA's column block of [k_u | v_u]

  const long long n = blockIdx.x;
  const int cb = blockIdx.y;                    // column block: cols [cb*64, cb*64+64) of [K|V]
  int b, h, t;
  split_frame(s, n, b, h, t);
  if (t < s.t0 || t >= s.t0 + s.Tn) return;     // an anchor frame: not scanned
  const Tio* wsrc = (cb * CB < D) ? k : v;
  const int wcol0 = (cb * CB) % D;

  const int tid = threadIdx.x;
  const int ig = tid / 16, cg = tid % 16;       // 16 row groups x 16 column groups
  float acc[TI][4];
#pragma unroll
  for (int r = 0; r < TI; ++r)
#pragma unroll
    for (int c = 0; c < 4; ++c) acc[r][c] = 0.f;

  for (int u0 = 0; u0 < s.F; u0 += TU) {
    // stage the tile
    for (int e = tid; e < TU * (D / 4); e += 256) {
      int uu = e / (D / 4), j4 = (e % (D / 4)) * 4;
      int u = u0 + uu;
      float4 kv = make_float4(0.f, 0.f, 0.f, 0.f);
      if (u < s.F) {
        float bu = beta[(((size_t)b * s.T + t) * s.F + u) * s.H + h];
        kv = load4(k + token_offset(s, b, t, u, h) + j4);
        kv.x *= bu; kv.y *= bu; kv.z *= bu; kv.w *= bu;
      }
      store4(&Ks[uu][j4], kv);
    }
    for (int e = tid; e < TU * (CB / 4); e += 256) {
      int uu = e / (CB / 4), j4 = (e % (CB / 4)) * 4;
      int u = u0 + uu;
      float4 w = make_float4(0.f, 0.f, 0.f, 0.f);
      if (u < s.F) w = load4(wsrc + token_offset(s, b, t, u, h) + wcol0 + j4);
      store4(&Ws[uu][j4], w);
    }
    __syncthreads();
#pragma unroll 4
    for (int uu = 0; uu < TU; ++uu) {
      float a[TI];
#pragma unroll
      for (int r = 0; r < TI; r += 4) {
        float4 x = load4(&Ks[uu][ig * TI + r]);
        a[r] = x.x; a[r + 1] = x.y; a[r + 2] = x.z; a[r + 3] = x.w;
      }
      float4 w = load4(&Ws[uu][cg * 4]);
#pragma unroll
      for (int r = 0; r < TI; ++r) {
        acc[r][0] = fmaf(a[r], w.x, acc[r][0]);
        acc[r][1] = fmaf(a[r], w.y, acc[r][1]);
        acc[r][2] = fmaf(a[r], w.z, acc[r][2]);
        acc[r][3] = fmaf(a[r], w.w, acc[r][3]);
      }
    }
    __syncthreads();
  }
  float* dst = stats + (size_t)n * 2 * D * D;
#pragma unroll
  for (int c = 0; c < 4; ++c) {
    float* row = dst + (size_t)(cb * CB + cg * 4 + c) * D + ig * TI;
#pragma unroll
    for (int r = 0; r < TI; r += 4) store4(row + r, make_float4(acc[r][c], acc[r + 1][c], acc[r + 2][c], acc[r + 3][c]));
  }
}

}  // namespace vdn

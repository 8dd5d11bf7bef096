// Read-out, RMSNorm and gate (Alg. 1 step 7; Eq. 1a, Eq. 1c) in plain fp32.
//
// One CTA per (frame, tile of 64 tokens).  The frame's read state arrives as float [d_k][d_v]
// (already the sum of the two directions), so  o[u][c] = sum_i q[u][i] * Zr[i][c].  A token's d_v
// outputs sit in 16 neighbouring lanes, which reduce the sum of squares with shuffles.
#pragma once
#include "common.cuh"

namespace vdn {

template <int D>
struct ReadoutSimtSmem {
  float Z[D][D];
  float Q[64][D + 1];
};

template <typename Tio, int D>
__global__ void __launch_bounds__(256) readout_simt_kernel(const Tio* __restrict__ q,
                                                            const float* __restrict__ read,
                                                            const float* __restrict__ gate,
                                                            Tio* __restrict__ out, Shape s, float eps) {
  constexpr int TU = 64;
  constexpr int DC = D / 16;   // output channels per thread
  extern __shared__ __align__(16) unsigned char smem_raw[];
  ReadoutSimtSmem<D>& sm = *reinterpret_cast<ReadoutSimtSmem<D>*>(smem_raw);

  const long long n = blockIdx.x;
  const int u0 = blockIdx.y * TU;
  int b, h, t;
  split_frame(s, n, b, h, t);
  const int tid = threadIdx.x;

  {
    const float* src = read + (size_t)n * D * D;
    float* dst = &sm.Z[0][0];
    for (int e = tid * 4; e < D * D; e += 256 * 4) cp_async16(dst + e, src + e);
    cp_async_commit();
  }
  for (int e = tid; e < TU * (D / 4); e += 256) {
    int uu = e / (D / 4), j4 = (e % (D / 4)) * 4;
    int u = u0 + uu;
    float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
    if (u < s.F) x = load4(q + token_offset(s, b, t, u, h) + j4);
    sm.Q[uu][j4] = x.x; sm.Q[uu][j4 + 1] = x.y; sm.Q[uu][j4 + 2] = x.z; sm.Q[uu][j4 + 3] = x.w;
  }
  cp_async_wait<0>();
  __syncthreads();

  const int tu = tid / 16, tc = tid % 16;
  float acc[4][DC];
#pragma unroll
  for (int r = 0; r < 4; ++r)
#pragma unroll
    for (int c = 0; c < DC; ++c) acc[r][c] = 0.f;

#pragma unroll 4
  for (int i = 0; i < D; ++i) {
    float qa[4];
#pragma unroll
    for (int r = 0; r < 4; ++r) qa[r] = sm.Q[tu * 4 + r][i];
    float zc[DC];
#pragma unroll
    for (int c = 0; c < DC; c += 4) {
      float4 x = load4(&sm.Z[i][tc * DC + c]);
      zc[c] = x.x; zc[c + 1] = x.y; zc[c + 2] = x.z; zc[c + 3] = x.w;
    }
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
      for (int c = 0; c < DC; ++c) acc[r][c] = fmaf(qa[r], zc[c], acc[r][c]);
  }

  const float g = gate[h];
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    float ss = 0.f;
#pragma unroll
    for (int c = 0; c < DC; ++c) ss = fmaf(acc[r][c], acc[r][c], ss);
#pragma unroll
    for (int off = 8; off >= 1; off >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, off);
    const float scale = g * rsqrtf(ss * (1.0f / D) + eps);
    const int u = u0 + tu * 4 + r;
    if (u < s.F) {
      Tio* dst = out + token_offset(s, b, t, u, h) + tc * DC;
#pragma unroll
      for (int c = 0; c < DC; c += 4)
        store4(dst + c, make_float4(acc[r][c] * scale, acc[r][c + 1] * scale, acc[r][c + 2] * scale,
                                    acc[r][c + 3] * scale));
    }
  }
}

}  // namespace vdn

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
                                                            Tio* __restrict__ out, Shape s, float eps,
                                                            const Tio* __restrict__ gate_elem,
                                                            const float* __restrict__ norm_weight,
                                                            float q_l2_eps) {
  constexpr int TU = 64;
  constexpr int DC = D / 16;   // output channels per thread
  extern __shared__ __align__(16) unsigned char smem_raw[];
  ReadoutSimtSmem<D>& sm = *reinterpret_cast<ReadoutSimtSmem<D>*>(smem_raw);

  const long long n = blockIdx.x;
  const int u0 = blockIdx.y * TU;
  int b, h, t;
  split_frame(s, n, b, h, t);
  if (t < s.t0 || t >= s.t0 + s.Tn) return;     // an anchor frame: its output rows are zeroed by the host
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

  // queries that arrive without their L2 normalisation (q_l2_eps > 0): o is linear in q, so scale the rows now
  if (q_l2_eps > 0.f) {
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      float qs = 0.f;
#pragma unroll
      for (int i = 0; i < DC; ++i) {
        const float x = sm.Q[tu * 4 + r][tc * DC + i];
        qs = fmaf(x, x, qs);
      }
#pragma unroll
      for (int off = 8; off >= 1; off >>= 1) qs += __shfl_xor_sync(0xffffffffu, qs, off);
      const float rs = rsqrtf(qs + q_l2_eps);
#pragma unroll
      for (int c = 0; c < DC; ++c) acc[r][c] *= rs;
    }
  }

  // Eq. 1c: per-head gate (null = 1), optional element-wise gate [B,T,F,H,d] and per-channel norm scale [H,d]
  const float g = gate ? gate[h] : 1.0f;
  float wn[DC];
#pragma unroll
  for (int c = 0; c < DC; ++c) wn[c] = norm_weight ? norm_weight[(size_t)h * D + tc * DC + c] : 1.0f;
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
      const size_t off = token_offset(s, b, t, u, h) + tc * DC;
      Tio* dst = out + off;
#pragma unroll
      for (int c = 0; c < DC; c += 4) {
        float4 ge = make_float4(1.f, 1.f, 1.f, 1.f);
        if (gate_elem) ge = load4(gate_elem + off + c);
        store4(dst + c, make_float4(acc[r][c] * scale * wn[c] * ge.x, acc[r][c + 1] * scale * wn[c + 1] * ge.y,
                                    acc[r][c + 2] * scale * wn[c + 2] * ge.z, acc[r][c + 3] * scale * wn[c + 3] * ge.w));
      }
    }
  }
}

}  // namespace vdn

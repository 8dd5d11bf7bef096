// Bidirectional frame scan + gather (Alg. 1 steps 5-6; Eq. A.1, Eq. A.4, Eq. 1a), plain fp32 FMA.
//
// With Z = S^T (d_k x d_v) and alpha = 1 the frame update  S_t = (S_{t-1} + B_t)(I + A_t)^{-1}
// reads  Z_t = C_t (Z_{t-1} + B_t^T).  The transition acts on the key index only, so the d_v columns
// of Z evolve independently: one CTA owns W columns of one (batch, head) chain, keeps them in
// registers for the whole clip and needs no communication with the CTAs that own the other columns.
//
// Pass 1 (the scanned frames first..last in order) stores P_t^T.  Pass 2 (last..first) carries R_{t+1}^T and, before
// it folds frame t in, emits the state read by every query frame whose local window [l, h] ends at h = t (Eq. A.4):
//     P_{l-1}^T bridged by prod_{r=l..q} alpha_r  +  R_{t+1}^T bridged by prod_{r=q..t} alpha_r
// (the initial state where a side has no distant frame; with the default window {t} this is
// alpha_t (P_{t-1} + R_{t+1})^T).  Both passes are written back by the very thread that computed them, so the
// second pass needs no inter-CTA ordering.
//
// C_t is symmetric; the kernel reads it as C_t[j][i] so that each thread's row group is contiguous.
#pragma once
#include "common.cuh"

namespace vdn {

template <int D, int W>
struct ScanSmem {
  float C[D][D];
  float X[2][D][W];
};

// The read state is written as float [d_k][d_v] (row i, column c).
template <int D, int W>
__global__ void __launch_bounds__(256, 2) scan_kernel(const float* __restrict__ stats,
                                                       const float* __restrict__ inv,
                                                       float* __restrict__ fwd, float* __restrict__ read,
                                                       int T, const float* __restrict__ alpha,
                                                       const float* __restrict__ s0, int H,
                                                       float additive_bscale, Window win) {
  constexpr int TI = D / 32;          // rows per thread
  constexpr int NCG = W / 4;          // column groups of 4
  static_assert(256 / NCG * TI == D, "thread tiling must cover D rows");
  extern __shared__ __align__(16) unsigned char smem_raw[];
  ScanSmem<D, W>& sm = *reinterpret_cast<ScanSmem<D, W>*>(smem_raw);

  const int bh = blockIdx.x;
  const int c0 = blockIdx.y * W;
  const int tid = threadIdx.x;
  const int cg = tid % NCG, ig = tid / NCG;
  const int i0 = ig * TI, cc0 = cg * 4;

  // Optional extras (Eq. A.1, Eq. 1b, Eq. A.4): alpha [B,T,H,d] decays key channel i of the inherited state
  // before frame t is folded in and bridges the state read by frame t; s0 [B,H,d_v,d_k] is the text state,
  // each scan starting from half of it.
  float zinit[TI][4];
#pragma unroll
  for (int r = 0; r < TI; ++r)
#pragma unroll
    for (int c = 0; c < 4; ++c)
      zinit[r][c] = s0 ? 0.5f * s0[((size_t)bh * D + c0 + cc0 + c) * D + i0 + r] : 0.f;
  auto alpha_of = [&](int t, float (&a)[TI]) {
#pragma unroll
    for (int r = 0; r < TI; ++r)
      a[r] = alpha ? alpha[(((size_t)(bh / H) * T + t) * H + (bh % H)) * D + i0 + r] : 1.0f;
  };

  float z[TI][4];
#pragma unroll
  for (int r = 0; r < TI; ++r)
#pragma unroll
    for (int c = 0; c < 4; ++c) z[r][c] = zinit[r][c];

  int buf = 0;
  const int Tn = win.last - win.first + 1;
  for (int step = 0; step < 2 * Tn; ++step) {
    const bool forward = step < Tn;
    const int t = forward ? win.first + step : win.last - (step - Tn);
    const size_t n = (size_t)bh * T + t;

    // C_t -> shared memory (asynchronously, 16 bytes per request)
    {
      const float* src = inv + n * D * D;
      float* dst = &sm.C[0][0];
      for (int e = tid * 4; e < D * D; e += 256 * 4) cp_async16(dst + e, src + e);
      cp_async_commit();
    }

    float al[TI];
    alpha_of(t, al);
    if (!forward && (t == win.last || (t + 1) % win.chunk == 0)) {
      // gather: the query frames whose window ends at t read the reverse state carried here
      for (int qf = max(win.first, t - win.span()); qf <= t; ++qf) {
        if (win.hi(qf) != t) continue;
        const int l = win.lo(qf);
        float af[TI], ab[TI], ar[TI];
#pragma unroll
        for (int r = 0; r < TI; ++r) af[r] = ab[r] = 1.0f;
        for (int fr = l; fr <= t; ++fr) {
          alpha_of(fr, ar);
#pragma unroll
          for (int r = 0; r < TI; ++r) {
            if (fr <= qf) af[r] *= ar[r];
            if (fr >= qf) ab[r] *= ar[r];
          }
        }
        float* dst = read + ((size_t)bh * T + qf) * D * D;
#pragma unroll
        for (int r = 0; r < TI; ++r) {
          float4 x = make_float4(zinit[r][0], zinit[r][1], zinit[r][2], zinit[r][3]);
          if (l > win.first) x = load4(fwd + ((size_t)bh * T + l - 1) * D * D + (size_t)(i0 + r) * D + c0 + cc0);
          store4(dst + (size_t)(i0 + r) * D + c0 + cc0,
                 make_float4(fmaf(af[r], x.x, ab[r] * z[r][0]), fmaf(af[r], x.y, ab[r] * z[r][1]),
                             fmaf(af[r], x.z, ab[r] * z[r][2]), fmaf(af[r], x.w, ab[r] * z[r][3])));
        }
      }
    }

    // X = alpha_t * Z + B_t^T (this CTA's columns).  Additive baseline (additive_bscale > 0, Eq. 3c): the write is
    // not resolved against the frame's keys, X = alpha_t * Z and Z_t = C_t X + B_t^T / sqrt(F), with C_t = I - A_t/F.
    const bool additive = additive_bscale > 0.f;
    float badd[TI][4];
    {
      // B_t is stored [d_v][d_k]: element (c, i) is B_t^T[i][c]
      const float* bsrc = stats + n * 2 * D * D + (size_t)(D + c0 + cc0) * D + i0;
      float bt[TI][4];
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        if constexpr (TI == 4) {
          float4 x = load4(bsrc + (size_t)c * D);
          bt[0][c] = x.x; bt[1][c] = x.y; bt[2][c] = x.z; bt[3][c] = x.w;
        } else {
          float2 x = *reinterpret_cast<const float2*>(bsrc + (size_t)c * D);
          bt[0][c] = x.x; bt[1][c] = x.y;
        }
      }
#pragma unroll
      for (int r = 0; r < TI; ++r)
      {
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          badd[r][c] = additive ? additive_bscale * bt[r][c] : 0.f;
          if (additive) bt[r][c] = 0.f;
        }
        store4(&sm.X[buf][i0 + r][cc0], make_float4(fmaf(al[r], z[r][0], bt[r][0]), fmaf(al[r], z[r][1], bt[r][1]),
                                                     fmaf(al[r], z[r][2], bt[r][2]), fmaf(al[r], z[r][3], bt[r][3])));
      }
    }
    cp_async_wait<0>();
    __syncthreads();

    // Z = C_t X  (+ the unresolved write of the additive baseline)
#pragma unroll
    for (int r = 0; r < TI; ++r)
#pragma unroll
      for (int c = 0; c < 4; ++c) z[r][c] = badd[r][c];
#pragma unroll 8
    for (int j = 0; j < D; ++j) {
      float a[TI];
      if constexpr (TI == 4) {
        float4 v = load4(&sm.C[j][i0]);
        a[0] = v.x; a[1] = v.y; a[2] = v.z; a[3] = v.w;
      } else {
        float2 v = *reinterpret_cast<const float2*>(&sm.C[j][i0]);
        a[0] = v.x; a[1] = v.y;
      }
      float4 x = load4(&sm.X[buf][j][cc0]);
#pragma unroll
      for (int r = 0; r < TI; ++r) {
        z[r][0] = fmaf(a[r], x.x, z[r][0]);
        z[r][1] = fmaf(a[r], x.y, z[r][1]);
        z[r][2] = fmaf(a[r], x.z, z[r][2]);
        z[r][3] = fmaf(a[r], x.w, z[r][3]);
      }
    }
    __syncthreads();   // everyone is done with C before the next step overwrites it
    buf ^= 1;

    if (forward) {
      float* dst = fwd + n * D * D;
#pragma unroll
      for (int r = 0; r < TI; ++r)
        store4(dst + (size_t)(i0 + r) * D + c0 + cc0, make_float4(z[r][0], z[r][1], z[r][2], z[r][3]));
    }
    if (step == Tn - 1) {
      // the reverse scan starts from the initial state as well
#pragma unroll
      for (int r = 0; r < TI; ++r)
#pragma unroll
        for (int c = 0; c < 4; ++c) z[r][c] = zinit[r][c];
    }
  }
}

}  // namespace vdn

// Resolve (Eq. 5, Alg. 1 step 4):  C_t = (I + A_t)^{-1}, d = 128, with the O(d^3) part of the elimination on
// the tcgen05 tensor cores at fp32 accuracy.  One CTA per frame; the matrix lives in TMEM.
//
// Blocked Gauss-Jordan, 16 pivots per step (8 steps), no pivot search (I + A_t is SPD, eigenvalues >= 1).
// With P the pivot indices of a step, G = M[P][P] and Gi = G^{-1}, the in-place inverse update is
//     rows outside P :  M[i][:] += c_i M[P][:],   c_i = -M[i][P] Gi,          then  M[i][P] = c_i
//     rows inside  P :  M[a][:] += (Gi[a] - e_a) M[P][:]   (= Gi[a] M[P][:]), then  M[a][P] = Gi[a]
// i.e. one rank-16 update  M += Cm * M[P][:]  of the whole matrix plus a 128 x 16 column fix.  The rank-16
// update is a 128 x 128 x 16 MMA accumulating into the TMEM-resident matrix.  Both factors are fp32 values
// split three-way into bf16 parts (24 mantissa bits); the six partial products of weight >= 2^-24 are
// accumulated in fp32, so the update carries fp32 accuracy.
//   * The 16 x 16 pivot block is inverted in plain fp32 inside the warp that owns those rows, one row per lane,
//     the pivot rows travelling by shuffle.
//   * Every thread owns one matrix row (its TMEM lane).  The 16 pivot rows M[P][:] are the B operand of the update,
//     K-major with one row per thread: thread j needs M[P_k][j], k = 0..15 -- a column of rows that sit in sixteen
//     other TMEM lanes.  The warp that owns those lanes reads them (tcgen05.ld) and puts them in shared memory as
//     plain fp32 rows (8 KB, sixteen 16-byte stores per lane); after one barrier every thread picks up its column
//     with sixteen conflict-free 4-byte reads.  (An earlier version took M[P_k][j] = +-M[j][P_k] from the thread's own
//     row instead -- exact while the matrix stays symmetric up to the sign pattern of in-place elimination, but the
//     rounding of the updates breaks that symmetry a little at every step, and pivot rows taken from the columns cost
//     a factor of the condition number in accuracy: a left residual of 8e-2 instead of 8e-5 at lambda_max = 2000 in
//     an fp32 emulation, 5e-6 instead of 1e-6 of the largest entry on benign matrices.)
//   * The 128 x 16 coefficients Cm = -M[:, P] Gi are a matrix product as well, in a first, 128 x 16 x 16 MMA into the
//     pivot columns themselves; each thread reads its row back and fixes the sign.  Its A operand is the pivot-row
//     operand just written: row i of it is M[P][i], which equals M[i][P] up to the sign pattern (minus for a row
//     whose block has been a pivot block already, plus otherwise) and up to rounding.  This direction of the
//     substitution is harmless -- the update stays an exact row operation with the true pivot rows, only its
//     coefficients are perturbed at rounding level (same fp32 emulation: left residual 1.1e-4 against 0.8e-4 with
//     the true columns at lambda_max = 2000) -- and it saves forming a second operand per step.  Formed with fp32
//     FMAs (256 per thread and step) the coefficients were the largest item of a kernel that is bound by
//     instruction issue.
//   * The operand rows of the 16 pivot rows themselves are never needed: as A rows they produce the pivot rows'
//     coefficients, which are replaced by Gi; as B rows they produce the update of the pivot columns, which the
//     column fix overwrites.  The warp that owns the pivot rows therefore writes no operand at all, and the sixteen
//     other rows of that warp are written by half of a neighbouring warp while the pivot block is being inverted.
// The matrix that is inverted is I + (A_t + A_t^T)/2: the stored statistics are symmetric only up to the bf16
// rounding of one factor, and the symmetric part is the natural reading of Eq. 3b (and keeps Proposition 1).
// The inverse is written as three bf16 parts C1 + C2 + C3 for the tensor-core scan.
#pragma once
#include <cuda_bf16.h>

#include "common.cuh"
#include "tc_common.cuh"

namespace vdn {

// 1/x for x >= 1 (a pivot of an SPD matrix with eigenvalues >= 1): hardware approximation plus one Newton
// step, good to about 1 ulp, on a much shorter dependency chain than the correctly rounded reciprocal.
__device__ __forceinline__ float fast_rcp(float x) {
  float r;
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
  return fmaf(r, fmaf(-x, r, 1.0f), r);
}

struct ResolveTc {
  static constexpr int D = 128;
  static constexpr int NB = 16;                       // pivots per step
  static constexpr int CM_BYTES = 128 * 128;          // coefficients, K-major: 128 rows x 128 B; part p of a row sits in
                                                      // bytes [32 p, 32 p + 32) (K = 16 bf16), 32 B unused
  static constexpr int PR_BYTES = 128 * 128;          // pivot rows, K-major as well: row j = column j of the 16 pivot
                                                      // rows, parts laid out like the coefficients
  static constexpr int OFF_CM = 0;
  static constexpr int PRF_STRIDE = D + 4;            // floats per fp32 pivot row: the sixteen lanes' 16-byte stores conflict two by two, the minimum
  static constexpr int OFF_PR = CM_BYTES;
  static constexpr int OFF_GIB = OFF_PR + PR_BYTES;   // Gi as an MMA operand: 16 rows x 128 B, three parts per row
  static constexpr int OFF_GI = OFF_GIB + 2048;       // Gi, 16 x 16 floats (for the pivot rows themselves)
  static constexpr int OFF_PRF = OFF_CM;              // the 16 pivot rows in fp32, [16][PRF_STRIDE]: in the coefficient
                                                      // operand's place until the coefficients exist (four CTAs per SM
                                                      // leave no room for a buffer of their own)
  static constexpr int OFF_BAR = OFF_GI + 1024;
  static_assert(16 * PRF_STRIDE * 4 <= CM_BYTES, "the fp32 pivot rows fit in the coefficient operand");
  static constexpr int SMEM_BYTES = OFF_BAR + 64 + 1024;
  static constexpr int THREADS = 160;                 // 4 row warps + 1 MMA warp
};

__global__ void __launch_bounds__(ResolveTc::THREADS, 4)
resolve_tc_kernel(const float* __restrict__ stats, __nv_bfloat16* __restrict__ csplit, long long nframes,
                  tc::DevStatus ds, Shape shp) {
  using namespace tc;
  using R = ResolveTc;
  constexpr int D = R::D;
  extern __shared__ unsigned char smem_dyn[];
  const uint32_t base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
  unsigned char* base_ptr = smem_dyn + (base - smem_u32(smem_dyn));
  const uint32_t OPREADY = base + R::OFF_BAR, MMADONE = base + R::OFF_BAR + 8;
  const uint32_t XREADY = base + R::OFF_BAR + 16, CDONE = base + R::OFF_BAR + 24;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(base_ptr + R::OFF_BAR + 32);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(base_ptr + R::OFF_BAR + 36);
  float* gi = reinterpret_cast<float*>(base_ptr + R::OFF_GI);
  const WaitCtx wc(abort_flag, ds);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const long long n = blockIdx.x;
  if (n >= nframes) return;
  if ((int)(n % shp.T) < shp.t0 || (int)(n % shp.T) >= shp.t0 + shp.Tn) return;   // an anchor frame: not scanned

  if (threadIdx.x == 0) {
    mbar_init(OPREADY, 4);                    // one arrival per row warp
    mbar_init(MMADONE, 1);
    mbar_init(XREADY, 4);
    mbar_init(CDONE, 1);
    *abort_flag = 0;
    mbar_fence_init();
  }
  if (warp == 4) {
    tmem_alloc(smem_u32(tmem_slot), 128);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 4) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = make_idesc_bf16(128, 128, false, false);
      constexpr int PA[6] = {0, 2, 1, 0, 1, 0};   // (coefficient part, pivot-row part), smallest first
      constexpr int PB[6] = {2, 0, 1, 1, 0, 0};
      constexpr uint32_t idesc_c = make_idesc_bf16(128, 16, false, false);
      for (int step = 0; step < D / R::NB; ++step) {
        // ---- coefficients: M[:, P] <- Y Gi (128 x 16 x 16), Y = the pivot-row operand the row threads just wrote
        // (row i = M[P][i] = +-M[i][P]), Gi = the inverse of the pivot block; each thread fixes the sign of its row
        const int p0c = (((int)(blockIdx.x & 3) * 2 + step) & 7) * R::NB;
        if (!mbar_wait(XREADY, step & 1, wc)) break;
        tc_fence_after_sync();
#pragma unroll
        for (int pr = 0; pr < 6; ++pr) {
          const uint64_t adesc = make_smem_desc(base + R::OFF_PR + PA[pr] * 32, 16, 1024);
          const uint64_t bdesc = make_smem_desc(base + R::OFF_GIB + PB[pr] * 32, 16, 1024);
          mma_bf16_ss(tmem_base + p0c, adesc, bdesc, idesc_c, pr == 0 ? 0u : 1u);
        }
        mma_commit(CDONE);
        // ---- the rank-16 update of the whole matrix
        if (!mbar_wait(OPREADY, step & 1, wc)) break;
        tc_fence_after_sync();
#pragma unroll
        for (int pr = 0; pr < 6; ++pr) {
          const uint64_t adesc = make_smem_desc(base + R::OFF_CM + PA[pr] * 32, 16, 1024);
          const uint64_t bdesc = make_smem_desc(base + R::OFF_PR + PB[pr] * 32, 16, 1024);
          mma_bf16_ss(tmem_base, adesc, bdesc, idesc, 1u);
        }
        mma_commit(MMADONE);
      }
    }
  } else {
    // ------------------------------------------------------------------ row threads
    const int row = warp * 32 + lane;
    const uint32_t trow = tmem_base + ((uint32_t)(warp * 32) << 16);
    // M = I + (A_t + A_t^T)/2 into TMEM.  The stored block is K^T (beta K) with one factor rounded to bf16,
    // symmetric only up to that rounding; its symmetric part is what gets inverted (the coefficients below
    // rely on the symmetry).  Column `row` is read with
    // consecutive lanes on consecutive addresses, row `row` as 16-byte pieces (mostly L1/L2 hits).
    {
      const float* col = stats + (size_t)n * (2 * D * D) + row;
      const float4* rw = reinterpret_cast<const float4*>(stats + (size_t)n * (2 * D * D) + (size_t)row * D);
#pragma unroll 1
      for (int cc = 0; cc < 4; ++cc) {
        float v[32];
#pragma unroll
        for (int e = 0; e < 32; ++e) v[e] = __ldg(col + (size_t)(cc * 32 + e) * D);
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          const float4 x = __ldg(rw + cc * 8 + e);
          v[4 * e] = 0.5f * (v[4 * e] + x.x);
          v[4 * e + 1] = 0.5f * (v[4 * e + 1] + x.y);
          v[4 * e + 2] = 0.5f * (v[4 * e + 2] + x.z);
          v[4 * e + 3] = 0.5f * (v[4 * e + 3] + x.w);
        }
#pragma unroll
        for (int e = 0; e < 32; ++e)
          if (cc * 32 + e == row) v[e] += 1.0f;
        tmem_st32(trow + cc * 32, v);
      }
      tmem_wait_st();
    }

    // Pivot blocks may be taken in any order (symmetric pivoting of an SPD matrix).  CTAs that share an SM start
    // at different blocks, so that their serial sections (the 16 x 16 inverse, done by the warp that owns the
    // pivot rows) fall on different warp schedulers instead of queueing on one.
    const int blk0 = (int)((blockIdx.x & 3) * 2);
    bool ok = true;
    float* prf = reinterpret_cast<float*>(base_ptr + R::OFF_PRF);  // fp32 pivot rows
    auto store_operand_row = [&](int off, int r, const float (&val)[16]) {
      uint4 w[3][2];
#pragma unroll
      for (int q = 0; q < 8; ++q) {
        uint32_t a1, a2, a3;
        split3_pair(val[2 * q], val[2 * q + 1], a1, a2, a3);
        reinterpret_cast<uint32_t*>(&w[0][q >> 2])[q & 3] = a1;
        reinterpret_cast<uint32_t*>(&w[1][q >> 2])[q & 3] = a2;
        reinterpret_cast<uint32_t*>(&w[2][q >> 2])[q & 3] = a3;
      }
      unsigned char* orow = base_ptr + off + r * 128;
#pragma unroll
      for (int part = 0; part < 3; ++part) {
        *reinterpret_cast<uint4*>(orow + (((2 * part) ^ (r & 7)) * 16)) = w[part][0];
        *reinterpret_cast<uint4*>(orow + (((2 * part + 1) ^ (r & 7)) * 16)) = w[part][1];
      }
    };
    // The pivot-row operand's rows that belong to the pivot rows themselves are never needed (see below); they are
    // zero from the start rather than whatever the memory held.
    {
      uint4* z = reinterpret_cast<uint4*>(base_ptr + R::OFF_PR + row * 128);
#pragma unroll
      for (int e = 0; e < 8; ++e) z[e] = make_uint4(0u, 0u, 0u, 0u);
    }
#pragma unroll 1
    for (int step = 0; step < D / R::NB; ++step) {
      const int blk = (blk0 + step) & 7;
      const int p0 = blk * R::NB;
      const bool owner = (row >> 4) == blk;               // rows p0 .. p0+15: 16 lanes of warp blk/2
      const bool eliminated = (((row >> 4) - blk0) & 7) < step;   // this row's block was a pivot block already
      float x[16];

      // ---- the 16 pivot rows, as they stand before this step, to shared memory in fp32 (the warp that owns them)
      if (warp == (blk >> 1)) {
        tmem_ld16(trow + p0, x);                          // the pivot block itself: this row's entries in the pivot columns
#pragma unroll 1
        for (int cc = 0; cc < 4; ++cc) {
          float v[32];
          tmem_ld32(trow + cc * 32, v);
          tmem_wait_ld();
          if (owner) {
            float* dst = prf + (row & 15) * R::PRF_STRIDE + cc * 32;
#pragma unroll
            for (int e = 0; e < 32; e += 4) store4(dst + e, make_float4(v[e], v[e + 1], v[e + 2], v[e + 3]));
          }
        }
      }
      // the pivot rows are in shared memory -- or a wait of the step before ran out somewhere: a thread that gave up
      // comes here all the same (`continue` below, not `break`), so that nobody is left standing at this barrier
      if (named_barrier_or(1, 128, !ok)) { ok = false; break; }
      // thread j's column of the pivot rows: one row of the K-major operand (row = output column).  The warp that
      // owns the pivot rows does this later, under the coefficient MMA: it is the one everybody waits for.
      float y[16];
      auto load_pivot_column = [&](int r) {
#pragma unroll
        for (int k = 0; k < 16; ++k) y[k] = prf[k * R::PRF_STRIDE + r];
      };
      if (warp != (blk >> 1)) { load_pivot_column(row); store_operand_row(R::OFF_PR, row, y); }
      if (warp == (((blk >> 1) + 1) & 3) && lane < 16) {
        // the sixteen rows that share a warp with the pivot rows: that warp is busy with the pivot block
        const int hrow = (blk ^ 1) * 16 + lane;
        load_pivot_column(hrow);
        store_operand_row(R::OFF_PR, hrow, y);
      }
      if (warp == (blk >> 1)) {
        // ---- invert the 16 x 16 pivot block: lane (l0 + a) holds row a; pivot rows travel by shuffle
        const int l0 = (blk & 1) * 16;
        float g[16];
#pragma unroll
        for (int j = 0; j < 16; ++j) g[j] = x[j];
#pragma unroll
        for (int p = 0; p < 16; ++p) {
          float rp[16];
#pragma unroll
          for (int j = 0; j < 16; ++j) rp[j] = __shfl_sync(0xffffffffu, g[j], l0 + p);
          const float ip = fast_rcp(rp[p]);
          const bool prow = lane == l0 + p;
          const float f = prow ? -1.0f : g[p];              // coefficient on the scaled pivot row
          const uint32_t keep = prow ? 0u : 0xFFFFFFFFu;    // the pivot row itself restarts from zero
          const float fi = f * ip;
#pragma unroll
          for (int j = 0; j < 16; ++j) g[j] = fmaf(-fi, rp[j], __uint_as_float(__float_as_uint(g[j]) & keep));
          g[p] = prow ? ip : -fi;
        }
        if (owner) {
          // Gi row a in fp32 for this pivot row's own coefficients, and Gi as three bf16 parts for the tensor cores
          const int a = row & 15;
          float* dst = gi + a * 16;
#pragma unroll
          for (int j = 0; j < 16; j += 4) store4(dst + j, make_float4(g[j], g[j + 1], g[j + 2], g[j + 3]));
        }
        __syncwarp();
        if (owner) {
          // ... whose rows must be the COLUMNS of Gi (c = -x Gi contracts x with a column).  The block of an
          // elimination in progress is symmetric only up to rounding, so the column is read back from the rows just
          // written, not taken to be the row.
          const int a = row & 15;
          float gc[16];
#pragma unroll
          for (int j = 0; j < 16; ++j) gc[j] = gi[j * 16 + a];
          uint4 w[3][2];
#pragma unroll
          for (int q = 0; q < 8; ++q) {
            uint32_t a1, a2, a3;
            split3_pair(gc[2 * q], gc[2 * q + 1], a1, a2, a3);
            reinterpret_cast<uint32_t*>(&w[0][q >> 2])[q & 3] = a1;
            reinterpret_cast<uint32_t*>(&w[1][q >> 2])[q & 3] = a2;
            reinterpret_cast<uint32_t*>(&w[2][q >> 2])[q & 3] = a3;
          }
          unsigned char* grow = base_ptr + R::OFF_GIB + a * 128;
#pragma unroll
          for (int part = 0; part < 3; ++part) {
            *reinterpret_cast<uint4*>(grow + (((2 * part) ^ (a & 7)) * 16)) = w[part][0];
            *reinterpret_cast<uint4*>(grow + (((2 * part + 1) ^ (a & 7)) * 16)) = w[part][1];
          }
        }
      }
      // (the fp32 pivot rows share their memory with the coefficient operand, which the warps write once the
      // coefficient MMA has completed, i.e. after all four arrivals below: every read of them comes before)
      fence_proxy_async_smem();
      tc_fence_before_sync();
      mbar_arrive_warp(XREADY);

      // ---- coefficients: c = -M[i][P] Gi = -+(Y Gi) from the tensor cores; a pivot row a takes Gi[a]
      if (!mbar_wait(CDONE, step & 1, wc)) { ok = false; continue; }
      tc_fence_after_sync();
      float c[16];
      tmem_ld16(trow + p0, c);
      tmem_wait_ld();
      if (owner) {
        const float* src = gi + (row & 15) * 16;
#pragma unroll
        for (int k = 0; k < 16; k += 4) {
          const float4 gq = load4(src + k);
          c[k] = gq.x; c[k + 1] = gq.y; c[k + 2] = gq.z; c[k + 3] = gq.w;
        }
      } else {
#pragma unroll
        for (int k = 0; k < 16; ++k) c[k] = eliminated ? c[k] : -c[k];
      }
      // ---- A operand: this row's 16 update coefficients (pivot rows: Gi[a] - e_a), three bf16 parts
      {
        float u[16];
#pragma unroll
        for (int k = 0; k < 16; ++k) u[k] = (owner && (row & 15) == k) ? c[k] - 1.0f : c[k];
        store_operand_row(R::OFF_CM, row, u);
      }
      fence_proxy_async_smem();
      tc_fence_before_sync();
      mbar_arrive_warp(OPREADY);
      if (!mbar_wait(MMADONE, step & 1, wc)) { ok = false; continue; }
      tc_fence_after_sync();
      // ---- column fix: M[i][P] = c (for a pivot row: Gi[a])
      tmem_st16(trow + p0, c);
      tmem_wait_st();
    }
    if (ok) {
      // ---- the inverse as three bf16 parts; this thread holds row `row` of it and stores it transposed (the
      // inverse is symmetric), so that the 32 lanes of a warp write 32 consecutive elements
      __nv_bfloat16* c1 = csplit + (size_t)n * (3 * D * D) + row;
#pragma unroll 1
      for (int cc = 0; cc < 4; ++cc) {
        float v[32];
        tmem_ld32(trow + cc * 32, v);
        tmem_wait_ld();
#pragma unroll
        for (int e = 0; e < 32; e += 2) {
          uint32_t w1, w2, w3;
          split3_pair(v[e], v[e + 1], w1, w2, w3);
          unsigned short* o = reinterpret_cast<unsigned short*>(c1 + (size_t)(cc * 32 + e) * D);
          o[0] = (unsigned short)(w1 & 0xFFFFu);
          o[D] = (unsigned short)(w1 >> 16);
          o[(size_t)D * D] = (unsigned short)(w2 & 0xFFFFu);
          o[(size_t)D * D + D] = (unsigned short)(w2 >> 16);
          o[(size_t)2 * D * D] = (unsigned short)(w3 & 0xFFFFu);
          o[(size_t)2 * D * D + D] = (unsigned short)(w3 >> 16);
        }
      }
    }
  }
  __syncwarp();
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 4) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, 128);
  }
}

}  // namespace vdn

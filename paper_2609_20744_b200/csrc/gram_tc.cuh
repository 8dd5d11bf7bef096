// Frame statistics (Eq. 3b) on the tcgen05 tensor cores, bf16 operands, fp32 accumulation in TMEM.
//
//   [ A_t | B_t^T ] = (Diag(beta_t) K_t)^T [ K_t | V_t ]          128 x 256 per frame (d = 128)
// (stored transposed: A_t is symmetric, and the second block becomes B_t itself, d_v x d_k)
//
// The contraction index is the token, so both operands are "MN-major": a token's 128 channels are
// contiguous in memory, and TMA drops each 128-token tile into shared memory as 64-channel boxes with
// the 128-byte swizzle, exactly the canonical MN-major layout the MMA reads.
//
// Persistent CTAs, one per SM, loop over frames (b,h,t).  Warp roles:
//   warp 0      TMA producer: K and V tiles (4 boxes of 16 KB) into a 3-stage ring
//   warp 1      MMA issuer (one thread) and TMEM owner
//   warps 2-9   weighting: K' = bf16(beta) * K in packed bf16 arithmetic, written to a second buffer in two halves of
//               64 tokens so the MMA of one half overlaps the weighting of the other.  A thread does 64 bytes of a
//               token row: the stage is held for the length of this chain (load, multiply, store, proxy fence,
//               arrive), and eight warps make it shorter than four (-3 %; sixteen are slower again)
//   warps 10-13 drain: once per frame, the finished accumulator (of two) TMEM -> registers -> global fp32 [2d][d]
//               (A_t, then B_t), while the other warps are already on the next frame
// Rows past the end of a frame are zero-filled by TMA (the map has F as its own dimension) and their
// beta is forced to zero.  Every mbarrier wait is bounded.
#pragma once
#include <cuda_bf16.h>

#include "common.cuh"
#include "tc_common.cuh"

namespace vdn {

// EXACT = true (VDN_FLAG_EXACT_STATS): the weighted key beta k is carried as TWO bf16 numbers, the rounded product and
// its rounding residue (beta k has 16 significant bits, so the pair holds it exactly), and every tile is contracted
// twice, once per part, into the same accumulator.  The statistics are then the exact fp32-accumulated sums of the
// 16-bit inputs -- what the plain-fp32 kernels compute -- with beta rounded to bf16 (a per-token weight change of
// 2^-9, the same in A_t and B_t).  Why it matters: rounding each token's weighted key to bf16 moves it by 2^-9 in a
// direction of its own; the update of Eq. 5 damps what a frame writes along a repeated key by 1 / (1 + lambda_max)
// but not those residues, so for frames of (nearly) identical keys (Sec. A.3) the error relative to the result grows
// like lambda_max 2^-10.  Costs: twice the tensor-core work, a second operand buffer (so a two-stage ring).
template <bool EXACT>
struct GramTcCfg {
  static constexpr int D = 128;
  static constexpr int TILE = 128;                 // tokens per tile
  static constexpr int STAGES = EXACT ? 2 : 3;
  static constexpr int PARTS = EXACT ? 2 : 1;      // bf16 parts of the weighted key
  static constexpr int BOX_BYTES = TILE * 128;     // one 64-channel box: 128 tokens x 128 B
  static constexpr int STAGE_BYTES = 4 * BOX_BYTES;       // K lo, K hi, V lo, V hi
  static constexpr int KP_HALF_BYTES = 2 * 64 * 128;      // 2 boxes x 64 tokens x 128 B
  static constexpr int OFF_KP = STAGES * STAGE_BYTES;     // [part][half]
  static constexpr int OFF_BAR = OFF_KP + PARTS * 2 * KP_HALF_BYTES;
  static constexpr int USED_BYTES = OFF_BAR + 128;
  static constexpr int SMEM_BYTES = EXACT ? USED_BYTES + 1024 : 232448;   // plain: everything an SM offers one CTA; the
                                                                          // slack absorbs the 1024-byte alignment
  static constexpr int THREADS = 448;
};
using GramTc = GramTcCfg<false>;

template <bool EXACT>
__global__ void __launch_bounds__(GramTcCfg<EXACT>::THREADS, 1)
gram_tc_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
               const float* __restrict__ beta, float* __restrict__ stats, Shape s, tc::DevStatus ds) {
  using namespace tc;
  using G = GramTcCfg<EXACT>;
  extern __shared__ unsigned char smem_dyn[];
  const uint32_t base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
  unsigned char* base_ptr = smem_dyn + (base - smem_u32(smem_dyn));

  // barrier block
  const uint32_t bar0 = base + G::OFF_BAR;
  auto FULL = [&](int i) { return bar0 + 8u * i; };            // 3
  auto EMPTY = [&](int i) { return bar0 + 8u * (3 + i); };     // 3
  auto SCALED = [&](int i) { return bar0 + 8u * (6 + i); };    // 2
  auto KPFREE = [&](int i) { return bar0 + 8u * (8 + i); };    // 2
  auto ACCFULL = [&](int i) { return bar0 + 8u * (10 + i); };  // 2
  auto ACCEMPTY = [&](int i) { return bar0 + 8u * (12 + i); }; // 2
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(base_ptr + G::OFF_BAR + 8 * 14);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(base_ptr + G::OFF_BAR + 8 * 14 + 4);
  const WaitCtx wc(abort_flag, ds);

  if ((base - smem_u32(smem_dyn)) + G::USED_BYTES > (uint32_t)G::SMEM_BYTES) {
    // the dynamic shared memory window starts too far from a 1024-byte boundary for the layout to fit
    if (threadIdx.x == 0) atomicExch(ds.word, kStatusInternal);
    return;
  }
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int ntiles = (s.F + G::TILE - 1) / G::TILE;
  const long long nitems = s.work_items();

  if (threadIdx.x == 0) {
    for (int i = 0; i < G::STAGES; ++i) { mbar_init(FULL(i), 1); mbar_init(EMPTY(i), 1); }
    for (int i = 0; i < 2; ++i) {
      mbar_init(SCALED(i), 8); mbar_init(KPFREE(i), 1);      // one arrival per weighting warp
      mbar_init(ACCFULL(i), 1);  mbar_init(ACCEMPTY(i), 4);   // ... per drain warp
    }
    *abort_flag = 0;
    mbar_fence_init();
    tma_prefetch_desc(&tmK);
    tma_prefetch_desc(&tmV);
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(tmem_slot), 512);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      for (long long item = blockIdx.x; item < nitems && ok; item += gridDim.x) {
        int b, h, t;
        split_work(s, item, b, h, t);
        for (int tile = 0; tile < ntiles; ++tile, ++it) {
          const int st = it % G::STAGES;
          if (!mbar_wait(EMPTY(st), ((it / G::STAGES) & 1) ^ 1, wc)) { ok = false; break; }
          mbar_arrive_expect_tx(FULL(st), G::STAGE_BYTES);
          const uint32_t dst = base + st * G::STAGE_BYTES;
          const int u0 = tile * G::TILE;
          tma_load_5d(dst + 0 * G::BOX_BYTES, &tmK, FULL(st), 0, h, u0, t, b);
          tma_load_5d(dst + 1 * G::BOX_BYTES, &tmK, FULL(st), 64, h, u0, t, b);
          tma_load_5d(dst + 2 * G::BOX_BYTES, &tmV, FULL(st), 0, h, u0, t, b);
          tma_load_5d(dst + 3 * G::BOX_BYTES, &tmV, FULL(st), 64, h, u0, t, b);
        }
      }
      if (!ok) {
        // give copies that are already in flight (`it` were issued) a bounded chance to land before the CTA retires
        mbar_drain_ring(FULL(0), G::STAGES, it);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = make_idesc_bf16(128, 256, true, true);
      uint32_t it = 0, ai = 0;
      bool ok = true;
      for (long long item = blockIdx.x; item < nitems && ok; item += gridDim.x, ++ai) {
        const int a = ai & 1;
        if (!mbar_wait(ACCEMPTY(a), ((ai >> 1) & 1) ^ 1, wc)) { ok = false; break; }
        tc_fence_after_sync();
        const uint32_t acc = tmem_base + a * 256;
        for (int tile = 0; tile < ntiles && ok; ++tile, ++it) {
          const int st = it % G::STAGES;
          if (!mbar_wait(FULL(st), (it / G::STAGES) & 1, wc)) { ok = false; break; }
          for (int half = 0; half < 2; ++half) {
            if (!mbar_wait(SCALED(half), it & 1, wc)) { ok = false; break; }
            tc_fence_after_sync();
            const uint32_t b_base = base + st * G::STAGE_BYTES + half * 64 * 128;
#pragma unroll
            for (int part = 0; part < G::PARTS; ++part) {     // EXACT: the residue part first (smallest terms first)
              const int pp = G::PARTS - 1 - part;
              const uint32_t a_base = base + G::OFF_KP + (pp * 2 + half) * G::KP_HALF_BYTES;
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                const uint64_t adesc = make_smem_desc(a_base + j * 2048, 64 * 128, 1024);
                const uint64_t bdesc = make_smem_desc(b_base + j * 2048, G::BOX_BYTES, 1024);
                mma_bf16_ss(acc, adesc, bdesc, idesc, (tile | half | j | part) != 0 ? 1u : 0u);
              }
            }
            mma_commit(KPFREE(half));
          }
          if (!ok) break;
          mma_commit(EMPTY(st));
        }
        if (ok) mma_commit(ACCFULL(a));
      }
    }
  } else if (warp >= 10) {
    // ------------------------------------------------------------------ drain warps
    // TMEM -> registers -> global fp32 [2d][d].  Accumulator lane = key channel i, column = column of [K|V];
    // stored transposed so that the 32 lanes of a warp write 32 consecutive floats.
    const int qd = warp & 3;                  // TMEM lane quarter this warp may read
    const int row = qd * 32 + lane;           // accumulator row drained by this thread
    uint32_t ai = 0;
    for (long long item = blockIdx.x; item < nitems; item += gridDim.x, ++ai) {
      const int a = ai & 1;
      if (!mbar_wait(ACCFULL(a), (ai >> 1) & 1, wc)) break;
      tc_fence_after_sync();
      const uint32_t taddr = tmem_base + ((uint32_t)(qd * 32) << 16) + a * 256;
      int b, h, t;
      const long long n = split_work(s, item, b, h, t);
      float* dst = stats + (size_t)n * (2 * G::D * G::D) + row;
#pragma unroll 1
      for (int cc = 0; cc < 8; ++cc) {
        float v[32];
        tmem_ld32(taddr + cc * 32, v);
        tmem_wait_ld();
#pragma unroll
        for (int e = 0; e < 32; ++e) dst[(size_t)(cc * 32 + e) * G::D] = v[e];
      }
      tc_fence_before_sync();
      mbar_arrive_warp(ACCEMPTY(a));            // the accumulator is free for the frame after next
    }
  } else {
    // ------------------------------------------------------------------ weighting warps: K' = beta * K
    const int ts = threadIdx.x - 64;          // 0..255
    const int r = ts >> 2, c = (ts >> 1) & 1; // row within the half, 64-channel box
    const int q4 = (ts & 1) * 4;              // which four 16-byte chunks of the 128-byte row
    uint32_t it = 0;
    bool ok = true;

    // beta of (frame, tile), one value per half for this thread's row; zero past the end of the frame.
    // Fetched one tile ahead: the loads are scattered 4-byte reads (one head out of H) whose L2 latency would
    // otherwise sit between a tile's arrival and its weighting.
    auto load_beta = [&](long long witem, int tile, float (&bw)[2]) {
      if (witem >= nitems) { bw[0] = bw[1] = 0.f; return; }
      int b, h, t;
      split_work(s, witem, b, h, t);
      const float* brow = beta + ((size_t)b * s.T + t) * s.F * s.H + h;
#pragma unroll
      for (int half = 0; half < 2; ++half) {
        const int u = tile * G::TILE + half * 64 + r;
        bw[half] = (u < s.F) ? __ldg(brow + (size_t)u * s.H) : 0.f;
      }
    };

    float bnext[2];
    load_beta(blockIdx.x, 0, bnext);
    for (long long item = blockIdx.x; item < nitems && ok; item += gridDim.x) {
      for (int tile = 0; tile < ntiles && ok; ++tile, ++it) {
        const int st = it % G::STAGES;
        const float bu[2] = {bnext[0], bnext[1]};
        if (tile + 1 < ntiles) load_beta(item, tile + 1, bnext);
        else load_beta(item + gridDim.x, 0, bnext);
        if (!mbar_wait(FULL(st), (it / G::STAGES) & 1, wc)) { ok = false; break; }
#pragma unroll
        for (int half = 0; half < 2; ++half) {
          if (!mbar_wait(KPFREE(half), (it & 1) ^ 1, wc)) { ok = false; break; }
          const unsigned char* src = base_ptr + st * G::STAGE_BYTES + c * G::BOX_BYTES + (half * 64 + r) * 128;
          unsigned char* dst = base_ptr + G::OFF_KP + half * G::KP_HALF_BYTES + c * (64 * 128) + r * 128;
          // beta rounded to bf16, then one packed bf16 multiply per channel pair (round to nearest): the
          // float->bf16 conversion instruction is slow on this GPU and kept this loop from hiding under HBM
          const __nv_bfloat162 w2 = __float2bfloat162_rn(bu[half]);
          const float wf = __low2float(w2);     // EXACT: the rounded gate, as the factor of the exact product
          // all eight loads first, then the stores: written as one load-store pair per chunk the compiler
          // must keep them in order (the two shared-memory pointers might alias) and every chunk pays the
          // full shared-memory latency
          uint4 raw[4], res[4];
#pragma unroll
          for (int j = 0; j < 4; ++j) raw[j] = *reinterpret_cast<const uint4*>(src + (((q4 + j) ^ (r & 7)) * 16));
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            __nv_bfloat162* x = reinterpret_cast<__nv_bfloat162*>(&raw[j]);
            uint32_t* ru = reinterpret_cast<uint32_t*>(&res[j]);
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              if constexpr (EXACT) {
                // the product's rounding residue beta k - rn(beta k): exact in fp32 (one FMA each), at most 8
                // significant bits, so its fp32 pattern has a zero low half and the bf16 is that pattern's top half
                const uint32_t ku = *reinterpret_cast<const uint32_t*>(&x[e]);
                const __nv_bfloat162 g = __hmul2(x[e], w2);
                const uint32_t gu = *reinterpret_cast<const uint32_t*>(&g);
                const float r0 = fmaf(wf, __uint_as_float(ku << 16), -__uint_as_float(gu << 16));
                const float r1 = fmaf(wf, __uint_as_float(ku & 0xFFFF0000u), -__uint_as_float(gu & 0xFFFF0000u));
                ru[e] = __byte_perm(__float_as_uint(r0), __float_as_uint(r1), 0x7632);
                x[e] = g;
              } else {
                x[e] = __hmul2(x[e], w2);
              }
            }
          }
#pragma unroll
          for (int j = 0; j < 4; ++j) {          // chunks staggered across rows: conflict-free
            *reinterpret_cast<uint4*>(dst + (((q4 + j) ^ (r & 7)) * 16)) = raw[j];
            if constexpr (EXACT) *reinterpret_cast<uint4*>(dst + 2 * G::KP_HALF_BYTES + (((q4 + j) ^ (r & 7)) * 16)) = res[j];
          }
          fence_proxy_async_smem();
          mbar_arrive_warp(SCALED(half));
        }
      }
    }
  }

  // ------------------------------------------------------------------ teardown
  __syncwarp();
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, 512);
  }
}

}  // namespace vdn

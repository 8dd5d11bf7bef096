// Read-out (Eq. 1a), RMSNorm and gate (Eq. 1c) on the tcgen05 tensor cores, d = 128, bf16 I/O.
//
//   O_t = Q_t (P_{t-1} + R_{t+1})^T      128-token tile x 128 channels, fp32 in TMEM
//   out = gate_h * O / sqrt(mean_c O^2 + eps)   -> bf16
//
// The two states a frame reads (forward state of the frames before it, reverse state of the frames after
// it) arrive as bf16 [d_v][d_k], i.e. K-major B operands; both products go into the same accumulator,
// which is the sum of Eq. 1a.  Q tiles are K-major as they sit in memory.  Persistent CTAs loop over
// frames (b,h,t).  Warp roles:
//   warp 0      TMA producer: the frame's two states (4 boxes of 16 KB) and Q tiles (2 boxes, 3-stage ring)
//   warp 1      MMA issuer (one thread), 4 accumulators of 128 TMEM columns
//   warps 2-5   epilogue: tcgen05.ld gives every thread one whole token row, so the sum of squares is
//               thread-local; the scaled row is packed to bf16, written to a swizzled staging tile and
//               sent out with a TMA store whose map has F as its own dimension (the tail is clipped)
//   warps 6-9   (QNORM only) the queries' L2 normalisation, for callers that skip the preparation pass over Q:
//               a thread sums the squares of one token's row of the Q tile in shared memory and leaves
//               1 / sqrt(|q|^2 + eps_q) for the epilogue thread of that token, which scales its row before the norm
// Every mbarrier wait is bounded.
#pragma once
#include <cuda_bf16.h>

#include "common.cuh"
#include "tc_common.cuh"

namespace vdn {

// SHORT: the layout for short frames (few token tiles per frame).  There a frame's two states are as many bytes as
// its queries, and with one state buffer the producer could fetch the next frame's states only after the last MMA
// of this frame had retired: their latency was exposed once per frame.  SHORT keeps two state buffers and pays for
// them with one Q stage and one staging tile.
template <bool EXTRAS, bool QNORM = false, bool GATE = false, bool SHORT = false>
struct ReadoutTcCfg {
  static_assert(EXTRAS || !GATE, "the element-wise gate is one of the optional factors");
  static_assert(!(SHORT && GATE), "the gate path keeps its three staging tiles");
  static constexpr int D = 128;
  static constexpr int TILE = 128;
  // GATE: gate tiles arrive by TMA in the output staging tiles, two tiles ahead; a third staging tile takes the
  // place of a Q stage (with 3 Q stages, 2 staging tiles and a one-tile lookahead the gate path takes 2.47 ms
  // instead of 1.76 ms on the 768p clip; without a gate the third Q stage is worth more: 1.24 against 1.37 ms)
  static constexpr int QSTAGES = (GATE || SHORT) ? 2 : 3;
  static constexpr int NOUT = GATE ? 3 : (SHORT ? 1 : 2);
  static constexpr int STSTAGES = SHORT ? 2 : 1;
  static constexpr int BOX_BYTES = 128 * 128;          // 128 rows x 128 B
  static constexpr int TILE_BYTES = 2 * BOX_BYTES;     // 32 KB: state, Q tile or output tile
  static constexpr int OFF_STATE = 0;
  static constexpr int OFF_Q = STSTAGES * 2 * TILE_BYTES;
  static constexpr int OFF_OUT = OFF_Q + QSTAGES * TILE_BYTES;
  static constexpr int OFF_NW = OFF_OUT + NOUT * TILE_BYTES;   // norm weights of the current head, 128 floats
  // QNORM: 1/|q| of the tokens of QSLOTS tiles, 128 floats each.  (Four slots instead of two for the variant with
  // two Q stages: no faster, 2.16 against 2.06 ms on the 768p clip.)
  static constexpr int QSLOTS = 2;
  static constexpr int OFF_QN = OFF_NW + (EXTRAS ? 512 : 0);
  static constexpr int OFF_BAR = OFF_QN + (QNORM ? QSLOTS * 512 : 0);
  static constexpr int USED_BYTES = OFF_BAR + 256;
  static constexpr int SMEM_BYTES = USED_BYTES + 1024 <= 227 * 1024 ? USED_BYTES + 1024 : 227 * 1024;
  static constexpr int THREADS = QNORM ? 320 : 192;
  static_assert(SMEM_BYTES <= 227 * 1024, "shared memory of one SM");
};
using ReadoutTc = ReadoutTcCfg<false>;
constexpr int kReadoutShortTiles = 4;     // frames of at most this many 128-token tiles take the SHORT layout

// EXTRAS = true adds the optional factors of Eq. 1c to the epilogue: a per-channel norm scale norm_weight [H,d]
// (kept in shared memory per frame; may be null), a per-head gate that may be null (read as 1) and, with GATE, an
// element-wise (content-dependent) gate gate_elem [B,T,F,H,d] bf16 (tensor map tmG; its tiles arrive by TMA in the
// very staging tile the output is then written to, two tiles ahead).  The plain instantiation carries none of that.
template <bool EXTRAS, bool QNORM = false, bool GATE = false, bool SHORT = false>
__global__ void __launch_bounds__(ReadoutTcCfg<EXTRAS, QNORM, GATE, SHORT>::THREADS, 1)
readout_tc_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmS,
                  const __grid_constant__ CUtensorMap tmO, const __grid_constant__ CUtensorMap tmG,
                  const float* __restrict__ gate, Shape s, float eps,
                  tc::DevStatus ds, const __nv_bfloat16* __restrict__ gate_elem, const float* __restrict__ norm_weight,
                  Window win, int bridged, float q_l2_eps) {
  using namespace tc;
  using R = ReadoutTcCfg<EXTRAS, QNORM, GATE, SHORT>;
  extern __shared__ unsigned char smem_dyn[];
  const uint32_t base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
  unsigned char* base_ptr = smem_dyn + (base - smem_u32(smem_dyn));

  const uint32_t bar0 = base + R::OFF_BAR;
  auto QFULL = [&](int i) { return bar0 + 8u * i; };             // 3
  auto QEMPTY = [&](int i) { return bar0 + 8u * (3 + i); };      // 3
  auto STFULL = [&](int i) { return bar0 + 8u * (6 + i); };      // 2
  auto STEMPTY = [&](int i) { return bar0 + 8u * (8 + i); };     // 2
  auto ACCFULL = [&](int i) { return bar0 + 8u * (10 + i); };    // 4
  auto ACCEMPTY = [&](int i) { return bar0 + 8u * (14 + i); };   // 4
  auto GFULL = [&](int i) { return bar0 + 8u * (18 + i); };      // 3 (EXTRAS: gate tile landed)
  auto QNFULL = [&](int i) { return bar0 + 8u * (21 + i); };     // up to 4 (QNORM: 1/|q| of a tile written)
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(base_ptr + R::OFF_BAR + 8 * 25);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(base_ptr + R::OFF_BAR + 8 * 25 + 8);
  constexpr uint32_t QS = R::QSLOTS;
  const WaitCtx wc(abort_flag, ds);

  if ((base - smem_u32(smem_dyn)) + R::USED_BYTES > (uint32_t)R::SMEM_BYTES) {
    // the dynamic shared memory window starts too far from a 1024-byte boundary for the layout to fit
    if (threadIdx.x == 0) atomicExch(ds.word, kStatusInternal);
    return;
  }
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int ntiles = (s.F + R::TILE - 1) / R::TILE;
  const long long nitems = s.work_items();

  if (threadIdx.x == 0) {
    // a Q stage is handed back by the MMA commit and, with QNORM, by the four warps that read its rows
    for (int i = 0; i < 3; ++i) { mbar_init(QFULL(i), 1); mbar_init(QEMPTY(i), QNORM ? 5 : 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(STFULL(i), 1); mbar_init(STEMPTY(i), 1); }
    for (int i = 0; i < 4; ++i) { mbar_init(ACCFULL(i), 1); mbar_init(ACCEMPTY(i), 4); }   // one arrival per epilogue warp
    for (int i = 0; i < 3; ++i) mbar_init(GFULL(i), 1);
    for (int i = 0; i < R::QSLOTS; ++i) mbar_init(QNFULL(i), 4);
    *abort_flag = 0;
    mbar_fence_init();
    tma_prefetch_desc(&tmQ);
    tma_prefetch_desc(&tmS);
    tma_prefetch_desc(&tmO);
    if (GATE) tma_prefetch_desc(&tmG);
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
      uint32_t qi = 0, si = 0, states_issued = 0;
      bool ok = true;
      for (long long item = blockIdx.x; item < nitems && ok; item += gridDim.x, ++si) {
        int b, h, t;
        const long long n = split_work(s, item, b, h, t);
        const int sb = si % R::STSTAGES;
        if (!mbar_wait(STEMPTY(sb), ((si / R::STSTAGES) & 1) ^ 1, wc)) { ok = false; break; }
        states_issued = si + 1;
        mbar_arrive_expect_tx(STFULL(sb), 2 * R::TILE_BYTES);
        const uint32_t sdst = base + R::OFF_STATE + sb * 2 * R::TILE_BYTES;
        // Slot of the forward state in rows [nf*128, +128), of the reverse state in rows [nrev*128, +128).  With
        // decay gates every frame has its own (bridged) pair; without, the frames of a window share the states
        // stored at the window's ends (slot l_t of the forward scan, slot h_t of the reverse scan; Eq. A.4).
        const long long nf = bridged ? n : n - t + win.lo(t);
        const long long nrev = s.frames() + (bridged ? n : n - t + win.hi(t));
        tma_load_2d(sdst, &tmS, STFULL(sb), 0, (int)(nf * R::D));
        tma_load_2d(sdst + R::BOX_BYTES, &tmS, STFULL(sb), 64, (int)(nf * R::D));
        tma_load_2d(sdst + 2 * R::BOX_BYTES, &tmS, STFULL(sb), 0, (int)(nrev * R::D));
        tma_load_2d(sdst + 3 * R::BOX_BYTES, &tmS, STFULL(sb), 64, (int)(nrev * R::D));
        for (int tile = 0; tile < ntiles; ++tile, ++qi) {
          const int st = qi % R::QSTAGES;
          if (!mbar_wait(QEMPTY(st), ((qi / R::QSTAGES) & 1) ^ 1, wc)) { ok = false; break; }
          mbar_arrive_expect_tx(QFULL(st), R::TILE_BYTES);
          const uint32_t dst = base + R::OFF_Q + st * R::TILE_BYTES;
          tma_load_5d(dst, &tmQ, QFULL(st), 0, h, tile * R::TILE, t, b);
          tma_load_5d(dst + R::BOX_BYTES, &tmQ, QFULL(st), 64, h, tile * R::TILE, t, b);
        }
      }
      if (!ok) {
        // give the copies already in flight (qi query tiles, states_issued pairs of states) a bounded chance to land
        // before the CTA retires
        mbar_drain_ring(QFULL(0), R::QSTAGES, qi);
        mbar_drain_ring(STFULL(0), R::STSTAGES, states_issued);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = make_idesc_bf16(128, 128, false, false);
      uint32_t qi = 0, si = 0;
      bool ok = true;
      for (long long item = blockIdx.x; item < nitems && ok; item += gridDim.x, ++si) {
        const int sb = si % R::STSTAGES;
        if (!mbar_wait(STFULL(sb), (si / R::STSTAGES) & 1, wc)) { ok = false; break; }
        const uint32_t sbase = base + R::OFF_STATE + sb * 2 * R::TILE_BYTES;
        for (int tile = 0; tile < ntiles; ++tile, ++qi) {
          const int st = qi % R::QSTAGES;
          const int a = qi & 3;
          if (!mbar_wait(QFULL(st), (qi / R::QSTAGES) & 1, wc)) { ok = false; break; }
          if (!mbar_wait(ACCEMPTY(a), ((qi >> 2) & 1) ^ 1, wc)) { ok = false; break; }
          tc_fence_after_sync();
          const uint32_t qbase = base + R::OFF_Q + st * R::TILE_BYTES;
#pragma unroll
          for (int dirn = 0; dirn < 2; ++dirn) {
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              // both operands K-major: 16 key channels = 32 B inside a swizzled row of Q / of the state
              const uint32_t off = (j >> 2) * R::BOX_BYTES + (j & 3) * 32;
              const uint64_t adesc = make_smem_desc(qbase + off, 16, 1024);
              const uint64_t bdesc = make_smem_desc(sbase + dirn * R::TILE_BYTES + off, 16, 1024);
              mma_bf16_ss(tmem_base + a * 128, adesc, bdesc, idesc, (dirn | j) != 0 ? 1u : 0u);
            }
          }
          mma_commit(QEMPTY(st));
          mma_commit(ACCFULL(a));
        }
        if (ok) mma_commit(STEMPTY(sb));
      }
    }
  } else if (QNORM && warp >= 6) {
    // ------------------------------------------------------------------ query norms
    const int qrow = threadIdx.x - 192;         // token row inside the tile
    float* qn = reinterpret_cast<float*>(base_ptr + R::OFF_QN);
    uint32_t qi = 0;
    bool ok = true;
    for (long long item = blockIdx.x; item < nitems && ok; item += gridDim.x) {
      for (int tile = 0; tile < ntiles; ++tile, ++qi) {
        const int st = qi % R::QSTAGES;
        // One lane polls, so that the other 31 take no issue slots from the epilogue warp on the same scheduler;
        // then every lane observes the completed phase itself.
        if (lane == 0) ok = mbar_wait(QFULL(st), (qi / R::QSTAGES) & 1, wc);
        ok = __shfl_sync(0xffffffffu, ok, 0);
        if (!ok) break;
        if (!mbar_wait(QFULL(st), (qi / R::QSTAGES) & 1, wc)) { ok = false; break; }
        const unsigned char* qrowp = base_ptr + R::OFF_Q + st * R::TILE_BYTES + qrow * 128;
        // packed fp32 pairs: these warps share their schedulers with the epilogue warps, whose per-tile chain sets
        // the pace of the kernel, so every instruction here counts
        unsigned long long acc2[2] = {0ull, 0ull};
#pragma unroll
        for (int bx = 0; bx < 2; ++bx)
#pragma unroll
          for (int c = 0; c < 8; ++c) {
            // the order of the channels does not matter here; walking the chunks in swizzled order keeps the
            // eight rows of a quarter-warp on different banks
            const uint4 x = *reinterpret_cast<const uint4*>(qrowp + bx * R::BOX_BYTES + ((c ^ (qrow & 7)) * 16));
            const uint32_t* u = reinterpret_cast<const uint32_t*>(&x);
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              unsigned long long pr;
              asm("mov.b64 %0, {%1, %2};" : "=l"(pr) : "r"(u[e] << 16), "r"(u[e] & 0xFFFF0000u));
              asm("fma.rn.f32x2 %0, %1, %1, %0;" : "+l"(acc2[e & 1]) : "l"(pr));
            }
          }
        float ss;
        {
          float a0, a1, b0, b1;
          asm("mov.b64 {%0, %1}, %2;" : "=f"(a0), "=f"(a1) : "l"(acc2[0]));
          asm("mov.b64 {%0, %1}, %2;" : "=f"(b0), "=f"(b1) : "l"(acc2[1]));
          ss = (a0 + a1) + (b0 + b1);
        }
        // Slot qi % QS was last read for tile qi - QS, whose epilogue threads arrived on that tile's ACCEMPTY after
        // the read (a later tile cannot have completed that barrier again: it needs this slot first).  The Q stage
        // goes back only after this wait: measured, handing it back before the wait is slower (768p clip, 148
        // CTAs: 1.39 instead of 1.25 ms) -- the producer running further ahead of the epilogue does not help.
        if (qi >= QS && !mbar_wait(ACCEMPTY((qi - QS) & 3), ((qi - QS) >> 2) & 1, wc)) { ok = false; break; }
        qn[(qi % QS) * 128 + qrow] = rsqrtf(ss + q_l2_eps);
        mbar_arrive_warp(QEMPTY(st));
        mbar_arrive_warp(QNFULL(qi % QS));
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue warps
    const int qd = warp & 3;
    const int row = qd * 32 + lane;             // token row inside the tile
    const int et = threadIdx.x - 64;            // 0..127
    uint32_t qi = 0;
    bool ok = true;
    constexpr bool use_ge = GATE;            // (gate_elem itself is read through its tensor map)
    float* nws = reinterpret_cast<float*>(base_ptr + R::OFF_NW);
    // A warp whose wait ran out does not just leave: the other three, whose wait may have been satisfied a moment
    // earlier, would stand at their next block barrier for ever.  It goes to that barrier -- between two barriers
    // every wait of a tile has the same next one: 1 without a gate tile, else 2 -- says so there, and all leave.
    auto give_up = [&]() {
      named_barrier_or(use_ge ? 2 : 1, 128, true);
      ok = false;
    };
    // EXTRAS: the gate tile of tile number q (counted over this CTA's tiles) is copied into staging tile q % NOUT,
    // where the output of that tile is then written; issued by one thread, two tiles ahead
    uint32_t gates_issued = 0;
    auto issue_gate = [&](uint32_t q, long long gitem, int gtile) {
      while (gtile >= ntiles) { gtile -= ntiles; gitem += gridDim.x; }
      if (gitem >= nitems) return;
      int gb, gh, gt;
      split_work(s, gitem, gb, gh, gt);
      const int ob = q % R::NOUT;
      const uint32_t dstg = base + R::OFF_OUT + ob * R::TILE_BYTES;
      gates_issued = q + 1;
      mbar_arrive_expect_tx(GFULL(ob), R::TILE_BYTES);
      tma_load_5d(dstg, &tmG, GFULL(ob), 0, gh, gtile * R::TILE, gt, gb);
      tma_load_5d(dstg + R::BOX_BYTES, &tmG, GFULL(ob), 64, gh, gtile * R::TILE, gt, gb);
    };
    if (use_ge && et == 0) {
      for (int i = 0; i < R::NOUT - 1; ++i) issue_gate(i, blockIdx.x, i);
    }
    for (long long item = blockIdx.x; item < nitems && ok; item += gridDim.x) {
      int b, h, t;
      split_work(s, item, b, h, t);
      const float g = (!EXTRAS || gate) ? __ldg(gate + h) : 1.0f;
      const bool use_nw = EXTRAS && norm_weight != nullptr;
      if (use_nw) {
        // this head's norm weights into shared memory (all epilogue threads are past the previous frame's reads:
        // they met at the barrier before its last store)
        nws[et] = __ldg(norm_weight + (size_t)h * R::D + et);
        if (named_barrier_or(1, 128, false)) { ok = false; break; }
      }
      for (int tile = 0; tile < ntiles; ++tile, ++qi) {
        const int a = qi & 3;
        if (!mbar_wait(ACCFULL(a), (qi >> 2) & 1, wc)) { give_up(); break; }
        tc_fence_after_sync();
        float qrs = 1.0f;
        if constexpr (QNORM) {
          if (!mbar_wait(QNFULL(qi % QS), (qi / QS) & 1, wc)) { give_up(); break; }
          qrs = reinterpret_cast<const float*>(base_ptr + R::OFF_QN)[(qi % QS) * 128 + row];
        }
        const uint32_t taddr = tmem_base + ((uint32_t)(qd * 32) << 16) + a * 128;
        float v[4][32];
        tmem_ld32(taddr + 0, v[0]);
        tmem_ld32(taddr + 32, v[1]);
        tmem_ld32(taddr + 64, v[2]);
        tmem_ld32(taddr + 96, v[3]);
        tmem_wait_ld();
        tc_fence_before_sync();
        mbar_arrive_warp(ACCEMPTY(a));

        // eight partial sums: one running sum would be a chain of 128 dependent FMAs (about 500 cycles) in the
        // per-tile critical path of these warps
        float sp[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) sp[e] = 0.f;
#pragma unroll
        for (int c = 0; c < 4; ++c)
#pragma unroll
          for (int e = 0; e < 32; ++e) sp[e & 7] = fmaf(v[c][e], v[c][e], sp[e & 7]);
        const float ss = ((sp[0] + sp[1]) + (sp[2] + sp[3])) + ((sp[4] + sp[5]) + (sp[6] + sp[7]));
        // with o = qrs * v (the read-out of the normalised query): mean o^2 = qrs^2 mean v^2
        const float scale = g * qrs * rsqrtf(ss * (qrs * qrs) * (1.0f / R::D) + eps);

        const int ob = qi % R::NOUT;
        if (use_ge) {
          // the gate tile sits in the staging tile (its copy was issued after the store that last used the tile
          // had been read)
          if (!mbar_wait(GFULL(ob), (qi / R::NOUT) & 1, wc)) { give_up(); break; }
        } else {
          if (et == 0) tma_store_wait_read<R::NOUT - 1>();   // the store that last used this staging tile has read it
          if (named_barrier_or(1, 128, false)) { ok = false; break; }
        }
        unsigned char* orow = base_ptr + R::OFF_OUT + ob * R::TILE_BYTES + row * 128;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const int chunk = (c & 1) * 4 + j;          // 16-byte chunk inside the 64-channel box
            const int boxi = c >> 1;                    // channels 0-63 / 64-127
            uint4* slot = reinterpret_cast<uint4*>(orow + boxi * R::BOX_BYTES + ((chunk ^ (row & 7)) * 16));
            float f[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) f[e] = v[c][j * 8 + e] * scale;
            if constexpr (EXTRAS) {
              if (use_nw) {
                const float4 w0 = *reinterpret_cast<const float4*>(nws + c * 32 + j * 8);
                const float4 w1 = *reinterpret_cast<const float4*>(nws + c * 32 + j * 8 + 4);
                f[0] *= w0.x; f[1] *= w0.y; f[2] *= w0.z; f[3] *= w0.w;
                f[4] *= w1.x; f[5] *= w1.y; f[6] *= w1.z; f[7] *= w1.w;
              }
              if (use_ge) {
                const uint4 gr = *slot;                 // this token's eight gate values for these channels
                const uint32_t* gu = reinterpret_cast<const uint32_t*>(&gr);
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                  f[2 * e] *= __uint_as_float(gu[e] << 16);
                  f[2 * e + 1] *= __uint_as_float(gu[e] & 0xFFFF0000u);
                }
              }
            }
            uint4 pk;
            uint32_t* x = reinterpret_cast<uint32_t*>(&pk);
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              __nv_bfloat162 p2 = __floats2bfloat162_rn(f[2 * e], f[2 * e + 1]);
              x[e] = *reinterpret_cast<uint32_t*>(&p2);
            }
            *slot = pk;
          }
        }
        fence_proxy_async_smem();
        if (named_barrier_or(2, 128, false)) { ok = false; break; }
        if (et == 0) {
          const uint32_t src = base + R::OFF_OUT + ob * R::TILE_BYTES;
          tma_store_5d(&tmO, src, 0, h, tile * R::TILE, t, b);
          tma_store_5d(&tmO, src + R::BOX_BYTES, 64, h, tile * R::TILE, t, b);
          tma_store_commit();
          if (use_ge) {
            // the staging tile of the tile after next was last used by the previous tile's store: once that one
            // has been read (only the newest may still be pending), the next gate tile may land there
            tma_store_wait_read<1>();
            issue_gate(qi + R::NOUT - 1, item, tile + R::NOUT - 1);
          }
        }
      }
    }
    if (et == 0) {
      tma_store_wait_all<0>();
      // a wait gave up: the gate tiles already on their way get a bounded chance to land before the CTA retires
      if (use_ge && !ok) mbar_drain_ring(GFULL(0), R::NOUT, gates_issued);
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

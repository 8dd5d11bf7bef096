// Frame scan (Alg. 1 step 5; Eq. A.1) with the d x d products on the tcgen05 tensor cores at fp32
// accuracy, d = 128.  One CTA per (batch, head, direction) chain; the state never leaves the SM.
//
// With Z = S^T the frame update reads  Z_t = C_t (alpha_t * Z_{t-1} + B_t^T),  C_t = (I+A_t)^{-1}  (alpha_t acts on
// the key rows of Z; it is 1 unless the caller passes a decay).
// Both factors are fp32.  Each is written as a sum of three bf16 numbers (x = x1 + x2 + x3, every part the
// bf16 rounding of what the earlier parts leave over: 24 mantissa bits, i.e. all of fp32), and the product
// is accumulated in fp32 (TMEM) from the six partial products whose weight is above 2^-24:
//        C1 X1 + C1 X2 + C2 X1 + C2 X2 + C1 X3 + C3 X1.
// The dropped terms are below 2^-24 relative to |C||X|, the rounding level of an fp32 dot product, so the
// state is carried at fp32 accuracy while the 2 d^3 flops per step run on the tensor pipe.
//
// C_t arrives already split (the resolve kernel writes the three parts), by TMA, K-major.  The state
// parts are produced on chip: after each step the 16 state warps read Z_t from TMEM (a thread owns one
// key row and 32 value columns), add
// the next frame's B^T, split the sum and write the three parts to shared memory as the next MN-major B
// operand.  The next frame's B^T row is fetched into registers while the MMAs run.
//
// Gather (Eq. A.4).  A chain covers the scanned frames win.first .. win.last (all frames, or the interior ones when
// the clip has boundary anchors).  Slot t of `pf` is what query frame t reads from the forward scan,
// P_{l_t - 1} Diag(prod_{r=l_t..t} alpha_r), slot t of `pb` what it reads from the reverse scan,
// R_{h_t + 1} Diag(prod_{r=t..h_t} alpha_r), [l_t, h_t] being the frame's local window: whenever a chain reaches a
// state that some frames read, it writes those frames' slots, bridged by their decay (with the default window
// {t} that is one slot per step: P_t into slot t+1, R_t into slot t-1).  Without a decay gate all readers of a
// state read the same matrix; it is then stored once, in slot l_t (forward) / h_t (reverse), where the read-out
// looks it up.  Frames whose window leaves no distant
// frame on a side read the initial state (zero unless a text state is passed).  A chain stops after the last
// state that anybody reads.  The read-out kernel adds the two slots in its accumulator (Eq. 1a).
//
// Chunk-wise scan (Sec. 5, "Chunk-wise scans").  With a chunk window, states are read at chunk edges only, so the
// frames of a chunk can be composed first:  Z_out = M Z_in + J  with  M = C_n D_n ... C_1 D_1  (D = Diag(alpha)) and
// J the chunk folded from a zero state.  The same pipeline runs in three modes:
//   SCAN_FRAMES   one CTA per chain, one step per frame (above).
//   SCAN_COMPOSE  one CTA per (chain, direction, chunk, half): the chunk's frames folded from Z = I without writes
//                 (-> M, written as three bf16 parts, the operand format of the scan) or from Z = 0 (-> J, fp32).
//                 All chunks run side by side, which is what shortens the critical path.
//   SCAN_CHUNKS   one CTA per chain, one step per chunk:  Z <- M Z + J,  the gather as above at chunk edges.
// The composed scan pays about four times the arithmetic of the frame scan for a chain of
// chunk + T/chunk steps instead of T: it wins when the chains leave most SMs idle (few heads per GPU).
#pragma once
#include <cuda_bf16.h>

#include "common.cuh"
#include "tc_common.cuh"

namespace vdn {

struct ScanTc {
  static constexpr int D = 128;
  static constexpr int BOX_BYTES = 128 * 128;        // 128 rows x 64 bf16
  static constexpr int PART_BYTES = 2 * BOX_BYTES;   // one 128 x 128 bf16 matrix
  static constexpr int OFF_C = 0;                    // C1, C2, C3
  static constexpr int OFF_X = 3 * PART_BYTES;       // X1, X2, X3
  static constexpr int OFF_BAR = 6 * PART_BYTES;
  static constexpr int SMEM_BYTES = OFF_BAR + 256 + 1024;
  static constexpr int CW = 32;                      // value columns per state thread
  static constexpr int THREADS = 64 + 4 * 32 * (D / CW);  // producer + MMA + state warps
  static constexpr int threads(int ns) { return 64 + 4 * 32 * (D / ns / CW); }
};

enum { SCAN_FRAMES = 0, SCAN_CHUNKS = 1, SCAN_COMPOSE = 2 };

struct ScanTcArgs {
  const float* stats;        // [B*H*T][2d][d] per-frame statistics; the scan reads the B_t half
  __nv_bfloat16* pf;         // [B*H*T][d_v][d_k] read slots of the forward scan
  __nv_bfloat16* pb;         // ... of the reverse scan
  const float* alpha;        // [B,T,H,d] or null
  const float* s0;           // [B,H,d_v,d_k] or null
  int T, H;
  int bh0;                   // first (batch, head) pair of this launch (CTA x works on pair bh0 + x / (2 NS))
  float additive_bscale;     // > 0: the additive baseline, Z_t = C_t (alpha Z) + bscale B_t^T
  Window win;
  // chunk composites (SCAN_COMPOSE writes, SCAN_CHUNKS reads); position p of a chain's direction is the p-th chunk
  // that direction folds
  int nseg;                  // chunks that overlap the scanned frames
  __nv_bfloat16* comp_m;     // [B*H][2][nseg][3][d][d]  M as three bf16 parts, row-major
  float* comp_j;             // [B*H][2][nseg][d_v][d_k] J (in the orientation of the B_t block)
};

// Chunks a direction's chunk-level scan folds: up to the last state that some frame reads.
__host__ __device__ inline int scan_chunk_steps(const Window& w, int dir) {
  if (dir == 0) return w.lo(w.last) == w.first ? 0 : w.lo(w.last) / w.chunk - w.first / w.chunk;
  return w.hi(w.first) == w.last ? 0 : w.last / w.chunk - w.hi(w.first) / w.chunk;
}

// NS = 2 splits the value columns of a chain over two CTAs (the columns of Z evolve independently; each CTA
// loads the whole C_t): for shapes whose chains would leave more than half of the SMs idle.  Such a CTA has half
// the state warps (launch it with threads(NS) threads) and issues MMAs of N = 64.
template <int MODE, int NS = 1>
__global__ void __launch_bounds__(ScanTc::THREADS, 1)
scan_tc_kernel(const __grid_constant__ CUtensorMap tmC, const ScanTcArgs a, tc::DevStatus ds) {
  using namespace tc;
  using S = ScanTc;
  constexpr int D = S::D;
  extern __shared__ unsigned char smem_dyn[];
  const uint32_t base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
  unsigned char* base_ptr = smem_dyn + (base - smem_u32(smem_dyn));

  const uint32_t bar0 = base + S::OFF_BAR;
  auto CFULL = [&](int p) { return bar0 + 8u * p; };          // one per part of C_t
  auto CFREE = [&](int p) { return bar0 + 8u * (3 + p); };
  const uint32_t XREADY = bar0 + 48, ACCFULL = bar0 + 56;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(base_ptr + S::OFF_BAR + 64);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(base_ptr + S::OFF_BAR + 72);
  const WaitCtx wc(abort_flag, ds);

  const Window& win = a.win;
  const int T = a.T;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  // ---- which sequence this CTA folds
  int bh, dir, nsteps;
  int f_lo = win.first, f_hi = win.last;     // frames of this CTA's sequence (SCAN_FRAMES, SCAN_COMPOSE)
  int half = 0, pos = 0;                     // SCAN_COMPOSE: 0 = J (from zero, with writes), 1 = M (from I, no writes)
  const int kfirst = win.first / win.chunk, klast = win.last / win.chunk;
  if constexpr (MODE == SCAN_COMPOSE) {
    half = blockIdx.x & 1;
    dir = (blockIdx.x >> 1) & 1;
    const int rest = blockIdx.x >> 2;
    pos = rest % a.nseg;
    bh = rest / a.nseg;
    if (pos >= scan_chunk_steps(win, dir)) return;           // nobody reads past this chunk
    const int kc = dir == 0 ? kfirst + pos : klast - pos;
    f_lo = max(win.first, kc * win.chunk);
    f_hi = min(win.last, (kc + 1) * win.chunk - 1);
    nsteps = f_hi - f_lo + 1;
  } else {
    bh = a.bh0 + (int)((blockIdx.x / NS) >> 1);
    dir = (blockIdx.x / NS) & 1;
    // steps this chain runs: up to the last state that some frame reads (P_{l-1} of the last frame's window,
    // R_{h+1} of the first frame's)
    if constexpr (MODE == SCAN_FRAMES) nsteps = dir == 0 ? win.lo(win.last) - win.first : win.last - win.hi(win.first);
    else nsteps = scan_chunk_steps(win, dir);
  }
  auto frame_of = [&](int s) { return dir == 0 ? f_lo + s : f_hi - s; };   // frame folded in at step s
  // index of step s's transition (three bf16 parts, 3*D rows of the tensor map) and of its write
  auto item_of = [&](int s) -> long long {
    if constexpr (MODE == SCAN_CHUNKS) return ((long long)bh * 2 + dir) * a.nseg + s;
    else return (long long)bh * T + frame_of(s);
  };

  if (threadIdx.x == 0) {
    for (int p = 0; p < 3; ++p) { mbar_init(CFULL(p), 1); mbar_init(CFREE(p), 1); }
    mbar_init(XREADY, (blockDim.x - 64) / 32);     // one arrival per state warp
    mbar_init(ACCFULL, 1);
    *abort_flag = 0;
    mbar_fence_init();
    tma_prefetch_desc(&tmC);
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(tmem_slot), 128);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer: C_t parts
    // Each part has its own pair of barriers and is re-loaded as soon as the MMAs that read it have retired:
    // the smallest part (C3) is used first and freed first, so every part's copy for the next step has most
    // of this step's MMA time plus the state warps' turn to arrive.
    if (lane == 0) {
      bool ok = true;
      uint32_t issued[3] = {0u, 0u, 0u};
      for (int s = 0; s < nsteps && ok; ++s) {
        const long long n = item_of(s);
#pragma unroll
        for (int p = 2; p >= 0; --p) {
          if (!mbar_wait(CFREE(p), (s & 1) ^ 1, wc)) { ok = false; break; }
          issued[p] = (uint32_t)s + 1u;
          mbar_arrive_expect_tx(CFULL(p), S::PART_BYTES);
          const uint32_t dst = base + S::OFF_C + p * S::PART_BYTES;
          const int row = (int)((n * 3 + p) * D);
          tma_load_2d(dst, &tmC, CFULL(p), 0, row);
          tma_load_2d(dst + S::BOX_BYTES, &tmC, CFULL(p), 64, row);
        }
      }
      if (!ok) {
        // give the copies already in flight a bounded chance to land before the CTA retires
#pragma unroll
        for (int p = 0; p < 3; ++p)
          if (issued[p]) mbar_drain(CFULL(p), (issued[p] - 1u) & 1u);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      // The transition as the A operand.  The resolve kernel eliminates by row operations, so the matrix M it ends
      // with is accurate as a LEFT inverse (M (I + A) - I is small; (I + A) M - I is larger by about the condition
      // number), and the right-hand side here is of the form (I + A) z.  The product must therefore be M X, not
      // M^T X -- in exact arithmetic the same thing.  The resolve stores M transposed (its threads own rows and write
      // coalesced columns), so the stored matrix is read MN-major, which transposes it back.  A composed chunk
      // (SCAN_CHUNKS) is stored as it is used: K-major.
      constexpr bool A_MN = MODE != SCAN_CHUNKS;
      constexpr uint32_t idesc = make_idesc_bf16(128, 128 / NS, A_MN, true);
      bool ok = true;
      for (int s = 0; s < nsteps && ok; ++s) {
        if (!mbar_wait(XREADY, s & 1, wc)) break;
        tc_fence_after_sync();
        // C3 X1, then C2 (X2, X1), then C1 (X3, X2, X1): smallest contributions first
#pragma unroll
        for (int pc = 2; pc >= 0; --pc) {
          if (!mbar_wait(CFULL(pc), s & 1, wc)) { ok = false; break; }
          const uint32_t cb = base + S::OFF_C + pc * S::PART_BYTES;
#pragma unroll
          for (int px = 2 - pc; px >= 0; --px) {
            const uint32_t xb = base + S::OFF_X + px * S::PART_BYTES;
#pragma unroll
            for (int k = 0; k < 8; ++k) {
              const uint64_t adesc = A_MN ? make_smem_desc(cb + k * 2048, S::BOX_BYTES, 1024)
                                          : make_smem_desc(cb + (k >> 2) * S::BOX_BYTES + (k & 3) * 32, 16, 1024);
              const uint64_t bdesc = make_smem_desc(xb + k * 2048, S::BOX_BYTES, 1024);
              mma_bf16_ss(tmem_base, adesc, bdesc, idesc, (pc == 2 && k == 0) ? 0u : 1u);
            }
          }
          mma_commit(CFREE(pc));
        }
        if (ok) mma_commit(ACCFULL);
      }
    }
  } else {
    // ------------------------------------------------------------------ state warps
    // 16 warps: 4 per TMEM lane quarter, each thread owns one key row and CW = 32 value columns.
    constexpr int CW = S::CW;
    const int qd = warp & 3;                 // TMEM lane quarter
    const int row = qd * 32 + lane;          // key channel (row of Z, row of X)
    const int slice = (warp - 2) >> 2;       // this CTA's value columns [CW*slice, CW*slice + CW)
    const int lc0 = slice * CW;              // ... counted inside the CTA (TMEM column, operand column)
    const int col0 = (MODE == SCAN_COMPOSE ? 0 : (int)(blockIdx.x % NS) * (D / NS)) + lc0;   // ... inside the state
    const uint32_t taddr = tmem_base + ((uint32_t)(qd * 32) << 16) + lc0;
    unsigned char* xrow = base_ptr + S::OFF_X + (lc0 >> 6) * S::BOX_BYTES + row * 128;
    const int ch0 = (lc0 & 63) >> 3;         // first 16-byte chunk of this thread inside the 64-column box
    const int sw = row & 7;

    auto load_bt = [&](int s, float (&bt)[CW]) {
      // the write of step s, stored [d_v][d_k]; lanes read consecutive key channels (scalar but coalesced: measured
      // faster than 16-byte loads of a thread-contiguous layout, whose lanes sit 512 bytes apart)
      const float* src;
      if constexpr (MODE == SCAN_CHUNKS) src = a.comp_j + (size_t)item_of(s) * (D * D) + (size_t)col0 * D + row;
      else src = a.stats + (size_t)item_of(s) * (2 * D * D) + (size_t)(D + col0) * D + row;
#pragma unroll
      for (int e = 0; e < CW; ++e) bt[e] = __ldg(src + (size_t)e * D);
    };
    auto publish_x = [&](const float (&x)[CW]) {
#pragma unroll
      for (int ch = 0; ch < CW / 8; ++ch) {
        uint4 w1, w2, w3;
        uint32_t* a1 = reinterpret_cast<uint32_t*>(&w1);
        uint32_t* a2 = reinterpret_cast<uint32_t*>(&w2);
        uint32_t* a3 = reinterpret_cast<uint32_t*>(&w3);
#pragma unroll
        for (int e = 0; e < 4; ++e) split3_pair(x[ch * 8 + 2 * e], x[ch * 8 + 2 * e + 1], a1[e], a2[e], a3[e]);
        const int off = ((ch0 + ch) ^ sw) * 16;
        *reinterpret_cast<uint4*>(xrow + off) = w1;
        *reinterpret_cast<uint4*>(xrow + S::PART_BYTES + off) = w2;
        *reinterpret_cast<uint4*>(xrow + 2 * S::PART_BYTES + off) = w3;
      }
      fence_proxy_async_smem();
      tc_fence_before_sync();
      mbar_arrive_warp(XREADY);
    };

    // Optional extras (Eq. A.1, Eq. 1b, Eq. A.4): alpha [B,T,H,d] decays key channel `row` of the inherited
    // state before a frame is folded in, and bridges the state that frame reads; s0 [B,H,d_v,d_k] is the text
    // state, each scan starting from half of it.  Both act on a thread's own row: one scalar per step.
    auto alpha_of = [&](int frame) {
      return a.alpha ? __ldg(a.alpha + (((size_t)(bh / a.H) * T + frame) * a.H + (bh % a.H)) * D + row) : 1.0f;
    };
    // decay applied to the inherited state at step s (inside M for a composed chunk)
    auto step_decay = [&](int s) { return MODE == SCAN_CHUNKS ? 1.0f : alpha_of(frame_of(s)); };
    // Additive form of a step: the write is added after the product, Z = C (decay * Z) + bscale * B^T.  That is the
    // additive baseline (additive_bscale = 1/sqrt(F) > 0; Eq. 3c with the key scaling of Sec. 3.3, C_t = I - A_t/F
    // prepared by the host's choice of kernel) and, with bscale = 1, a composed chunk (Z = M Z + J).
    // Otherwise Z = C (decay * Z + B^T), the joint solve of Eq. 5.
    const bool additive = MODE == SCAN_CHUNKS || a.additive_bscale > 0.f;
    const float bscale = MODE == SCAN_CHUNKS ? 1.0f : a.additive_bscale;
    const bool writes = !(MODE == SCAN_COMPOSE && half == 1);     // M is the chunk without its writes
    const int lead = additive ? 0 : 1;       // bt holds the write of step (s + lead) when step s's MMAs retire

    // Gather: `z` is the state that the frames t with l_t = bound (forward chain) / h_t = bound (reverse chain)
    // read; write their slots, each bridged by the decay of the frames between the state and the query
    // (Eq. A.4).  Readers are visited walking away from the state, so the bridge is a running product.
    auto store_readers = [&](int bound, const float (&z)[CW]) {
      // only a chunk edge (or the end of the scanned range) is the end of anybody's window
      if (dir == 0 ? (bound != win.first && bound % win.chunk != 0) : (bound != win.last && (bound + 1) % win.chunk != 0))
        return;
      __nv_bfloat16* slots = (dir == 0 ? a.pf : a.pb) + (size_t)bh * T * (D * D) + (size_t)col0 * D + row;
      if (a.alpha == nullptr) {
        // no decay, no bridge: every reader of this state reads the same matrix, stored once in slot `bound`
        // (the read-out looks up slot l_t / h_t)
        __nv_bfloat16* dst = slots + (size_t)bound * (D * D);
#pragma unroll
        for (int e = 0; e < CW; e += 2) {
          const __nv_bfloat162 v2 = __floats2bfloat162_rn(z[e], z[e + 1]);
          dst[(size_t)e * D] = v2.x;
          dst[(size_t)(e + 1) * D] = v2.y;
        }
        return;
      }
      float bridge = 1.0f;
      int r = bound;                           // next frame whose decay enters the bridge
      const int far = dir == 0 ? min(win.last, bound + win.span()) : max(win.first, bound - win.span());
      for (int t = bound; dir == 0 ? t <= far : t >= far; t += dir == 0 ? 1 : -1) {
        if ((dir == 0 ? win.lo(t) : win.hi(t)) != bound) continue;
        for (; dir == 0 ? r <= t : r >= t; r += dir == 0 ? 1 : -1) bridge *= alpha_of(r);
        __nv_bfloat16* dst = slots + (size_t)t * (D * D);
#pragma unroll
        for (int e = 0; e < CW; e += 2) {
          const __nv_bfloat162 v2 = __floats2bfloat162_rn(bridge * z[e], bridge * z[e + 1]);
          dst[(size_t)e * D] = v2.x;
          dst[(size_t)(e + 1) * D] = v2.y;
        }
      }
    };
    // the state that the frames beyond step s's last frame read sits at this window bound
    auto bound_after = [&](int s) {
      if constexpr (MODE == SCAN_CHUNKS) {
        const int kc = dir == 0 ? kfirst + s : klast - s;
        return dir == 0 ? min(win.last, (kc + 1) * win.chunk - 1) + 1 : max(win.first, kc * win.chunk) - 1;
      } else {
        return dir == 0 ? frame_of(s) + 1 : frame_of(s) - 1;
      }
    };
    // SCAN_COMPOSE: the folded chunk goes to position `pos` of this direction's composites
    auto store_composite = [&](const float (&z)[CW]) {
      const size_t slot = ((size_t)bh * 2 + dir) * a.nseg + pos;
      if (half == 0) {
        float* dst = a.comp_j + slot * (D * D) + (size_t)col0 * D + row;      // [d_v][d_k], as the B_t block
#pragma unroll
        for (int e = 0; e < CW; ++e) dst[(size_t)e * D] = z[e];
      } else {
        // row `row`, columns col0 .. col0+31 of M, three bf16 parts, row-major (the K-major A operand of the scan)
        __nv_bfloat16* dst = a.comp_m + slot * (3 * D * D) + (size_t)row * D + col0;
#pragma unroll
        for (int ch = 0; ch < CW / 8; ++ch) {
          uint4 w1, w2, w3;
          uint32_t* a1 = reinterpret_cast<uint32_t*>(&w1);
          uint32_t* a2 = reinterpret_cast<uint32_t*>(&w2);
          uint32_t* a3 = reinterpret_cast<uint32_t*>(&w3);
#pragma unroll
          for (int e = 0; e < 4; ++e) split3_pair(z[ch * 8 + 2 * e], z[ch * 8 + 2 * e + 1], a1[e], a2[e], a3[e]);
          *reinterpret_cast<uint4*>(dst + ch * 8) = w1;
          *reinterpret_cast<uint4*>(dst + (size_t)D * D + ch * 8) = w2;
          *reinterpret_cast<uint4*>(dst + (size_t)2 * D * D + ch * 8) = w3;
        }
      }
    };

    float bt[CW];
    if (nsteps > 0 && writes) load_bt(0, bt);
    {
      // the state the sequence starts from: half the text state for a scan (the frames with no distant frame on
      // this chain's side read it), zero or the identity for the two halves of a composed chunk
      float zi[CW];
#pragma unroll
      for (int e = 0; e < CW; ++e) {
        if constexpr (MODE == SCAN_COMPOSE) zi[e] = (half == 1 && col0 + e == row) ? 1.0f : 0.0f;
        else zi[e] = a.s0 ? 0.5f * __ldg(a.s0 + ((size_t)bh * D + col0 + e) * D + row) : 0.f;
      }
      if constexpr (MODE != SCAN_COMPOSE) store_readers(dir == 0 ? win.first : win.last, zi);
      if (nsteps > 0) {
        // X_0 = decay_0 * Z_init (+ the first write)
        const float a0 = step_decay(0);
        if (additive || !writes) {
#pragma unroll
          for (int e = 0; e < CW; ++e) zi[e] *= a0;
          publish_x(zi);
        } else {
#pragma unroll
          for (int e = 0; e < CW; ++e) bt[e] = fmaf(a0, zi[e], bt[e]);
          publish_x(bt);
        }
      }
    }
    if (!additive && writes && nsteps > 1) load_bt(1, bt);
    float a_next = nsteps > 1 ? step_decay(1) : 1.0f;
    for (int s = 0; s < nsteps; ++s) {
      if (!mbar_wait(ACCFULL, s & 1, wc)) break;
      tc_fence_after_sync();
      float z[CW];
      tmem_ld32(taddr, z);
      tmem_wait_ld();
      if (additive && writes) {
#pragma unroll
        for (int e = 0; e < CW; ++e) z[e] = fmaf(bscale, bt[e], z[e]);
      }
      // first what the next MMAs are waiting for: X = decay * Z (+ the next write), split, into shared memory
      if (s + 1 < nsteps) {
        if (additive || !writes) {
          float xn[CW];
#pragma unroll
          for (int e = 0; e < CW; ++e) xn[e] = a_next * z[e];
          publish_x(xn);
        } else {                               // in place: bt is dead once it has been added
#pragma unroll
          for (int e = 0; e < CW; ++e) bt[e] = fmaf(a_next, z[e], bt[e]);
          publish_x(bt);
        }
      }
      // then, under the next step's MMAs: the state after step s goes to the frames that read it.
      // Stored as bf16 [d_v][d_k] (the paper's orientation), so the 32 lanes of a warp (consecutive key
      // channels) write 64 contiguous bytes per value column.
      // (the write and the decay for the step after are requested first: their latency passes under the stores)
      if (writes && s + 1 + lead < nsteps) load_bt(s + 1 + lead, bt);
      if (s + 2 < nsteps) a_next = step_decay(s + 2);
      if constexpr (MODE == SCAN_COMPOSE) {
        if (s + 1 == nsteps) store_composite(z);
      } else {
        store_readers(bound_after(s), z);
      }
    }
  }

  // ------------------------------------------------------------------ teardown
  __syncwarp();
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, 128);
  }
}

}  // namespace vdn

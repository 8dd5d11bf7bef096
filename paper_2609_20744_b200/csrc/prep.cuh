// Feature preparation in front of the recurrence (Sec. 2.3; "VDA-Prep", Sec. 5):
//     K, V : depthwise 5 x 5 spatial filter and five-tap temporal filter (one pair per channel, taps centred,
//            zero padding), then SiLU;      K, Q : L2 normalisation over the d channels of a (token, head).
//
// prep_spatial_kernel: the 5 x 5 spatial filter, 25 fused multiply-adds per element: bound by the fp32 pipe.
// prep_kv_temporal_kernel: the temporal filter, SiLU and the norm of K, one read and one write per element: bound
//     by HBM.  Run in place on the spatial kernel's result, or alone when no spatial filters are passed (the
//     operation of the paper's VDA-Prep).
// prep_q_kernel: L2 normalisation of Q; bound by HBM.
//
// A single kernel that did all of it in one pass over K and V (tile + halo in shared memory, the spatial results of
// five frames in a register ring) was the first version: 242 registers, one CTA of eight warps per SM, 8.9 ms on
// the 768p shape where the two kernels take 4.2 + 2.3 ms.
#pragma once
#include <cuda_bf16.h>

#include <type_traits>

#include "common.cuh"
#include "tc_common.cuh"

namespace vdn {

// ---- packed fp32 pairs (the two channels a thread owns)
typedef unsigned long long f32x2;
__device__ __forceinline__ f32x2 pack2(float lo, float hi) {
  f32x2 r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpack2(f32x2 v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ f32x2 fma2(f32x2 a, f32x2 b, f32x2 c) {
  f32x2 d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ f32x2 mul2(f32x2 a, f32x2 b) {
  f32x2 d;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}

// two neighbouring channels from shared / to global memory
__device__ __forceinline__ f32x2 load_pair(const __nv_bfloat16* p) {
  const uint32_t u = *reinterpret_cast<const uint32_t*>(p);
  return pack2(__uint_as_float(u << 16), __uint_as_float(u & 0xFFFF0000u));
}
__device__ __forceinline__ f32x2 load_pair(const float* p) {
  const float2 v = *reinterpret_cast<const float2*>(p);
  return pack2(v.x, v.y);
}
__device__ __forceinline__ void store_pair(__nv_bfloat16* p, float lo, float hi) {
  const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  *reinterpret_cast<__nv_bfloat162*>(p) = v;
}
__device__ __forceinline__ void store_pair(float* p, float lo, float hi) {
  *reinterpret_cast<float2*>(p) = make_float2(lo, hi);
}

// SiLU(x) = x / (1 + 2^(-x log2 e)) with the hardware exponential and reciprocal (each good to about 2^-22
// relative): five instructions per element, and this kernel is bound by instruction issue.
__device__ __forceinline__ float silu_f(float x) {
  float e, r;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"(-1.4426950408889634f * x));
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(1.0f + e));
  return x * r;
}

// For 16-bit outputs: SiLU(x) = h + h tanh(h), h = x / 2, with the hardware tanh (specified to about 2^-11 relative,
// three bits below the bf16 rounding of the result; measured, 0.04 % of the outputs differ from the correctly
// rounded value): five instructions per pair instead of eight, in kernels that are bound by instruction issue.
__device__ __forceinline__ void silu2_tanh(f32x2 x, float& y0, float& y1) {
  float h0, h1, t0, t1;
  const f32x2 h = mul2(x, pack2(0.5f, 0.5f));
  unpack2(h, h0, h1);
  asm("tanh.approx.f32 %0, %1;" : "=f"(t0) : "f"(h0));
  asm("tanh.approx.f32 %0, %1;" : "=f"(t1) : "f"(h1));
  unpack2(fma2(h, pack2(t0, t1), h), y0, y1);
}

// the same for a packed pair: the scale, the "+ 1" and the final product as packed operations
__device__ __forceinline__ void silu2(f32x2 x, float& y0, float& y1) {
  float t0, t1, e0, e1, r0, r1;
  unpack2(mul2(x, pack2(-1.4426950408889634f, -1.4426950408889634f)), t0, t1);
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e0) : "f"(t0));
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e1) : "f"(t1));
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r0) : "f"(1.0f + e0));
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r1) : "f"(1.0f + e1));
  unpack2(mul2(x, pack2(r0, r1)), y0, y1);
}

struct PrepArgs {
  const void* in[2];          // k, v   [B,T,F,H,d]
  void* out[2];
  const float* ws[2];         // spatial filters  [H*d][5][5]
  const float* wt[2];         // temporal filters [H*d][5]
  int Y, X;                   // F = Y * X, tokens of a frame in row-major (y, x) order
  float l2_eps;
};

// The spatial filter alone: out[t, y, x, c] = sum_{i,j} ws[c, i, j] in[t, y+i-2, x+j-2, c]  (the first half of the
// preparation; prep_kv_temporal_kernel, run in place on the result, is the second).  Splitting the fused kernel in
// two costs one more round trip of K and V through HBM (the temporal half streams at copy speed) and, for 16-bit
// I/O, one rounding of the intermediate to the I/O type; it frees the 80 registers of the fused kernel's five-frame
// ring, which held it to one CTA of eight warps per SM, its fp32 pipe idle through every barrier and every
// temporal / SiLU / norm phase.
//
// One CTA per (head, 12 x 8 token tile, batch, tensor) walks the frames.  The tile and its 2-token halo arrive by TMA,
// double buffered: the tensor is mapped as (channel, head, x, y, frame) so that one box is the halo tile of one head,
// and whatever hangs over the frame's edge (negative x or y included) is zero-filled by the copy engine -- one
// instruction of one thread per frame, where sixteen-byte asynchronous copies with their bounds checks cost 131 of
// the kernel's 900 instructions per warp and tile.  A thread owns two neighbouring channels (the lanes of the packed
// fp32 FMA) and three tile rows of eight tokens: seven input rows per column feed fifteen tap rows, 600 packed FMAs
// for 84 shared-memory reads (with two rows: 400 for 72, and 4.44 ms instead of 4.22 ms on the 768p shape).  Two CTAs per SM.  The wait for a tile is bounded like every other.
struct PrepSpatial {
  static constexpr int TX = 8, RPT = 3, HALO = 2;            // columns and rows per thread
  static constexpr int THREADS = 256;
  __host__ __device__ static constexpr int rows(int D) { return RPT * THREADS / (D / 2); }      // tile rows
  __host__ __device__ static constexpr int tile_tokens(int D) { return (rows(D) + 2 * HALO) * (TX + 2 * HALO); }
  // two tiles, the barriers, and slack for the 128-byte alignment of the tiles
  static constexpr size_t smem_bytes(int D, int es) { return (size_t)2 * tile_tokens(D) * D * es + 64 + 128; }
};

template <typename Tio, int D>
__global__ void __launch_bounds__(PrepSpatial::THREADS, sizeof(Tio) == 2 ? 2 : 1)
prep_spatial_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV, PrepArgs a, Shape s,
                    tc::DevStatus ds) {
  using namespace tc;
  using P = PrepSpatial;
  constexpr int ROWS = P::rows(D);
  constexpr int TX = P::TX, HALO = P::HALO, RPT = P::RPT;
  constexpr int SW = TX + 2 * HALO, SH = ROWS + 2 * HALO;       // tile with halo
  constexpr int GT = D / 2;                                      // threads per row pair (one head's channel pairs)
  constexpr uint32_t TILE_BYTES = (uint32_t)(SH * SW * D * sizeof(Tio));
  extern __shared__ unsigned char smem_dyn[];
  const uint32_t base = (smem_u32(smem_dyn) + 127u) & ~127u;
  unsigned char* base_ptr = smem_dyn + (base - smem_u32(smem_dyn));
  const Tio* tile = reinterpret_cast<const Tio*>(base_ptr);      // [2][SH][SW][D]
  const uint32_t bar0 = base + 2 * TILE_BYTES;                   // FULL[2]
  volatile int* abort_flag = reinterpret_cast<volatile int*>(base_ptr + 2 * TILE_BYTES + 16);
  const WaitCtx wc(abort_flag, ds);

  const int h = blockIdx.x;
  const int tiles_x = (a.X + TX - 1) / TX;
  const int x0 = (blockIdx.y % tiles_x) * TX, y0 = (blockIdx.y / tiles_x) * ROWS;
  const int which = blockIdx.z & 1;                              // 0 = K, 1 = V
  const int b = blockIdx.z >> 1;
  const CUtensorMap* tm = which == 0 ? &tmK : &tmV;
  Tio* __restrict__ dst = static_cast<Tio*>(which == 0 ? a.out[0] : a.out[1]);

  const int tid = threadIdx.x;
  const int g = tid / GT;                   // row group of this thread: tile rows RPT g .. RPT g + RPT - 1
  const int cp = tid % GT;                  // channel pair within the head
  const int ch = h * D + 2 * cp;

  if (tid == 0) {
    mbar_init(bar0, 1);
    mbar_init(bar0 + 8, 1);
    *abort_flag = 0;
    mbar_fence_init();
    tma_prefetch_desc(tm);
  }
  __syncthreads();

  f32x2 wsp[5][5];
  {
    const float* w0 = (which == 0 ? a.ws[0] : a.ws[1]) + (size_t)ch * 25;
#pragma unroll
    for (int i = 0; i < 5; ++i)
#pragma unroll
      for (int j = 0; j < 5; ++j) wsp[i][j] = pack2(__ldg(w0 + i * 5 + j), __ldg(w0 + 25 + i * 5 + j));
  }

  const int first = s.t0, last = s.t0 + s.Tn - 1;
  const size_t frame_elems = (size_t)s.F * s.H * D;
  const int yr = y0 + RPT * g;              // first of this thread's output rows
  Tio* pdst = dst + token_offset(s, b, first, min(yr, a.Y - 1) * a.X + x0, h) + 2 * cp;

  // frame t's halo tile -> buffer t & 1 (one thread; the engine zero-fills what lies outside the frame)
  int last_staged = first - 1;
  auto stage = [&](int t) {
    last_staged = t;
    const uint32_t bar = bar0 + 8u * (t & 1);
    mbar_arrive_expect_tx(bar, TILE_BYTES);
    tma_load_5d(base + (uint32_t)(t & 1) * TILE_BYTES, tm, bar, 0, h, x0 - HALO, y0 - HALO, b * s.T + t);
  };

  if (tid == 0) stage(first);
#pragma unroll 1
  for (int t = first; t <= last; ++t) {
    // the other buffer was last read for frame t - 1; every thread passed the barrier that closed that frame
    if (tid == 0 && t + 1 <= last) stage(t + 1);
    // frame t's tile has landed -- or the wait ran out: such a thread skips the frame and says so at the barrier
    // that closes it, where all leave together (a lone `break` would leave the others standing at that barrier)
    const bool landed = mbar_wait(bar0 + 8u * (t & 1), ((t - first) >> 1) & 1, wc);
    if (landed) {
      const Tio* tbase = tile + (size_t)(t & 1) * SH * SW * D + (size_t)(RPT * g) * SW * D + 2 * cp;
      f32x2 acc[RPT][TX];
#pragma unroll
      for (int r = 0; r < RPT; ++r)
#pragma unroll
        for (int j = 0; j < TX; ++j) acc[r][j] = 0ull;
#pragma unroll
      for (int xi = 0; xi < SW; ++xi) {       // input column xi sits at x0 - 2 + xi
        f32x2 in[4 + RPT];
#pragma unroll
        for (int i = 0; i < 4 + RPT; ++i) in[i] = load_pair(tbase + ((size_t)i * SW + xi) * D);
#pragma unroll
        for (int i = 0; i < 5; ++i) {
#pragma unroll
          for (int j = 0; j < 5; ++j) {       // tap column j: output column xo = xi - j
            const int xo = xi - j;
            if (xo < 0 || xo >= TX) continue;
#pragma unroll
            for (int r = 0; r < RPT; ++r) acc[r][xo] = fma2(wsp[i][j], in[i + r], acc[r][xo]);
          }
        }
      }
#pragma unroll
      for (int r = 0; r < RPT; ++r) {
        if (yr + r < a.Y) {
#pragma unroll
          for (int j = 0; j < TX; ++j) {
            if (x0 + j < a.X) {
              float o0, o1;
              unpack2(acc[r][j], o0, o1);
              store_pair(pdst + ((size_t)r * a.X + j) * (s.H * D), o0, o1);
            }
          }
        }
      }
    }
    pdst += frame_elems;
    // this frame's buffer may be overwritten by the copy issued two frames on
    if (__syncthreads_or(landed ? 0 : 1)) break;
  }
  if (tid == 0 && *abort_flag) {
    // a wait gave up: give the copies that may still be in flight a bounded chance to land before the CTA retires
    for (int tt = max(first, last_staged - 1); tt <= last_staged; ++tt) mbar_drain(bar0 + 8u * (tt & 1), ((tt - first) >> 1) & 1);
  }
}

// The same preparation without the spatial filter (its filters passed as null: the spatial part is then the
// identity, e.g. because it was applied elsewhere): five-tap temporal filter, SiLU, L2 normalisation of K.  This is
// the operation the paper's VDA-Prep kernel fuses (Sec. 5).  No neighbours in space, so no shared memory: a thread
// owns one 16-byte piece of a (token, head) row and walks the frames with a five-frame ring in registers; the
// lanes that share a row reduce the sum of squares by shuffles.  One read and one write of K and V: bound by HBM.
struct PrepKvTemporal {
  static constexpr int PF = 5;                                   // queue slots per thread (4, 6, 8: the same; 12: 7 % slower)
  static constexpr int THREADS = 256;
  static constexpr int SMEM_BYTES = PF * THREADS * 16;
};

template <typename Tio, int D>
__global__ void __launch_bounds__(PrepKvTemporal::THREADS, 512 / PrepKvTemporal::THREADS)
prep_kv_temporal_kernel(PrepArgs a, Shape s) {
  constexpr int NT = PrepKvTemporal::THREADS;
  constexpr int EPL = 16 / (int)sizeof(Tio);   // channels per thread
  constexpr int LPR = D / EPL;                 // lanes per (token, head) row
  const int which = blockIdx.y & 1;            // 0 = K (normalised), 1 = V
  const int b = blockIdx.y >> 1;
  const long long gid = (long long)blockIdx.x * NT + threadIdx.x;
  const long long rows = (long long)s.F * s.H;
  // whole warps stay together for the shuffles: threads past the end work on the last row and do not store
  const bool live = gid < rows * LPR;
  const long long g2 = live ? gid : rows * LPR - 1;
  const int piece = (int)(g2 % LPR);
  const long long row = g2 / LPR;              // u * H + h
  const int h = (int)(row % s.H);
  const int ch = h * D + piece * EPL;

  // Channels are handled two at a time as packed fp32 pairs (fma.rn.f32x2 and friends): the kernel would
  // otherwise be bound by instruction issue, at about 22 instructions per element, not by HBM.
  constexpr int NP = EPL / 2;                  // channel pairs per thread
  f32x2 wt[5][NP];
  {
    // the thread's EPL x 5 taps are contiguous (and 16-byte aligned): 16-byte loads, a quarter of the L1 wavefronts
    // of tap-by-tap loads, which otherwise cost a fifth of a CTA's lifetime
    const float4* t0 = reinterpret_cast<const float4*>((which == 0 ? a.wt[0] : a.wt[1]) + (size_t)ch * 5);
    float w[EPL * 5];
#pragma unroll
    for (int i = 0; i < EPL * 5 / 4; ++i) {
      const float4 x = __ldg(t0 + i);
      w[4 * i] = x.x; w[4 * i + 1] = x.y; w[4 * i + 2] = x.z; w[4 * i + 3] = x.w;
    }
#pragma unroll
    for (int c = 0; c < NP; ++c)
#pragma unroll
      for (int i = 0; i < 5; ++i) wt[i][c] = pack2(w[(2 * c) * 5 + i], w[(2 * c + 1) * 5 + i]);
  }
  const size_t frame_elems = (size_t)rows * D;
  const Tio* src = static_cast<const Tio*>(which == 0 ? a.in[0] : a.in[1]) + (size_t)b * s.T * frame_elems +
                   (size_t)row * D + piece * EPL;
  Tio* dst = static_cast<Tio*>(which == 0 ? a.out[0] : a.out[1]) + (size_t)b * s.T * frame_elems + (size_t)row * D +
             piece * EPL;
  const int first = s.t0, last = s.t0 + s.Tn - 1;

  f32x2 ring[5][NP];
#pragma unroll
  for (int i = 0; i < 5; ++i)
#pragma unroll
    for (int c = 0; c < NP; ++c) ring[i][c] = 0ull;

  // Frames arrive through a queue of asynchronous copies in shared memory, PF - 1 frames ahead; a thread only ever
  // reads the 16 bytes it copied itself, so no barrier is needed.  (Held in registers, the same number of bytes
  // in flight would cost a quarter of the register file.)  The queue is as long as the ring, so both slots of a
  // step are static in the loop unrolled by five.
  constexpr int PF = PrepKvTemporal::PF;
  static_assert(PF == 5, "queue slot = ring slot = step % 5");
  extern __shared__ uint4 stg[];               // [PF][NT]
  uint4* const myq = stg + threadIdx.x;
  const int nsteps = s.Tn + 2;
  const Tio* psrc = src + (size_t)first * frame_elems;      // next frame to request
  Tio* pdst = dst + (size_t)first * frame_elems;            // next frame to write
#pragma unroll
  for (int i = 0; i < PF - 1; ++i) {
    if (first + i <= last) cp_async16(myq + i * NT, psrc);
    psrc += frame_elems;
    cp_async_commit();
  }

  // One step: request frame t + 4, take frame t = first + step into ring slot r, write frame t - 2.  EDGE = false
  // is the steady state, where every frame involved exists; EDGE = true checks each of them.
  auto one_step = [&](auto rc, auto ec, int step) {
    constexpr int r = decltype(rc)::value;
    constexpr bool EDGE = decltype(ec)::value;
    const int t = first + step;
    if (!EDGE || t + PF - 1 <= last) cp_async16(myq + ((r + PF - 1) % PF) * NT, psrc);
    psrc += frame_elems;
    cp_async_commit();
    cp_async_wait<PF - 1>();                   // frame t has landed
    if (!EDGE || t <= last) {
      const uint4 cur = myq[r * NT];
      if constexpr (sizeof(Tio) == 2) {
        const uint32_t* u = reinterpret_cast<const uint32_t*>(&cur);
#pragma unroll
        for (int i = 0; i < 4; ++i)
          ring[r][i] = pack2(__uint_as_float(u[i] << 16), __uint_as_float(u[i] & 0xFFFF0000u));
      } else {
        const float* u = reinterpret_cast<const float*>(&cur);
#pragma unroll
        for (int i = 0; i < 2; ++i) ring[r][i] = pack2(u[2 * i], u[2 * i + 1]);
      }
    } else {
#pragma unroll
      for (int c = 0; c < NP; ++c) ring[r][c] = 0ull;
    }
    // output frame to = t - 2: sum_i wt[i] x[to + i - 2], x[to + i - 2] in slot (r + i + 1) % 5
    if (EDGE && step < 2) return;
    f32x2 y[NP];
    f32x2 ss2 = 0ull;
#pragma unroll
    for (int c = 0; c < NP; ++c) {
      f32x2 v = mul2(wt[0][c], ring[(r + 1) % 5][c]);
#pragma unroll
      for (int i = 1; i < 5; ++i) v = fma2(wt[i][c], ring[(r + i + 1) % 5][c], v);
      float y0, y1;
      if constexpr (sizeof(Tio) == 2) silu2_tanh(v, y0, y1); else silu2(v, y0, y1);
      y[c] = pack2(y0, y1);
      ss2 = fma2(y[c], y[c], ss2);
    }
    if (which == 0) {
      float s0, s1;
      unpack2(ss2, s0, s1);
      float ss = s0 + s1;
#pragma unroll
      for (int off = LPR / 2; off >= 1; off >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, off);
      const float sc = rsqrtf(ss + a.l2_eps);
      const f32x2 sc2 = pack2(sc, sc);
#pragma unroll
      for (int c = 0; c < NP; ++c) y[c] = mul2(y[c], sc2);
    }
    float o[EPL];
#pragma unroll
    for (int c = 0; c < NP; ++c) unpack2(y[c], o[2 * c], o[2 * c + 1]);
    uint4 res;
    if constexpr (sizeof(Tio) == 2) {
      uint32_t* w = reinterpret_cast<uint32_t*>(&res);
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const __nv_bfloat162 v2 = __floats2bfloat162_rn(o[2 * i], o[2 * i + 1]);
        w[i] = *reinterpret_cast<const uint32_t*>(&v2);
      }
    } else {
      float* w = reinterpret_cast<float*>(&res);
#pragma unroll
      for (int i = 0; i < 4; ++i) w[i] = o[i];
    }
    if (live) *reinterpret_cast<uint4*>(pdst) = res;
    pdst += frame_elems;
  };
  using std::integral_constant;
#pragma unroll 1
  for (int sb = 0; sb < nsteps; sb += 5) {
    // ring slot r = step % 5 is static: sb is a multiple of five
    if (sb >= 5 && sb + 4 + PF - 1 <= s.Tn - 1) {
      one_step(integral_constant<int, 0>{}, integral_constant<bool, false>{}, sb);
      one_step(integral_constant<int, 1>{}, integral_constant<bool, false>{}, sb + 1);
      one_step(integral_constant<int, 2>{}, integral_constant<bool, false>{}, sb + 2);
      one_step(integral_constant<int, 3>{}, integral_constant<bool, false>{}, sb + 3);
      one_step(integral_constant<int, 4>{}, integral_constant<bool, false>{}, sb + 4);
    } else {
      if (sb + 0 < nsteps) one_step(integral_constant<int, 0>{}, integral_constant<bool, true>{}, sb);
      if (sb + 1 < nsteps) one_step(integral_constant<int, 1>{}, integral_constant<bool, true>{}, sb + 1);
      if (sb + 2 < nsteps) one_step(integral_constant<int, 2>{}, integral_constant<bool, true>{}, sb + 2);
      if (sb + 3 < nsteps) one_step(integral_constant<int, 3>{}, integral_constant<bool, true>{}, sb + 3);
      if (sb + 4 < nsteps) one_step(integral_constant<int, 4>{}, integral_constant<bool, true>{}, sb + 4);
    }
  }
}

// L2 normalisation of Q over the d channels of each (token, head).  A (token, head) row is D * sizeof(Tio) / 16
// 16-byte pieces, one per lane; a warp covers 32 / that many rows at once and four such groups per trip, so that
// enough loads are in flight to stream from HBM.  In place is fine.
template <typename Tio, int D>
__global__ void __launch_bounds__(256) prep_q_kernel(const Tio* __restrict__ q, Tio* __restrict__ out, Shape s,
                                                      float eps) {
  constexpr int EPL = 16 / (int)sizeof(Tio);   // elements per lane
  constexpr int LPR = D / EPL;                 // lanes per row
  constexpr int RPW = 32 / LPR;                // rows per warp
  constexpr int UN = 4;
  const int lane = threadIdx.x & 31;
  const int sub = lane / LPR, li = lane % LPR;
  const long long per_frame = (long long)s.F * s.H;
  const long long total = (long long)s.B * s.Tn * per_frame;
  const long long stride = (long long)gridDim.x * 8 * RPW * UN;
  for (long long w0 = ((long long)blockIdx.x * 8 + (threadIdx.x >> 5)) * RPW * UN; w0 < total; w0 += stride) {
    uint4 raw[UN];
    size_t off[UN];
    bool ok[UN];
#pragma unroll
    for (int u = 0; u < UN; ++u) {
      const long long w = w0 + u * RPW + sub;
      ok[u] = w < total;
      const long long ww = ok[u] ? w : 0;
      const long long bt = ww / per_frame;
      const int b = (int)(bt / s.Tn), t = s.t0 + (int)(bt % s.Tn);
      off[u] = (((size_t)b * s.T + t) * per_frame + (size_t)(ww % per_frame)) * D + li * EPL;
      raw[u] = ok[u] ? __ldg(reinterpret_cast<const uint4*>(q + off[u])) : make_uint4(0u, 0u, 0u, 0u);
    }
#pragma unroll
    for (int u = 0; u < UN; ++u) {
      float x[EPL];
      if constexpr (sizeof(Tio) == 2) {
        const uint32_t* r = reinterpret_cast<const uint32_t*>(&raw[u]);
#pragma unroll
        for (int i = 0; i < 4; ++i) { x[2 * i] = __uint_as_float(r[i] << 16); x[2 * i + 1] = __uint_as_float(r[i] & 0xFFFF0000u); }
      } else {
        const float* r = reinterpret_cast<const float*>(&raw[u]);
#pragma unroll
        for (int i = 0; i < 4; ++i) x[i] = r[i];
      }
      float ss = 0.f;
#pragma unroll
      for (int i = 0; i < EPL; ++i) ss = fmaf(x[i], x[i], ss);
#pragma unroll
      for (int o = LPR / 2; o >= 1; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
      const float sc = rsqrtf(ss + eps);
      uint4 res;
      if constexpr (sizeof(Tio) == 2) {
        uint32_t* r = reinterpret_cast<uint32_t*>(&res);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const __nv_bfloat162 v = __floats2bfloat162_rn(x[2 * i] * sc, x[2 * i + 1] * sc);
          r[i] = *reinterpret_cast<const uint32_t*>(&v);
        }
      } else {
        float* r = reinterpret_cast<float*>(&res);
#pragma unroll
        for (int i = 0; i < 4; ++i) r[i] = x[i] * sc;
      }
      if (ok[u]) *reinterpret_cast<uint4*>(out + off[u]) = res;
    }
  }
}

}  // namespace vdn

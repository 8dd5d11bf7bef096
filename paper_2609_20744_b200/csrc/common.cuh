// Shared device helpers for the VDA forward kernels (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace vdn {

// Problem shape in the library's naming: T latent frames of F tokens, H heads, d = d_k = d_v.
// t0 / Tn: the frames the linear branch works on, t0 .. t0+Tn-1 (all T frames, or the interior frames when the
// first and the last frame are boundary anchors, Sec. A.4).  Workspace indices always count all T frames.
// bh0 / bhn: the (batch, head) pairs a persistent kernel works on, pair index b*H + h in bh0 .. bh0+bhn-1 (bhn = 0: all
// of them).  The read-out of a layer with more scan chains than SMs is launched in two parts.
struct Shape {
  int B, T, F, H, d;
  int t0, Tn;
  int bh0 = 0, bhn = 0;
  __host__ __device__ int pairs() const { return bhn > 0 ? bhn : B * H; }
  __host__ __device__ long long frames() const { return (long long)B * H * T; }          // (b,h,t) triples
  __host__ __device__ long long work_items() const { return (long long)pairs() * Tn; }   // ... that are worked on
};

// Local window of a query frame in temporal chunks (Sec. 2.1), clipped to the scanned frames first..last
// (Sec. A.4): chunks of `chunk` frames counted from frame 0 of the clip, `radius` chunks on either side.
// chunk = 1, radius = 0 is the window {t}.
struct Window {
  int chunk, radius, first, last;
  __host__ __device__ int lo(int t) const {
    const int x = (t / chunk - radius) * chunk;
    return x > first ? x : first;
  }
  __host__ __device__ int hi(int t) const {
    const int x = (t / chunk + radius + 1) * chunk - 1;
    return x < last ? x : last;
  }
  __host__ __device__ int span() const { return (radius + 1) * chunk; }   // frames from a window end to its query chunk's far end
};

// Element offset of token (b,t,u), head h in a [B,T,F,H,d] tensor.
__device__ __forceinline__ size_t token_offset(const Shape& s, int b, int t, int u, int h) {
  return ((((size_t)b * s.T + t) * s.F + u) * s.H + h) * (size_t)s.d;
}

// Frame index n = (b*H + h)*T + t  ->  (b, h, t)
__device__ __forceinline__ void split_frame(const Shape& s, long long n, int& b, int& h, int& t) {
  t = (int)(n % s.T);
  long long bh = n / s.T;
  h = (int)(bh % s.H);
  b = (int)(bh / s.H);
}

// Work order of the persistent tensor-core kernels: work item w (of s.work_items()) -> (b, h, t) with the (batch,
// head) pair fastest, so that CTAs running side by side stream the same token rows (a token's H heads are contiguous
// in memory: neighbouring 256-byte pieces of one DRAM page, and shared 32-byte sectors of beta).  Returns the frame
// index n = (b*H + h)*T + t that addresses the workspace.
__device__ __forceinline__ long long split_work(const Shape& s, long long w, int& b, int& h, int& t) {
  const int np = s.pairs();
  const int pair = s.bh0 + (int)(w % np);
  t = s.t0 + (int)(w / np);
  h = pair % s.H;
  b = pair / s.H;
  return (long long)pair * s.T + t;
}

__device__ __forceinline__ float to_float(float x) { return x; }
__device__ __forceinline__ float to_float(__nv_bfloat16 x) { return __bfloat162float(x); }

template <typename T>
__device__ __forceinline__ T from_float(float x);
template <>
__device__ __forceinline__ float from_float<float>(float x) { return x; }
template <>
__device__ __forceinline__ __nv_bfloat16 from_float<__nv_bfloat16>(float x) { return __float2bfloat16_rn(x); }

// Load 4 consecutive elements (16-byte aligned for float, 8-byte for bf16) as floats.
__device__ __forceinline__ float4 load4(const float* p) { return *reinterpret_cast<const float4*>(p); }
__device__ __forceinline__ float4 load4(const __nv_bfloat16* p) {
  uint2 raw = *reinterpret_cast<const uint2*>(p);
  __nv_bfloat162 a = *reinterpret_cast<__nv_bfloat162*>(&raw.x);
  __nv_bfloat162 b = *reinterpret_cast<__nv_bfloat162*>(&raw.y);
  float2 fa = __bfloat1622float2(a), fb = __bfloat1622float2(b);
  return make_float4(fa.x, fa.y, fb.x, fb.y);
}
__device__ __forceinline__ void store4(float* p, float4 v) { *reinterpret_cast<float4*>(p) = v; }
__device__ __forceinline__ void store4(__nv_bfloat16* p, float4 v) {
  __nv_bfloat162 a = __floats2bfloat162_rn(v.x, v.y);
  __nv_bfloat162 b = __floats2bfloat162_rn(v.z, v.w);
  uint2 raw;
  raw.x = *reinterpret_cast<uint32_t*>(&a);
  raw.y = *reinterpret_cast<uint32_t*>(&b);
  *reinterpret_cast<uint2*>(p) = raw;
}

// 16-byte asynchronous global->shared copy (LDGSTS) and its group fences.
__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gmem_src) {
  uint32_t s = (uint32_t)__cvta_generic_to_shared(smem_dst);
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(s), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory"); }

}  // namespace vdn

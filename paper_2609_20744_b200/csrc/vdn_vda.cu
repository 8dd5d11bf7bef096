// Host side of the VDA forward library: handle, argument checks, workspace layout, kernel dispatch.
// The exported functions are documented in include/vdn_vda.h.
#include "../../include/vdn_vda.h"

#include <cuda.h>
#include <cudaTypedefs.h>
#include <cuda_runtime.h>

#include <cmath>
#include <cstdio>
#include <atomic>
#include <cstdlib>
#include <cstring>
#include <new>
#include <string>

#include "common.cuh"
#include "gram_simt.cuh"
#include "gram_tc.cuh"
#include "prep.cuh"
#include "readout_simt.cuh"
#include "readout_tc.cuh"
#include "resolve.cuh"
#include "resolve_tc.cuh"
#include "scan.cuh"
#include "scan_tc.cuh"
#include "wait_selftest.cuh"

namespace {

using vdn::Shape;

constexpr size_t kAlign = 256;
inline size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

// Offsets of the workspace regions (bytes).
//   plain-fp32 path : stats f32 [n][2d][d] | inv f32 [n][d][d] | fwd f32 [n][d][d] | read f32 [n][d][d]
//   tensor-core path: stats f32 [n][2d][d] | inv bf16 [n][3][d][d] (C1,C2,C3) | fwd bf16 [n][d][d] (P_{t-1}^T)
//                     | read bf16 [n][d][d] (R_{t+1}^T), the last two contiguous
struct Layout {
  size_t stats, inv, fwd, read, total;
  size_t inv_bytes, state_bytes;
  size_t comp_m = 0, comp_j = 0;   // chunk composites of the chunk-wise scan (0 = not laid out)
  int nseg_max = 0;
};

struct StagingLayout {
  size_t q, k, v, out, beta, gate, alpha, s0, norm_weight, gate_elem, total;
};

// The optional inputs of vdn_vda_forward_opt, checked and with defaults filled in.
struct Extras {
  const float* alpha = nullptr;
  const float* s0 = nullptr;
  const void* gate_elem = nullptr;
  const float* norm_weight = nullptr;
  float q_l2_eps = 0.f;    // > 0: the read-out normalises the queries itself
  vdn::Window win{1, 0, 0, -1};
  bool anchors = false;
  bool composed = false;   // run the scan chunk-wise (tensor-core path, chunk >= 2)
  // vdn_vda_forward_host runs the layer in pieces: everything up to the scans once the keys and values have
  // arrived, then the read-out of one group of frames after another as their queries arrive
  int phase = 0;           // 0 = whole layer, 1 = statistics, resolve and scans only, 2 = read-out only
  int ro_first = 0, ro_count = 0;   // phase 2: the frames to read out
};

}  // namespace

// Optional per-kernel timing: a ring of CUDA-event sets recorded on the caller's stream, one set per
// forward call, folded into running sums when read (or when the ring wraps).
struct Profiler {
  static constexpr int kMaxKernels = 8;
  static constexpr int kSets = 128;
  bool on = false;
  cudaEvent_t ev[kSets][kMaxKernels + 1];
  int marks[kSets];          // events recorded in each pending set
  int head = 0, pending = 0; // ring state
  const char* names[kMaxKernels] = {};
  double sum_ms[kMaxKernels] = {};
  int count[kMaxKernels] = {};
  int cur = -1;
};

struct vdn_vda_s {
  vdn_vda_config cfg;
  Profiler prof;
  int sm_count = 0;
  void* workspace = nullptr;
  size_t workspace_bytes = 0;
  void* staging = nullptr;
  size_t staging_bytes = 0;
  int* status_host = nullptr;  // pinned, device-mapped: word 0 = status, word 1 = marker of the wait self-test
  int* status_dev = nullptr;
  unsigned long long wait_ns = 2000000000ull;   // limit of any single device-side wait
  int launches = 0;
  // where the last chunk-wise scan left its composites (views VDN_VIEW_COMP_M / _J); nseg = 0: it did not run
  size_t last_comp_m = 0, last_comp_j = 0;
  int last_nseg = 0;
  bool attrs_set = false;
  bool tc_attrs_set = false;
  unsigned ro_attrs_set = 0;       // read-out instantiations whose shared-memory attribute has been set
  int ro_short = 1;                // use the short-frame read-out layout where it applies (VDN_RO_SHORT=0 turns it off)
  // More scan chains than SMs: the surplus chains run on a side stream beside the read-out of the others
  // (stream and events made on first use; VDN_SCAN_SPLIT=0 turns it off)
  int scan_split = 1;
  cudaStream_t side_stream = nullptr;
  cudaEvent_t side_ev[2] = {};
  PFN_cuTensorMapEncodeTiled_v12000 encode = nullptr;  // driver entry point, resolved at create
  // vdn_vda_forward_host: inputs arrive on one stream of the handle's own and results leave on another, in groups of
  // frames (streams and events made on first use)
  static constexpr int kHostGroups = 32;
  cudaStream_t copy_stream = nullptr;                  // device -> host
  cudaEvent_t copy_ev[kHostGroups + 1] = {};
  cudaStream_t in_stream = nullptr;                    // host -> device
  cudaEvent_t in_ev[kHostGroups + 2] = {};             // call entered, keys/values landed, query group g landed
  std::string err = "no error";
};

namespace {

vdn_status fail(vdn_vda_t h, vdn_status st, const std::string& msg) {
  if (h) h->err = msg;
  return st;
}

vdn::tc::DevStatus dev_status(const vdn_vda_s* h) { return vdn::tc::DevStatus{h->status_dev, h->wait_ns}; }

// bf16 I/O with d = 128 runs on the tcgen05 kernels unless the handle asks for the plain-fp32 ones.
bool use_tensor_cores(const vdn_vda_s* h, int d) {
  return h->cfg.io_dtype == VDN_BF16 && d == 128 && !(h->cfg.flags & VDN_FLAG_FORCE_SIMT);
}

size_t elem_size(const vdn_vda_s* h) { return h->cfg.io_dtype == VDN_BF16 ? 2 : 4; }

bool shape_ok(const vdn_vda_s* h, int B, int T, int F, int H, int d, std::string* why) {
  if (B <= 0 || T <= 0 || F <= 0 || H <= 0) { *why = "B, T, F, H must be positive"; return false; }
  if (d != h->cfg.d) { *why = "d differs from the handle's configured head dimension"; return false; }
  const long long tok = (long long)B * T * F;
  if (tok > 0x7fffffffLL / 2) { *why = "B*T*F exceeds the 32-bit token index range"; return false; }
  if ((long long)B * H * T > (1LL << 22)) { *why = "B*H*T exceeds 2^22 frames"; return false; }
  if ((long long)B * H > 65535LL * 1024) { *why = "B*H too large"; return false; }
  return true;
}

// chunk >= 2 adds room for the composites of the chunk-wise scan (tensor-core path): per (batch, head, direction)
// and chunk, M as three bf16 parts and J in fp32.
Layout make_layout(const vdn_vda_s* h, int B, int T, int H, int d, int chunk = 1) {
  const size_t n = (size_t)B * H * T;
  const size_t dd = (size_t)d * d;
  Layout L;
  size_t off = kAlign;  // a reserved header line
  const bool tcp = use_tensor_cores(h, d);
  L.inv_bytes = tcp ? n * dd * 3 * 2 : n * dd * sizeof(float);
  L.state_bytes = tcp ? n * dd * 2 : n * dd * sizeof(float);
  L.stats = off; off += align_up(n * dd * 2 * sizeof(float));
  L.inv = off;   off += align_up(L.inv_bytes);
  L.fwd = off;   off += L.state_bytes;             // fwd and read stay contiguous (n*d*d*es is 256-aligned)
  L.read = off;  off += align_up(L.state_bytes);
  if (tcp && chunk >= 2 && !(h->cfg.flags & VDN_FLAG_SCAN_FRAMEWISE)) {
    L.nseg_max = (T - 1) / chunk + 1;
    const size_t nc = (size_t)B * H * 2 * L.nseg_max;
    L.comp_m = off; off += align_up(nc * dd * 3 * 2);
    L.comp_j = off; off += align_up(nc * dd * sizeof(float));
  }
  L.total = off;
  return L;
}

StagingLayout make_staging(const vdn_vda_s* h, int B, int T, int F, int H, int d, bool with_gate_elem = false) {
  const size_t tokh = (size_t)B * T * F * H;
  const size_t big = align_up(tokh * d * elem_size(h));
  StagingLayout S;
  size_t off = 0;
  S.q = off; off += big;
  S.k = off; off += big;
  S.v = off; off += big;
  S.out = off; off += big;
  S.beta = off; off += align_up(tokh * sizeof(float));
  S.gate = off; off += align_up((size_t)H * sizeof(float));
  // the optional inputs of vdn_vda_forward_host_opt: the small ones always have their place
  S.alpha = off; off += align_up((size_t)B * T * H * d * sizeof(float));
  S.s0 = off; off += align_up((size_t)B * H * d * d * sizeof(float));
  S.norm_weight = off; off += align_up((size_t)H * d * sizeof(float));
  S.gate_elem = off; if (with_gate_elem) off += big;
  S.total = off;
  return S;
}

struct DeviceGuard {
  int prev = -1;
  bool ok = true;
  explicit DeviceGuard(int dev) {
    if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
    if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
  }
  ~DeviceGuard() { if (prev >= 0) cudaSetDevice(prev); }
};

#define VDN_CUDA(h, call)                                                                      \
  do {                                                                                         \
    cudaError_t e_ = (call);                                                                   \
    if (e_ != cudaSuccess)                                                                     \
      return fail((h), VDN_ERR_CUDA, std::string(#call) + ": " + cudaGetErrorString(e_));      \
  } while (0)

void prof_fold_oldest(Profiler& p) {
  const int set = (p.head - p.pending + Profiler::kSets) % Profiler::kSets;
  const int m = p.marks[set];
  if (m > 0 && cudaEventSynchronize(p.ev[set][m]) == cudaSuccess) {
    for (int i = 0; i < m; ++i) {
      float ms = 0.f;
      if (cudaEventElapsedTime(&ms, p.ev[set][i], p.ev[set][i + 1]) == cudaSuccess) {
        p.sum_ms[i] += ms;
        p.count[i] += 1;
      }
    }
  }
  cudaGetLastError();
  p.pending -= 1;
}

// Opens a new event set for this forward call and records its first event.
void prof_begin(vdn_vda_t h, cudaStream_t st) {
  Profiler& p = h->prof;
  if (!p.on) return;
  if (p.pending == Profiler::kSets) prof_fold_oldest(p);
  p.cur = p.head;
  p.head = (p.head + 1) % Profiler::kSets;
  p.pending += 1;
  p.marks[p.cur] = 0;
  cudaEventRecord(p.ev[p.cur][0], st);
}

// Records the event that closes kernel number `idx` of this forward call.
void prof_mark(vdn_vda_t h, cudaStream_t st, int idx, const char* name) {
  Profiler& p = h->prof;
  if (!p.on || p.cur < 0 || idx >= Profiler::kMaxKernels) return;
  p.names[idx] = name;
  cudaEventRecord(p.ev[p.cur][idx + 1], st);
  p.marks[p.cur] = idx + 1;
}

template <typename Tio, int D>
vdn_status set_attrs_simt(vdn_vda_t h) {
  VDN_CUDA(h, cudaFuncSetAttribute(vdn::scan_kernel<D, 32>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                   (int)sizeof(vdn::ScanSmem<D, 32>)));
  VDN_CUDA(h, cudaFuncSetAttribute(vdn::readout_simt_kernel<Tio, D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                   (int)sizeof(vdn::ReadoutSimtSmem<D>)));
  return VDN_OK;
}

// The plain-fp32 path: four launches.
template <typename Tio, int D>
vdn_status forward_simt(vdn_vda_t h, const void* q, const void* k, const void* v, const float* beta,
                        const float* gate, const Extras& x, void* out, const Shape& s,
                        const Layout& L, cudaStream_t st) {
  if (!h->attrs_set) {
    vdn_status r = set_attrs_simt<Tio, D>(h);
    if (r != VDN_OK) return r;
    h->attrs_set = true;
  }
  char* ws = static_cast<char*>(h->workspace);
  float* stats = reinterpret_cast<float*>(ws + L.stats);
  float* inv = reinterpret_cast<float*>(ws + L.inv);
  float* fwd = reinterpret_cast<float*>(ws + L.fwd);
  float* read = reinterpret_cast<float*>(ws + L.read);
  const long long n = s.frames();

  if (x.phase != 2) {
    prof_begin(h, st);
    vdn::gram_simt_kernel<Tio, D><<<dim3((unsigned)n, 2 * D / 64), 256, 0, st>>>(
        static_cast<const Tio*>(k), static_cast<const Tio*>(v), beta, stats, s);
    prof_mark(h, st, 0, "gram_simt");
    const bool additive = (h->cfg.flags & VDN_FLAG_ADDITIVE_RULE) != 0;
    const float bscale = additive ? 1.0f / sqrtf((float)s.F) : 0.f;
    if (additive) {
      vdn::additive_transition_kernel<D><<<(unsigned)n, 256, 0, st>>>(stats, inv, nullptr, n, 1.0f / (float)s.F, s);
      prof_mark(h, st, 1, "additive_transition");
    } else {
      vdn::resolve_kernel<D><<<(unsigned)n, 256, 0, st>>>(stats, inv, nullptr, n, s);
      prof_mark(h, st, 1, "resolve");
    }
    vdn::scan_kernel<D, 32><<<dim3((unsigned)(s.B * s.H), D / 32), 256, sizeof(vdn::ScanSmem<D, 32>), st>>>(
        stats, inv, fwd, read, s.T, x.alpha, x.s0, s.H, bscale, x.win);
    prof_mark(h, st, 2, "scan");
    h->launches = 3;
  } else {
    h->prof.cur = -1;
  }
  if (x.phase != 1) {
    Shape sr = s;                                     // the frames to read out (the kernel skips the others)
    if (x.phase == 2) { sr.t0 = x.ro_first; sr.Tn = x.ro_count; }
    vdn::readout_simt_kernel<Tio, D><<<dim3((unsigned)n, (s.F + 63) / 64), 256, sizeof(vdn::ReadoutSimtSmem<D>), st>>>(
        static_cast<const Tio*>(q), read, gate, static_cast<Tio*>(out), sr, h->cfg.rms_eps,
        static_cast<const Tio*>(x.gate_elem), x.norm_weight, x.q_l2_eps);
    prof_mark(h, st, 3, "readout_simt");
    h->launches += 1;
  }
  VDN_CUDA(h, cudaGetLastError());
  return VDN_OK;
}

// ---------------------------------------------------------------------------------------------------
// Tensor-core path (bf16, d = 128): TMA tensor maps + four launches.

// [B,T,F,H,d] bf16 tensor as a 5-D map (d, H, F, T, B) with a (64, 1, box_tokens, 1, 1) box and the 128-byte
// swizzle: one box is box_tokens tokens x 64 channels of one head.  F is its own dimension so that a tile
// hanging over the end of a frame is zero-filled on load and clipped on store.
vdn_status make_token_map(vdn_vda_t h, CUtensorMap* m, const void* ptr, const Shape& s, unsigned box_tokens = 128) {
  const cuuint64_t dims[5] = {(cuuint64_t)s.d, (cuuint64_t)s.H, (cuuint64_t)s.F, (cuuint64_t)s.T, (cuuint64_t)s.B};
  const cuuint64_t es = 2;
  const cuuint64_t strides[4] = {s.d * es, (cuuint64_t)s.H * s.d * es, (cuuint64_t)s.F * s.H * s.d * es,
                                 (cuuint64_t)s.T * s.F * s.H * s.d * es};
  const cuuint32_t box[5] = {64, 1, box_tokens, 1, 1};
  const cuuint32_t estr[5] = {1, 1, 1, 1, 1};
  CUresult r = h->encode(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(ptr), dims, strides, box, estr,
                         CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return fail(h, VDN_ERR_CUDA, "cuTensorMapEncodeTiled (token tensor) failed: " + std::to_string((int)r));
  return VDN_OK;
}

// A stack of 128 x 128 bf16 matrices, [rows][128], as a 2-D map with a (64, 128) box.
vdn_status make_matrix_map(vdn_vda_t h, CUtensorMap* m, const void* ptr, long long rows) {
  const cuuint64_t dims[2] = {128, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {256};
  const cuuint32_t box[2] = {64, 128};
  const cuuint32_t estr[2] = {1, 1};
  CUresult r = h->encode(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
                         CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return fail(h, VDN_ERR_CUDA, "cuTensorMapEncodeTiled (matrix stack) failed: " + std::to_string((int)r));
  return VDN_OK;
}

vdn_status forward_tc(vdn_vda_t h, const void* q, const void* k, const void* v, const float* beta,
                      const float* gate, const Extras& x, void* out, const Shape& s,
                      const Layout& L, cudaStream_t st) {
  constexpr int D = 128;
  if (!h->encode) return fail(h, VDN_ERR_CUDA, "cuTensorMapEncodeTiled is not available from this driver");
  if (!h->tc_attrs_set) {
    VDN_CUDA(h, cudaFuncSetAttribute(vdn::gram_tc_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     vdn::GramTcCfg<false>::SMEM_BYTES));
    VDN_CUDA(h, cudaFuncSetAttribute(vdn::gram_tc_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     vdn::GramTcCfg<true>::SMEM_BYTES));
    VDN_CUDA(h, cudaFuncSetAttribute(vdn::scan_tc_kernel<vdn::SCAN_FRAMES>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     vdn::ScanTc::SMEM_BYTES));
    VDN_CUDA(h, (cudaFuncSetAttribute(vdn::scan_tc_kernel<vdn::SCAN_FRAMES, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      vdn::ScanTc::SMEM_BYTES)));
    VDN_CUDA(h, cudaFuncSetAttribute(vdn::scan_tc_kernel<vdn::SCAN_CHUNKS>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     vdn::ScanTc::SMEM_BYTES));
    VDN_CUDA(h, cudaFuncSetAttribute(vdn::scan_tc_kernel<vdn::SCAN_COMPOSE>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     vdn::ScanTc::SMEM_BYTES));
    VDN_CUDA(h, cudaFuncSetAttribute(vdn::resolve_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     vdn::ResolveTc::SMEM_BYTES));
    h->tc_attrs_set = true;
  }
  char* ws = static_cast<char*>(h->workspace);
  float* stats = reinterpret_cast<float*>(ws + L.stats);
  __nv_bfloat16* csplit = reinterpret_cast<__nv_bfloat16*>(ws + L.inv);
  __nv_bfloat16* pf = reinterpret_cast<__nv_bfloat16*>(ws + L.fwd);
  __nv_bfloat16* pb = reinterpret_cast<__nv_bfloat16*>(ws + L.read);
  const long long n = s.frames();

  CUtensorMap tmQ, tmK, tmV, tmO, tmS, tmC;
  vdn_status r;
  if ((r = make_token_map(h, &tmK, k, s, vdn::GramTc::TILE)) != VDN_OK) return r;
  if ((r = make_token_map(h, &tmV, v, s, vdn::GramTc::TILE)) != VDN_OK) return r;
  if ((r = make_token_map(h, &tmQ, q, s)) != VDN_OK) return r;
  if ((r = make_token_map(h, &tmO, out, s)) != VDN_OK) return r;
  if ((r = make_matrix_map(h, &tmS, pf, 2 * n * D)) != VDN_OK) return r;      // pf then pb
  if ((r = make_matrix_map(h, &tmC, csplit, 3 * n * D)) != VDN_OK) return r;

  const long long nwork = s.work_items();
  const unsigned persistent = (unsigned)(nwork < h->sm_count ? nwork : h->sm_count);
  int nk = 0, nk_side = 0;
  const int pairs_a = h->sm_count / 2;
  const bool split_scan = x.phase == 0 && !x.composed && h->scan_split && 2LL * s.B * s.H > h->sm_count &&
                          s.B * s.H < 2 * pairs_a;      // worth it while the surplus is less than a full wave
  if (split_scan && !h->side_stream) {
    VDN_CUDA(h, cudaStreamCreateWithFlags(&h->side_stream, cudaStreamNonBlocking));
    for (cudaEvent_t& e : h->side_ev) VDN_CUDA(h, cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
  }
  if (x.phase != 2) {
    prof_begin(h, st);
    if (h->cfg.flags & VDN_FLAG_EXACT_STATS)
      vdn::gram_tc_kernel<true><<<persistent, vdn::GramTcCfg<true>::THREADS, vdn::GramTcCfg<true>::SMEM_BYTES, st>>>(
          tmK, tmV, beta, stats, s, dev_status(h));
    else
      vdn::gram_tc_kernel<false><<<persistent, vdn::GramTc::THREADS, vdn::GramTc::SMEM_BYTES, st>>>(
          tmK, tmV, beta, stats, s, dev_status(h));
    prof_mark(h, st, nk++, (h->cfg.flags & VDN_FLAG_EXACT_STATS) ? "gram_tc_exact" : "gram_tc");
    const bool additive = (h->cfg.flags & VDN_FLAG_ADDITIVE_RULE) != 0;
    const float bscale = additive ? 1.0f / sqrtf((float)s.F) : 0.f;
    if (additive) {
      vdn::additive_transition_kernel<D><<<(unsigned)n, 256, 0, st>>>(stats, nullptr, csplit, n, 1.0f / (float)s.F, s);
      prof_mark(h, st, nk++, "additive_transition");
    } else if (h->cfg.flags & VDN_FLAG_FP32_RESOLVE) {
      // the plain-fp32 Gauss-Jordan (true pivot rows and columns), writing the three bf16 parts the scan reads
      vdn::resolve_kernel<D><<<(unsigned)n, 256, 0, st>>>(stats, nullptr, csplit, n, s);
      prof_mark(h, st, nk++, "resolve");
    } else {
      vdn::resolve_tc_kernel<<<(unsigned)n, vdn::ResolveTc::THREADS, vdn::ResolveTc::SMEM_BYTES, st>>>(
          stats, csplit, n, dev_status(h), s);
      prof_mark(h, st, nk++, "resolve_tc");
    }
    vdn::ScanTcArgs sa{};
    sa.stats = stats; sa.pf = pf; sa.pb = pb; sa.alpha = x.alpha; sa.s0 = x.s0;
    sa.T = s.T; sa.H = s.H; sa.additive_bscale = bscale; sa.win = x.win;
    if (x.composed) {
      // chunk-wise scan: compose every chunk (all at once), then scan the chunk sequence
      sa.nseg = x.win.last / x.win.chunk - x.win.first / x.win.chunk + 1;
      sa.comp_m = reinterpret_cast<__nv_bfloat16*>(ws + L.comp_m);
      sa.comp_j = reinterpret_cast<float*>(ws + L.comp_j);
      h->last_comp_m = L.comp_m; h->last_comp_j = L.comp_j; h->last_nseg = sa.nseg;
      CUtensorMap tmM;
      if ((r = make_matrix_map(h, &tmM, sa.comp_m, (long long)3 * s.B * s.H * 2 * sa.nseg * D)) != VDN_OK) return r;
      vdn::scan_tc_kernel<vdn::SCAN_COMPOSE><<<(unsigned)(4 * s.B * s.H * sa.nseg), vdn::ScanTc::THREADS,
                                               vdn::ScanTc::SMEM_BYTES, st>>>(tmC, sa, dev_status(h));
      prof_mark(h, st, nk++, "compose_tc");
      vdn::scan_tc_kernel<vdn::SCAN_CHUNKS><<<(unsigned)(2 * s.B * s.H), vdn::ScanTc::THREADS,
                                              vdn::ScanTc::SMEM_BYTES, st>>>(tmM, sa, dev_status(h));
      prof_mark(h, st, nk++, "scan_chunks_tc");
    } else if (4LL * s.B * s.H <= h->sm_count) {
      // few chains: two CTAs per chain, half of the value columns each
      vdn::scan_tc_kernel<vdn::SCAN_FRAMES, 2><<<(unsigned)(4 * s.B * s.H), vdn::ScanTc::threads(2),
                                                 vdn::ScanTc::SMEM_BYTES, st>>>(tmC, sa, dev_status(h));
      prof_mark(h, st, nk++, "scan_tc");
    } else if (split_scan) {
      // More chains than SMs (one CTA per SM): a second wave would hold the whole GPU for a handful of chains.
      // The first sm_count / 2 pairs are scanned here; the rest on the side stream once these are done, beside the
      // read-out of the first part, which leaves SMs free (see below).
      vdn::scan_tc_kernel<vdn::SCAN_FRAMES><<<(unsigned)(2 * pairs_a), vdn::ScanTc::THREADS,
                                              vdn::ScanTc::SMEM_BYTES, st>>>(tmC, sa, dev_status(h));
      prof_mark(h, st, nk++, "scan_tc");
      VDN_CUDA(h, cudaEventRecord(h->side_ev[0], st));
      VDN_CUDA(h, cudaStreamWaitEvent(h->side_stream, h->side_ev[0], 0));
      sa.bh0 = pairs_a;
      vdn::scan_tc_kernel<vdn::SCAN_FRAMES><<<(unsigned)(2 * (s.B * s.H - pairs_a)), vdn::ScanTc::THREADS,
                                              vdn::ScanTc::SMEM_BYTES, h->side_stream>>>(tmC, sa, dev_status(h));
      VDN_CUDA(h, cudaEventRecord(h->side_ev[1], h->side_stream));
      nk_side = 1;
    } else {
      vdn::scan_tc_kernel<vdn::SCAN_FRAMES><<<(unsigned)(2 * s.B * s.H), vdn::ScanTc::THREADS,
                                              vdn::ScanTc::SMEM_BYTES, st>>>(tmC, sa, dev_status(h));
      prof_mark(h, st, nk++, "scan_tc");
    }
    h->launches = nk;
  } else {
    h->prof.cur = -1;
    nk = h->launches;
  }
  if (x.phase == 1) { VDN_CUDA(h, cudaGetLastError()); return VDN_OK; }
  // The plain read-out streams reads and writes in equal parts and is fastest on about five SMs out of six
  // (measured on three workloads: 124 CTAs beat 148 by 5 %; fewer interleaved read/write streams at the DRAM).
  // With the optional factors or the query norms it is paced by its epilogue warps and wants every SM (768p clip,
  // warm GPU, 124 -> 148 CTAs: queries normalised 1.36 -> 1.25 ms, gate + norm weight 2.09 -> 1.87 ms).
  const bool extras = x.gate_elem || x.norm_weight || !gate;
  const long long ro_target = (extras || x.q_l2_eps > 0.f) ? h->sm_count : ((long long)h->sm_count * 27 + 16) / 32;
  CUtensorMap tmG = tmO;                                        // the gate tensor has the layout of the output
  if (x.gate_elem && (r = make_token_map(h, &tmG, x.gate_elem, s)) != VDN_OK) return r;
  // short frames (at most kReadoutShortTiles token tiles): the plain read-out with two state buffers
  const bool short_frames = (s.F + 127) / 128 <= vdn::kReadoutShortTiles && h->ro_short != 0;
  auto launch_readout = [&](const Shape& sr, auto ex, auto qn, auto ge, auto sh) {
    constexpr bool EX = decltype(ex)::value, QN = decltype(qn)::value, GE = decltype(ge)::value, SH = decltype(sh)::value;
    using RX = vdn::ReadoutTcCfg<EX, QN, GE, SH>;
    constexpr unsigned bit = 1u << ((EX ? 1 : 0) | (QN ? 2 : 0) | (GE ? 4 : 0) | (SH ? 8 : 0));
    if (!(h->ro_attrs_set & bit)) {        // per handle, i.e. per device
      if (cudaFuncSetAttribute(vdn::readout_tc_kernel<EX, QN, GE, SH>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                               RX::SMEM_BYTES) != cudaSuccess)
        return false;
      h->ro_attrs_set |= bit;
    }
    const long long nread = sr.work_items();
    const unsigned persistent_ro = (unsigned)(nread < ro_target ? nread : ro_target);
    vdn::readout_tc_kernel<EX, QN, GE, SH><<<persistent_ro, RX::THREADS, RX::SMEM_BYTES, st>>>(
        tmQ, tmS, tmO, tmG, gate, sr, h->cfg.rms_eps, dev_status(h), static_cast<const __nv_bfloat16*>(x.gate_elem),
        x.norm_weight, x.win, x.alpha != nullptr, x.q_l2_eps);
    return true;
  };
  using std::true_type;
  using std::false_type;
  auto readout = [&](const Shape& sr) {
    if (x.q_l2_eps > 0.f) {
      if (x.gate_elem) return launch_readout(sr, true_type{}, true_type{}, true_type{}, false_type{});
      if (extras) return launch_readout(sr, true_type{}, true_type{}, false_type{}, false_type{});
      return launch_readout(sr, false_type{}, true_type{}, false_type{}, false_type{});
    }
    if (x.gate_elem) return launch_readout(sr, true_type{}, false_type{}, true_type{}, false_type{});
    if (extras) return launch_readout(sr, true_type{}, false_type{}, false_type{}, false_type{});
    if (short_frames) return launch_readout(sr, false_type{}, false_type{}, false_type{}, true_type{});
    return launch_readout(sr, false_type{}, false_type{}, false_type{}, false_type{});
  };
  Shape sr = s;                                       // the frames to read out
  if (x.phase == 2) { sr.t0 = x.ro_first; sr.Tn = x.ro_count; }
  bool launched;
  if (split_scan) {
    // the pairs whose chains are done; then, once the side stream's chains are done too, the others
    sr.bh0 = 0; sr.bhn = pairs_a;
    launched = readout(sr);
    prof_mark(h, st, nk++, "readout_tc");
    VDN_CUDA(h, cudaStreamWaitEvent(st, h->side_ev[1], 0));
    sr.bh0 = pairs_a; sr.bhn = s.B * s.H - pairs_a;
    launched = launched && readout(sr);
  } else {
    launched = readout(sr);
  }
  if (!launched) return fail(h, VDN_ERR_CUDA, "cudaFuncSetAttribute failed for the read-out kernel");
  prof_mark(h, st, nk++, split_scan ? "readout_tc_rest" : "readout_tc");
  h->launches = nk + nk_side;
  VDN_CUDA(h, cudaGetLastError());
  return VDN_OK;
}

// ---------------------------------------------------------------------------------------------------
// Scratch for vdn_vda_scan_static: lives in the library image, one copy on every GPU that loads it.
// In host code the array's name is only a handle for cudaGetSymbolAddress, never a device address.
constexpr size_t kStaticScanFloats = VDN_SCAN_STATIC_MAX_BYTES / sizeof(float);
static __device__ __align__(256) float g_scan_static_scratch[kStaticScanFloats];
constexpr int kMaxDevices = 64;
// Device address of the array, per device ordinal.  Host threads may race to fill an entry; every one of them
// would store the same value (the lookup is a pure function of the device), and the atomic makes the publication
// well defined.
std::atomic<float*> g_scan_static_ptr[kMaxDevices];

void put_msg(char* buf, size_t len, const std::string& msg) {
  if (!buf || len == 0) return;
  const size_t n = msg.size() < len - 1 ? msg.size() : len - 1;
  std::memcpy(buf, msg.data(), n);
  buf[n] = 0;
}

template <int D>
vdn_status launch_scan_static(const float* stats, const float* inv, float* read, int BH, int T, float* scratch,
                              cudaStream_t st, std::string* why) {
  cudaError_t e = cudaFuncSetAttribute(vdn::scan_kernel<D, 32>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)sizeof(vdn::ScanSmem<D, 32>));
  if (e != cudaSuccess) { *why = std::string("cudaFuncSetAttribute: ") + cudaGetErrorString(e); return VDN_ERR_CUDA; }
  vdn::scan_kernel<D, 32><<<dim3((unsigned)BH, D / 32), 256, sizeof(vdn::ScanSmem<D, 32>), st>>>(
      stats, inv, scratch, read, T, nullptr, nullptr, 1, 0.f, vdn::Window{1, 0, 0, T - 1});
  e = cudaGetLastError();
  if (e != cudaSuccess) { *why = std::string("kernel launch: ") + cudaGetErrorString(e); return VDN_ERR_CUDA; }
  return VDN_OK;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Feature preparation: the spatial filter of K and V (when filters are passed), their temporal half in place, Q.
template <typename Tio, int D>
vdn_status launch_prepare(vdn_vda_t h, const void* q_in, const void* k_in, const void* v_in, void* q_out, void* k_out,
                          void* v_out, const Shape& s, const vdn_vda_prep_params& p, cudaStream_t st) {
  vdn::PrepArgs a;
  a.in[0] = k_in; a.in[1] = v_in; a.out[0] = k_out; a.out[1] = v_out;
  a.ws[0] = p.wk_spatial; a.ws[1] = p.wv_spatial; a.wt[0] = p.wk_temporal; a.wt[1] = p.wv_temporal;
  a.Y = p.Y; a.X = p.X;
  a.l2_eps = p.l2_eps > 0.f ? p.l2_eps : 1e-6f;
  prof_begin(h, st);
  int nk = 0;
  {
    if (p.wk_spatial) {
      // spatial filter into the outputs, then the temporal half in place on them
      using P = vdn::PrepSpatial;
      if (!h->encode) return fail(h, VDN_ERR_CUDA, "cuTensorMapEncodeTiled is not available from this driver");
      const size_t smem = P::smem_bytes(D, (int)sizeof(Tio));
      VDN_CUDA(h, cudaFuncSetAttribute(vdn::prep_spatial_kernel<Tio, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
      // [B,T,F,H,d] with F = Y * X as a 5-D map (d, H, X, Y, B*T): one box = the halo tile of one head in one frame
      CUtensorMap tmk, tmv;
      {
        const cuuint64_t es = sizeof(Tio);
        const cuuint64_t dims[5] = {(cuuint64_t)D, (cuuint64_t)s.H, (cuuint64_t)p.X, (cuuint64_t)p.Y, (cuuint64_t)s.B * s.T};
        const cuuint64_t strides[4] = {D * es, (cuuint64_t)s.H * D * es, (cuuint64_t)p.X * s.H * D * es,
                                       (cuuint64_t)s.F * s.H * D * es};
        const cuuint32_t box[5] = {(cuuint32_t)D, 1, (cuuint32_t)(P::TX + 2 * P::HALO), (cuuint32_t)(P::rows(D) + 2 * P::HALO), 1};
        const cuuint32_t estr[5] = {1, 1, 1, 1, 1};
        const CUtensorMapDataType dt = sizeof(Tio) == 2 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32;
        const void* srcs[2] = {k_in, v_in};
        CUtensorMap* maps[2] = {&tmk, &tmv};
        for (int i = 0; i < 2; ++i) {
          CUresult cr = h->encode(maps[i], dt, 5, const_cast<void*>(srcs[i]), dims, strides, box, estr,
                                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                                  CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
          if (cr != CUDA_SUCCESS)
            return fail(h, VDN_ERR_CUDA, "cuTensorMapEncodeTiled (preparation input) failed: " + std::to_string((int)cr));
        }
      }
      const int tiles = ((p.X + P::TX - 1) / P::TX) * ((p.Y + P::rows(D) - 1) / P::rows(D));
      vdn::prep_spatial_kernel<Tio, D><<<dim3((unsigned)s.H, (unsigned)tiles, (unsigned)(2 * s.B)), P::THREADS, smem, st>>>(
          tmk, tmv, a, s, dev_status(h));
      prof_mark(h, st, nk++, "prep_spatial");
      a.in[0] = k_out; a.in[1] = v_out;
    }
    VDN_CUDA(h, cudaFuncSetAttribute(vdn::prep_kv_temporal_kernel<Tio, D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     vdn::PrepKvTemporal::SMEM_BYTES));
    const long long threads = (long long)s.F * s.H * (D * (int)sizeof(Tio) / 16);
    constexpr int NT = vdn::PrepKvTemporal::THREADS;
    vdn::prep_kv_temporal_kernel<Tio, D><<<dim3((unsigned)((threads + NT - 1) / NT), (unsigned)(2 * s.B)), NT,
                                           vdn::PrepKvTemporal::SMEM_BYTES, st>>>(a, s);
    prof_mark(h, st, nk++, "prep_kv_temporal");
  }
  h->launches = nk;
  if (!q_in) { VDN_CUDA(h, cudaGetLastError()); return VDN_OK; }   // the queries are normalised by the read-out
  const long long rows = (long long)s.B * s.Tn * s.F * s.H;
  const long long per_cta = 8LL * (32 / (D * (int)sizeof(Tio) / 16)) * 4;       // rows one CTA covers per trip
  const long long want = (rows + per_cta - 1) / per_cta;
  const unsigned grid = (unsigned)(want < (long long)h->sm_count * 8 ? want : (long long)h->sm_count * 8);
  vdn::prep_q_kernel<Tio, D><<<grid, 256, 0, st>>>(static_cast<const Tio*>(q_in), static_cast<Tio*>(q_out), s, a.l2_eps);
  prof_mark(h, st, nk++, "prep_q");
  h->launches = nk;
  VDN_CUDA(h, cudaGetLastError());
  return VDN_OK;
}

}  // namespace

extern "C" {

vdn_status vdn_vda_create(const vdn_vda_config* cfg, vdn_vda_t* out_handle) {
  if (!cfg || !out_handle) return VDN_ERR_INVALID_ARG;
  *out_handle = nullptr;
  if (cfg->struct_size != sizeof(vdn_vda_config)) return VDN_ERR_INVALID_ARG;
  if (cfg->io_dtype != VDN_F32 && cfg->io_dtype != VDN_BF16) return VDN_ERR_INVALID_ARG;
  if (cfg->d != 64 && cfg->d != 128) return VDN_ERR_UNSUPPORTED;
  if (cfg->device < 0) return VDN_ERR_INVALID_ARG;
  int count = 0;
  if (cudaGetDeviceCount(&count) != cudaSuccess) { cudaGetLastError(); return VDN_ERR_CUDA; }
  if (cfg->device >= count) return VDN_ERR_INVALID_ARG;
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, cfg->device) != cudaSuccess) { cudaGetLastError(); return VDN_ERR_CUDA; }
  if (prop.major != 10) return VDN_ERR_ARCH;

  vdn_vda_s* h = new (std::nothrow) vdn_vda_s();
  if (!h) return VDN_ERR_CUDA;
  h->cfg = *cfg;
  if (!(h->cfg.rms_eps > 0.f)) h->cfg.rms_eps = 1e-6f;
  h->sm_count = prop.multiProcessorCount;
  if (const char* e = std::getenv("VDN_RO_SHORT")) h->ro_short = std::atoi(e);
  if (const char* e = std::getenv("VDN_SCAN_SPLIT")) h->scan_split = std::atoi(e);
  DeviceGuard guard(cfg->device);
  if (!guard.ok || cudaHostAlloc(reinterpret_cast<void**>(&h->status_host), 64, cudaHostAllocMapped) != cudaSuccess ||
      cudaHostGetDevicePointer(reinterpret_cast<void**>(&h->status_dev), h->status_host, 0) != cudaSuccess) {
    cudaGetLastError();
    if (h->status_host) cudaFreeHost(h->status_host);
    delete h;
    return VDN_ERR_CUDA;
  }
  std::memset(h->status_host, 0, 64);
  {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      h->encode = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(fn);
    else
      cudaGetLastError();
  }
  *out_handle = h;
  return VDN_OK;
}

size_t vdn_vda_workspace_bytes(vdn_vda_t h, int B, int T, int F, int H, int d) {
  std::string why;
  if (!h || !shape_ok(h, B, T, F, H, d, &why)) return 0;
  return make_layout(h, B, T, H, d).total;
}

size_t vdn_vda_workspace_bytes_opt(vdn_vda_t h, int B, int T, int F, int H, int d, const vdn_vda_options* opt) {
  std::string why;
  if (!h || !shape_ok(h, B, T, F, H, d, &why)) return 0;
  if (opt && (opt->struct_size != sizeof(vdn_vda_options) || opt->chunk < 0)) return 0;
  return make_layout(h, B, T, H, d, opt ? opt->chunk : 1).total;
}

vdn_status vdn_vda_set_workspace(vdn_vda_t h, void* dev_ptr, size_t bytes) {
  if (!h) return VDN_ERR_INVALID_ARG;
  if (dev_ptr && (reinterpret_cast<uintptr_t>(dev_ptr) % kAlign) != 0)
    return fail(h, VDN_ERR_INVALID_ARG, "workspace must be 256-byte aligned");
  h->workspace = dev_ptr;
  h->workspace_bytes = dev_ptr ? bytes : 0;
  return VDN_OK;
}

size_t vdn_vda_staging_bytes(vdn_vda_t h, int B, int T, int F, int H, int d) {
  std::string why;
  if (!h || !shape_ok(h, B, T, F, H, d, &why)) return 0;
  return make_staging(h, B, T, F, H, d).total;
}

size_t vdn_vda_staging_bytes_opt(vdn_vda_t h, int B, int T, int F, int H, int d, const vdn_vda_options* opt) {
  std::string why;
  if (!h || !shape_ok(h, B, T, F, H, d, &why)) return 0;
  if (opt && opt->struct_size != sizeof(vdn_vda_options)) return 0;
  return make_staging(h, B, T, F, H, d, opt && opt->gate_elem).total;
}

vdn_status vdn_vda_set_staging(vdn_vda_t h, void* dev_ptr, size_t bytes) {
  if (!h) return VDN_ERR_INVALID_ARG;
  if (dev_ptr && (reinterpret_cast<uintptr_t>(dev_ptr) % kAlign) != 0)
    return fail(h, VDN_ERR_INVALID_ARG, "staging buffer must be 256-byte aligned");
  h->staging = dev_ptr;
  h->staging_bytes = dev_ptr ? bytes : 0;
  return VDN_OK;
}

}  // extern "C"

namespace {

// Everything about a forward call that the host can check, checked, and the call laid out: nothing is enqueued
// and no CUDA call is made.  Fills x (optional inputs with defaults, window), L (workspace layout), s (shape).
vdn_status plan_forward(vdn_vda_t h, const void* q, const void* k, const void* v, const float* beta,
                        const float* gate, void* out, int B, int T, int F, int H, int d,
                        const vdn_vda_options* opt, Extras& x, Layout& L, Shape& s) {
  if (!h) return VDN_ERR_INVALID_ARG;
  if (opt) {
    if (opt->struct_size != sizeof(vdn_vda_options))
      return fail(h, VDN_ERR_INVALID_ARG, "vdn_vda_options.struct_size does not match this library");
    if (opt->chunk < 0 || opt->radius < 0) return fail(h, VDN_ERR_INVALID_ARG, "chunk and radius must be non-negative");
    x.alpha = opt->alpha;
    x.s0 = opt->s0;
    x.gate_elem = opt->gate_elem;
    x.norm_weight = opt->norm_weight;
    if (!(opt->q_l2_eps >= 0.f) || opt->q_l2_eps > 1e30f)
      return fail(h, VDN_ERR_INVALID_ARG, "q_l2_eps must be a finite non-negative number");
    x.q_l2_eps = opt->q_l2_eps;
    x.win.chunk = opt->chunk > 0 ? opt->chunk : 1;
    x.win.radius = opt->radius;
    x.anchors = opt->anchors != 0;
  }
  if (!q || !k || !v || !beta || !out || (!gate && !x.gate_elem))
    return fail(h, VDN_ERR_INVALID_ARG, "null tensor pointer");
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out) || !aligned16(beta) ||
      !aligned16(x.alpha) || !aligned16(x.s0) || !aligned16(x.gate_elem) || !aligned16(x.norm_weight))
    return fail(h, VDN_ERR_INVALID_ARG, "q, k, v, beta, alpha, s0, gate_elem, norm_weight, out must be 16-byte aligned");
  if (out == q || out == k || out == v || out == x.gate_elem)
    return fail(h, VDN_ERR_INVALID_ARG, "out must not alias an input");
  std::string why;
  if (!shape_ok(h, B, T, F, H, d, &why)) return fail(h, VDN_ERR_INVALID_ARG, why);
  if ((long long)(x.win.radius + 1) * x.win.chunk > (1 << 20))
    return fail(h, VDN_ERR_INVALID_ARG, "(radius + 1) * chunk is unreasonably large");
  // The scanned frames: all of them, or the interior ones when frames 0 and T-1 are boundary anchors.
  x.win.first = x.anchors ? 1 : 0;
  x.win.last = x.anchors ? T - 2 : T - 1;
  L = make_layout(h, B, T, H, d);
  if (!h->workspace || h->workspace_bytes < L.total)
    return fail(h, VDN_ERR_WORKSPACE, "workspace not set or smaller than vdn_vda_workspace_bytes");
  if (use_tensor_cores(h, d) && !h->encode)
    return fail(h, VDN_ERR_CUDA, "cuTensorMapEncodeTiled is not available from this driver");
  if (use_tensor_cores(h, d) && x.win.chunk >= 2 && x.win.last >= x.win.first &&
      !(h->cfg.flags & VDN_FLAG_SCAN_FRAMEWISE)) {
    // Chunk-wise scan (Sec. 5): worth it when the chains leave most SMs idle.  Costs in scan steps: one chain
    // step per frame, against the waves of chunk compositions plus one chain step per chunk plus a launch.
    const Layout Lc = make_layout(h, B, T, H, d, x.win.chunk);
    const bool forced = (h->cfg.flags & VDN_FLAG_SCAN_CHUNKWISE) != 0;
    const int cf = vdn::scan_chunk_steps(x.win, 0), cb = vdn::scan_chunk_steps(x.win, 1);
    const int ff = x.win.lo(x.win.last) - x.win.first, fb = x.win.last - x.win.hi(x.win.first);
    const long long ctas = (long long)B * H * (cf + cb) * 2;
    const long long waves = (ctas + h->sm_count - 1) / h->sm_count;
    const long long cost_chunks = waves * x.win.chunk + (cf > cb ? cf : cb) + 2;
    const long long cost_frames = ff > fb ? ff : fb;
    if (forced && h->workspace_bytes < Lc.total)
      return fail(h, VDN_ERR_WORKSPACE, "VDN_FLAG_SCAN_CHUNKWISE needs a workspace of vdn_vda_workspace_bytes_opt");
    if ((forced || cost_chunks < cost_frames) && h->workspace_bytes >= Lc.total && cf + cb > 0) {
      x.composed = true;
      L = Lc;
    }
  }
  s = Shape{B, T, F, H, d, x.win.first, x.win.last - x.win.first + 1};
  return VDN_OK;
}

// Enqueues a planned call, whole (phase 0) or in the two pieces vdn_vda_forward_host interleaves with its copies
// (phase 1: statistics, resolve, scans; phase 2: read-out of frames ro_first .. ro_first + ro_count - 1).
// The handle's device is current.
vdn_status run_forward(vdn_vda_t h, const void* q, const void* k, const void* v, const float* beta,
                       const float* gate, void* out, Extras x, const Layout& L, const Shape& s, cudaStream_t st,
                       int phase, int ro_first, int ro_count) {
  const int B = s.B, T = s.T, F = s.F, H = s.H, d = s.d;
  x.phase = phase;
  if (phase == 2) {
    // clip the requested frames to the scanned ones (anchor rows were zeroed in phase 1)
    const int lo = ro_first > x.win.first ? ro_first : x.win.first;
    const int hi = ro_first + ro_count - 1 < x.win.last ? ro_first + ro_count - 1 : x.win.last;
    if (hi < lo) return VDN_OK;
    x.ro_first = lo;
    x.ro_count = hi - lo + 1;
  } else {
    h->launches = 0;
    h->last_nseg = 0;
  }
  if (x.anchors && phase != 2) {
    // Alg. 1 step 7: anchor rows of the linear output are zero (frames 0 and T-1 of every clip)
    const size_t frame_bytes = (size_t)F * H * d * elem_size(h);
    char* o = static_cast<char*>(out);
    for (int b = 0; b < B; ++b) {
      VDN_CUDA(h, cudaMemsetAsync(o + (size_t)b * T * frame_bytes, 0, frame_bytes, st));
      if (T > 1) VDN_CUDA(h, cudaMemsetAsync(o + ((size_t)b * T + T - 1) * frame_bytes, 0, frame_bytes, st));
    }
  }
  if (s.Tn <= 0) return VDN_OK;        // a clip of anchor frames only has no linear output (Sec. A.4)
  if (use_tensor_cores(h, d)) return forward_tc(h, q, k, v, beta, gate, x, out, s, L, st);
  if (h->cfg.io_dtype == VDN_F32) {
    return d == 64 ? forward_simt<float, 64>(h, q, k, v, beta, gate, x, out, s, L, st)
                   : forward_simt<float, 128>(h, q, k, v, beta, gate, x, out, s, L, st);
  }
  return d == 64 ? forward_simt<__nv_bfloat16, 64>(h, q, k, v, beta, gate, x, out, s, L, st)
                 : forward_simt<__nv_bfloat16, 128>(h, q, k, v, beta, gate, x, out, s, L, st);
}

}  // namespace

extern "C" {

vdn_status vdn_vda_forward_opt(vdn_vda_t h, const void* q, const void* k, const void* v, const float* beta,
                               const float* gate, void* out, int B, int T, int F, int H, int d,
                               const vdn_vda_options* opt, void* cuda_stream) {
  Extras x;
  Layout L;
  Shape s;
  const vdn_status r = plan_forward(h, q, k, v, beta, gate, out, B, T, F, H, d, opt, x, L, s);
  if (r != VDN_OK) return r;
  DeviceGuard guard(h->cfg.device);
  if (!guard.ok) return fail(h, VDN_ERR_CUDA, "cannot make the handle's device current");
  return run_forward(h, q, k, v, beta, gate, out, x, L, s, static_cast<cudaStream_t>(cuda_stream), 0, 0, 0);
}

vdn_status vdn_vda_prepare(vdn_vda_t h, const void* q_in, const void* k_in, const void* v_in, void* q_out, void* k_out,
                           void* v_out, int B, int T, int F, int H, int d, const vdn_vda_prep_params* p,
                           void* cuda_stream) {
  if (!h) return VDN_ERR_INVALID_ARG;
  if (!p || p->struct_size != sizeof(vdn_vda_prep_params))
    return fail(h, VDN_ERR_INVALID_ARG, "vdn_vda_prep_params missing or of the wrong struct_size");
  if (!k_in || !v_in || !k_out || !v_out || !p->wk_temporal || !p->wv_temporal || (q_in == nullptr) != (q_out == nullptr))
    return fail(h, VDN_ERR_INVALID_ARG, "null tensor pointer");
  if ((p->wk_spatial == nullptr) != (p->wv_spatial == nullptr))
    return fail(h, VDN_ERR_INVALID_ARG, "pass both spatial filters or neither");
  if (!aligned16(q_in) || !aligned16(k_in) || !aligned16(v_in) || !aligned16(q_out) || !aligned16(k_out) ||
      !aligned16(v_out) || !aligned16(p->wk_spatial) || !aligned16(p->wk_temporal) || !aligned16(p->wv_spatial) ||
      !aligned16(p->wv_temporal))
    return fail(h, VDN_ERR_INVALID_ARG, "tensors and filters must be 16-byte aligned");
  if (k_out == k_in || k_out == v_in || v_out == k_in || v_out == v_in || k_out == v_out || k_out == q_in ||
      v_out == q_in || (q_out && (q_out == k_in || q_out == v_in || q_out == k_out || q_out == v_out)))
    return fail(h, VDN_ERR_INVALID_ARG, "k_out and v_out must not alias anything (only q_out may equal q_in)");
  std::string why;
  if (!shape_ok(h, B, T, F, H, d, &why)) return fail(h, VDN_ERR_INVALID_ARG, why);
  if (p->Y <= 0 || p->X <= 0 || (long long)p->Y * p->X != F)
    return fail(h, VDN_ERR_INVALID_ARG, "Y * X must equal F");
  if ((long long)F * H * d * (long long)elem_size(h) > 0x7fffffffLL)
    return fail(h, VDN_ERR_UNSUPPORTED, "one frame of a tensor must stay below 2 GiB");
  if (H > 65535 || 2LL * B > 65535 || ((long long)(p->X + 7) / 8) * ((p->Y + 7) / 8) > 65535)
    return fail(h, VDN_ERR_UNSUPPORTED, "grid too large for the preparation kernel");
  DeviceGuard guard(h->cfg.device);
  if (!guard.ok) return fail(h, VDN_ERR_CUDA, "cannot make the handle's device current");
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const bool anchors = p->anchors != 0;
  const Shape s{B, T, F, H, d, anchors ? 1 : 0, anchors ? T - 2 : T};
  h->launches = 0;
  if (anchors) {
    // anchor frames are removed before the preparation (Alg. 1 step 2): they come out as zeros
    const size_t frame_bytes = (size_t)F * H * d * elem_size(h);
    void* outs[3] = {q_out, k_out, v_out};
    for (void* o : outs)
      for (int b = 0; o && b < B; ++b) {
        VDN_CUDA(h, cudaMemsetAsync(static_cast<char*>(o) + (size_t)b * T * frame_bytes, 0, frame_bytes, st));
        if (T > 1)
          VDN_CUDA(h, cudaMemsetAsync(static_cast<char*>(o) + ((size_t)b * T + T - 1) * frame_bytes, 0, frame_bytes, st));
      }
    if (s.Tn <= 0) return VDN_OK;
  }
  if (h->cfg.io_dtype == VDN_F32)
    return d == 64 ? launch_prepare<float, 64>(h, q_in, k_in, v_in, q_out, k_out, v_out, s, *p, st)
                   : launch_prepare<float, 128>(h, q_in, k_in, v_in, q_out, k_out, v_out, s, *p, st);
  return d == 64 ? launch_prepare<__nv_bfloat16, 64>(h, q_in, k_in, v_in, q_out, k_out, v_out, s, *p, st)
                 : launch_prepare<__nv_bfloat16, 128>(h, q_in, k_in, v_in, q_out, k_out, v_out, s, *p, st);
}

vdn_status vdn_vda_forward_ex(vdn_vda_t h, const void* q, const void* k, const void* v, const float* beta,
                              const float* gate, const float* alpha, const float* s0, void* out, int B, int T,
                              int F, int H, int d, void* cuda_stream) {
  if (!gate) return h ? fail(h, VDN_ERR_INVALID_ARG, "null tensor pointer") : VDN_ERR_INVALID_ARG;
  vdn_vda_options opt;
  std::memset(&opt, 0, sizeof(opt));
  opt.struct_size = sizeof(opt);
  opt.alpha = alpha;
  opt.s0 = s0;
  opt.chunk = 1;
  return vdn_vda_forward_opt(h, q, k, v, beta, gate, out, B, T, F, H, d, &opt, cuda_stream);
}

vdn_status vdn_vda_forward(vdn_vda_t h, const void* q, const void* k, const void* v, const float* beta,
                           const float* gate, void* out, int B, int T, int F, int H, int d,
                           void* cuda_stream) {
  return vdn_vda_forward_ex(h, q, k, v, beta, gate, nullptr, nullptr, out, B, T, F, H, d, cuda_stream);
}

vdn_status vdn_vda_forward_host_opt(vdn_vda_t h, const void* q, const void* k, const void* v,
                                    const float* beta, const float* gate, void* out, int B, int T, int F,
                                    int H, int d, const vdn_vda_options* opt, void* cuda_stream) {
  if (!h) return VDN_ERR_INVALID_ARG;
  if (!q || !k || !v || !beta || !out) return fail(h, VDN_ERR_INVALID_ARG, "null tensor pointer");
  std::string why;
  if (!shape_ok(h, B, T, F, H, d, &why)) return fail(h, VDN_ERR_INVALID_ARG, why);
  if (opt && opt->struct_size != sizeof(vdn_vda_options))
    return fail(h, VDN_ERR_INVALID_ARG, "vdn_vda_options.struct_size does not match this library");
  const bool with_ge = opt && opt->gate_elem;
  const StagingLayout S = make_staging(h, B, T, F, H, d, with_ge);
  if (!h->staging || h->staging_bytes < S.total)
    return fail(h, VDN_ERR_WORKSPACE, "staging buffer not set or smaller than vdn_vda_staging_bytes(_opt)");
  char* sg = static_cast<char*>(h->staging);
  // The call as the kernels will see it: every tensor in the staging buffer.  Planned (and refused, if it must
  // be) before the first copy is queued, so an error return never leaves copies reading the caller's buffers.
  vdn_vda_options dopt;
  std::memset(&dopt, 0, sizeof(dopt));
  dopt.struct_size = sizeof(dopt);
  if (opt) {
    dopt = *opt;
    dopt.alpha = opt->alpha ? reinterpret_cast<const float*>(sg + S.alpha) : nullptr;
    dopt.s0 = opt->s0 ? reinterpret_cast<const float*>(sg + S.s0) : nullptr;
    dopt.norm_weight = opt->norm_weight ? reinterpret_cast<const float*>(sg + S.norm_weight) : nullptr;
    dopt.gate_elem = opt->gate_elem ? sg + S.gate_elem : nullptr;
  }
  const float* dbeta = reinterpret_cast<const float*>(sg + S.beta);
  const float* dgate = gate ? reinterpret_cast<const float*>(sg + S.gate) : nullptr;
  Extras x;
  Layout L;
  Shape s;
  vdn_status r = plan_forward(h, sg + S.q, sg + S.k, sg + S.v, dbeta, dgate, sg + S.out, B, T, F, H, d,
                              opt ? &dopt : nullptr, x, L, s);
  if (r != VDN_OK) return r;
  DeviceGuard guard(h->cfg.device);
  if (!guard.ok) return fail(h, VDN_ERR_CUDA, "cannot make the handle's device current");
  if (!h->copy_stream) {
    // a second stream and a few events, made on first use: results travel back while later queries still arrive
    VDN_CUDA(h, cudaStreamCreateWithFlags(&h->copy_stream, cudaStreamNonBlocking));
    for (int i = 0; i <= vdn_vda_s::kHostGroups; ++i)
      VDN_CUDA(h, cudaEventCreateWithFlags(&h->copy_ev[i], cudaEventDisableTiming));
    VDN_CUDA(h, cudaStreamCreateWithFlags(&h->in_stream, cudaStreamNonBlocking));
    for (int i = 0; i < vdn_vda_s::kHostGroups + 2; ++i)
      VDN_CUDA(h, cudaEventCreateWithFlags(&h->in_ev[i], cudaEventDisableTiming));
  }
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const size_t tokh = (size_t)B * T * F * H;
  const size_t big = tokh * d * elem_size(h);
  const size_t frame_bytes = (size_t)F * H * d * elem_size(h);
  cudaStream_t in = h->in_stream;
  // From here on work is queued on the handle's own streams.  Whatever goes wrong later, the caller's stream is
  // made to wait for the tail of both before the error is returned, so that synchronising it still means that
  // nothing of this call touches the caller's buffers any more.
  auto join = [&]() {
    if (cudaEventRecord(h->in_ev[0], in) == cudaSuccess) cudaStreamWaitEvent(st, h->in_ev[0], 0);
    if (cudaEventRecord(h->copy_ev[vdn_vda_s::kHostGroups], h->copy_stream) == cudaSuccess)
      cudaStreamWaitEvent(st, h->copy_ev[vdn_vda_s::kHostGroups], 0);
    cudaGetLastError();
  };
#define VDN_CUDA_J(call)                                                                       \
  do {                                                                                         \
    cudaError_t e_ = (call);                                                                   \
    if (e_ != cudaSuccess) {                                                                   \
      join();                                                                                  \
      return fail(h, VDN_ERR_CUDA, std::string(#call) + ": " + cudaGetErrorString(e_));        \
    }                                                                                          \
  } while (0)
  // All copies in are queued at once on the handle's input stream, in the order the layer needs them, so that the
  // host link never waits for a kernel: keys, values and write gates first (the statistics, the resolve and both
  // scans need nothing else), then the queries, one group of frames after another.  The input stream starts where
  // the caller's stream stands now (earlier work on it may still be reading the staging buffer).
  VDN_CUDA_J(cudaEventRecord(h->in_ev[0], st));
  VDN_CUDA_J(cudaStreamWaitEvent(in, h->in_ev[0], 0));
  VDN_CUDA_J(cudaMemcpyAsync(sg + S.k, k, big, cudaMemcpyHostToDevice, in));
  VDN_CUDA_J(cudaMemcpyAsync(sg + S.v, v, big, cudaMemcpyHostToDevice, in));
  VDN_CUDA_J(cudaMemcpyAsync(sg + S.beta, beta, tokh * sizeof(float), cudaMemcpyHostToDevice, in));
  if (gate) VDN_CUDA_J(cudaMemcpyAsync(sg + S.gate, gate, (size_t)H * sizeof(float), cudaMemcpyHostToDevice, in));
  if (opt && opt->alpha)
    VDN_CUDA_J(cudaMemcpyAsync(sg + S.alpha, opt->alpha, (size_t)B * T * H * d * sizeof(float), cudaMemcpyHostToDevice, in));
  if (opt && opt->s0)
    VDN_CUDA_J(cudaMemcpyAsync(sg + S.s0, opt->s0, (size_t)B * H * d * d * sizeof(float), cudaMemcpyHostToDevice, in));
  if (opt && opt->norm_weight)
    VDN_CUDA_J(cudaMemcpyAsync(sg + S.norm_weight, opt->norm_weight, (size_t)H * d * sizeof(float), cudaMemcpyHostToDevice, in));
  VDN_CUDA_J(cudaEventRecord(h->in_ev[1], in));
  const int groups = T < vdn_vda_s::kHostGroups ? T : vdn_vda_s::kHostGroups;
  for (int g = 0; g < groups; ++g) {
    const int t0 = (int)((long long)T * g / groups), t1 = (int)((long long)T * (g + 1) / groups);
    const size_t off = (size_t)t0 * frame_bytes, len = (size_t)(t1 - t0) * frame_bytes;
    for (int b = 0; b < B; ++b) {
      const size_t o = (size_t)b * T * frame_bytes + off;
      VDN_CUDA_J(cudaMemcpyAsync(sg + S.q + o, static_cast<const char*>(q) + o, len, cudaMemcpyHostToDevice, in));
      if (with_ge)
        VDN_CUDA_J(cudaMemcpyAsync(sg + S.gate_elem + o, static_cast<const char*>(opt->gate_elem) + o, len,
                                   cudaMemcpyHostToDevice, in));
    }
    VDN_CUDA_J(cudaEventRecord(h->in_ev[2 + g], in));
  }
  VDN_CUDA_J(cudaStreamWaitEvent(st, h->in_ev[1], 0));
  r = run_forward(h, sg + S.q, sg + S.k, sg + S.v, dbeta, dgate, sg + S.out, x, L, s, st, 1, 0, 0);
  if (r != VDN_OK) { join(); return r; }
  // Each group is read out as soon as its queries have landed, and its finished rows go to the second stream,
  // whose copy back to the host runs beside the copies in (the link is full duplex).
  for (int g = 0; g < groups; ++g) {
    const int t0 = (int)((long long)T * g / groups), t1 = (int)((long long)T * (g + 1) / groups);
    const size_t off = (size_t)t0 * frame_bytes, len = (size_t)(t1 - t0) * frame_bytes;
    VDN_CUDA_J(cudaStreamWaitEvent(st, h->in_ev[2 + g], 0));
    r = run_forward(h, sg + S.q, sg + S.k, sg + S.v, dbeta, dgate, sg + S.out, x, L, s, st, 2, t0, t1 - t0);
    if (r != VDN_OK) { join(); return r; }
    VDN_CUDA_J(cudaEventRecord(h->copy_ev[g], st));
    VDN_CUDA_J(cudaStreamWaitEvent(h->copy_stream, h->copy_ev[g], 0));
    for (int b = 0; b < B; ++b) {
      const size_t o = (size_t)b * T * frame_bytes + off;
      VDN_CUDA_J(cudaMemcpyAsync(static_cast<char*>(out) + o, sg + S.out + o, len, cudaMemcpyDeviceToHost,
                                 h->copy_stream));
    }
  }
  // the caller's stream is done when the last rows have landed
  VDN_CUDA_J(cudaEventRecord(h->copy_ev[vdn_vda_s::kHostGroups], h->copy_stream));
  VDN_CUDA_J(cudaStreamWaitEvent(st, h->copy_ev[vdn_vda_s::kHostGroups], 0));
#undef VDN_CUDA_J
  return VDN_OK;
}

vdn_status vdn_vda_forward_host(vdn_vda_t h, const void* q, const void* k, const void* v,
                                const float* beta, const float* gate, void* out, int B, int T, int F,
                                int H, int d, void* cuda_stream) {
  if (h && !gate) return fail(h, VDN_ERR_INVALID_ARG, "null tensor pointer");
  return vdn_vda_forward_host_opt(h, q, k, v, beta, gate, out, B, T, F, H, d, nullptr, cuda_stream);
}

vdn_status vdn_vda_workspace_view(vdn_vda_t h, int which, int B, int T, int F, int H, int d,
                                  size_t* offset_bytes, size_t* size_bytes) {
  if (!h || !offset_bytes || !size_bytes) return VDN_ERR_INVALID_ARG;
  std::string why;
  if (!shape_ok(h, B, T, F, H, d, &why)) return fail(h, VDN_ERR_INVALID_ARG, why);
  const Layout L = make_layout(h, B, T, H, d);
  (void)F;
  const size_t n = (size_t)B * H * T, dd = (size_t)d * d;
  const bool tcp = use_tensor_cores(h, d);
  switch (which) {
    case VDN_VIEW_STATS: *offset_bytes = L.stats; *size_bytes = n * dd * 2 * sizeof(float); break;
    case VDN_VIEW_INV:
      if (tcp) return fail(h, VDN_ERR_UNSUPPORTED, "this handle keeps the inverse as three bf16 parts (VDN_VIEW_INV_SPLIT)");
      *offset_bytes = L.inv; *size_bytes = L.inv_bytes; break;
    case VDN_VIEW_FWD:
    case VDN_VIEW_READ:
      if (tcp) return fail(h, VDN_ERR_UNSUPPORTED, "this handle keeps the two read states apart (VDN_VIEW_READ_FWD / _BWD)");
      *offset_bytes = which == VDN_VIEW_FWD ? L.fwd : L.read; *size_bytes = L.state_bytes; break;
    case VDN_VIEW_INV_SPLIT:
      if (!tcp) return fail(h, VDN_ERR_UNSUPPORTED, "only the tensor-core kernels split the inverse");
      *offset_bytes = L.inv; *size_bytes = L.inv_bytes; break;
    case VDN_VIEW_READ_FWD:
    case VDN_VIEW_READ_BWD:
      if (!tcp) return fail(h, VDN_ERR_UNSUPPORTED, "the plain-fp32 kernels store the summed read state (VDN_VIEW_READ)");
      *offset_bytes = which == VDN_VIEW_READ_FWD ? L.fwd : L.read; *size_bytes = L.state_bytes; break;
    case VDN_VIEW_COMP_M:
    case VDN_VIEW_COMP_J:
      if (!tcp || h->last_nseg == 0) return fail(h, VDN_ERR_UNSUPPORTED, "the last forward call did not scan chunk-wise");
      *offset_bytes = which == VDN_VIEW_COMP_M ? h->last_comp_m : h->last_comp_j;
      *size_bytes = (size_t)B * H * 2 * h->last_nseg * dd * (which == VDN_VIEW_COMP_M ? 3 * 2 : sizeof(float));
      break;
    default: return fail(h, VDN_ERR_INVALID_ARG, "unknown view");
  }
  return VDN_OK;
}

int vdn_vda_last_launch_count(vdn_vda_t h) { return h ? h->launches : 0; }

vdn_status vdn_vda_profile(vdn_vda_t h, int enable) {
  if (!h) return VDN_ERR_INVALID_ARG;
  Profiler& p = h->prof;
  DeviceGuard guard(h->cfg.device);
  if (!guard.ok) return fail(h, VDN_ERR_CUDA, "cannot make the handle's device current");
  if (enable && !p.on) {
    for (int s = 0; s < Profiler::kSets; ++s)
      for (int i = 0; i <= Profiler::kMaxKernels; ++i) VDN_CUDA(h, cudaEventCreate(&p.ev[s][i]));
    p.on = true;
  } else if (!enable && p.on) {
    for (int s = 0; s < Profiler::kSets; ++s)
      for (int i = 0; i <= Profiler::kMaxKernels; ++i) cudaEventDestroy(p.ev[s][i]);
    p.on = false;
  }
  p.head = p.pending = 0;
  p.cur = -1;
  for (int i = 0; i < Profiler::kMaxKernels; ++i) { p.sum_ms[i] = 0.0; p.count[i] = 0; p.names[i] = nullptr; }
  return VDN_OK;
}

int vdn_vda_kernel_times(vdn_vda_t h, int max_kernels, const char** names, float* mean_ms, int* launches) {
  if (!h || !names || !mean_ms || !launches || max_kernels <= 0) return 0;
  Profiler& p = h->prof;
  if (!p.on) return 0;
  DeviceGuard guard(h->cfg.device);
  while (p.pending > 0) prof_fold_oldest(p);
  int n = 0;
  for (int i = 0; i < Profiler::kMaxKernels && n < max_kernels; ++i) {
    if (!p.names[i] || p.count[i] == 0) continue;
    names[n] = p.names[i];
    mean_ms[n] = (float)(p.sum_ms[i] / p.count[i]);
    launches[n] = p.count[i];
    ++n;
  }
  return n;
}

vdn_status vdn_vda_status(vdn_vda_t h) {
  if (!h) return VDN_ERR_INVALID_ARG;
  const int v = *const_cast<volatile int*>(h->status_host);
  if (v == 0) return VDN_OK;
  return v == VDN_ERR_INTERNAL ? VDN_ERR_INTERNAL : VDN_ERR_TIMEOUT;
}

vdn_status vdn_vda_clear_status(vdn_vda_t h) {
  if (!h) return VDN_ERR_INVALID_ARG;
  const vdn_status prev = vdn_vda_status(h);
  *const_cast<volatile int*>(h->status_host) = 0;
  return prev;
}

vdn_status vdn_vda_set_wait_limit_us(vdn_vda_t h, unsigned long long microseconds) {
  if (!h) return VDN_ERR_INVALID_ARG;
  if (microseconds == 0 || microseconds > 3600ull * 1000000ull)
    return fail(h, VDN_ERR_INVALID_ARG, "the wait limit must lie between 1 microsecond and 1 hour");
  h->wait_ns = microseconds * 1000ull;
  return VDN_OK;
}

vdn_status vdn_vda_selftest_wait_expiry(vdn_vda_t h, unsigned long long limit_us, void* cuda_stream) {
  if (!h) return VDN_ERR_INVALID_ARG;
  if (limit_us == 0 || limit_us > 1000000ull)
    return fail(h, VDN_ERR_INVALID_ARG, "the self-test's wait limit must lie between 1 microsecond and 1 second");
  DeviceGuard guard(h->cfg.device);
  if (!guard.ok) return fail(h, VDN_ERR_CUDA, "cannot make the handle's device current");
  const_cast<volatile int*>(h->status_host)[1] = 0;
  vdn::wait_expiry_selftest_kernel<<<1, 64, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
      vdn::tc::DevStatus{h->status_dev, limit_us * 1000ull}, h->status_dev + 1);
  VDN_CUDA(h, cudaGetLastError());
  return VDN_OK;
}

int vdn_vda_selftest_marker(vdn_vda_t h) { return h ? const_cast<volatile int*>(h->status_host)[1] : -1; }

vdn_status vdn_vda_scan_static(const float* stats, const float* inv, float* read, int BH, int T, int d,
                               int device, void* cuda_stream, char* errbuf, size_t errbuf_len) {
  if (!stats || !inv || !read) { put_msg(errbuf, errbuf_len, "null tensor pointer"); return VDN_ERR_INVALID_ARG; }
  if (!aligned16(stats) || !aligned16(inv) || !aligned16(read)) {
    put_msg(errbuf, errbuf_len, "stats, inv, read must be 16-byte aligned");
    return VDN_ERR_INVALID_ARG;
  }
  if (BH <= 0 || T <= 0) { put_msg(errbuf, errbuf_len, "BH and T must be positive"); return VDN_ERR_INVALID_ARG; }
  if (d != 64 && d != 128) { put_msg(errbuf, errbuf_len, "d must be 64 or 128"); return VDN_ERR_UNSUPPORTED; }
  if (device < 0 || device >= kMaxDevices) { put_msg(errbuf, errbuf_len, "device ordinal out of range"); return VDN_ERR_INVALID_ARG; }
  const size_t need = (size_t)BH * T * d * d * sizeof(float);
  if ((size_t)BH * T > kStaticScanFloats / ((size_t)d * d)) {
    put_msg(errbuf, errbuf_len,
            "BH*T*d*d*4 = " + std::to_string(need) + " bytes of scan scratch exceed the built-in " +
                std::to_string((size_t)VDN_SCAN_STATIC_MAX_BYTES) + " bytes (VDN_SCAN_STATIC_MAX_BYTES); use vdn_vda_forward with a workspace");
    return VDN_ERR_WORKSPACE;
  }
  DeviceGuard guard(device);
  if (!guard.ok) { put_msg(errbuf, errbuf_len, "cannot make the device current"); return VDN_ERR_CUDA; }
  float* ptr = g_scan_static_ptr[device].load(std::memory_order_acquire);
  if (!ptr) {
    // first call on this device: look up where the array lives on it (the device is current here)
    cudaError_t e = cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_scan_static_scratch);
    if (e != cudaSuccess || !ptr) {
      put_msg(errbuf, errbuf_len, std::string("cudaGetSymbolAddress: ") + cudaGetErrorString(e));
      cudaGetLastError();
      return VDN_ERR_CUDA;
    }
    g_scan_static_ptr[device].store(ptr, std::memory_order_release);
  }
  std::string why;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const vdn_status r = d == 64 ? launch_scan_static<64>(stats, inv, read, BH, T, ptr, st, &why)
                               : launch_scan_static<128>(stats, inv, read, BH, T, ptr, st, &why);
  if (r != VDN_OK) put_msg(errbuf, errbuf_len, why);
  return r;
}

const char* vdn_vda_last_error(vdn_vda_t h) { return h ? h->err.c_str() : "null handle"; }

vdn_status vdn_vda_destroy(vdn_vda_t h) {
  if (!h) return VDN_ERR_INVALID_ARG;
  if (h->prof.on) vdn_vda_profile(h, 0);
  if (h->copy_stream) {
    for (cudaEvent_t e : h->copy_ev)
      if (e) cudaEventDestroy(e);
    cudaStreamDestroy(h->copy_stream);
    for (cudaEvent_t e : h->in_ev)
      if (e) cudaEventDestroy(e);
    if (h->in_stream) cudaStreamDestroy(h->in_stream);
  }
  if (h->side_stream) {
    for (cudaEvent_t e : h->side_ev)
      if (e) cudaEventDestroy(e);
    cudaStreamDestroy(h->side_stream);
  }
  if (h->status_host) cudaFreeHost(h->status_host);
  delete h;
  return VDN_OK;
}

}  // extern "C"

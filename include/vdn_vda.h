/*
 * vdn_vda.h -- C ABI of the bidirectional Video Delta Attention (VDA) forward pass for NVIDIA B200.
 *
 * The layer (Video DeltaNet, Sec. 2.2, Sec. 3 and Algorithm 1 steps 3-7), per (batch, head):
 *
 *   frame statistics (Eq. 3b)        A_t = K_t^T Diag(beta_t) K_t,   B_t = V_t^T Diag(beta_t) K_t
 *   joint frame update (Eq. 5, A.1)  S_t = (S_{t-1} + B_t)(I + A_t)^{-1}   (decay alpha_t = 1; see forward_ex)
 *   two scans (Sec. 2.2)             P_t: frames 0..t in order,  R_t: frames T-1..t in reverse order,
 *                                    both started from the zero state (vdn_vda_forward_ex: from S_T / 2)
 *   gather (Eq. A.4, Eq. 1a)         the queries of frame t read  P_{t-1} + R_{t+1}  (P_{-1} = R_T = 0):
 *                                    the local window is the query frame itself, so no frame is counted
 *                                    twice and a frame never reads its own write
 *   read-out, norm, gate (Eq. 1c)    o = S q;  out = gate_h * o / sqrt(mean_j o_j^2 + rms_eps)
 *
 * No patch order inside a frame, no 1/sqrt(F) key scaling (Sec. 3.3).  The statistics are contracted on
 * the tensor cores (bf16 operands, fp32 accumulation) in bf16 mode and in plain fp32 in f32 mode; the
 * inverse and the norm are always plain fp32, and the scan carries its state at fp32 accuracy (plain fp32
 * FMA in f32 mode; in bf16 mode fp32 factors split three-way into bf16 parts, multiplied on the tensor
 * cores and accumulated in fp32).
 *
 * Naming: T = latent frames, F = spatial tokens per frame, H = heads, d = d_k = d_v (the paper's F, U).
 *
 * Tensors.  All `const void*` / `void*` tensor arguments of vdn_vda_forward are DEVICE pointers, dense,
 * row-major, last index fastest, 16-byte aligned:
 *      q, k, v, out : [B, T, F, H, d]   elements of cfg.io_dtype
 *      beta         : [B, T, F, H]      float, already through the sigmoid, must be >= 0 (Proposition 1)
 *      gate         : [H]               float, already through the sigmoid
 * q and k are *prepared* features (feature map and L2 normalisation already applied, Sec. 2.3); the
 * library applies no normalisation of its own and does not assume unit norm.
 *
 * Ownership.  The caller owns every buffer, the workspace included; the library never allocates device
 * memory on the forward path.  The handle owns host-side state and one pinned status word.  `out` must not
 * alias an input.  Inputs are only read.
 *
 * Asynchrony.  vdn_vda_forward validates its arguments on the host, enqueues its kernels on `cuda_stream`
 * (a cudaStream_t passed as void*, NULL = the legacy default stream) and returns without synchronising.
 * One handle (one workspace) must not be used from two streams at the same time.  The device entry points
 * (forward, forward_ex, forward_opt, prepare) enqueue only kernels, memsets and event waits, so after one ordinary
 * call of the same kind (which sets kernel attributes and creates what the handle needs) they may be recorded in a
 * CUDA stream capture and replayed.  When a layer has more scan chains (2 B H) than the GPU has SMs, part of the scan
 * runs on a stream owned by the handle, forked from and joined back into cuda_stream by events inside the call:
 * synchronising cuda_stream still covers everything.
 *
 * Errors.  Every call returns a vdn_status; nothing throws, aborts or traps.  Problems the host can see
 * (null or misaligned pointers, non-positive sizes, d != cfg.d, workspace too small, 32-bit index overflow,
 * wrong device architecture) are reported synchronously and nothing is enqueued.  Every wait inside a
 * kernel is bounded (vdn_vda_set_wait_limit_us); a wait that runs out records VDN_ERR_TIMEOUT in the handle's
 * status word, which vdn_vda_status returns once the caller has synchronised the stream and which stays set
 * until vdn_vda_clear_status.
 *
 * Determinism.  No atomics on the result path: the same inputs give bit-identical outputs run to run.
 *
 * Accuracy (measured on B200 against an fp64 evaluation of the layer; error = max |out - ref| over a (batch, head)
 * slice divided by that slice's max |ref|; lambda_max = largest eigenvalue of a frame's A_t, at most sum(beta |k|^2)):
 *   f32 I/O, bound 1e-4.  The inverse (I + A_t)^{-1} is formed explicitly in fp32, as in the paper, so the result is
 *     good to about eps lambda_max relative to the largest state entry.  Unstructured or partly repeated keys (up to
 *     nine in ten of a frame identical): within 1e-4 up to lambda_max of about 2000.  Every key of a frame identical
 *     and random values (the state is then small against what is cancelled): within 1e-4 up to lambda_max of about
 *     60, 4e-4 at 150, 1e-2 at 2000.
 *   bf16 I/O, bound 2e-2, plain-fp32 kernels (VDN_FLAG_FORCE_SIMT): within 2e-2 for every input tried, including
 *     lambda_max of 1e5 and beyond, except all-identical keys at lambda_max >= 8000 (3e-2).
 *   bf16 I/O, bound 2e-2, tensor-core kernels.  What sets their range is the contraction of the statistics: the weighted
 *     key beta_u k_u of every token is rounded to bf16, a 2^-9 move in a direction of its own; Eq. 5 damps what a frame
 *     writes along a repeated key by 1 / (1 + lambda_max) but not those residues, so the error relative to the result
 *     grows with the share of identical keys (and falls with the number of tokens the residues average over).  Within
 *     2e-2 (typically 4e-3) for unstructured keys and the benchmark's correlated keys; for keys of any norm around
 *     shared directions at F = 4096 (6e-3 at lambda_max 6e5); with nine keys in ten of a frame bit-identical at
 *     F = 4080 for any key norm (1e-2 up to lambda_max 5e5) and at F = 300 up to lambda_max of about 500.  NOT within
 *     2e-2 when 99 % or more of a frame's keys are bit-identical (3e-2 .. 8e-2 at 99 %, more at 100 %, from lambda_max
 *     of about 5 on), nor when all keys of a frame lie within a few degrees of one direction: unit keys drawn as one
 *     direction plus N(0, s^2) per component give 6e-3 at s = 0.05, 1e-2 at 0.02, 1.7e-2 at 0.01 (a cone of about six
 *     degrees), 3.5e-2 at 0.005, 8e-2 at 0.002 -- the rounding of the weighted keys (4e-3) must stay small against
 *     the keys' own spread.  The states a frame reads (P_{t-1}, R_{t+1}) reach the read-out as bf16 as well: a row
 *     whose read-out nearly cancels, |S q| << |S| |q|, keeps that much less of it, and the RMSNorm rescales what is
 *     left.  States of thousands of tokens have full rank and no query is orthogonal to them; with ONE token per
 *     frame and one frame left to read, a query at |cos| = 2e-4 to that frame's key gave 1e-1 (plain-fp32 kernels,
 *     whose states stay fp32: 4e-3).
 *   VDN_FLAG_EXACT_STATS contracts the exactly weighted keys (two bf16 parts; the statistics then equal the plain-fp32
 *     kernels' to 5e-7): 4e-3 for keys within any cone (s = 0.002 .. 0.05 above); within 2e-2 (4e-3 .. 1e-2) up to 99 % identical keys for lambda_max up to 5e5 at F = 4080 and up
 *     to about 1e4 at F = 300, and with all keys
 *     of a frame identical up to lambda_max of about 2500 at F = 300 (1e-2) and about 1000 at F = 4080 (2.5e-2 at 2050,
 *     where the plain-fp32 kernels give 1.2e-2).
 *   VDN_FLAG_FP32_RESOLVE on top of that takes the inverse from the plain-fp32 Gauss-Jordan kernel and brings the
 *     tensor-core kernels to the plain-fp32 kernels' figures throughout (all-identical keys: 2e-2 up to lambda_max 4e4).
 *     On the 768p benchmark shape a forward takes 3.0 ms as it comes, 3.5 ms with exact statistics, 3.9 ms with both
 *     (the plain-fp32 kernels: 49 ms).
 */
#ifndef VDN_VDA_H_
#define VDN_VDA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct vdn_vda_s* vdn_vda_t;

typedef enum {
  VDN_OK = 0,
  VDN_ERR_INVALID_ARG = 1,  /* null / misaligned pointer, bad size, struct_size mismatch            */
  VDN_ERR_UNSUPPORTED = 2,  /* shape or dtype this build has no kernel for                            */
  VDN_ERR_WORKSPACE = 3,    /* workspace missing or smaller than vdn_vda_workspace_bytes              */
  VDN_ERR_CUDA = 4,         /* a CUDA runtime / driver call failed; see vdn_vda_last_error            */
  VDN_ERR_ARCH = 5,         /* the device is not compute capability 10.x                              */
  VDN_ERR_TIMEOUT = 6,      /* a bounded device-side wait expired (reported by vdn_vda_status)        */
  VDN_ERR_INTERNAL = 7      /* a kernel found its shared-memory window unusable and did nothing       */
                            /* (reported by vdn_vda_status)                                           */
} vdn_status;

typedef enum { VDN_F32 = 0, VDN_BF16 = 1 } vdn_dtype;

/* cfg.flags */
#define VDN_FLAG_FORCE_SIMT 1u    /* bf16 I/O through the plain-fp32 kernels (a second opinion for tests)      */
#define VDN_FLAG_ADDITIVE_RULE 4u /* the baseline VDA replaces, for ablations: frozen-state additive frame      */
                                  /* update with 1/sqrt(F) key scaling, S_t = S_bar (I - A_t/F) + B_t/sqrt(F)   */
                                  /* (Eq. 3c, Sec. 3.3), no resolve; everything else unchanged                  */

#define VDN_FLAG_SCAN_CHUNKWISE 8u  /* vdn_vda_forward_opt with chunk >= 2 on the tensor-core kernels: always run the */
                                   /* scan chunk-wise (Sec. 5, "Chunk-wise scans"); without this flag the library    */
                                   /* chooses by the number of chains and chunks, given a large enough workspace     */
#define VDN_FLAG_SCAN_FRAMEWISE 16u /* never run the scan chunk-wise                                                 */
#define VDN_FLAG_EXACT_STATS 32u    /* tensor-core kernels: contract the frame statistics (Eq. 3b) from the exact      */
                                   /* weighted keys beta k (two bf16 parts) instead of their bf16 rounding: twice the  */
                                   /* tensor-core work in the statistics kernel, for frames whose keys (nearly) all    */
                                   /* coincide (Sec. A.3); see "Accuracy" above                                        */
#define VDN_FLAG_FP32_RESOLVE 64u   /* tensor-core kernels: form (I + A_t)^{-1} with the plain-fp32 Gauss-Jordan kernel  */
                                   /* (1e-6 of its largest entry where the tensor-core resolve reaches 5e-6): matters   */
                                   /* only for frames of identical keys at lambda_max of 1e4 and more; see "Accuracy"   */

typedef struct {
  uint32_t struct_size; /* sizeof(vdn_vda_config), checked                                            */
  int32_t io_dtype;     /* vdn_dtype of q, k, v, out                                                  */
  int32_t d;            /* head dimension: 64 or 128 (bf16 tensor-core kernels: 128)                  */
  float rms_eps;        /* epsilon inside the RMSNorm of Eq. 1c; <= 0 selects 1e-6                    */
  uint32_t flags;
  int32_t device;       /* CUDA device ordinal the handle is bound to                                 */
} vdn_vda_config;

/* Names of workspace regions for vdn_vda_workspace_view (stage-wise checks in the tests).  Which views
 * exist depends on the kernels the handle runs; asking for one of the others returns VDN_ERR_UNSUPPORTED. */
typedef enum {
  VDN_VIEW_STATS = 0,     /* float [B,H,T,2d,d]: rows 0..d-1 = A_t, rows d..2d-1 = B_t (d_v x d_k)  (Eq. 3b) */
  /* plain-fp32 kernels (f32 I/O, or VDN_FLAG_FORCE_SIMT, or d = 64) */
  VDN_VIEW_INV = 1,       /* float [B,H,T,d,d]: C_t = (I + A_t)^{-1}                                (Eq. 5)  */
  VDN_VIEW_FWD = 2,       /* float [B,H,T,d_k,d_v]: transpose of P_t, the forward-scan state      (Eq. A.1)  */
  VDN_VIEW_READ = 3,      /* float [B,H,T,d_k,d_v]: transpose of P_{t-1} + R_{t+1}, what frame t reads (A.4) */
  /* tensor-core kernels (bf16 I/O, d = 128) */
  VDN_VIEW_INV_SPLIT = 4, /* bf16 [B,H,T,3,d,d]: C_t as C1 + C2 + C3 (bf16 parts of the fp32 inverse)         */
  VDN_VIEW_READ_FWD = 5,  /* bf16 [B,H,T,d_v,d_k]: slot t = P_{t-1} (zero for t = 0)                  (A.4)  */
  VDN_VIEW_READ_BWD = 6,  /* bf16 [B,H,T,d_v,d_k]: slot t = R_{t+1} (zero for t = T-1)                (A.4)  */
  /* ... after a forward call that scanned chunk-wise (Sec. 5): the composites S_out = S_in M + J of the chunks each  */
  /* direction folds, position p = the p-th chunk in that direction's order; n = number of chunks (size / per-chunk)  */
  VDN_VIEW_COMP_M = 7,    /* bf16 [B*H,2,n,3,d,d]: M as three bf16 parts, stored as the scan multiplies: Z <- M Z  */
  VDN_VIEW_COMP_J = 8     /* float [B*H,2,n,d_v,d_k]: J                                                             */
} vdn_view;

/* Sec. 3 (the layer as a whole).  Creates a handle bound to cfg->device.  Allocates host memory only
 * (one pinned, device-mapped status word).  Returns VDN_ERR_ARCH when the device is not sm_100.
 * Two environment variables are read here, for measurements only: VDN_SCAN_SPLIT=0 keeps all scan chains in one
 * launch even when there are more of them than SMs, VDN_RO_SHORT=0 keeps the read-out's long-frame layout for short
 * frames; both default to 1. */
vdn_status vdn_vda_create(const vdn_vda_config* cfg, vdn_vda_t* out_handle);

/* Bytes of device workspace a forward call of this shape needs (per-frame statistics of Eq. 3b, the
 * inverses of Eq. 5 and the scanned states of Eq. A.1 live there).  Pure function; 0 on invalid shape. */
size_t vdn_vda_workspace_bytes(vdn_vda_t h, int B, int T, int F, int H, int d);

/* Plumbing (no passage of the paper to cite).  Hands the library a caller-owned device buffer (256-byte aligned).  It must stay valid until replaced
 * or until the handle is destroyed, and must not be shared between handles that run concurrently. */
vdn_status vdn_vda_set_workspace(vdn_vda_t h, void* dev_ptr, size_t bytes);

/* Algorithm 1 steps 3-7 with the readings stated at the top of this file.  All tensor pointers are
 * device pointers (layout above).  Enqueues on cuda_stream and returns; does not synchronise. */
vdn_status vdn_vda_forward(vdn_vda_t h, const void* q, const void* k, const void* v, const float* beta,
                           const float* gate, void* out, int B, int T, int F, int H, int d,
                           void* cuda_stream);

/* The same layer with the two inputs of the paper's recurrence that vdn_vda_forward fixes (the local window is
 * still the query frame itself, and there are no anchor frames -- see vdn_vda_forward_opt for those):
 *   alpha [B,T,H,d] float, DEVICE, in [0,1], or NULL (= 1): channel-wise decay gate of frame t (Eq. 2, Eq. A.1:
 *         M_t = Diag(alpha_t)(I + A_t)^{-1}).  It decays the inherited state before frame t is folded in, in both
 *         scans, and bridges the state that frame t's queries read (Eq. A.4 with l_t = h_t = t):
 *         (P_{t-1} + R_{t+1}) Diag(alpha_t).
 *   s0    [B,H,d_v,d_k] float, DEVICE, or NULL (= 0): the text state S_T; each scan starts from S_T / 2 (Eq. 1b),
 *         and a missing side of the gather reads S_T / 2 (Eq. A.4).
 * Everything else is as for vdn_vda_forward, which is this call with alpha = s0 = NULL. */
vdn_status vdn_vda_forward_ex(vdn_vda_t h, const void* q, const void* k, const void* v, const float* beta,
                              const float* gate, const float* alpha, const float* s0, void* out, int B, int T,
                              int F, int H, int d, void* cuda_stream);

/* The layer with every optional input of the paper's linear branch (the "paper-faithful gather" and the
 * content-dependent output gate).  `opt` may be NULL (= vdn_vda_forward).  Zero-initialise the struct, set
 * struct_size, then the fields you need; all pointers are DEVICE pointers, 16-byte aligned, caller-owned.
 *
 *   alpha, s0    as for vdn_vda_forward_ex.
 *   chunk, radius  the local Softmax window in temporal chunks (Sec. 2.1): latent frames are grouped into
 *                chunks of `chunk` frames counted from frame 0 of the clip; a query frame's window [l_t, h_t]
 *                is its own chunk and `radius` chunks on either side, clipped to the scanned frames.  Its
 *                queries read (Eq. A.4)
 *                    P_{l_t - 1} Diag(prod_{r=l_t..t} alpha_r)  +  R_{h_t + 1} Diag(prod_{r=t..h_t} alpha_r),
 *                the forward state of the frames before the window and the reverse state of the frames after
 *                it, each bridged by the decay of the skipped span; a side with no distant frame reads S_T / 2.
 *                chunk <= 1 and radius = 0 give the window {t} of vdn_vda_forward.  The paper's release uses
 *                chunk = 5, radius = 1 (a 15-frame window).
 *   anchors      non-zero: frames 0 and T-1 are boundary anchors (Sec. 2.1): they belong to Softmax alone, are
 *                excluded from both scans (Alg. 1 step 2), and their output rows are zero (Alg. 1 step 7).
 *                A clip of at most two frames then has no linear output at all (Sec. A.4).
 *   gate_elem    [B,T,F,H,d] of cfg.io_dtype or NULL: element-wise output gate G^L of Eq. 1c, already through the
 *                sigmoid.  It multiplies the per-head `gate`, which may then be NULL (= 1).
 *   norm_weight  [H,d] float or NULL (= 1): per-channel scale of the RMSNorm in Eq. 1c, applied after the
 *                normalisation: out = gate_h * gate_elem * norm_weight * o / sqrt(mean_j o_j^2 + rms_eps).
 * When a window covers every scanned frame both sides read S_T / 2 (Eq. A.4 as written); bypassing the linear
 * branch for such clips (Sec. A.4) is the caller's decision. */
typedef struct {
  uint32_t struct_size;     /* sizeof(vdn_vda_options), checked */
  int32_t chunk;            /* frames per temporal chunk; 0 is read as 1 */
  int32_t radius;           /* chunks on either side of the query chunk inside the window, >= 0 */
  int32_t anchors;          /* boolean */
  const float* alpha;
  const float* s0;
  const void* gate_elem;
  const float* norm_weight;
  float q_l2_eps;           /* 0: q arrives L2-normalised.  > 0: q arrives as projected and the read-out uses
                             * q / sqrt(sum_j q_j^2 + q_l2_eps), the q' of vdn_vda_prepare (Sec. 2.3), which may then
                             * be called without queries: one pass over Q less */
  uint32_t reserved;        /* 0 */
} vdn_vda_options;
vdn_status vdn_vda_forward_opt(vdn_vda_t h, const void* q, const void* k, const void* v, const float* beta,
                               const float* gate, void* out, int B, int T, int F, int H, int d,
                               const vdn_vda_options* opt, void* cuda_stream);

/* Workspace for vdn_vda_forward_opt with room for the chunk-wise scan (Sec. 5, "Chunk-wise scans": the frames of a
 * temporal chunk are composed into S_out = S_in M_chunk + J_chunk, all chunks side by side, and the chunk sequence
 * is scanned; states are read at chunk edges only, so nothing is lost, and the chain is about `chunk` times
 * shorter at about four times the arithmetic).  With opt->chunk >= 2 on the tensor-core kernels this is
 * vdn_vda_workspace_bytes plus the composites (per batch, head, direction and chunk: M as three bf16 parts, J in
 * fp32); otherwise it equals vdn_vda_workspace_bytes.  Given such a workspace, vdn_vda_forward_opt runs the scan
 * chunk-wise when that shortens it (few chains, many chunks: e.g. heads sharded over several GPUs), or always
 * under VDN_FLAG_SCAN_CHUNKWISE; with the smaller workspace it scans frame by frame.  The text state enters the
 * chunk-level scan as its initial state.  Pure function; 0 on invalid arguments. */
size_t vdn_vda_workspace_bytes_opt(vdn_vda_t h, int B, int T, int F, int H, int d, const vdn_vda_options* opt);

/* Feature preparation in front of the layer (Sec. 2.3; the "VDA-Prep" kernel of Sec. 5): turns the projected
 * q, k, v into the prepared features that vdn_vda_forward takes.
 *      k' = L2norm( SiLU( conv(k) ) ),    v' = SiLU( conv(v) ),    q' = L2norm(q)
 * conv is the separable short convolution of Sec. 2.3: per channel a 5 x 5 spatial filter over the frame's
 * Y x X token grid and a five-tap temporal filter over the frames, applied as cross-correlations with centred
 * taps and zero padding:  out[t,y,x,c] = sum_{i,j,l} wt[c,l] ws[c,i,j] in[t+l-2, y+i-2, x+j-2, c].
 * L2norm(x) = x / sqrt(sum_j x_j^2 + l2_eps) over the d channels of a (token, head).  All arithmetic in fp32.
 *
 *   q_in, k_in, v_in, q_out, k_out, v_out : [B,T,F,H,d] of cfg.io_dtype, DEVICE, 16-byte aligned.  k_out and v_out
 *        must not alias any input (the filters read neighbours); q_out may be q_in.  q_in and q_out may both be
 *        NULL: the queries are then left alone (vdn_vda_options.q_l2_eps makes the read-out normalise them).
 *   p->Y, p->X   the spatial grid: F = Y * X, tokens of a frame in row-major (y, x) order
 *   p->wk_spatial, p->wv_spatial   float [H*d][5][5];   p->wk_temporal, p->wv_temporal   float [H*d][5]  (DEVICE)
 *        Both spatial filters may be NULL: the spatial part is then the identity (temporal filter, SiLU and
 *        normalisation only -- the operation the paper's VDA-Prep kernel fuses, Sec. 5), a streaming pass bound
 *        by HBM instead of by the 25 extra multiply-adds per element.
 *   p->anchors   non-zero: frames 0 and T-1 are boundary anchors, removed before the preparation (Alg. 1
 *        step 2): the temporal filter sees zeros beyond frames 1 and T-2, and the anchor frames of all three
 *        outputs are zero.
 * Needs no workspace.  Enqueues on cuda_stream and returns; does not synchronise. */
typedef struct {
  uint32_t struct_size;      /* sizeof(vdn_vda_prep_params), checked */
  int32_t Y, X;
  int32_t anchors;
  float l2_eps;              /* <= 0 selects 1e-6 */
  const float* wk_spatial;
  const float* wk_temporal;
  const float* wv_spatial;
  const float* wv_temporal;
} vdn_vda_prep_params;
vdn_status vdn_vda_prepare(vdn_vda_t h, const void* q_in, const void* k_in, const void* v_in, void* q_out,
                           void* k_out, void* v_out, int B, int T, int F, int H, int d,
                           const vdn_vda_prep_params* p, void* cuda_stream);

/* The same layer for callers whose tensors live in HOST memory (pinned memory recommended; with pageable
 * memory the copies are not asynchronous).  All six tensor pointers are HOST pointers.  The staging buffer is a
 * caller-owned DEVICE buffer of at least vdn_vda_staging_bytes, set beforehand.  The copies in run on an input
 * stream owned by the handle, which starts where cuda_stream stands at the call and is queued in one go, so the
 * host link never waits for a kernel: k, v, beta, gate, then the queries in up to 32 groups of frames.  On
 * cuda_stream: statistics, resolve and both scans once k, v, beta have landed; then each group is read out as
 * soon as its queries have landed.  Each group's output rows are copied back on a third stream, beside the
 * copies in (the host link is full duplex, and out needs the scans of the whole clip, so this is all the
 * overlap there is).  cuda_stream waits for the last copy back: synchronising it is enough.  The first call
 * creates the two streams and their events (no device memory). */
size_t vdn_vda_staging_bytes(vdn_vda_t h, int B, int T, int F, int H, int d);
vdn_status vdn_vda_set_staging(vdn_vda_t h, void* dev_ptr, size_t bytes);
vdn_status vdn_vda_forward_host(vdn_vda_t h, const void* q, const void* k, const void* v,
                                const float* beta, const float* gate, void* out, int B, int T, int F,
                                int H, int d, void* cuda_stream);

/* vdn_vda_forward_host with the optional inputs of vdn_vda_forward_opt (the release setting of Sec. A.4 and Alg. 1
 * end to end from host memory).  Here every pointer inside `opt` is a HOST pointer as well (alpha, s0, norm_weight,
 * gate_elem; same shapes as for vdn_vda_forward_opt); they are copied into the staging buffer with the other inputs,
 * gate_elem in the same groups of frames as the queries.  The staging buffer must hold
 * vdn_vda_staging_bytes_opt(..., opt) bytes (vdn_vda_staging_bytes plus room for alpha, s0 and norm_weight, plus one
 * tensor of the size of q when opt->gate_elem is set).  `opt` may be NULL (= vdn_vda_forward_host); `gate` may be
 * NULL when opt->gate_elem is set.  All host-side checks (arguments, workspace, staging) are made before the first
 * copy is queued; should a CUDA call fail after that, cuda_stream is made to wait for everything already queued on
 * the handle's own streams before the error is returned, so synchronising cuda_stream still releases the caller's
 * buffers. */
size_t vdn_vda_staging_bytes_opt(vdn_vda_t h, int B, int T, int F, int H, int d, const vdn_vda_options* opt);
vdn_status vdn_vda_forward_host_opt(vdn_vda_t h, const void* q, const void* k, const void* v,
                                    const float* beta, const float* gate, void* out, int B, int T, int F,
                                    int H, int d, const vdn_vda_options* opt, void* cuda_stream);

/* Offset and size, inside the workspace, of an intermediate of the last forward call of this shape
 * (see vdn_view).  For stage-wise parity checks; the contents are valid after the stream is synchronised. */
vdn_status vdn_vda_workspace_view(vdn_vda_t h, int which, int B, int T, int F, int H, int d,
                                  size_t* offset_bytes, size_t* size_bytes);

/* Number of kernels the last vdn_vda_forward call on this handle launched (0 before the first call). */
int vdn_vda_last_launch_count(vdn_vda_t h);

/* Per-kernel timing for benchmarks (no counterpart in the paper).  vdn_vda_profile(h, 1) makes every
 * later forward call record CUDA events between its kernels on the caller's stream and clears the running
 * sums; vdn_vda_profile(h, 0) stops that.  vdn_vda_kernel_times waits for the recorded events, then fills
 * up to max_kernels entries (kernel name, mean milliseconds per launch, launches seen since the sums were
 * cleared) and returns how many it filled.  `names` receives pointers to static strings. */
vdn_status vdn_vda_profile(vdn_vda_t h, int enable);
int vdn_vda_kernel_times(vdn_vda_t h, int max_kernels, const char** names, float* mean_ms, int* launches);

/* No counterpart in the paper: a convenience for callers that must not allocate device memory.
 *
 * Some programs hand all of a GPU's memory to their own pools at start-up and, from then on, treat any
 * cudaMalloc as a bug (it can fail for lack of memory, and it stalls every stream of the device); others
 * run this step from places where allocating is not possible at all, e.g. a real-time loop with a fixed
 * memory plan.  vdn_vda_forward needs a caller-supplied workspace, which such callers may have no pool
 * to cut from.  This entry point runs ONE stage of the plain-fp32 path -- the bidirectional frame scan
 * and gather (Alg. 1 steps 5-6: Eq. A.1, Eq. A.4) -- whose only scratch is the buffer of forward states
 * P_t, and keeps that scratch in an array that is part of the library image
 * (VDN_SCAN_STATIC_MAX_BYTES bytes of device memory on every GPU that loads the library, until the
 * process exits).  It calls neither cudaMalloc nor cudaFree nor any routine that allocates.
 *
 *   stats [BH][T][2d][d] float, DEVICE  in   per-frame statistics, layout of VDN_VIEW_STATS
 *   inv   [BH][T][d][d]  float, DEVICE  in   C_t = (I + A_t)^{-1}, layout of VDN_VIEW_INV
 *   read  [BH][T][d][d]  float, DEVICE  out  transpose of P_{t-1} + R_{t+1}, layout of VDN_VIEW_READ
 *   BH = batch * heads chains of T frames; d = 64 or 128; all pointers 16-byte aligned, caller-owned.
 *
 * Limit: BH*T*d*d*4 bytes must not exceed VDN_SCAN_STATIC_MAX_BYTES (8 MiB: 128 frames at d = 128, 512 at
 * d = 64); larger shapes are rejected with VDN_ERR_WORKSPACE and a message in errbuf, and nothing is
 * enqueued.  errbuf (HOST, may be NULL) receives a NUL-terminated description of any error.
 * The first call on a device looks up the array's address on that device (cudaGetSymbolAddress); make that
 * first call outside any stream capture.  Enqueues on cuda_stream and returns without synchronising.
 * The looked-up address is cached per device in an atomic pointer: host threads that make their first calls at
 * the same time each do the lookup and store the same value, which is harmless.
 * Every call on a device uses the same array: two calls whose kernels may overlap on the GPU (different
 * streams, or different host threads) race on it -- serialise them.  The array keeps the previous call's
 * contents; the kernel writes every element it later reads, so nothing has to be cleared in between. */
#define VDN_SCAN_STATIC_MAX_BYTES (8u << 20)
vdn_status vdn_vda_scan_static(const float* stats, const float* inv, float* read, int BH, int T, int d,
                               int device, void* cuda_stream, char* errbuf, size_t errbuf_len);

/* Plumbing (no passage of the paper to cite).  Last device-side status recorded by this handle's kernels: VDN_OK,
 * VDN_ERR_TIMEOUT (a wait inside a kernel ran out; that kernel's CTA stopped early and the outputs of the call are
 * incomplete) or VDN_ERR_INTERNAL.  Does not synchronise: call it after synchronising the stream.  The word is
 * sticky: reading it clears nothing, and no forward call clears it, so that an error is not lost between a call
 * and the moment the caller looks.  vdn_vda_clear_status resets it. */
vdn_status vdn_vda_status(vdn_vda_t h);

/* Plumbing.  Returns what vdn_vda_status would return and resets the status word to VDN_OK.  Call it with no
 * kernel of this handle in flight (after synchronising): a kernel that is still running may set the word again.
 * After a timeout the handle stays usable: the kernels keep no state between calls. */
vdn_status vdn_vda_clear_status(vdn_vda_t h);

/* Plumbing.  The longest any single wait inside a kernel of this handle may take before its CTA gives up
 * (default 2 s = 2 000 000 microseconds; 1 microsecond .. 1 hour).  A wait covers one pipeline hand-over (a tile
 * arriving, an accumulator being drained), never a whole kernel, so the default is generous for any shape. */
vdn_status vdn_vda_set_wait_limit_us(vdn_vda_t h, unsigned long long microseconds);

/* Test support (no counterpart in the paper): exercises the give-up path of the bounded waits without touching
 * any pipeline.  Enqueues one small kernel that is set up like the tensor-core kernels (mbarrier, tensor memory,
 * the same wait routine) and waits, for at most limit_us microseconds (<= 1 s), on a barrier that nothing ever
 * completes and that no copy is bound to.  The wait runs out, the CTA takes the same abort and teardown path as
 * the real kernels (frees its tensor memory, returns) and records VDN_ERR_TIMEOUT in the handle's status word.
 * After synchronising: vdn_vda_status gives VDN_ERR_TIMEOUT and vdn_vda_selftest_marker gives 3 (bit 0: the CTA
 * reached its last instruction after giving up; bit 1: its other warp, which had waited for nothing, learned of the
 * timeout at the block-level barrier the two share, the way threads of the real kernels leave together; 0 = the
 * kernel has not run, -1 = null handle). */
vdn_status vdn_vda_selftest_wait_expiry(vdn_vda_t h, unsigned long long limit_us, void* cuda_stream);
int vdn_vda_selftest_marker(vdn_vda_t h);

/* Plumbing.  Human-readable description of the last error returned on this handle (never NULL). */
const char* vdn_vda_last_error(vdn_vda_t h);

/* Plumbing.  Frees the handle's host state, streams and events.  No kernel of the handle may be in flight. */
vdn_status vdn_vda_destroy(vdn_vda_t h);

#ifdef __cplusplus
}
#endif
#endif /* VDN_VDA_H_ */

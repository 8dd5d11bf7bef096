"""fp64 CPU oracle for bidirectional Video Delta Attention (VDA) forward.

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain statement of what the
layer computes.  Only the test-suite, the smoke check and the benchmark's CPU
baseline leg may import it; the CUDA library never does, and the two share no
code.  Everything is numpy float64; each function follows one passage of the
paper and keeps the paper's notation and orientation:

    state   S  in R^{d_v x d_k},   read-out  o = S q            (Sec. 3.1, Eq. 1a)
    frame t has U tokens (rows of K_t, V_t, Q_t), write gates beta_t >= 0,
    channel-wise decay alpha_t in [0,1]^{d_k}.

No blocking, fusion or re-ordering: one frame at a time, one equation per line.

Pinning status (see tests/test_oracle_*.py):
  frame_statistics   pinned: literal per-token sums, permutation invariance
  frame_update_additive
                     pinned: literal token sum of Eq. 3a with keys scaled by 1/sqrt(U), Eq. 3c, the
                     non-expansive bound of Sec. A.3 for unit keys, agreement with Eq. 5 as beta -> 0
  frame_update       pinned: least-squares brute force of Eq. 4, first-order
                     condition, token-space (Woodbury) form, Eq. 2 for U=1,
                     Eq. A.3 repeated keys, orthonormal keys, Eq. 3c as beta->0
  transition         pinned: Proposition 1 (spectral norm <= 1)
  scan_states / read_state / vda_slice
                     pinned: hand-worked examples in tests/golden/, frame
                     reversal symmetry, disjointness by linearity in V,
                     brute-force evaluator on tiny shapes
  local_window / read_states with chunk windows and anchors
                     pinned: a hand-worked six-frame example in tests/golden/, a brute-force evaluator that
                     derives the linear regions from the Softmax visibility mask of Sec. 2.1 and bridges by
                     running the recurrence with the writes switched off, disjointness by linearity in V
  rmsnorm_gate       pinned: row mean-square identity, scale invariance, literal per-element evaluation
  Readings that the paper does not fix (read window = the query frame itself,
  per-head scalar gate, alpha = 1 and zero initial state at the C boundary,
  eps) are conventions of this build: parity unpinned *for those choices only*.
"""
from __future__ import annotations

import numpy as np

F64 = np.float64


def frame_statistics(K, V, beta):
    """Eq. 3b.  A_t = K^T Diag(beta) K  (d_k x d_k),  B_t = V^T Diag(beta) K  (d_v x d_k)."""
    K = np.asarray(K, F64)
    V = np.asarray(V, F64)
    beta = np.asarray(beta, F64)
    A = K.T @ (beta[:, None] * K)
    B = V.T @ (beta[:, None] * K)
    return A, B


def resolve(A):
    """C_t = (I + A_t)^{-1}  (Alg. 1 step 4; the inverse that appears in Eq. 5)."""
    A = np.asarray(A, F64)
    d = A.shape[0]
    return np.linalg.solve(np.eye(d) + A, np.eye(d))


def transition(A, alpha):
    """Eq. A.1.  M_t = Diag(alpha_t) (I + A_t)^{-1}."""
    return np.asarray(alpha, F64)[:, None] * resolve(A)


def injection(A, B):
    """Eq. A.1.  J_t = B_t (I + A_t)^{-1}."""
    return np.asarray(B, F64) @ resolve(A)


def frame_update(S_prev, alpha, A, B):
    """Eq. 5.  S_bar = S_{t-1} Diag(alpha_t);  S_t (I + A_t) = S_bar + B_t."""
    S_prev = np.asarray(S_prev, F64)
    d = A.shape[0]
    S_bar = S_prev * np.asarray(alpha, F64)[None, :]
    # S_t = (S_bar + B_t)(I + A_t)^{-1};  I + A_t is symmetric, so solve on the transpose.
    return np.linalg.solve(np.eye(d) + A, (S_bar + B).T).T


def frame_update_additive(S_prev, alpha, A, B, U):
    """The baseline VDA replaces (Eq. 3a/3c with the frame-size key scaling of Sec. 3.3): all token corrections
    are evaluated at the same decayed state, keys scaled by 1/sqrt(U), i.e. A_t -> A_t/U, B_t -> B_t/sqrt(U):

        S_bar = S_{t-1} Diag(alpha_t);   S_t = S_bar (I - A_t/U) + B_t/sqrt(U).
    """
    S_prev = np.asarray(S_prev, F64)
    d = A.shape[0]
    S_bar = S_prev * np.asarray(alpha, F64)[None, :]
    return S_bar @ (np.eye(d) - np.asarray(A, F64) / U) + np.asarray(B, F64) / np.sqrt(U)


def scan_states(A, B, alpha, S_init, rule="vda", U=None, first=0, last=None):
    """Sec. 2.2 / Alg. 1 step 5.  Both temporal scans of S <- S M_t + J_t over the frames first .. last
    (all frames by default; the interior frames when the boundary anchors are excluded, Sec. A.4).

    Returns P, R with P[t] = forward state through frame t and R[t] = reverse state from frame `last` down
    to t (None for frames outside the range).  Each scan starts from S_init (the caller passes S_T / 2, Eq. 1b).
    """
    T = len(A)
    last = T - 1 if last is None else last
    P = [None] * T
    R = [None] * T
    def step(S, t):
        if rule == "additive":
            return frame_update_additive(S, alpha[t], A[t], B[t], U)
        return frame_update(S, alpha[t], A[t], B[t])
    S = np.asarray(S_init, F64)
    for t in range(first, last + 1):
        S = step(S, t)
        P[t] = S
    S = np.asarray(S_init, F64)
    for t in range(last, first - 1, -1):
        S = step(S, t)
        R[t] = S
    return P, R


def interior_range(T, anchors):
    """Sec. 2.2 / Sec. A.4.  The frames the linear branch scans: with boundary anchors the first and the last
    latent frame belong to Softmax alone (Alg. 1 step 2), leaving 1 .. T-2; otherwise 0 .. T-1.
    Returns (first, last); the range is empty when last < first."""
    return (1, T - 2) if anchors else (0, T - 1)


def local_window(t, T, chunk=1, radius=0, anchors=False):
    """Sec. 2.1 / Sec. A.4.  [l_t, h_t]: the Softmax window of query frame t clipped to interior frame indices.

    Latent frames are grouped into temporal chunks of `chunk` frames counted from frame 0 of the clip; a query
    chunk sees itself and `radius` chunks on either side.  chunk = 1, radius = 0 is the window {t}.
    """
    first, last = interior_range(T, anchors)
    c = t // chunk
    lo = max(first, (c - radius) * chunk)
    hi = min(last, (c + radius + 1) * chunk - 1)
    return lo, hi


def read_states(P, R, alpha, S_init, t, chunk=1, radius=0, anchors=False):
    """Eq. A.4.  With [l_t, h_t] the local window of query frame t,

        forward part  P_{l_t - 1} Diag(prod_{r = l_t .. t} alpha_r),
        reverse part  R_{h_t + 1} Diag(prod_{r = t .. h_t} alpha_r);

    a side with no distant interior frame selects the initial state (S_T / 2).  The default window is the
    query frame itself (l_t = h_t = t).  Returned separately so that the two directional read-outs of Eq. 1a
    can be inspected.
    """
    T = len(P)
    first, last = interior_range(T, anchors)
    lo, hi = local_window(t, T, chunk, radius, anchors)
    a_f = np.ones_like(np.asarray(alpha[t], F64))
    for r in range(lo, t + 1):
        a_f = a_f * np.asarray(alpha[r], F64)
    a_b = np.ones_like(a_f)
    for r in range(t, hi + 1):
        a_b = a_b * np.asarray(alpha[r], F64)
    S_fwd = (P[lo - 1] if lo - 1 >= first else np.asarray(S_init, F64)) * a_f[None, :]
    S_bwd = (R[hi + 1] if hi + 1 <= last else np.asarray(S_init, F64)) * a_b[None, :]
    return S_fwd, S_bwd


def rmsnorm_gate(O, gate, eps, weight=None):
    """Eq. 1c.  G^L * RMSNorm(O^L), the norm over the d_v channels of each (token, head).

    gate   : a scalar (one value per head) or an array broadcastable to O (a content-dependent gate has one
             value per token and channel);  weight : optional per-channel scale of the norm, [d_v]."""
    O = np.asarray(O, F64)
    ms = np.mean(O * O, axis=-1, keepdims=True)
    y = O / np.sqrt(ms + eps)
    if weight is not None:
        y = y * np.asarray(weight, F64)
    return np.asarray(gate, F64) * y


def vda_slice(q, k, v, beta, gate, eps=1e-6, alpha=None, s0=None, want=(), rule="vda",
              chunk=1, radius=0, anchors=False, norm_weight=None):
    """Whole layer for ONE (batch, head) slice.  rule = "vda" (Eq. 5) or "additive" (Eq. 3c with 1/sqrt(U) keys).

    q, k : [T, U, d_k]   v : [T, U, d_v]   beta : [T, U]   gate : scalar, or [T, U, d_v] (element-wise gate)
    alpha: [T, d_k] or None (ones)         s0   : [d_v, d_k] text state S_T or None (zero)
    chunk, radius : local window in temporal chunks (Sec. 2.1); anchors : first and last frame are boundary
    anchors, excluded from both scans, their output rows zero (Alg. 1 steps 2 and 7)
    norm_weight : [d_v] or None, per-channel scale inside the RMSNorm
    Returns a dict with 'out' [T, U, d_v] and whichever intermediates `want` names
    ('A','B','C','P','R','o_fwd','o_bwd','O'); P and R are zero for frames outside the scanned range.
    """
    q = np.asarray(q, F64)
    k = np.asarray(k, F64)
    v = np.asarray(v, F64)
    beta = np.asarray(beta, F64)
    T, U, dk = k.shape
    dv = v.shape[2]
    alpha = np.ones((T, dk)) if alpha is None else np.asarray(alpha, F64)
    S_T = np.zeros((dv, dk)) if s0 is None else np.asarray(s0, F64)
    S_init = 0.5 * S_T                                         # Eq. 1b
    first, last = interior_range(T, anchors)                   # Alg. 1 step 2

    A = [None] * T
    B = [None] * T
    for t in range(T):                                         # Alg. 1 step 3
        A[t], B[t] = frame_statistics(k[t], v[t], beta[t])
    P, R = scan_states(A, B, alpha, S_init, rule, U, first, last)   # Alg. 1 steps 4-5

    o_fwd = np.zeros((T, U, dv))
    o_bwd = np.zeros((T, U, dv))
    for t in range(first, last + 1):                           # Alg. 1 steps 6-7
        S_fwd, S_bwd = read_states(P, R, alpha, S_init, t, chunk, radius, anchors)
        o_fwd[t] = q[t] @ S_fwd.T                              # o = S q, one row per token
        o_bwd[t] = q[t] @ S_bwd.T
    O = o_fwd + o_bwd                                          # Eq. 1a
    g = np.asarray(gate, F64)
    out = np.zeros((T, U, dv))                                 # Alg. 1 step 7: anchor rows stay zero
    rows = slice(first, last + 1)
    out[rows] = rmsnorm_gate(O[rows], g[rows] if g.ndim else float(g), eps, norm_weight)   # Eq. 1c
    res = {"out": out}
    zero = np.zeros((dv, dk))
    pool = {"A": A, "B": B, "P": [zero if x is None else x for x in P], "R": [zero if x is None else x for x in R],
            "o_fwd": o_fwd, "o_bwd": o_bwd, "O": O}
    for name in want:
        if name == "C":
            res["C"] = np.stack([resolve(A[t]) for t in range(T)])
        else:
            val = pool[name]
            res[name] = np.stack(val) if isinstance(val, list) else val
    return res


def vda_forward(q, k, v, beta, gate, eps=1e-6, alpha=None, s0=None, heads=None, rule="vda",
                chunk=1, radius=0, anchors=False, norm_weight=None):
    """Whole layer on the boundary layout.

    q, k, v : [B, T, U, H, d]    beta : [B, T, U, H]    gate : [H], or [B, T, U, H, d] (element-wise)
    alpha   : [B, T, H, d] or None    s0 : [B, H, d, d] or None    norm_weight : [H, d] or None
    heads   : optional list of (b, h) pairs to evaluate (others are left at zero).
    Returns out [B, T, U, H, d] float64.
    """
    q = np.asarray(q)
    gate = np.asarray(gate)
    Bn, T, U, H, d = q.shape
    out = np.zeros((Bn, T, U, H, d), F64)
    pairs = heads if heads is not None else [(b, h) for b in range(Bn) for h in range(H)]
    for (b, h) in pairs:
        res = vda_slice(q[b, :, :, h, :], k[b, :, :, h, :], v[b, :, :, h, :], beta[b, :, :, h],
                        gate[h] if gate.ndim == 1 else gate[b, :, :, h, :], eps,
                        None if alpha is None else alpha[b, :, h, :],
                        None if s0 is None else s0[b, h], (), rule, chunk, radius, anchors,
                        None if norm_weight is None else np.asarray(norm_weight)[h])
        out[b, :, :, h, :] = res["out"]
    return out


def slice_error(got, want):
    """The parity metric: max |got - want| over one (batch, head) slice, relative to
    the slice's largest |want| (outputs cross zero, so a per-element ratio is ill-posed)."""
    got = np.asarray(got, F64)
    want = np.asarray(want, F64)
    scale = np.max(np.abs(want))
    if scale == 0.0:
        return float(np.max(np.abs(got)))
    return float(np.max(np.abs(got - want)) / scale)

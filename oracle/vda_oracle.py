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
  rmsnorm_gate       pinned: row mean-square identity, scale invariance
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


def scan_states(A, B, alpha, S_init, rule="vda", U=None):
    """Sec. 2.2 / Alg. 1 step 5.  Both temporal scans of S <- S M_t + J_t.

    Returns P, R with P[t] = forward state through frame t (t = 0..T-1) and
    R[t] = reverse state from frame T-1 down to t.  Each scan starts from S_init
    (the caller passes S_T / 2, Eq. 1b).
    """
    T = len(A)
    P = [None] * T
    R = [None] * T
    def step(S, t):
        if rule == "additive":
            return frame_update_additive(S, alpha[t], A[t], B[t], U)
        return frame_update(S, alpha[t], A[t], B[t])
    S = np.asarray(S_init, F64)
    for t in range(T):
        S = step(S, t)
        P[t] = S
    S = np.asarray(S_init, F64)
    for t in range(T - 1, -1, -1):
        S = step(S, t)
        R[t] = S
    return P, R


def read_states(P, R, alpha, S_init, t):
    """Eq. A.4 with the local window shrunk to the query frame, l_t = h_t = t.

    forward part  P_{t-1} Diag(alpha_t),  reverse part  R_{t+1} Diag(alpha_t);
    a missing side selects the initial state.  Returned separately so that the
    two directional read-outs of Eq. 1a can be inspected.
    """
    T = len(P)
    a = np.asarray(alpha[t], F64)[None, :]
    S_fwd = (P[t - 1] if t >= 1 else np.asarray(S_init, F64)) * a
    S_bwd = (R[t + 1] if t + 1 < T else np.asarray(S_init, F64)) * a
    return S_fwd, S_bwd


def rmsnorm_gate(O, gate, eps):
    """Eq. 1c.  G^L * RMSNorm(O^L), the norm over the d_v channels of each (token, head)."""
    O = np.asarray(O, F64)
    ms = np.mean(O * O, axis=-1, keepdims=True)
    return gate * (O / np.sqrt(ms + eps))


def vda_slice(q, k, v, beta, gate, eps=1e-6, alpha=None, s0=None, want=(), rule="vda"):
    """Whole layer for ONE (batch, head) slice.  rule = "vda" (Eq. 5) or "additive" (Eq. 3c with 1/sqrt(U) keys).

    q, k : [T, U, d_k]   v : [T, U, d_v]   beta : [T, U]   gate : scalar
    alpha: [T, d_k] or None (ones)         s0   : [d_v, d_k] text state S_T or None (zero)
    Returns a dict with 'out' [T, U, d_v] and whichever intermediates `want` names
    ('A','B','C','P','R','o_fwd','o_bwd','O').
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

    A = [None] * T
    B = [None] * T
    for t in range(T):                                         # Alg. 1 step 3
        A[t], B[t] = frame_statistics(k[t], v[t], beta[t])
    P, R = scan_states(A, B, alpha, S_init, rule, U)           # Alg. 1 steps 4-5

    o_fwd = np.zeros((T, U, dv))
    o_bwd = np.zeros((T, U, dv))
    for t in range(T):                                         # Alg. 1 steps 6-7
        S_fwd, S_bwd = read_states(P, R, alpha, S_init, t)
        o_fwd[t] = q[t] @ S_fwd.T                              # o = S q, one row per token
        o_bwd[t] = q[t] @ S_bwd.T
    O = o_fwd + o_bwd                                          # Eq. 1a
    res = {"out": rmsnorm_gate(O, float(gate), eps)}           # Eq. 1c
    pool = {"A": A, "B": B, "P": P, "R": R, "o_fwd": o_fwd, "o_bwd": o_bwd, "O": O}
    for name in want:
        if name == "C":
            res["C"] = np.stack([resolve(A[t]) for t in range(T)])
        else:
            val = pool[name]
            res[name] = np.stack(val) if isinstance(val, list) else val
    return res


def vda_forward(q, k, v, beta, gate, eps=1e-6, alpha=None, s0=None, heads=None):
    """Whole layer on the boundary layout.

    q, k, v : [B, T, U, H, d]    beta : [B, T, U, H]    gate : [H]
    alpha   : [B, T, H, d] or None    s0 : [B, H, d, d] or None
    heads   : optional list of (b, h) pairs to evaluate (others are left at zero).
    Returns out [B, T, U, H, d] float64.
    """
    q = np.asarray(q)
    Bn, T, U, H, d = q.shape
    out = np.zeros((Bn, T, U, H, d), F64)
    pairs = heads if heads is not None else [(b, h) for b in range(Bn) for h in range(H)]
    for (b, h) in pairs:
        res = vda_slice(q[b, :, :, h, :], k[b, :, :, h, :], v[b, :, :, h, :], beta[b, :, :, h],
                        gate[h], eps,
                        None if alpha is None else alpha[b, :, h, :],
                        None if s0 is None else s0[b, h])
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

"""Direct, unoptimised evaluation of the layer's equations on tiny shapes.

An independent second opinion for the fp64 checker in `oracle/`: different algebra
(the frame update is obtained by handing the joint objective, Eq. 4, to a
least-squares routine row by row -- no normal equations, no inverse), explicit
Python loops over frames and tokens, and the read indices written out from the
text of Sec. 2.2 (forward state = frames strictly before the query frame, reverse
state = frames strictly after it).  Imports nothing from `oracle/`.
"""
import numpy as np


def lstsq_frame_update(S_bar, K, V, beta):
    """argmin_S 1/2 ||S - S_bar||_F^2 + 1/2 sum_u beta_u ||S k_u - v_u||^2   (Eq. 4).

    Row r of S only meets row r of S_bar and component r of each v_u, so each row
    is its own least-squares problem  [I ; Diag(sqrt beta) K] s = [s_bar ; sqrt(beta) v_r].
    """
    dv, dk = S_bar.shape
    rb = np.sqrt(beta)
    lhs = np.vstack([np.eye(dk), rb[:, None] * K])
    S = np.zeros_like(S_bar)
    for r in range(dv):
        rhs = np.concatenate([S_bar[r], rb * V[:, r]])
        S[r] = np.linalg.lstsq(lhs, rhs, rcond=None)[0]
    return S


def state_after(frames, k, v, beta, alpha, S_init):
    """Fold the frames listed in `frames` (in that order) into a state starting from S_init."""
    S = S_init.copy()
    for t in frames:
        S = lstsq_frame_update(S * alpha[t][None, :], k[t], v[t], beta[t])
    return S


def vda_bruteforce(q, k, v, beta, gate, eps, alpha=None, s0=None):
    """q,k [T,U,dk], v [T,U,dv], beta [T,U] -> out [T,U,dv], o_fwd, o_bwd (pre-norm parts)."""
    T, U, dk = k.shape
    dv = v.shape[2]
    alpha = np.ones((T, dk)) if alpha is None else alpha
    S_init = np.zeros((dv, dk)) if s0 is None else 0.5 * s0
    out = np.zeros((T, U, dv))
    o_fwd = np.zeros((T, U, dv))
    o_bwd = np.zeros((T, U, dv))
    for t in range(T):
        # states are recomputed from scratch for every query frame on purpose
        S_before = state_after(list(range(0, t)), k, v, beta, alpha, S_init)
        S_after = state_after(list(range(T - 1, t, -1)), k, v, beta, alpha, S_init)
        for u in range(U):
            for c in range(dv):
                acc_f = 0.0
                acc_b = 0.0
                for j in range(dk):
                    acc_f += S_before[c, j] * alpha[t][j] * q[t, u, j]
                    acc_b += S_after[c, j] * alpha[t][j] * q[t, u, j]
                o_fwd[t, u, c] = acc_f
                o_bwd[t, u, c] = acc_b
            o = o_fwd[t, u] + o_bwd[t, u]
            ms = sum(x * x for x in o) / dv
            out[t, u] = gate * o / np.sqrt(ms + eps)
    return out, o_fwd, o_bwd


def softmax_sees(t, j, T, chunk, radius, anchors):
    """Sec. 2.1: is frame j visible to the Softmax branch of query frame t?  Frames are grouped into temporal
    chunks of `chunk` frames from the start of the clip; a query chunk attends to itself and `radius` chunks on
    either side; with boundary anchors every frame also attends to the first and the last frame and those two
    attend to everything."""
    if abs(t // chunk - j // chunk) <= radius:
        return True
    if anchors and (j in (0, T - 1) or t in (0, T - 1)):
        return True
    return False


def vda_bruteforce_windowed(q, k, v, beta, gate, eps, alpha=None, s0=None, chunk=1, radius=0, anchors=False,
                            norm_weight=None):
    """The layer with chunk windows and boundary anchors, from the text of Sec. 2.1-2.2 and Sec. A.4.

    For every query frame the two linear regions are whatever Softmax does not see, before and after the frame;
    each is folded from the initial state in scan order, and the decay across the skipped local span is applied
    by running the same frame update over that span with every write gate set to zero.  `gate` may be a scalar
    or an array [T, U, dv]; `norm_weight` an optional [dv] vector.
    """
    T, U, dk = k.shape
    dv = v.shape[2]
    alpha = np.ones((T, dk)) if alpha is None else alpha
    S_init = np.zeros((dv, dk)) if s0 is None else 0.5 * s0
    gate = np.broadcast_to(np.asarray(gate, float), (T, U, dv))
    w = np.ones(dv) if norm_weight is None else norm_weight
    anchor_frames = (0, T - 1) if anchors else ()
    interior = [j for j in range(T) if j not in anchor_frames]
    out = np.zeros((T, U, dv))
    o_fwd = np.zeros((T, U, dv))
    o_bwd = np.zeros((T, U, dv))
    no_write = np.zeros(U)
    for t in interior:
        far_before = [j for j in interior if j < t and not softmax_sees(t, j, T, chunk, radius, anchors)]
        far_after = [j for j in interior if j > t and not softmax_sees(t, j, T, chunk, radius, anchors)]
        near_before = [j for j in interior if j <= t and j not in far_before]       # skipped span, ends at t
        near_after = [j for j in interior if j >= t and j not in far_after]         # skipped span, starts at t
        S_f = state_after(far_before, k, v, beta, alpha, S_init)
        for j in near_before:
            S_f = lstsq_frame_update(S_f * alpha[j][None, :], k[j], v[j], no_write)
        S_b = state_after(far_after[::-1], k, v, beta, alpha, S_init)
        for j in near_after[::-1]:
            S_b = lstsq_frame_update(S_b * alpha[j][None, :], k[j], v[j], no_write)
        for u in range(U):
            for c in range(dv):
                o_fwd[t, u, c] = sum(S_f[c, j] * q[t, u, j] for j in range(dk))
                o_bwd[t, u, c] = sum(S_b[c, j] * q[t, u, j] for j in range(dk))
            o = o_fwd[t, u] + o_bwd[t, u]
            ms = sum(x * x for x in o) / dv
            for c in range(dv):
                out[t, u, c] = gate[t, u, c] * w[c] * o[c] / np.sqrt(ms + eps)
    return out, o_fwd, o_bwd

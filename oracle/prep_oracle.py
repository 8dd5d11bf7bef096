"""fp64 CPU oracle for the feature preparation in front of Video Delta Attention (Sec. 2.3; "VDA-Prep", Sec. 5).

TEST INFRASTRUCTURE ONLY, like vda_oracle.py: only the tests, the smoke check and the benchmark's CPU baseline
may import it; the CUDA library never does and shares no code with it.  numpy float64 throughout.

What the linear branch does to the projected q, k, v before the recurrence (Sec. 2.3):
    K, V : a separable short convolution -- a depthwise 5 x 5 spatial filter and a five-tap temporal filter,
           one filter pair per channel -- followed by SiLU;
    Q, K : L2 normalisation over the d channels of each (token, head).
Readings where the text is silent:
  * "convolution" is the cross-correlation of deep-learning libraries, taps centred on the output position
    (the model is bidirectional, so the temporal filter is centred too), zero padding, no bias;
  * the SiLU belongs to the convolved tensors (K and V); Q is only normalised;
  * L2 normalisation is x / sqrt(sum_j x_j^2 + eps) with a small eps (1e-6 by default);
  * with boundary anchors the anchor frames are removed before the preparation (Alg. 1 step 2): the temporal
    filter sees zeros beyond the first and the last scanned frame, and anchor frames come out as zeros.

Pinning status (tests/test_prep_oracle_pins.py):
  depthwise_spatial / depthwise_temporal / short_conv
                 pinned: literal five-fold loops on tiny shapes, scipy.ndimage.correlate (a library routine with
                 its own padding logic) per channel, the 3-D outer-product form of the separable filter,
                 delta filters, shift filters, linearity
  silu           pinned: printed values (silu(0) = 0, silu(1) = 0.7310585786300049), the large-|x| limits
  l2_normalise   pinned: unit rows, scale invariance, a 3-4-5 triangle
  prepare        pinned: a hand-worked single-channel example in tests/golden/prep_examples.json
"""
from __future__ import annotations

import numpy as np

F64 = np.float64
TAPS = 5
HALF = TAPS // 2


def depthwise_spatial(x, w):
    """x [T, Y, X, C], w [C, 5, 5]:  out[t,y,x,c] = sum_{i,j} w[c,i,j] x[t, y+i-2, x+j-2, c]  (zero outside)."""
    x = np.asarray(x, F64)
    w = np.asarray(w, F64)
    T, Y, X, C = x.shape
    xp = np.zeros((T, Y + 2 * HALF, X + 2 * HALF, C))
    xp[:, HALF:HALF + Y, HALF:HALF + X, :] = x
    out = np.zeros_like(x)
    for i in range(TAPS):
        for j in range(TAPS):
            out += w[None, None, None, :, i, j] * xp[:, i:i + Y, j:j + X, :]
    return out


def depthwise_temporal(x, w):
    """x [T, ..., C], w [C, 5]:  out[t,...,c] = sum_i w[c,i] x[t+i-2, ..., c]  (zero outside)."""
    x = np.asarray(x, F64)
    w = np.asarray(w, F64)
    T = x.shape[0]
    xp = np.zeros((T + 2 * HALF,) + x.shape[1:])
    xp[HALF:HALF + T] = x
    out = np.zeros_like(x)
    for i in range(TAPS):
        out += w[:, i] * xp[i:i + T]
    return out


def short_conv(x, w_spatial, w_temporal):
    """Sec. 2.3: the separable short convolution, spatial filter then temporal filter (they act on different
    axes, so the order does not matter)."""
    return depthwise_temporal(depthwise_spatial(x, w_spatial), w_temporal)


def silu(x):
    """SiLU(x) = x * sigmoid(x)."""
    x = np.asarray(x, F64)
    return x / (1.0 + np.exp(-x))


def l2_normalise(x, eps=1e-6):
    """x / sqrt(sum_j x_j^2 + eps) over the last axis (the d channels of one token and head)."""
    x = np.asarray(x, F64)
    return x / np.sqrt(np.sum(x * x, axis=-1, keepdims=True) + eps)


def prepare(q, k, v, wk_s, wk_t, wv_s, wv_t, Y, X, eps=1e-6, anchors=False):
    """Feature preparation of ONE (batch, head) slice.

    q, k, v : [T, Y*X, d] projected features, tokens of a frame in row-major (y, x) order
    wk_s, wv_s : [d, 5, 5] spatial filters;  wk_t, wv_t : [d, 5] temporal filters (one per channel)
    Returns prepared (q, k, v) of the same shape:
        q' = l2_normalise(q),   k' = l2_normalise(silu(short_conv(k))),   v' = silu(short_conv(v)).
    With `anchors` the first and the last frame are removed first and come back as zeros.
    """
    q = np.asarray(q, F64)
    k = np.asarray(k, F64)
    v = np.asarray(v, F64)
    T, U, d = k.shape
    assert U == Y * X
    first, last = (1, T - 2) if anchors else (0, T - 1)
    qo = np.zeros_like(q)
    ko = np.zeros_like(k)
    vo = np.zeros_like(v)
    if last < first:
        return qo, ko, vo
    rows = slice(first, last + 1)
    n = last - first + 1
    kc = short_conv(k[rows].reshape(n, Y, X, d), wk_s, wk_t).reshape(n, U, d)
    vc = short_conv(v[rows].reshape(n, Y, X, d), wv_s, wv_t).reshape(n, U, d)
    qo[rows] = l2_normalise(q[rows], eps)
    ko[rows] = l2_normalise(silu(kc), eps)
    vo[rows] = silu(vc)
    return qo, ko, vo

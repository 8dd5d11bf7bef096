"""Pins for the feature-preparation checker (oracle/prep_oracle.py): literal loops, a library routine with its
own padding logic, identities of the filters, printed SiLU values and a hand-worked example."""
import json
import os

import numpy as np
import pytest
from scipy import ndimage

from oracle import prep_oracle as po

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "prep_examples.json")


def rng(seed):
    return np.random.default_rng(seed)


def literal_short_conv(x, ws, wt):
    """out[t,y,x,c] = sum_{dt,dy,dx} wt[c,dt+2] ws[c,dy+2,dx+2] x[t+dt,y+dy,x+dx,c], zero outside; plain loops."""
    T, Y, X, C = x.shape
    out = np.zeros_like(x)
    for t in range(T):
        for y in range(Y):
            for xx in range(X):
                for c in range(C):
                    acc = 0.0
                    for dt in range(-2, 3):
                        for dy in range(-2, 3):
                            for dx in range(-2, 3):
                                tt, yy, x2 = t + dt, y + dy, xx + dx
                                if 0 <= tt < T and 0 <= yy < Y and 0 <= x2 < X:
                                    acc += wt[c, dt + 2] * ws[c, dy + 2, dx + 2] * x[tt, yy, x2, c]
                    out[t, y, xx, c] = acc
    return out


@pytest.mark.parametrize("T,Y,X,C", [(1, 1, 1, 2), (3, 2, 4, 3), (6, 5, 3, 2), (2, 7, 7, 1)])
def test_short_conv_matches_literal_loops(T, Y, X, C):
    r = rng(T * 100 + Y * 10 + X)
    x = r.standard_normal((T, Y, X, C))
    ws = r.standard_normal((C, 5, 5))
    wt = r.standard_normal((C, 5))
    assert np.allclose(po.short_conv(x, ws, wt), literal_short_conv(x, ws, wt), atol=1e-12)


def test_filters_match_scipy_correlate_per_channel():
    r = rng(1)
    T, Y, X, C = 7, 6, 9, 3
    x = r.standard_normal((T, Y, X, C))
    ws = r.standard_normal((C, 5, 5))
    wt = r.standard_normal((C, 5))
    sp = po.depthwise_spatial(x, ws)
    tp = po.depthwise_temporal(x, wt)
    full = po.short_conv(x, ws, wt)
    for c in range(C):
        for t in range(T):
            assert np.allclose(sp[t, :, :, c], ndimage.correlate(x[t, :, :, c], ws[c], mode="constant", cval=0.0),
                               atol=1e-12)
        assert np.allclose(tp[..., c], ndimage.correlate1d(x[..., c], wt[c], axis=0, mode="constant", cval=0.0),
                           atol=1e-12)
        # the separable pair is one 3-D filter: the outer product of the temporal and the spatial taps
        w3 = wt[c][:, None, None] * ws[c][None, :, :]
        assert np.allclose(full[..., c], ndimage.correlate(x[..., c], w3, mode="constant", cval=0.0), atol=1e-12)


def test_delta_and_shift_filters():
    r = rng(2)
    x = r.standard_normal((5, 4, 6, 2))
    delta_s = np.zeros((2, 5, 5)); delta_s[:, 2, 2] = 1.0
    delta_t = np.zeros((2, 5)); delta_t[:, 2] = 1.0
    assert np.array_equal(po.short_conv(x, delta_s, delta_t), x)
    # a tap at (i, j) = (2, 3) reads the right-hand neighbour (x + 1); a temporal tap at index 0 reads frame t - 2
    sh = np.zeros((2, 5, 5)); sh[:, 2, 3] = 1.0
    out = po.depthwise_spatial(x, sh)
    assert np.array_equal(out[:, :, :-1], x[:, :, 1:]) and not out[:, :, -1].any()
    st = np.zeros((2, 5)); st[:, 0] = 1.0
    out = po.depthwise_temporal(x, st)
    assert np.array_equal(out[2:], x[:-2]) and not out[:2].any()
    # channels never mix
    x2 = x.copy(); x2[..., 1] = 0.0
    ws = r.standard_normal((2, 5, 5)); wt = r.standard_normal((2, 5))
    assert np.array_equal(po.short_conv(x2, ws, wt)[..., 0], po.short_conv(x, ws, wt)[..., 0])
    # linear in the input
    y = r.standard_normal(x.shape)
    assert np.allclose(po.short_conv(2.0 * x - y, ws, wt), 2.0 * po.short_conv(x, ws, wt) - po.short_conv(y, ws, wt),
                       atol=1e-12)


def test_silu_values_and_limits():
    assert po.silu(0.0) == 0.0
    assert abs(po.silu(1.0) - 0.7310585786300049) < 1e-15
    assert abs(po.silu(-1.0) + 0.2689414213699951) < 1e-15
    assert abs(po.silu(40.0) - 40.0) < 1e-12 and abs(po.silu(-40.0)) < 1e-12
    x = np.linspace(-6, 6, 41)
    assert np.allclose(po.silu(x) - po.silu(-x), x, atol=1e-14)          # x s(x) + x s(-x) = x


def test_l2_normalise():
    assert np.allclose(po.l2_normalise(np.array([3.0, 4.0]), 0.0), [0.6, 0.8])
    r = rng(3)
    x = r.standard_normal((4, 5, 16))
    y = po.l2_normalise(x, 1e-12)
    assert np.allclose(np.sum(y * y, axis=-1), 1.0, atol=1e-9)
    assert np.allclose(po.l2_normalise(7.0 * x, 1e-12), y, atol=1e-9)
    assert np.array_equal(po.l2_normalise(np.zeros((2, 8)), 1e-6), np.zeros((2, 8)))


def test_golden_prepare_example():
    with open(GOLDEN) as f:
        g = json.load(f)["single_channel_3x1x3"]
    arr = lambda n: np.array(g[n], float)
    wk_s = np.zeros((1, 5, 5)); wk_s[0, 2] = g["wk_s_middle_row"]
    wv_s = np.zeros((1, 5, 5)); wv_s[0, 2, 2] = 1.0
    wk_t = np.array([g["wk_t"]], float)
    wv_t = np.array([g["wv_t"]], float)
    Y, X = g["Y"], g["X"]
    kc = po.short_conv(arr("k").reshape(3, Y, X, 1), wk_s, wk_t).reshape(3, Y * X, 1)
    vc = po.short_conv(arr("v").reshape(3, Y, X, 1), wv_s, wv_t).reshape(3, Y * X, 1)
    assert np.array_equal(kc, arr("k_conv")) and np.array_equal(vc, arr("v_conv"))
    q, k, v = po.prepare(arr("q"), arr("k"), arr("v"), wk_s, wk_t, wv_s, wv_t, Y, X, eps=1e-30)
    assert np.allclose(v, arr("v_out"), atol=1e-15)
    assert np.allclose(k, arr("k_out"), atol=1e-12)
    assert np.allclose(q, arr("q_out"), atol=1e-12)


def test_prepare_with_anchors_removes_the_boundary_frames_first():
    r = rng(4)
    T, Y, X, d = 6, 3, 4, 5
    q, k, v = (r.standard_normal((T, Y * X, d)) for _ in range(3))
    ws = r.standard_normal((d, 5, 5)); wt = r.standard_normal((d, 5))
    qa, ka, va = po.prepare(q, k, v, ws, wt, ws, wt, Y, X, anchors=True)
    qi, ki, vi = po.prepare(q[1:-1], k[1:-1], v[1:-1], ws, wt, ws, wt, Y, X)
    assert np.array_equal(ka[1:-1], ki) and np.array_equal(va[1:-1], vi) and np.array_equal(qa[1:-1], qi)
    for z in (qa, ka, va):
        assert not z[0].any() and not z[-1].any()
    # changing an anchor frame changes nothing
    k2 = k.copy(); k2[0] += 5.0; k2[-1] -= 3.0
    assert np.array_equal(po.prepare(q, k2, v, ws, wt, ws, wt, Y, X, anchors=True)[1], ka)

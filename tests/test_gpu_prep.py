"""Parity of vdn_vda_prepare (Sec. 2.3 feature preparation) against the fp64 checker, element by element.

Same metric and tolerances as the layer itself: oracle.slice_error (max |gpu - ref| over a (batch, head) slice
divided by the slice's max |ref|) <= 1e-4 for f32 I/O and <= 2e-2 for bf16 I/O, for each of q', k', v'.
"""
import numpy as np
import pytest
import torch

from oracle import prep_oracle as po
from oracle import vda_oracle as orc
from paper_2609_20744_b200 import binding, build, inputs

pytestmark = pytest.mark.gpu

TOL = {"f32": 1e-4, "bf16": 2e-2}


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    binding.load_library()


def f64(t):
    return t.detach().double().cpu().numpy()


def check(w, p, got, Y, X, anchors=False):
    C = w.d
    for b in range(w.B):
        for h in range(w.H):
            sl = slice(h * C, (h + 1) * C)
            ref = po.prepare(f64(p["q"][b, :, :, h]), f64(p["k"][b, :, :, h]), f64(p["v"][b, :, :, h]),
                             f64(p["wk_spatial"][sl]), f64(p["wk_temporal"][sl]), f64(p["wv_spatial"][sl]),
                             f64(p["wv_temporal"][sl]), Y, X, 1e-6, anchors)
            for name, g, r in zip("qkv", got, ref):
                gg = f64(g[b, :, :, h])
                assert np.isfinite(gg).all()
                e = orc.slice_error(gg, r)
                assert e <= TOL[w.dtype], f"{name}' slice (b={b}, h={h}) error {e:.3e} > {TOL[w.dtype]}"


@pytest.mark.parametrize("dtype,d", [("f32", 64), ("f32", 128), ("bf16", 128), ("bf16", 64)])
@pytest.mark.parametrize("T,Y,X,anchors", [
    (6, 9, 11, False),     # several tiles with ragged edges in both directions
    (1, 3, 5, False),      # one frame, one partial tile: every tap but the centre frame's hits padding
    (2, 4, 8, False),      # exactly one tile at d = 128
    (3, 1, 1, False),      # a single token per frame
    (7, 5, 17, True),      # anchors: frames 1..5 prepared, 0 and 6 zero
    (4, 2, 30, False),
])
def test_prepare_matches_oracle(dtype, d, T, Y, X, anchors):
    w = inputs.TINY.scaled(dtype=dtype, d=d, B=2, H=3, T=T, F=Y * X, seed=T * 100 + Y * 10 + X)
    p = inputs.generate_projected(w, "cuda")
    vda = binding.Vda(w.d, w.dtype)
    got = vda.prepare(p["q"], p["k"], p["v"], p, Y, X, anchors=anchors)
    torch.cuda.synchronize()
    assert vda.status() == binding.VDN_OK and vda.launch_count() == 3      # spatial filter, temporal half, queries
    check(w, p, got, Y, X, anchors)
    if anchors:
        for g in got:
            assert torch.count_nonzero(g[:, 0]) == 0 and torch.count_nonzero(g[:, -1]) == 0


@pytest.mark.parametrize("dtype,d", [("f32", 64), ("f32", 128), ("bf16", 128), ("bf16", 64)])
@pytest.mark.parametrize("T,Y,X,anchors", [(6, 9, 11, False), (1, 3, 5, False), (2, 1, 1, False), (9, 5, 7, True)])
def test_prepare_without_spatial_filter_matches_oracle(dtype, d, T, Y, X, anchors):
    # spatial filters left out: temporal filter + SiLU + normalisation; the checker gets centre-tap spatial filters
    w = inputs.TINY.scaled(dtype=dtype, d=d, B=2, H=3, T=T, F=Y * X, seed=T * 100 + Y * 10 + X + 1)
    p = inputs.generate_projected(w, "cuda")
    vda = binding.Vda(w.d, w.dtype)
    flt = dict(wk_temporal=p["wk_temporal"], wv_temporal=p["wv_temporal"])
    got = vda.prepare(p["q"], p["k"], p["v"], flt, Y, X, anchors=anchors)
    torch.cuda.synchronize()
    assert vda.status() == binding.VDN_OK
    for n in ("wk", "wv"):
        p[n + "_spatial"].zero_(); p[n + "_spatial"][:, 2, 2] = 1.0
    check(w, p, got, Y, X, anchors)


def test_prepare_identity_filters_and_in_place_q():
    # centre-tap filters: k' = L2norm(SiLU(k)), v' = SiLU(v); q normalised in place
    w = inputs.TINY.scaled(dtype="f32", d=64, B=1, H=2, T=3, F=6 * 7)
    p = inputs.generate_projected(w, "cuda")
    for n in ("wk", "wv"):
        p[n + "_spatial"].zero_(); p[n + "_spatial"][:, 2, 2] = 1.0
        p[n + "_temporal"].zero_(); p[n + "_temporal"][:, 2] = 1.0
    vda = binding.Vda(w.d, w.dtype)
    q0 = p["q"].clone()
    ko, vo = torch.empty_like(p["k"]), torch.empty_like(p["v"])
    vda.prepare(p["q"], p["k"], p["v"], p, 6, 7, out=(p["q"], ko, vo))
    torch.cuda.synchronize()
    sk = torch.nn.functional.silu(p["k"].double())
    assert torch.allclose(vo.double(), torch.nn.functional.silu(p["v"].double()), atol=2e-6)
    assert torch.allclose(ko.double(), sk / torch.sqrt((sk * sk).sum(-1, keepdim=True) + 1e-6), atol=2e-6)
    assert torch.allclose(p["q"].double(), q0.double() / torch.sqrt((q0.double() ** 2).sum(-1, keepdim=True) + 1e-6),
                          atol=2e-6)
    assert torch.allclose(ko.pow(2).sum(-1), torch.ones_like(ko[..., 0]), atol=1e-4)


def test_prepared_features_feed_the_layer():
    # projected q, k, v -> vdn_vda_prepare -> vdn_vda_forward_opt, against the two checkers chained the same way
    w = inputs.TINY.scaled(dtype="bf16", d=128, B=1, H=2, T=7, F=10 * 13, seed=21)
    Y, X = 10, 13
    p = inputs.generate_projected(w, "cuda")
    x = inputs.generate(w, "cuda")                     # beta and gate from the layer's own recipe
    vda = binding.Vda(w.d, w.dtype)
    q, k, v = vda.prepare(p["q"], p["k"], p["v"], p, Y, X, anchors=True)
    out = vda.forward(q, k, v, x["beta"], x["gate"], chunk=2, radius=0, anchors=True)
    torch.cuda.synchronize()
    assert vda.status() == binding.VDN_OK
    for h in range(w.H):
        # the layer's checker consumes the GPU's prepared (rounded) features: each stage is checked on its own inputs
        ref = orc.vda_slice(f64(q[0, :, :, h]), f64(k[0, :, :, h]), f64(v[0, :, :, h]), f64(x["beta"][0, :, :, h]),
                            float(x["gate"][h]), 1e-6, chunk=2, radius=0, anchors=True)["out"]
        assert orc.slice_error(f64(out[0, :, :, h]), ref) <= TOL["bf16"]
    check(w, p, (q, k, v), Y, X, anchors=True)


@pytest.mark.parametrize("dtype,d,F,extras", [
    ("bf16", 128, 300, False),     # tensor-core read-out, three tiles with a ragged tail
    ("bf16", 128, 130, True),      # ... with the element-wise gate and the norm weight on top
    ("bf16", 64, 70, False),       # plain-fp32 kernels
    ("f32", 128, 45, True),
])
def test_readout_normalises_the_queries(dtype, d, F, extras):
    # q arrives as projected (norms far from one); with q_l2_eps the read-out applies q / sqrt(|q|^2 + eps) itself.
    # Checker: the preparation's L2 normalisation in fp64, unrounded, in front of the layer.  A large RMSNorm eps
    # makes the scale of q matter (with a tiny eps the norm would hide a wrong or missing factor).
    w = inputs.TINY.scaled(dtype=dtype, d=d, B=2, H=2, T=5, F=F, seed=77)
    x = inputs.generate(w, "cuda")
    p = inputs.generate_projected(w, "cuda")
    scale = torch.linspace(0.05, 20.0, w.T * w.F, device="cuda").view(1, w.T, w.F, 1, 1)
    q_raw = (p["q"].float() * scale).to(p["q"].dtype)
    rms_eps = 1e-2
    vda = binding.Vda(w.d, w.dtype, rms_eps=rms_eps)
    kw = {}
    if extras:
        ge, nw = inputs.generate_output_extras(w, "cuda")
        kw = dict(gate_elem=ge, norm_weight=nw)
    out = vda.forward(q_raw, x["k"], x["v"], x["beta"], x["gate"], chunk=2, radius=1, q_l2_eps=1e-6, **kw)
    torch.cuda.synchronize()
    assert vda.status() == binding.VDN_OK
    for b in range(w.B):
        for h in range(w.H):
            qn = po.l2_normalise(f64(q_raw[b, :, :, h]), 1e-6)
            gate = float(x["gate"][h]) * (f64(kw["gate_elem"][b, :, :, h]) if extras else 1.0)
            ref = orc.vda_slice(qn, f64(x["k"][b, :, :, h]), f64(x["v"][b, :, :, h]), f64(x["beta"][b, :, :, h]),
                                gate, rms_eps, chunk=2, radius=1,
                                norm_weight=f64(kw["norm_weight"][h]) if extras else None)["out"]
            assert orc.slice_error(f64(out[b, :, :, h]), ref) <= TOL[dtype]
    # and it is not a no-op: without the option the same inputs give a different answer
    out2 = vda.forward(q_raw, x["k"], x["v"], x["beta"], x["gate"], chunk=2, radius=1, **kw)
    torch.cuda.synchronize()
    assert (out2.float() - out.float()).abs().max() > 1e-2 * out.float().abs().max()


def test_prepare_without_queries():
    w = inputs.TINY.scaled(dtype="bf16", d=128, B=1, H=2, T=4, F=6 * 7, seed=5)
    p = inputs.generate_projected(w, "cuda")
    vda = binding.Vda(w.d, w.dtype)
    q1, k1, v1 = vda.prepare(p["q"], p["k"], p["v"], p, 6, 7)
    q2, k2, v2 = vda.prepare(None, p["k"], p["v"], p, 6, 7)
    torch.cuda.synchronize()
    assert q2 is None and torch.equal(k1, k2) and torch.equal(v1, v2)


def test_prepare_argument_errors():
    import ctypes
    w = inputs.TINY.scaled(F=4 * 5)
    p = inputs.generate_projected(w, "cuda")
    vda = binding.Vda(w.d, w.dtype)
    with pytest.raises(binding.VdnError):
        vda.prepare(p["q"], p["k"], p["v"], p, 4, 6)                       # Y * X != F
    with pytest.raises(binding.VdnError):
        vda.prepare(p["q"], p["k"], p["v"], p, 4, 5, out=(p["q"], p["k"], torch.empty_like(p["v"])))   # k in place
    torch.cuda.synchronize()


@pytest.mark.parametrize("dtype,d", [("bf16", 128), ("f32", 64)])
def test_random_preparation_shapes(dtype, d):
    # seeded sweep over clip length, token grid (whole tiles, ragged tiles, single rows and columns), anchors and the
    # two variants (with and without the spatial filter)
    import random
    rnd = random.Random(744)
    for trial in range(12):
        T = rnd.randint(1, 9)
        Y, X = rnd.choice([(1, 1), (1, 9), (9, 1), (4, 8), (5, 9), (8, 16), (3, 17), (13, 5)])
        anchors = rnd.random() < 0.4
        spatial = rnd.random() < 0.6
        w = inputs.TINY.scaled(dtype=dtype, d=d, B=rnd.choice([1, 2]), H=rnd.choice([1, 2, 3]), T=T, F=Y * X,
                               seed=3000 + trial)
        p = inputs.generate_projected(w, "cuda")
        vda = binding.Vda(w.d, w.dtype)
        flt = p if spatial else dict(wk_temporal=p["wk_temporal"], wv_temporal=p["wv_temporal"])
        got = vda.prepare(p["q"], p["k"], p["v"], flt, Y, X, anchors=anchors)
        torch.cuda.synchronize()
        assert vda.status() == binding.VDN_OK
        if not spatial:
            for n in ("wk", "wv"):
                p[n + "_spatial"].zero_(); p[n + "_spatial"][:, 2, 2] = 1.0
        try:
            check(w, p, got, Y, X, anchors)
        except AssertionError as e:
            raise AssertionError(f"trial {trial}: T={T} grid={Y}x{X} anchors={anchors} spatial={spatial}: {e}")
        vda.close()

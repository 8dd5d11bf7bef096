"""Parity at the benchmark's full sizes, in the launch configuration bench.py times.

Heads never interact, so checking whole (batch, head) slices against the fp64 checker is exact for those
slices; which slices are checked is fixed (first, last, one seeded).  Every slice is additionally covered by
a property that holds at any size: each output row has mean square gate_h^2 (Eq. 1c), and rows of a
single-frame-free clip are finite.
"""
import gc

import numpy as np
import pytest
import torch

from oracle import vda_oracle as orc
from paper_2609_20744_b200 import binding, build, inputs

pytestmark = pytest.mark.gpu
TOL_BF16 = 2e-2


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    binding.load_library()


def sampled_pairs(w, count):
    pairs = [(0, 0), (w.B - 1, w.H - 1)]
    rng = np.random.default_rng(w.seed + 1234)
    while len(pairs) < count:
        p = (int(rng.integers(w.B)), int(rng.integers(w.H)))
        if p not in pairs:
            pairs.append(p)
    return pairs[:count]


def run_and_check(w, nheads, flags=0):
    x = inputs.generate(w, "cuda")
    vda = binding.Vda(w.d, w.dtype, flags=flags)
    assert vda.uses_tensor_cores()
    out = vda.forward(x["q"], x["k"], x["v"], x["beta"], x["gate"])
    torch.cuda.synchronize()
    assert vda.status() == binding.VDN_OK
    worst = 0.0
    for (b, h) in sampled_pairs(w, nheads):
        q, k, v, beta, gate = inputs.head_slice(x, b, h)
        ref = orc.vda_slice(q, k, v, beta, gate, 1e-6)["out"]
        got = out[b, :, :, h, :].double().cpu().numpy()
        e = orc.slice_error(got, ref)
        worst = max(worst, e)
        assert e <= TOL_BF16, f"{w.name} slice (b={b}, h={h}): error {e:.3e}"
        del q, k, v, ref, got
    # all slices: finite, and every row's mean square equals gate^2 (bf16 output rounding: 2^-8 relative)
    for b in range(w.B):
        for t0 in range(0, w.T, 16):
            blk = out[b, t0:t0 + 16].float()
            assert torch.isfinite(blk).all()
            ms = blk.pow(2).mean(dim=-1)
            want = x["gate"].pow(2)[None, None, :].expand_as(ms)
            assert torch.allclose(ms, want, rtol=2e-2), f"{w.name}: row mean-square off in frames {t0}.."
    del x, out, vda
    gc.collect()
    torch.cuda.empty_cache()
    return worst


def test_768p_config_full_size():
    run_and_check(inputs.CLIP_768P, 4)       # first, last and two seeded (batch, head) slices


@pytest.mark.parametrize("flags", [binding.VDN_FLAG_EXACT_STATS,
                                   binding.VDN_FLAG_EXACT_STATS | binding.VDN_FLAG_FP32_RESOLVE])
def test_768p_config_full_size_accuracy_options(flags):
    # the statistics from exact weighted keys, and with the plain-fp32 inverse behind them: other kernels in the same
    # launch configuration; the error is the default path's less the share of the bf16-rounded weighted keys
    worst = run_and_check(inputs.CLIP_768P, 2, flags=flags)
    assert worst <= 6e-3, f"flags={flags}: {worst:.3e}"


@pytest.mark.parametrize("idx", [0, 1, 2, 3])
def test_scan_depth_sweep_full_size(idx):
    run_and_check(inputs.SWEEP[idx], 4)      # first, last and two seeded slices


def test_cfg_long_clip_full_size():
    free, _ = torch.cuda.mem_get_info()
    w = inputs.CFG_LONG
    need = 4 * w.tokens * w.H * w.d * 2 + (5 << 30)
    if free < need:
        pytest.skip(f"needs {need >> 30} GiB of free device memory")
    run_and_check(w, 4)


def test_768p_release_window_full_size():
    # the release setting of the paper (chunk 5, radius 1, boundary anchors, decay bridge, text state) at the
    # benchmark's size; both scan schedules
    w = inputs.CLIP_768P
    x = inputs.generate(w, "cuda")
    alpha, s0 = inputs.generate_recurrence_extras(w, "cuda")
    kw = dict(chunk=5, radius=1, anchors=True)
    pairs = sampled_pairs(w, 2)
    refs = {}
    for (b, h) in pairs:
        q, k, v, beta, gate = inputs.head_slice(x, b, h)
        refs[(b, h)] = orc.vda_slice(q, k, v, beta, gate, 1e-6, alpha=alpha[b, :, h].double().cpu().numpy(),
                                     s0=s0[b, h].double().cpu().numpy(), **kw)["out"]
        del q, k, v
    for flags in (binding.VDN_FLAG_SCAN_FRAMEWISE, binding.VDN_FLAG_SCAN_CHUNKWISE):
        vda = binding.Vda(w.d, w.dtype, flags=flags)
        out = vda.forward(x["q"], x["k"], x["v"], x["beta"], x["gate"], alpha=alpha, s0=s0, **kw)
        torch.cuda.synchronize()
        assert vda.status() == binding.VDN_OK
        for (b, h) in pairs:
            e = orc.slice_error(out[b, :, :, h, :].double().cpu().numpy(), refs[(b, h)])
            assert e <= TOL_BF16, f"flags={flags} slice (b={b}, h={h}): error {e:.3e}"
        assert torch.count_nonzero(out[:, 0]) == 0 and torch.count_nonzero(out[:, -1]) == 0
        assert torch.isfinite(out.float()).all()
        del out, vda
    del x
    gc.collect()
    torch.cuda.empty_cache()


def test_768p_queries_normalised_by_the_readout_full_size():
    # projected queries (token norms spread over two decades) with vdn_vda_options.q_l2_eps: the read-out applies
    # the preparation's L2 normalisation itself; checker = that normalisation in fp64 in front of the layer
    from oracle import prep_oracle as po
    w = inputs.CLIP_768P
    x = inputs.generate(w, "cuda")
    g = torch.Generator(device="cuda")
    g.manual_seed(991)
    scale = torch.exp(torch.empty((w.B, w.T, w.F, w.H, 1), device="cuda").uniform_(-2.3, 2.3, generator=g))
    q_raw = (x["q"].float() * scale).to(x["q"].dtype)
    del scale
    vda = binding.Vda(w.d, w.dtype)
    out = vda.forward(q_raw, x["k"], x["v"], x["beta"], x["gate"], q_l2_eps=1e-6)
    torch.cuda.synchronize()
    assert vda.status() == binding.VDN_OK
    assert vda.uses_tensor_cores()
    again = vda.forward(q_raw, x["k"], x["v"], x["beta"], x["gate"], q_l2_eps=1e-6)
    torch.cuda.synchronize()
    assert torch.equal(out, again)          # the norms travel between warps through shared memory: no race
    del again
    for (b, h) in sampled_pairs(w, 2):
        q, k, v, beta, gate = inputs.head_slice(x, b, h)
        qn = po.l2_normalise(q_raw[b, :, :, h, :].double().cpu().numpy(), 1e-6)
        ref = orc.vda_slice(qn, k, v, beta, gate, 1e-6)["out"]
        e = orc.slice_error(out[b, :, :, h, :].double().cpu().numpy(), ref)
        assert e <= TOL_BF16, f"slice (b={b}, h={h}): error {e:.3e}"
        del q, k, v, qn, ref
    for t0 in range(0, w.T, 16):
        blk = out[:, t0:t0 + 16].float()
        assert torch.isfinite(blk).all()
        ms = blk.pow(2).mean(dim=-1)
        assert torch.allclose(ms, x["gate"].pow(2)[None, None, None, :].expand_as(ms), rtol=2e-2)
    del x, out, q_raw, vda
    gc.collect()
    torch.cuda.empty_cache()


@pytest.mark.parametrize("spatial", [True, False])
def test_768p_preparation_full_size(spatial):
    # vdn_vda_prepare on the 768p shape (48 x 85 tokens per frame): sampled output frames of sampled heads against
    # the checker (which gets the five input frames the temporal filter reaches), plus properties on everything
    from oracle import prep_oracle as po
    w = inputs.CLIP_768P
    Y, X = 48, 85
    p = inputs.generate_projected(w, "cuda")
    vda = binding.Vda(w.d, w.dtype)
    flt = p if spatial else dict(wk_temporal=p["wk_temporal"], wv_temporal=p["wv_temporal"])
    q, k, v = vda.prepare(p["q"], p["k"], p["v"], flt, Y, X)
    torch.cuda.synchronize()
    assert vda.status() == binding.VDN_OK
    if not spatial:
        for n in ("wk", "wv"):
            p[n + "_spatial"].zero_(); p[n + "_spatial"][:, 2, 2] = 1.0
    f = lambda t: t.detach().double().cpu().numpy()
    for (b, h, tc) in [(0, 0, 0), (0, w.H - 1, w.T - 1), (0, 17, 40), (0, 5, 1)]:
        lo, hi = max(0, tc - 2), min(w.T, tc + 3)
        sl = slice(h * w.d, (h + 1) * w.d)
        # frames outside the clip are zero padding for the checker too: hand it exactly the frames that exist
        ref = po.prepare(f(p["q"][b, lo:hi, :, h]), f(p["k"][b, lo:hi, :, h]), f(p["v"][b, lo:hi, :, h]),
                         f(p["wk_spatial"][sl]), f(p["wk_temporal"][sl]), f(p["wv_spatial"][sl]),
                         f(p["wv_temporal"][sl]), Y, X)
        # the cropped clip pads with zeros where the real clip has frames: only exact when the crop reaches as far
        # as the filter does, i.e. at the clip's own ends or with two frames on either side
        assert lo == max(0, tc - 2) and hi == min(w.T, tc + 3)
        for name, g, r in zip("qkv", (q, k, v), ref):
            e = orc.slice_error(f(g[b, tc, :, h]), r[tc - lo])
            assert e <= TOL_BF16, f"{name}' (b={b}, h={h}, t={tc}): error {e:.3e}"
    for t0 in range(0, w.T, 16):
        assert torch.isfinite(v[:, t0:t0 + 16].float()).all()
        for g in (q, k):
            n2 = g[:, t0:t0 + 16].float().pow(2).sum(-1)
            assert torch.allclose(n2, torch.ones_like(n2), atol=2e-2)       # unit rows (bf16 rounding)
    del p, q, k, v
    gc.collect()
    torch.cuda.empty_cache()

"""Parity on seeded random configurations: shapes that straddle the 128-token tile and the SM count, with a random
choice of kernel path, window, anchors, decay gates, text state, element-wise gate, norm weight, rule, value scale
and gate sign.

The hand-picked cases of test_gpu_parity.py and test_gpu_window.py name the edges one at a time; this file draws
combinations of them.  The draws are fixed by the case number, so a failure names a reproducible configuration.
Every (batch, head) slice of every case is compared with the fp64 checker, element by element, at the usual bounds
(1e-4 for f32 I/O, 2e-2 for bf16 I/O).
"""
import numpy as np
import pytest
import torch

from oracle import vda_oracle as orc
from paper_2609_20744_b200 import binding, build, inputs

pytestmark = pytest.mark.gpu

TOL = {"f32": 1e-4, "bf16": 2e-2}
TOKENS = [1, 2, 31, 64, 127, 128, 129, 200, 255, 256, 257, 383, 385, 511, 513, 640]
PATHS = [
    ("bf16", 128, 0),
    ("bf16", 128, binding.VDN_FLAG_EXACT_STATS),
    ("bf16", 128, binding.VDN_FLAG_EXACT_STATS | binding.VDN_FLAG_FP32_RESOLVE),
    ("bf16", 128, binding.VDN_FLAG_FORCE_SIMT),
    ("f32", 128, 0),
    ("f32", 64, 0),
]


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    binding.load_library()


def draw(case):
    rng = np.random.default_rng(7000 + case)
    dtype, d, flags = PATHS[case % len(PATHS)]
    cfg = dict(dtype=dtype, d=d, flags=flags)
    cfg["B"] = int(rng.integers(1, 4))
    cfg["H"] = int(rng.integers(1, 6))
    cfg["T"] = int(rng.integers(1, 12))
    cfg["F"] = int(rng.choice(TOKENS))
    tensor_cores = dtype == "bf16" and not (flags & binding.VDN_FLAG_FORCE_SIMT)
    if tensor_cores and cfg["F"] < 31:
        # The tensor-core read-out takes the states a frame reads as bf16.  With one or two tokens per frame such a
        # state has rank one or two, a query can be orthogonal to all of it, and the RMSNorm then rescales rounding
        # (seen: |cos(q, k)| = 2e-4 -> 0.1).  The 2e-2 bound is stated for states of some rank.
        cfg["F"] = 31
    if case % 7 == 3:                                  # more scan chains than SMs, short frames
        cfg["B"], cfg["H"], cfg["F"] = 2, int(rng.integers(75, 90)), int(rng.choice([1, 31, 129]) if not tensor_cores else 129)
        cfg["T"] = int(rng.integers(2, 6))
    cfg["additive"] = bool(rng.random() < 0.15)
    cfg["use_alpha"] = bool(rng.random() < 0.5)
    cfg["use_s0"] = bool(rng.random() < 0.5)
    cfg["use_gate_elem"] = bool(rng.random() < 0.3)
    cfg["use_norm_weight"] = bool(rng.random() < 0.3)
    cfg["chunk"] = int(rng.choice([1, 1, 2, 3, 5]))
    cfg["radius"] = int(rng.choice([0, 0, 1, 2]))
    cfg["anchors"] = bool(rng.random() < 0.4) and cfg["T"] >= 3
    if rng.random() < 0.4:                             # the unwindowed layer
        cfg["chunk"], cfg["radius"], cfg["anchors"] = 1, 0, False
    if cfg["additive"]:
        cfg["flags"] = (cfg["flags"] & binding.VDN_FLAG_FORCE_SIMT) | binding.VDN_FLAG_ADDITIVE_RULE
    cfg["sched"] = int(rng.choice([0, binding.VDN_FLAG_SCAN_CHUNKWISE, binding.VDN_FLAG_SCAN_FRAMEWISE]))
    cfg["via_host"] = bool(rng.random() < 0.25)        # through the host-buffer entry point (pinned memory)
    cfg["v_scale_log2"] = int(rng.choice([0, 0, -10, 10]))   # values far from unit scale (exact in bf16): the RMSNorm's
    cfg["negative_gates"] = bool(rng.random() < 0.25)        # epsilon against small read-outs; gates of either sign
    return cfg


@pytest.mark.parametrize("case", range(120))
def test_random_configuration_matches_oracle(case):
    c = draw(case)
    w = inputs.TINY.scaled(dtype=c["dtype"], d=c["d"], B=c["B"], H=c["H"], T=c["T"], F=c["F"], seed=9000 + case)
    x = inputs.generate(w, "cuda")
    alpha, s0 = inputs.generate_recurrence_extras(w, "cuda")
    x["v"] = x["v"] * (2.0 ** c["v_scale_log2"])
    s0 = s0 * (2.0 ** c["v_scale_log2"])
    if c["negative_gates"]:
        x["gate"] = x["gate"] * (1.0 - 2.0 * (torch.arange(w.H, device="cuda") % 2)).to(x["gate"].dtype)
    gen = torch.Generator(device="cpu").manual_seed(9100 + case)
    io = torch.bfloat16 if c["dtype"] == "bf16" else torch.float32
    ge = nw = None
    if c["use_gate_elem"]:
        ge = torch.sigmoid(torch.randn(w.B, w.T, w.F, w.H, w.d, generator=gen)).to(io).cuda()
    if c["use_norm_weight"]:
        nw = (1.0 + 0.25 * torch.randn(w.H, w.d, generator=gen)).float().cuda()
    kw = dict(chunk=c["chunk"], radius=c["radius"], anchors=c["anchors"])
    flags = c["flags"]
    windowed = c["chunk"] >= 2
    if windowed and not (flags & binding.VDN_FLAG_FORCE_SIMT) and c["d"] == 128 and c["dtype"] == "bf16":
        flags |= c["sched"]
    vda = binding.Vda(w.d, w.dtype, flags=flags)
    opt = dict(alpha=alpha if c["use_alpha"] else None, s0=s0 if c["use_s0"] else None, gate_elem=ge, norm_weight=nw)
    if c["via_host"]:
        pin = lambda t: None if t is None else t.cpu().pin_memory()
        out_h = torch.empty(x["q"].shape, dtype=io).pin_memory()
        vda.forward_host(pin(x["q"]), pin(x["k"]), pin(x["v"]), pin(x["beta"]), pin(x["gate"]), out_h,
                         **{n: pin(t) for n, t in opt.items()}, **kw)
        torch.cuda.synchronize()
        out = out_h
    else:
        out = vda.forward(x["q"], x["k"], x["v"], x["beta"], x["gate"], **opt, **kw)
        torch.cuda.synchronize()
    assert vda.status() == binding.VDN_OK, c
    rule = "additive" if c["additive"] else "vda"
    for b in range(w.B):
        for h in (range(w.H) if w.H <= 6 else (0, 36, 37, 73, 74, w.H - 1)):
            q, k, v, beta, gate = inputs.head_slice(x, b, h)
            if ge is not None:
                gate = ge[b, :, :, h, :].double().cpu().numpy() * gate
            a = alpha[b, :, h, :].double().cpu().numpy() if c["use_alpha"] else None
            s = s0[b, h].double().cpu().numpy() if c["use_s0"] else None
            n = nw[h].double().cpu().numpy() if nw is not None else None
            ref = orc.vda_slice(q, k, v, beta, gate, 1e-6, alpha=a, s0=s, rule=rule, norm_weight=n, **kw)["out"]
            got = out[b, :, :, h, :].double().cpu().numpy()
            assert np.isfinite(got).all(), c
            e = orc.slice_error(got, ref)
            assert e <= TOL[w.dtype], f"case {case} {c}: slice (b={b}, h={h}) error {e:.3e}"
    vda.close()

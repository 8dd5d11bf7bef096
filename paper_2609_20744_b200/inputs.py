"""Seeded synthetic inputs for the VDA forward path.

This module only draws random tensors with the shapes and value distributions of
the benchmark workloads; it contains none of the layer's arithmetic.  It serves
both the CUDA library's tests/benchmark and the CPU checker's tests.

Layout (the library's boundary layout): q, k, v : [B, T, F, H, d], beta : [B, T, F, H],
gate : [H]; T latent frames of F spatial tokens each.  Values are drawn in fp32,
normalised in fp32 and then rounded once to the I/O dtype, so a checker that reads
the rounded tensors sees exactly what the GPU sees.

Streams are seeded per (config seed, batch index, frame index) on the device the
tensors are drawn on.  torch's CPU and CUDA generators produce different streams
for the same seed, so a parity check always hands the checker a host copy of the
very tensors the GPU consumed.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Optional

import torch


@dataclass(frozen=True)
class VdaWorkload:
    name: str
    B: int
    H: int
    d: int
    T: int
    F: int
    dtype: str = "bf16"            # "f32" | "bf16"
    seed: int = 0
    beta_std: float = 1.0          # beta = sigmoid(beta_std * N(0,1))
    corr_frac: float = 0.0         # fraction of each frame's keys drawn near shared directions
    corr_sigma: float = 0.05       # per-component perturbation before re-normalisation
    corr_dirs: int = 8             # shared unit directions per (batch, head)
    # Degenerate and out-of-the-ordinary inputs the layer must still handle (all off by default):
    key_repeat_frac: float = 0.0   # fraction of a frame's tokens that carry ONE unit key, drawn per (batch, frame, head)
    key_norm_lo: float = 1.0       # key norms log-uniform in [key_norm_lo, key_norm_hi] instead of 1
    key_norm_hi: float = 1.0
    zero_beta_frames: tuple = ()   # frames whose write gates are all zero (nothing is written)
    beta_const: float = -1.0       # >= 0: every write gate has this value

    @property
    def tokens(self) -> int:
        return self.B * self.T * self.F

    @property
    def torch_dtype(self):
        return torch.float32 if self.dtype == "f32" else torch.bfloat16

    def scaled(self, **kw) -> "VdaWorkload":
        return replace(self, **kw)


# The five benchmark configurations.
TINY = VdaWorkload("tiny", B=1, H=2, d=64, T=4, F=64, dtype="f32", seed=0)
CLIP_480P = VdaWorkload("480p", B=1, H=8, d=128, T=21, F=1560, seed=1)
CLIP_768P = VdaWorkload("768p", B=1, H=40, d=128, T=86, F=4080, seed=2,
                        beta_std=1.5, corr_frac=0.30, corr_sigma=0.05, corr_dirs=8)
SWEEP = tuple(VdaWorkload(f"sweep_T{T}_F{F}", B=1, H=24, d=128, T=T, F=F, seed=3)
              for (T, F) in ((16, 16384), (64, 4096), (256, 1024), (1024, 256)))
CFG_LONG = VdaWorkload("cfg_long", B=2, H=40, d=128, T=172, F=4080, seed=4)

WORKLOADS = {w.name: w for w in (TINY, CLIP_480P, CLIP_768P, *SWEEP, CFG_LONG)}


def _seed(*parts: int) -> int:
    s = 0x9E3779B97F4A7C15
    for p in parts:
        s = (s ^ (int(p) + 0x9E3779B97F4A7C15 + ((s << 6) & 0xFFFFFFFFFFFFFFFF) + (s >> 2))) & 0xFFFFFFFFFFFFFFFF
    return s & 0x7FFFFFFFFFFFFFFF


def _unit(x: torch.Tensor) -> torch.Tensor:
    return x / x.norm(dim=-1, keepdim=True).clamp_min(1e-12)


def generate(w: VdaWorkload, device="cpu", pin: bool = False):
    """Draw q, k, v, beta, gate for workload `w` on `device`.

    Returns a dict of tensors in the boundary layout.  `pin` places CPU tensors in
    pinned memory (for timing host->device copies).
    """
    dev = torch.device(device)
    dt = w.torch_dtype
    kw = dict(device=dev, dtype=dt)
    if dev.type == "cpu" and pin:
        kw["pin_memory"] = True
    q = torch.empty((w.B, w.T, w.F, w.H, w.d), **kw)
    k = torch.empty_like(q, pin_memory=pin and dev.type == "cpu")
    v = torch.empty_like(q, pin_memory=pin and dev.type == "cpu")
    fkw = dict(device=dev, dtype=torch.float32)
    if dev.type == "cpu" and pin:
        fkw["pin_memory"] = True
    beta = torch.empty((w.B, w.T, w.F, w.H), **fkw)

    g = torch.Generator(device=dev)
    g.manual_seed(_seed(w.seed, 0xA7E))
    gate = torch.sigmoid(torch.randn((w.H,), generator=g, device=dev, dtype=torch.float32))

    for b in range(w.B):
        dirs = None
        if w.corr_frac > 0.0:
            g.manual_seed(_seed(w.seed, b, 0xD1F))
            dirs = _unit(torch.randn((w.H, w.corr_dirs, w.d), generator=g, device=dev))
        for t in range(w.T):
            g.manual_seed(_seed(w.seed, b, t))
            shp = (w.F, w.H, w.d)
            qf = _unit(torch.randn(shp, generator=g, device=dev))
            kf = torch.randn(shp, generator=g, device=dev)
            vf = torch.randn(shp, generator=g, device=dev)
            bf = torch.sigmoid(w.beta_std * torch.randn((w.F, w.H), generator=g, device=dev))
            if dirs is not None:
                pick = torch.rand((w.F, w.H), generator=g, device=dev) < w.corr_frac
                j = torch.randint(0, w.corr_dirs, (w.F, w.H), generator=g, device=dev)
                hidx = torch.arange(w.H, device=dev)[None, :].expand(w.F, w.H)
                near = dirs[hidx, j] + w.corr_sigma * torch.randn(shp, generator=g, device=dev)
                kf = torch.where(pick[..., None], near, kf)
            kf = _unit(kf)
            # the optional recipes draw after everything else, so the default streams do not move
            if w.key_repeat_frac > 0.0:
                shared = _unit(torch.randn((1, w.H, w.d), generator=g, device=dev))
                if w.key_repeat_frac >= 1.0:
                    kf = shared.expand(shp).clone()
                else:
                    rep = torch.rand((w.F, w.H), generator=g, device=dev) < w.key_repeat_frac
                    kf = torch.where(rep[..., None], shared.expand(shp), kf)
            if (w.key_norm_lo, w.key_norm_hi) != (1.0, 1.0):
                import math
                lo, hi = math.log(w.key_norm_lo), math.log(w.key_norm_hi)
                kf = kf * torch.exp(lo + (hi - lo) * torch.rand((w.F, w.H, 1), generator=g, device=dev))
            if w.beta_const >= 0.0:
                bf = torch.full_like(bf, w.beta_const)
            if t in w.zero_beta_frames:
                bf = torch.zeros_like(bf)
            q[b, t].copy_(qf)
            k[b, t].copy_(kf)
            v[b, t].copy_(vf)
            beta[b, t].copy_(bf)
    return {"q": q, "k": k, "v": v, "beta": beta, "gate": gate}


def generate_recurrence_extras(w: VdaWorkload, device="cpu"):
    """Seeded decay gates alpha [B,T,H,d] = sigmoid(N(2,1)) (mostly close to 1, as decay gates are) and a text
    state s0 [B,H,d,d] ~ N(0, 1/d), for the extended entry point.  float32."""
    dev = torch.device(device)
    g = torch.Generator(device=dev)
    g.manual_seed(_seed(w.seed, 0xA1FA))
    alpha = torch.sigmoid(2.0 + torch.randn((w.B, w.T, w.H, w.d), generator=g, device=dev))
    s0 = torch.randn((w.B, w.H, w.d, w.d), generator=g, device=dev) / (w.d ** 0.5)
    return alpha.contiguous(), s0.contiguous()


def generate_output_extras(w: VdaWorkload, device="cpu"):
    """Seeded element-wise output gate gate_elem [B,T,F,H,d] = sigmoid(N(0,1)) in the I/O dtype (the output of a
    content-dependent gate network) and a per-channel norm scale norm_weight [H,d] = 1 + 0.1 N(0,1), float32."""
    dev = torch.device(device)
    g = torch.Generator(device=dev)
    g.manual_seed(_seed(w.seed, 0x6A7E))
    gate_elem = torch.sigmoid(torch.randn((w.B, w.T, w.F, w.H, w.d), generator=g, device=dev)).to(w.torch_dtype)
    norm_weight = 1.0 + 0.1 * torch.randn((w.H, w.d), generator=g, device=dev)
    return gate_elem.contiguous(), norm_weight.contiguous()


def generate_projected(w: VdaWorkload, device="cpu"):
    """Seeded stand-ins for the projected (not yet prepared) q, k, v [B,T,F,H,d] ~ N(0,1) in the I/O dtype and
    for the short-convolution filters of the feature preparation: per channel a 5 x 5 spatial and a five-tap
    temporal filter, drawn as a unit centre tap plus N(0, 0.15^2) on every tap (a trained short filter stays
    close to the identity it is initialised with).  Filters are float32."""
    dev = torch.device(device)
    g = torch.Generator(device=dev)
    out = {}
    for i, n in enumerate(("q", "k", "v")):
        x = torch.empty((w.B, w.T, w.F, w.H, w.d), device=dev, dtype=w.torch_dtype)
        for b in range(w.B):
            for t in range(w.T):
                g.manual_seed(_seed(w.seed, 0x9E0 + i, b, t))
                x[b, t].copy_(torch.randn((w.F, w.H, w.d), generator=g, device=dev))
        out[n] = x
    g.manual_seed(_seed(w.seed, 0xF17))
    C = w.H * w.d
    for n in ("wk", "wv"):
        ws = 0.15 * torch.randn((C, 5, 5), generator=g, device=dev)
        ws[:, 2, 2] += 1.0
        wt = 0.15 * torch.randn((C, 5), generator=g, device=dev)
        wt[:, 2] += 1.0
        out[n + "_spatial"] = ws.contiguous()
        out[n + "_temporal"] = wt.contiguous()
    return out


def head_slice(x: dict, b: int, h: int):
    """Host float64 numpy copies of one (batch, head) slice: q,k,v [T,F,d], beta [T,F], gate scalar."""
    import numpy as np

    def f64(t):
        return t.detach().to("cpu").to(torch.float64).numpy()

    return (f64(x["q"][b, :, :, h, :]), f64(x["k"][b, :, :, h, :]), f64(x["v"][b, :, :, h, :]),
            f64(x["beta"][b, :, :, h]), float(x["gate"][h].item()))

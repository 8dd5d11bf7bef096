"""Parity of the CUDA library (through the C ABI) against the fp64 checker, element by element.

Tolerances (the metric is oracle.slice_error: max |gpu - ref| over one (batch, head) slice divided
by that slice's max |ref|):  1e-4 for f32 I/O,  2e-2 for bf16 I/O.
"""
import numpy as np
import pytest
import torch

from oracle import vda_oracle as orc
from paper_2609_20744_b200 import binding, build, inputs

pytestmark = pytest.mark.gpu

TOL = {"f32": 1e-4, "bf16": 2e-2}


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    binding.load_library()


def run_gpu(w, x, flags=0):
    vda = binding.Vda(w.d, w.dtype, flags=flags)
    out = vda.forward(x["q"], x["k"], x["v"], x["beta"], x["gate"])
    torch.cuda.synchronize()
    assert vda.status() == binding.VDN_OK
    assert vda.launch_count() > 0
    return vda, out


def check_heads(w, x, out, pairs, tol):
    worst = 0.0
    for (b, h) in pairs:
        q, k, v, beta, gate = inputs.head_slice(x, b, h)
        ref = orc.vda_slice(q, k, v, beta, gate, 1e-6)["out"]
        got = out[b, :, :, h, :].double().cpu().numpy()
        assert np.isfinite(got).all()
        e = orc.slice_error(got, ref)
        worst = max(worst, e)
        assert e <= tol, f"slice (b={b}, h={h}) error {e:.3e} > {tol}"
    return worst


def kernel_names(vda, x):
    vda.profile(True)
    vda.forward(x["q"], x["k"], x["v"], x["beta"], x["gate"])
    torch.cuda.synchronize()
    times = vda.kernel_times()
    vda.profile(False)
    return times


def all_pairs(w):
    return [(b, h) for b in range(w.B) for h in range(w.H)]


# ------------------------------------------------------------------------------ whole layer
@pytest.mark.parametrize("name,kw", [
    ("tiny", {}),                                              # the f32 benchmark config
    ("tiny", dict(d=128, F=100, T=5, H=3)),                    # d=128, ragged token tail
    ("tiny", dict(T=1)),                                       # single frame -> all zeros
    ("tiny", dict(T=2, F=1)),                                  # one token per frame
    ("tiny", dict(B=2, H=1, T=3, F=257)),                      # several tiles + tail, two batches
    ("tiny", dict(dtype="bf16", d=128, T=6, F=300, H=2)),      # bf16 I/O
    ("tiny", dict(dtype="bf16", d=64, T=3, F=70, H=2)),
    ("tiny", dict(dtype="bf16", d=128, B=2, T=5, F=3100, H=3)),  # long frames, ragged last tile
])
def test_forward_matches_oracle_small(name, kw):
    w = inputs.WORKLOADS[name].scaled(**kw)
    x = inputs.generate(w, "cuda")
    _, out = run_gpu(w, x)
    if w.T == 1:
        assert torch.count_nonzero(out) == 0
    check_heads(w, x, out, all_pairs(w), TOL[w.dtype])


@pytest.mark.parametrize("B,H,T,F", [
    (1, 1, 1, 5),        # one frame: nothing to read, all zeros
    (1, 1, 2, 1),        # one token per frame
    (2, 3, 3, 127),      # one short tile, several batches and heads
    (1, 2, 4, 129),      # one full tile + one token
    (3, 1, 2, 256),      # exact tiles, batch > heads
    (1, 5, 7, 64),       # more chains than frames
    (1, 2, 33, 40),      # a deeper scan than anything else in this file
])
def test_tensor_core_path_edge_shapes(B, H, T, F):
    w = inputs.TINY.scaled(dtype="bf16", d=128, B=B, H=H, T=T, F=F, seed=B * 1000 + H * 100 + T * 10 + F)
    x = inputs.generate(w, "cuda")
    vda, out = run_gpu(w, x)
    assert vda.uses_tensor_cores()
    if T == 1:
        assert torch.count_nonzero(out) == 0
    check_heads(w, x, out, all_pairs(w), TOL["bf16"])
    # the plain-fp32 kernels on the same bf16 inputs are a second GPU opinion
    _, out2 = run_gpu(w, x, flags=binding.VDN_FLAG_FORCE_SIMT)
    scale = out2.float().abs().amax().clamp_min(1e-30)
    assert float((out.float() - out2.float()).abs().amax() / scale) < 2e-2


# ------------------------------------------------------------------------------ decay gates and text state
@pytest.mark.parametrize("dtype,d,flags,use_alpha,use_s0", [
    ("f32", 64, 0, True, True), ("f32", 128, 0, True, False), ("f32", 64, 0, False, True),
    ("bf16", 128, 0, True, True), ("bf16", 128, 0, True, False), ("bf16", 128, 0, False, True),
    ("bf16", 128, binding.VDN_FLAG_FORCE_SIMT, True, True),
])
def test_forward_ex_decay_and_text_state(dtype, d, flags, use_alpha, use_s0):
    w = inputs.TINY.scaled(dtype=dtype, d=d, B=2, H=2, T=5, F=140, seed=77)
    x = inputs.generate(w, "cuda")
    alpha, s0 = inputs.generate_recurrence_extras(w, "cuda")
    alpha = alpha if use_alpha else None
    s0 = s0 if use_s0 else None
    vda = binding.Vda(w.d, w.dtype, flags=flags)
    out = vda.forward(x["q"], x["k"], x["v"], x["beta"], x["gate"], alpha=alpha, s0=s0)
    torch.cuda.synchronize()
    assert vda.status() == binding.VDN_OK
    for (b, h) in all_pairs(w):
        q, k, v, beta, gate = inputs.head_slice(x, b, h)
        a = None if alpha is None else alpha[b, :, h, :].double().cpu().numpy()
        s = None if s0 is None else s0[b, h].double().cpu().numpy()
        ref = orc.vda_slice(q, k, v, beta, gate, 1e-6, alpha=a, s0=s)["out"]
        e = orc.slice_error(out[b, :, :, h, :].double().cpu().numpy(), ref)
        assert e <= TOL[dtype], f"slice (b={b}, h={h}) error {e:.3e}"
    # the extras matter: the plain call gives something else
    plain = vda.forward(x["q"], x["k"], x["v"], x["beta"], x["gate"])
    torch.cuda.synchronize()
    assert not torch.allclose(plain.float(), out.float(), atol=1e-2)


def test_forward_ex_single_frame_reads_the_text_state():
    # T = 1: nothing but S_T is read (both halves), bridged by alpha_0 (Eq. 1b, Eq. A.4)
    w = inputs.TINY.scaled(dtype="bf16", d=128, T=1, F=70, H=2)
    x = inputs.generate(w, "cuda")
    alpha, s0 = inputs.generate_recurrence_extras(w, "cuda")
    vda = binding.Vda(w.d, w.dtype)
    out = vda.forward(x["q"], x["k"], x["v"], x["beta"], x["gate"], alpha=alpha, s0=s0)
    torch.cuda.synchronize()
    o = torch.einsum("bhck,bfhk->bfhc", s0, (alpha[:, 0][:, None] * x["q"][:, 0].float()))
    want = x["gate"][None, None, :, None] * o / torch.sqrt(o.pow(2).mean(-1, keepdim=True) + 1e-6)
    assert torch.allclose(out[:, 0].float(), want, atol=3e-2, rtol=3e-2)


# ------------------------------------------------------------------------------ the additive baseline (ablation)
@pytest.mark.parametrize("dtype,d,flags,extras", [
    ("f32", 64, 0, False), ("f32", 128, 0, True), ("bf16", 128, 0, False), ("bf16", 128, 0, True),
    ("bf16", 128, binding.VDN_FLAG_FORCE_SIMT, True),
])
def test_additive_rule_matches_oracle(dtype, d, flags, extras):
    w = inputs.TINY.scaled(dtype=dtype, d=d, B=1, H=2, T=6, F=200, seed=91)
    x = inputs.generate(w, "cuda")
    alpha, s0 = inputs.generate_recurrence_extras(w, "cuda") if extras else (None, None)
    vda = binding.Vda(w.d, w.dtype, flags=flags | binding.VDN_FLAG_ADDITIVE_RULE)
    out = vda.forward(x["q"], x["k"], x["v"], x["beta"], x["gate"], alpha=alpha, s0=s0)
    torch.cuda.synchronize()
    assert vda.status() == binding.VDN_OK
    for (b, h) in all_pairs(w):
        q, k, v, beta, gate = inputs.head_slice(x, b, h)
        a = None if alpha is None else alpha[b, :, h, :].double().cpu().numpy()
        s = None if s0 is None else s0[b, h].double().cpu().numpy()
        ref = orc.vda_slice(q, k, v, beta, gate, 1e-6, alpha=a, s0=s, rule="additive")["out"]
        e = orc.slice_error(out[b, :, :, h, :].double().cpu().numpy(), ref)
        assert e <= TOL[dtype], f"slice (b={b}, h={h}) error {e:.3e}"
    # and it is not the joint solve
    vda2 = binding.Vda(w.d, w.dtype, flags=flags)
    out2 = vda2.forward(x["q"], x["k"], x["v"], x["beta"], x["gate"], alpha=alpha, s0=s0)
    torch.cuda.synchronize()
    assert not torch.allclose(out.float(), out2.float(), atol=1e-2)


@pytest.mark.parametrize("B,H", [(1, 80), (2, 45)])
def test_more_scan_chains_than_sms(B, H):
    # 2 B H chains on 148 SMs: the surplus chains are scanned on the library's side stream beside the read-out of
    # the first 74 (batch, head) pairs; pairs on both sides of the split, and the ends, against the checker
    w = inputs.TINY.scaled(dtype="bf16", d=128, B=B, H=H, T=5, F=130, seed=61)
    x = inputs.generate(w, "cuda")
    vda, out = run_gpu(w, x)
    assert vda.uses_tensor_cores()
    pairs = [(0, 0), (B - 1, H - 1)] + [divmod(p, H) for p in (72, 73, 74, 75)]
    check_heads(w, x, out, pairs, TOL["bf16"])
    ms = out.float().pow(2).mean(dim=-1)                      # every pair was read out: rows have gate-sized rms
    assert torch.allclose(ms, x["gate"].pow(2)[None, None, None, :].expand_as(ms), rtol=3e-2)
    again = vda.forward(x["q"], x["k"], x["v"], x["beta"], x["gate"])
    torch.cuda.synchronize()
    assert torch.equal(again, out)


def test_bf16_through_plain_fp32_kernels():
    w = inputs.TINY.scaled(dtype="bf16", d=128, T=4, F=200, H=2)
    x = inputs.generate(w, "cuda")
    _, out = run_gpu(w, x, flags=binding.VDN_FLAG_FORCE_SIMT)
    check_heads(w, x, out, all_pairs(w), TOL["bf16"])


def test_480p_config_all_heads():
    w = inputs.CLIP_480P
    x = inputs.generate(w, "cuda")
    _, out = run_gpu(w, x)
    check_heads(w, x, out, all_pairs(w), TOL[w.dtype])


# ------------------------------------------------------------------------------ stage-wise
def rel(g, r):
    return np.max(np.abs(g - r)) / max(np.max(np.abs(r)), 1e-30)


@pytest.mark.parametrize("dtype,d,flags", [("f32", 64, 0), ("f32", 128, 0), ("bf16", 128, binding.VDN_FLAG_FORCE_SIMT)])
def test_stagewise_intermediates_plain_fp32_kernels(dtype, d, flags):
    w = inputs.TINY.scaled(dtype=dtype, d=d, T=5, F=150, H=2)
    x = inputs.generate(w, "cuda")
    vda, out = run_gpu(w, x, flags=flags)
    assert not vda.uses_tensor_cores()
    B, T, F, H = w.B, w.T, w.F, w.H
    stats = vda.view(binding.VIEW_STATS, B, T, F, H).double().cpu().numpy()
    inv = vda.view(binding.VIEW_INV, B, T, F, H).double().cpu().numpy()
    fwd = vda.view(binding.VIEW_FWD, B, T, F, H).double().cpu().numpy()
    read = vda.view(binding.VIEW_READ, B, T, F, H).double().cpu().numpy()
    for h in range(H):
        q, k, v, beta, gate = inputs.head_slice(x, 0, h)
        ref = orc.vda_slice(q, k, v, beta, gate, 1e-6, want=("A", "B", "C", "P", "R"))
        for t in range(T):
            assert rel(stats[0, h, t, :d, :], ref["A"][t]) < 1e-5
            assert rel(stats[0, h, t, d:, :], ref["B"][t]) < 1e-5
            assert rel(inv[0, h, t], ref["C"][t]) < 1e-5
            assert rel(fwd[0, h, t], ref["P"][t].T) < 1e-5
            want = np.zeros((d, d))
            if t > 0:
                want = want + ref["P"][t - 1]
            if t + 1 < T:
                want = want + ref["R"][t + 1]
            assert rel(read[0, h, t].T, want) < 1e-5


@pytest.mark.parametrize("F", [300, 3200])
def test_stagewise_intermediates_tensor_core_kernels(F):
    d = 128
    w = inputs.TINY.scaled(dtype="bf16", d=d, T=6, F=F, H=2)
    x = inputs.generate(w, "cuda")
    vda, out = run_gpu(w, x)
    assert [n for (n, _, _) in kernel_names(vda, x)] == ["gram_tc", "resolve_tc", "scan_tc", "readout_tc"]
    assert vda.uses_tensor_cores()
    B, T, F, H = w.B, w.T, w.F, w.H
    stats = vda.view(binding.VIEW_STATS, B, T, F, H).double().cpu().numpy()
    split = vda.view(binding.VIEW_INV_SPLIT, B, T, F, H).double().cpu().numpy()
    pf = vda.view(binding.VIEW_READ_FWD, B, T, F, H).double().cpu().numpy()
    pb = vda.view(binding.VIEW_READ_BWD, B, T, F, H).double().cpu().numpy()
    for h in range(H):
        q, k, v, beta, gate = inputs.head_slice(x, 0, h)
        ref = orc.vda_slice(q, k, v, beta, gate, 1e-6, want=("A", "B", "C", "P", "R"))
        # the checker's states from the GPU's own statistics isolate the scan's arithmetic from the
        # bf16 rounding of the weighted keys in the Gram stage
        Pg, Rg = orc.scan_states([0.5 * (stats[0, h, t, :d, :] + stats[0, h, t, :d, :].T) for t in range(T)], [stats[0, h, t, d:, :] for t in range(T)],
                                 np.ones((T, d)), np.zeros((d, d)))
        for t in range(T):
            # bf16 products are exact in fp32; only the beta-weighted key operand is rounded (2^-9 relative)
            assert rel(stats[0, h, t, :d, :], ref["A"][t]) < 4e-3
            assert rel(stats[0, h, t, d:, :], ref["B"][t]) < 4e-3
            # (the stored A block is K^T (beta K) with only one factor rounded to bf16, hence symmetric up to
            # that rounding only; the resolve inverts I + its symmetric part)
            a_sym = 0.5 * (stats[0, h, t, :d, :] + stats[0, h, t, :d, :].T)
            inv_g = np.linalg.inv(np.eye(d) + a_sym)
            # three parts carry fp32 accuracy: an fp32 inverse is good to a few eps times the condition number
            assert rel(split[0, h, t].sum(axis=0), inv_g) < 5e-6 * np.linalg.cond(np.eye(d) + a_sym)
            assert rel(split[0, h, t, 0], inv_g) < 8e-3                     # the leading part alone: bf16, truncated (2^-7)
            want_f = ref["P"][t - 1] if t > 0 else np.zeros((d, d))
            want_b = ref["R"][t + 1] if t + 1 < T else np.zeros((d, d))
            assert rel(pf[0, h, t], want_f) < 1e-2 or not want_f.any()
            assert rel(pb[0, h, t], want_b) < 1e-2 or not want_b.any()
            if t == 0:
                assert not pf[0, h, t].any()
            if t == T - 1:
                assert not pb[0, h, t].any()
            # against the checker fed with the GPU's statistics the stored states differ by their own bf16
            # rounding (2^-9 relative per element) plus an fp32-level absolute term (a few eps times the condition
            # number, relative to the largest entry): the inverse and the scan run at fp32 accuracy
            if t > 0:
                assert np.all(np.abs(pf[0, h, t] - Pg[t - 1]) <= 2.0 ** -8 * np.abs(Pg[t - 1]) + 2e-5 * np.abs(Pg[t - 1]).max())
            if t + 1 < T:
                assert np.all(np.abs(pb[0, h, t] - Rg[t + 1]) <= 2.0 ** -8 * np.abs(Rg[t + 1]) + 2e-5 * np.abs(Rg[t + 1]).max())


# ------------------------------------------------------------------------------ properties
def test_run_to_run_bitwise_determinism_and_canaries():
    w = inputs.TINY.scaled(dtype="bf16", d=128, T=4, F=333, H=3)
    x = inputs.generate(w, "cuda")
    vda = binding.Vda(w.d, w.dtype)
    n = x["q"].numel()
    pad = 4096
    buf = torch.full((n + 2 * pad,), 7.0, dtype=x["q"].dtype, device="cuda")
    out = buf[pad: pad + n].view_as(x["q"])
    vda.forward(x["q"], x["k"], x["v"], x["beta"], x["gate"], out=out)
    torch.cuda.synchronize()
    first = out.clone()
    vda.forward(x["q"], x["k"], x["v"], x["beta"], x["gate"], out=out)
    torch.cuda.synchronize()
    assert torch.equal(first, out)
    assert torch.all(buf[:pad] == 7.0) and torch.all(buf[pad + n:] == 7.0)


def test_one_handle_across_shapes_and_two_handles_on_two_streams():
    # a handle carries no shape: calls of different shapes in turn give what a fresh handle gives, bit for bit; and
    # two handles (each with its own workspace) run side by side on two streams without touching each other
    shapes = [dict(T=4, F=333, H=3), dict(T=7, F=128, H=1, B=2), dict(T=2, F=1000, H=5), dict(T=4, F=333, H=3)]
    ws = [inputs.TINY.scaled(dtype="bf16", d=128, seed=300 + i, **kw) for i, kw in enumerate(shapes)]
    xs = [inputs.generate(w, "cuda") for w in ws]
    fresh = []
    for w, x in zip(ws, xs):
        v = binding.Vda(w.d, w.dtype)
        fresh.append(v.forward(x["q"], x["k"], x["v"], x["beta"], x["gate"]).clone())
        torch.cuda.synchronize()
        v.close()
    vda = binding.Vda(128, "bf16")
    for w, x, want in zip(ws, xs, fresh):
        got = vda.forward(x["q"], x["k"], x["v"], x["beta"], x["gate"])
        torch.cuda.synchronize()
        assert torch.equal(got, want), f"shape {w.T}x{w.F}x{w.H} after another shape on the same handle"
    a, b = binding.Vda(128, "bf16"), binding.Vda(128, "bf16")
    sa, sb = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    outs_a, outs_b = [], []
    for _ in range(3):
        with torch.cuda.stream(sa):
            outs_a.append(a.forward(xs[0]["q"], xs[0]["k"], xs[0]["v"], xs[0]["beta"], xs[0]["gate"]).clone())
        with torch.cuda.stream(sb):
            outs_b.append(b.forward(xs[2]["q"], xs[2]["k"], xs[2]["v"], xs[2]["beta"], xs[2]["gate"]).clone())
    torch.cuda.synchronize()
    assert a.status() == binding.VDN_OK and b.status() == binding.VDN_OK
    for o in outs_a:
        assert torch.equal(o, fresh[0])
    for o in outs_b:
        assert torch.equal(o, fresh[2])


def test_forward_can_be_captured_in_a_cuda_graph():
    # the layer only enqueues kernels and memsets on the caller's stream (tensor maps travel as kernel parameters):
    # after one eager call (which sets the kernels' attributes) it can be captured and replayed; replays are
    # bitwise the eager result, also after the inputs change in place
    w = inputs.TINY.scaled(dtype="bf16", d=128, T=6, F=200, H=3, seed=12)
    x = inputs.generate(w, "cuda")
    alpha, s0 = inputs.generate_recurrence_extras(w, "cuda")
    vda = binding.Vda(w.d, w.dtype)
    kw = dict(alpha=alpha, s0=s0, chunk=2, radius=1, anchors=True)
    out = torch.empty_like(x["q"])
    eager = vda.forward(x["q"], x["k"], x["v"], x["beta"], x["gate"], **kw).clone()
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            vda.forward(x["q"], x["k"], x["v"], x["beta"], x["gate"], out=out, stream=side, **kw)
    graph.replay()
    torch.cuda.synchronize()
    assert vda.status() == binding.VDN_OK
    assert torch.equal(out, eager)
    x["v"].mul_(0.5)                       # same buffers, new contents
    graph.replay()
    torch.cuda.synchronize()
    eager2 = vda.forward(x["q"], x["k"], x["v"], x["beta"], x["gate"], **kw)
    torch.cuda.synchronize()
    assert torch.equal(out, eager2) and not torch.equal(out, eager)


def test_split_scan_can_be_captured_in_a_cuda_graph():
    # more chains than SMs: the forward forks to the handle's side stream and joins again; captured, the fork becomes
    # two branches of the graph.  After one eager call (which creates the side stream and its events).
    w = inputs.TINY.scaled(dtype="bf16", d=128, B=1, H=80, T=4, F=130, seed=62)
    x = inputs.generate(w, "cuda")
    vda = binding.Vda(w.d, w.dtype)
    eager = vda.forward(x["q"], x["k"], x["v"], x["beta"], x["gate"]).clone()
    torch.cuda.synchronize()
    out = torch.empty_like(x["q"])
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            vda.forward(x["q"], x["k"], x["v"], x["beta"], x["gate"], out=out, stream=side)
    for _ in range(2):
        out.zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert vda.status() == binding.VDN_OK
        assert torch.equal(out, eager)


def test_token_permutation_within_frames_permutes_rows_only():
    w = inputs.TINY.scaled(d=128, T=3, F=96, H=2)
    x = inputs.generate(w, "cuda")
    _, out = run_gpu(w, x)
    perm = torch.randperm(w.F, generator=torch.Generator().manual_seed(5)).cuda()
    xp = {n: (t[:, :, perm] if t.dim() >= 4 else t).contiguous() for n, t in x.items()}
    _, outp = run_gpu(w, xp)
    assert torch.allclose(outp, out[:, :, perm], atol=2e-5)


def test_frame_reversal_reverses_output():
    w = inputs.TINY.scaled(d=64, T=5, F=64, H=2)
    x = inputs.generate(w, "cuda")
    _, out = run_gpu(w, x)
    xr = {n: (t.flip(1) if t.dim() >= 4 else t).contiguous() for n, t in x.items()}
    _, outr = run_gpu(w, xr)
    assert torch.allclose(outr.flip(1), out, atol=2e-5)


def test_output_rows_have_gate_sized_rms():
    w = inputs.TINY.scaled(dtype="bf16", d=128, T=4, F=130, H=3)
    x = inputs.generate(w, "cuda")
    _, out = run_gpu(w, x)
    ms = out.float().pow(2).mean(dim=-1)                      # [B,T,F,H]
    want = x["gate"].pow(2)[None, None, None, :].expand_as(ms)
    assert torch.allclose(ms, want, rtol=3e-2)


# ------------------------------------------------------------------------------ host-buffer entry point
@pytest.mark.parametrize("dtype,d,B,T", [("bf16", 128, 1, 3), ("bf16", 128, 2, 11), ("f32", 64, 2, 9), ("bf16", 128, 1, 1)])
def test_forward_host_matches_device_entry_point(dtype, d, B, T):
    # the host entry point copies the queries in and the results out in groups of frames, on two streams
    w = inputs.TINY.scaled(dtype=dtype, d=d, B=B, T=T, F=200, H=2)
    xh = inputs.generate(w, "cpu", pin=True)
    xd = {n: t.cuda() for n, t in xh.items()}
    vda, out_d = run_gpu(w, xd)
    out_h = torch.empty_like(xh["q"]).pin_memory()
    out_h.fill_(7.0)
    for _ in range(2):                                  # twice: the second call reuses the stream and events
        vda.forward_host(xh["q"], xh["k"], xh["v"], xh["beta"], xh["gate"], out_h)
        torch.cuda.current_stream().synchronize()       # the caller's stream alone covers the copies back
        assert torch.equal(out_h, out_d.cpu())
        out_h.fill_(7.0)


@pytest.mark.parametrize("dtype,d,flags", [("bf16", 128, 0), ("bf16", 128, binding.VDN_FLAG_SCAN_CHUNKWISE), ("f32", 64, 0)])
def test_forward_host_opt_release_setting_matches_device_entry_point(dtype, d, flags):
    # every optional input from host memory: chunk window, anchors, decay gates, text state, element-wise gate,
    # norm weight, queries normalised by the read-out
    w = inputs.TINY.scaled(dtype=dtype, d=d, B=2, T=13, F=150, H=2, seed=41)
    xh = inputs.generate(w, "cpu", pin=True)
    alpha, s0 = inputs.generate_recurrence_extras(w, "cpu")
    ge, nw = inputs.generate_output_extras(w, "cpu")
    kw = dict(chunk=3, radius=1, anchors=True, q_l2_eps=1e-6)
    host_extras = dict(alpha=alpha.pin_memory(), s0=s0.pin_memory(), gate_elem=ge.pin_memory(), norm_weight=nw.pin_memory())
    vda = binding.Vda(w.d, w.dtype, flags=flags)
    out_d = vda.forward(*(xh[n].cuda() for n in ("q", "k", "v", "beta", "gate")),
                        **{n: t.cuda() for n, t in host_extras.items()}, **kw)
    torch.cuda.synchronize()
    assert vda.status() == binding.VDN_OK
    out_h = torch.empty_like(xh["q"]).pin_memory()
    for _ in range(2):
        out_h.fill_(7.0)
        vda.forward_host(xh["q"], xh["k"], xh["v"], xh["beta"], xh["gate"], out_h, **host_extras, **kw)
        torch.cuda.current_stream().synchronize()
        assert torch.equal(out_h, out_d.cpu())
    assert torch.count_nonzero(out_h[:, 0]) == 0 and torch.count_nonzero(out_h[:, -1]) == 0
    # and against the checker, one slice
    q, k, v, beta, gate = inputs.head_slice(xh, 1, 1)
    from oracle import prep_oracle as po
    ref = orc.vda_slice(po.l2_normalise(q, 1e-6), k, v, beta, gate * ge[1, :, :, 1].double().numpy(), 1e-6,
                        alpha=alpha[1, :, 1].double().numpy(), s0=s0[1, 1].double().numpy(),
                        norm_weight=nw[1].double().numpy(), chunk=3, radius=1, anchors=True)["out"]
    assert orc.slice_error(out_h[1, :, :, 1].double().numpy(), ref) <= TOL[dtype]


def test_forward_host_refuses_before_queuing_any_copy():
    # a staging buffer that is too small is a host-side error: nothing may be enqueued, `out` stays untouched
    w = inputs.TINY.scaled(dtype="bf16", d=128, T=3, F=100, H=2)
    xh = inputs.generate(w, "cpu", pin=True)
    vda = binding.Vda(w.d, w.dtype)
    vda.ensure_workspace(w.B, w.T, w.F, w.H)
    small = torch.empty(4096, dtype=torch.uint8, device="cuda")
    import ctypes
    vda.lib.vdn_vda_set_staging(vda.h, ctypes.c_void_p(small.data_ptr()), 4096)
    out_h = torch.full(xh["q"].shape, 7.0, dtype=xh["q"].dtype).pin_memory()
    p = lambda t: ctypes.c_void_p(t.data_ptr())
    st = vda.lib.vdn_vda_forward_host(vda.h, p(xh["q"]), p(xh["k"]), p(xh["v"]), p(xh["beta"]), p(xh["gate"]), p(out_h),
                                      w.B, w.T, w.F, w.H, w.d, None)
    assert st == 3
    torch.cuda.synchronize()
    assert torch.all(out_h == 7.0)


# ------------------------------------------------------------------------------ argument errors (host side)
def test_argument_errors_enqueue_nothing():
    w = inputs.TINY
    x = inputs.generate(w, "cuda")
    vda = binding.Vda(w.d, w.dtype)
    with pytest.raises(binding.VdnError) as e:
        vda.forward(x["q"], x["k"], x["v"], x["beta"], x["gate"], out=x["q"])      # aliasing
    assert e.value.status == 1
    vda2 = binding.Vda(128, "f32")
    with pytest.raises(binding.VdnError):
        vda2.forward(x["q"], x["k"], x["v"], x["beta"], x["gate"])                 # d mismatch
    import ctypes
    vda3 = binding.Vda(w.d, w.dtype)
    small = torch.empty(1024, dtype=torch.uint8, device="cuda")
    vda3.lib.vdn_vda_set_workspace(vda3.h, ctypes.c_void_p(small.data_ptr()), 1024)
    p = lambda t: ctypes.c_void_p(t.data_ptr())
    out = torch.empty_like(x["q"])
    st = vda3.lib.vdn_vda_forward(vda3.h, p(x["q"]), p(x["k"]), p(x["v"]), p(x["beta"]), p(x["gate"]), p(out),
                                  w.B, w.T, w.F, w.H, w.d, None)
    assert st == 3                                                                  # workspace too small
    st = vda3.lib.vdn_vda_forward(vda3.h, None, p(x["k"]), p(x["v"]), p(x["beta"]), p(x["gate"]), p(out),
                                  w.B, w.T, w.F, w.H, w.d, None)
    assert st == 1
    st = vda3.lib.vdn_vda_forward(vda3.h, ctypes.c_void_p(x["q"].data_ptr() + 4), p(x["k"]), p(x["v"]),
                                  p(x["beta"]), p(x["gate"]), p(out), w.B, w.T, w.F, w.H, w.d, None)
    assert st == 1                                                                  # misaligned
    torch.cuda.synchronize()

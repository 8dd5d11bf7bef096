"""Parity of vdn_vda_forward_opt (chunk windows, boundary anchors, decay bridge, element-wise gate, norm
weight) against the fp64 checker, element by element, on every kernel path.

Tolerances as in test_gpu_parity.py: 1e-4 for f32 I/O, 2e-2 for bf16 I/O (oracle.slice_error).
"""
import numpy as np
import pytest
import torch

from oracle import vda_oracle as orc
from paper_2609_20744_b200 import binding, build, inputs

pytestmark = pytest.mark.gpu

TOL = {"f32": 1e-4, "bf16": 2e-2}
SIMT = binding.VDN_FLAG_FORCE_SIMT


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    binding.load_library()


def check(w, x, out, alpha=None, s0=None, gate_elem=None, norm_weight=None, use_gate=True, rule="vda", **win):
    worst = 0.0
    for b in range(w.B):
        for h in range(w.H):
            q, k, v, beta, gate = inputs.head_slice(x, b, h)
            if gate_elem is not None:
                ge = gate_elem[b, :, :, h, :].double().cpu().numpy()
                gate = ge * gate if use_gate else ge
            a = None if alpha is None else alpha[b, :, h, :].double().cpu().numpy()
            s = None if s0 is None else s0[b, h].double().cpu().numpy()
            nw = None if norm_weight is None else norm_weight[h].double().cpu().numpy()
            ref = orc.vda_slice(q, k, v, beta, gate, 1e-6, alpha=a, s0=s, rule=rule, norm_weight=nw, **win)["out"]
            got = out[b, :, :, h, :].double().cpu().numpy()
            assert np.isfinite(got).all()
            e = orc.slice_error(got, ref)
            worst = max(worst, e)
            assert e <= TOL[w.dtype], f"slice (b={b}, h={h}) error {e:.3e} > {TOL[w.dtype]}"
    return worst


@pytest.mark.parametrize("dtype,d,flags", [("f32", 64, 0), ("bf16", 128, 0), ("bf16", 128, SIMT)])
@pytest.mark.parametrize("T,chunk,radius,anchors", [
    (12, 5, 1, True),      # the release setting on a short clip: every window touches a clip end
    (23, 5, 1, True),      # long enough for full 15-frame windows in the middle
    (9, 2, 0, True), (10, 2, 1, False), (7, 3, 0, False), (6, 1, 1, True), (5, 1, 0, True),
    (4, 5, 1, True),       # one window covers every scanned frame: both sides read the text state
    (3, 1, 0, True),       # a single scanned frame
])
def test_window_anchor_bridge_matches_oracle(dtype, d, flags, T, chunk, radius, anchors):
    w = inputs.TINY.scaled(dtype=dtype, d=d, B=1, H=2, T=T, F=140, seed=100 * T + 10 * chunk + radius)
    x = inputs.generate(w, "cuda")
    alpha, s0 = inputs.generate_recurrence_extras(w, "cuda")
    vda = binding.Vda(w.d, w.dtype, flags=flags)
    out = vda.forward(x["q"], x["k"], x["v"], x["beta"], x["gate"], alpha=alpha, s0=s0,
                      chunk=chunk, radius=radius, anchors=anchors)
    torch.cuda.synchronize()
    assert vda.status() == binding.VDN_OK and vda.launch_count() > 0
    check(w, x, out, alpha, s0, chunk=chunk, radius=radius, anchors=anchors)
    if anchors:
        assert torch.count_nonzero(out[:, 0]) == 0 and torch.count_nonzero(out[:, -1]) == 0


@pytest.mark.parametrize("dtype,d,flags", [("f32", 128, 0), ("bf16", 128, 0)])
def test_window_without_decay_or_text_state(dtype, d, flags):
    # alpha = 1, S_T = 0: frames of one chunk read the same pair of states; frames near a clip end read zero on that side
    w = inputs.TINY.scaled(dtype=dtype, d=d, B=2, H=2, T=17, F=130, seed=5)
    x = inputs.generate(w, "cuda")
    vda = binding.Vda(w.d, w.dtype, flags=flags)
    out = vda.forward(x["q"], x["k"], x["v"], x["beta"], x["gate"], chunk=5, radius=1, anchors=True)
    torch.cuda.synchronize()
    assert vda.status() == binding.VDN_OK
    check(w, x, out, chunk=5, radius=1, anchors=True)


@pytest.mark.parametrize("T", [1, 2])
def test_clip_of_anchor_frames_only_has_no_linear_output(T):
    w = inputs.TINY.scaled(dtype="bf16", d=128, T=T, F=70, H=2)
    x = inputs.generate(w, "cuda")
    _, s0 = inputs.generate_recurrence_extras(w, "cuda")
    vda = binding.Vda(w.d, w.dtype)
    out = torch.full_like(x["q"], 3.0)
    vda.forward(x["q"], x["k"], x["v"], x["beta"], x["gate"], out=out, s0=s0, anchors=True)
    torch.cuda.synchronize()
    assert torch.count_nonzero(out) == 0


@pytest.mark.parametrize("dtype,d,flags", [("f32", 64, 0), ("bf16", 128, 0), ("bf16", 128, SIMT)])
@pytest.mark.parametrize("use_gate_elem,use_weight,use_head_gate", [
    (True, True, True), (True, False, False), (False, True, True)])
def test_elementwise_gate_and_norm_weight_match_oracle(dtype, d, flags, use_gate_elem, use_weight, use_head_gate):
    w = inputs.TINY.scaled(dtype=dtype, d=d, B=2, H=3, T=4, F=150, seed=31)
    x = inputs.generate(w, "cuda")
    ge, nw = inputs.generate_output_extras(w, "cuda")
    ge = ge if use_gate_elem else None
    nw = nw if use_weight else None
    vda = binding.Vda(w.d, w.dtype, flags=flags)
    out = vda.forward(x["q"], x["k"], x["v"], x["beta"], x["gate"] if use_head_gate else None,
                      gate_elem=ge, norm_weight=nw)
    torch.cuda.synchronize()
    assert vda.status() == binding.VDN_OK
    check(w, x, out, gate_elem=ge, norm_weight=nw, use_gate=use_head_gate)
    plain = vda.forward(x["q"], x["k"], x["v"], x["beta"], x["gate"])
    torch.cuda.synchronize()
    assert not torch.allclose(plain.float(), out.float(), atol=1e-2)


def test_everything_at_once_on_the_tensor_core_path():
    # release setting (chunk 5, radius 1, anchors, decay bridge, text state) + content-dependent gate + norm weight,
    # several token tiles with a ragged tail, two batches
    w = inputs.TINY.scaled(dtype="bf16", d=128, B=2, H=2, T=13, F=300, seed=8)
    x = inputs.generate(w, "cuda")
    alpha, s0 = inputs.generate_recurrence_extras(w, "cuda")
    ge, nw = inputs.generate_output_extras(w, "cuda")
    vda = binding.Vda(w.d, w.dtype)
    assert vda.uses_tensor_cores()
    kw = dict(chunk=5, radius=1, anchors=True)
    out = vda.forward(x["q"], x["k"], x["v"], x["beta"], x["gate"], alpha=alpha, s0=s0, gate_elem=ge,
                      norm_weight=nw, **kw)
    torch.cuda.synchronize()
    assert vda.status() == binding.VDN_OK
    check(w, x, out, alpha, s0, ge, nw, **kw)
    # bit-identical run to run
    out2 = vda.forward(x["q"], x["k"], x["v"], x["beta"], x["gate"], alpha=alpha, s0=s0, gate_elem=ge,
                       norm_weight=nw, **kw)
    torch.cuda.synchronize()
    assert torch.equal(out, out2)


def test_additive_rule_with_window():
    w = inputs.TINY.scaled(dtype="bf16", d=128, B=1, H=2, T=11, F=200, seed=12)
    x = inputs.generate(w, "cuda")
    alpha, s0 = inputs.generate_recurrence_extras(w, "cuda")
    for flags in (0, SIMT):
        vda = binding.Vda(w.d, w.dtype, flags=flags | binding.VDN_FLAG_ADDITIVE_RULE)
        out = vda.forward(x["q"], x["k"], x["v"], x["beta"], x["gate"], alpha=alpha, s0=s0,
                          chunk=2, radius=1, anchors=True)
        torch.cuda.synchronize()
        assert vda.status() == binding.VDN_OK
        check(w, x, out, alpha, s0, rule="additive", chunk=2, radius=1, anchors=True)


def test_default_window_through_the_options_entry_is_bitwise_the_plain_call():
    w = inputs.TINY.scaled(dtype="bf16", d=128, T=6, F=260, H=2)
    x = inputs.generate(w, "cuda")
    vda = binding.Vda(w.d, w.dtype)
    a = vda.forward(x["q"], x["k"], x["v"], x["beta"], x["gate"]).clone()
    nw = torch.ones((w.H, w.d), device="cuda")
    b = vda.forward(x["q"], x["k"], x["v"], x["beta"], x["gate"], norm_weight=nw)     # forces forward_opt, extras path
    torch.cuda.synchronize()
    assert torch.equal(a, b)


def test_options_argument_errors():
    import ctypes
    w = inputs.TINY
    x = inputs.generate(w, "cuda")
    vda = binding.Vda(w.d, w.dtype)
    vda.ensure_workspace(w.B, w.T, w.F, w.H)
    p = lambda t: ctypes.c_void_p(t.data_ptr())
    out = torch.empty_like(x["q"])
    opt = binding.VdnOptions(ctypes.sizeof(binding.VdnOptions) - 4, 1, 0, 0, None, None, None, None)
    args = (vda.h, p(x["q"]), p(x["k"]), p(x["v"]), p(x["beta"]), p(x["gate"]), p(out), w.B, w.T, w.F, w.H, w.d)
    assert vda.lib.vdn_vda_forward_opt(*args, ctypes.byref(opt), None) == 1          # struct_size mismatch
    opt = binding.VdnOptions(ctypes.sizeof(binding.VdnOptions), 1, -1, 0, None, None, None, None)
    assert vda.lib.vdn_vda_forward_opt(*args, ctypes.byref(opt), None) == 1          # negative radius
    args_nogate = args[:5] + (None,) + args[6:]
    opt = binding.VdnOptions(ctypes.sizeof(binding.VdnOptions), 1, 0, 0, None, None, None, None)
    assert vda.lib.vdn_vda_forward_opt(*args_nogate, ctypes.byref(opt), None) == 1   # neither gate given
    assert vda.lib.vdn_vda_forward_opt(*args, None, None) == 0                       # NULL options = plain forward
    torch.cuda.synchronize()


# ------------------------------------------------------------------------------ chunk-wise scan (Sec. 5)
CHUNKWISE = binding.VDN_FLAG_SCAN_CHUNKWISE


@pytest.mark.parametrize("T,chunk,radius,anchors,extras", [
    (23, 5, 1, True, True),       # release setting; first and last chunk clipped by the anchors
    (23, 5, 1, True, False),      # alpha = 1, zero text state
    (20, 5, 0, False, True),      # exact chunks, no anchors
    (14, 2, 1, False, True), (17, 3, 0, True, True), (9, 4, 0, True, True),
    (12, 5, 1, True, True),       # one (clipped) chunk folded each way
    (9, 5, 1, True, True),        # no chunk is ever folded: every frame reads the text state on both sides
])
def test_chunkwise_scan_matches_oracle(T, chunk, radius, anchors, extras):
    w = inputs.TINY.scaled(dtype="bf16", d=128, B=1, H=2, T=T, F=140, seed=7 * T + chunk)
    x = inputs.generate(w, "cuda")
    alpha, s0 = inputs.generate_recurrence_extras(w, "cuda") if extras else (None, None)
    vda = binding.Vda(w.d, w.dtype, flags=CHUNKWISE)
    kw = dict(chunk=chunk, radius=radius, anchors=anchors)
    out = vda.forward(x["q"], x["k"], x["v"], x["beta"], x["gate"], alpha=alpha, s0=s0, **kw)
    torch.cuda.synchronize()
    assert vda.status() == binding.VDN_OK
    names = [n for (n, _, _) in _kernel_names(vda, x, alpha, s0, kw)]
    folds = any(orc.local_window(t, T, chunk, radius, anchors)[0] > (1 if anchors else 0) for t in range(T))
    assert ("compose_tc" in names) == folds
    check(w, x, out, alpha, s0, **kw)
    # frame by frame on the same inputs: the same result up to rounding
    vda2 = binding.Vda(w.d, w.dtype, flags=binding.VDN_FLAG_SCAN_FRAMEWISE)
    out2 = vda2.forward(x["q"], x["k"], x["v"], x["beta"], x["gate"], alpha=alpha, s0=s0, **kw)
    torch.cuda.synchronize()
    scale = out2.float().abs().amax()
    assert float((out.float() - out2.float()).abs().amax() / scale) < 2e-2


def _kernel_names(vda, x, alpha, s0, kw):
    vda.profile(True)
    vda.forward(x["q"], x["k"], x["v"], x["beta"], x["gate"], alpha=alpha, s0=s0, **kw)
    torch.cuda.synchronize()
    times = vda.kernel_times()
    vda.profile(False)
    return times


def test_chunkwise_scan_with_the_additive_rule():
    w = inputs.TINY.scaled(dtype="bf16", d=128, B=1, H=2, T=16, F=200, seed=3)
    x = inputs.generate(w, "cuda")
    alpha, s0 = inputs.generate_recurrence_extras(w, "cuda")
    vda = binding.Vda(w.d, w.dtype, flags=CHUNKWISE | binding.VDN_FLAG_ADDITIVE_RULE)
    kw = dict(chunk=3, radius=0, anchors=True)
    out = vda.forward(x["q"], x["k"], x["v"], x["beta"], x["gate"], alpha=alpha, s0=s0, **kw)
    torch.cuda.synchronize()
    assert vda.status() == binding.VDN_OK
    check(w, x, out, alpha, s0, rule="additive", **kw)


def test_chunkwise_scan_is_chosen_for_few_chains_and_needs_its_workspace():
    import ctypes
    w = inputs.TINY.scaled(dtype="bf16", d=128, B=1, H=1, T=52, F=64, seed=9)
    x = inputs.generate(w, "cuda")
    kw = dict(chunk=5, radius=1, anchors=True)
    vda = binding.Vda(w.d, w.dtype)                                   # no flag: the library decides
    assert vda.workspace_bytes(w.B, w.T, w.F, w.H, chunk=5) > vda.workspace_bytes(w.B, w.T, w.F, w.H)
    out = vda.forward(x["q"], x["k"], x["v"], x["beta"], x["gate"], **kw)
    torch.cuda.synchronize()
    assert "compose_tc" in [n for (n, _, _) in _kernel_names(vda, x, None, None, kw)]   # 2 chains, 9 chunks each way
    check(w, x, out, **kw)
    # with the plain workspace the same call scans frame by frame
    vda2 = binding.Vda(w.d, w.dtype)
    vda2.ensure_workspace(w.B, w.T, w.F, w.H)
    small = vda2._ws[: vda2.workspace_bytes(w.B, w.T, w.F, w.H)]
    vda2.lib.vdn_vda_set_workspace(vda2.h, ctypes.c_void_p(small.data_ptr()), small.numel())
    p = lambda t: ctypes.c_void_p(t.data_ptr())
    opt = binding.VdnOptions(ctypes.sizeof(binding.VdnOptions), 5, 1, 1, None, None, None, None)
    out2 = torch.empty_like(x["q"])
    vda2.profile(True)
    st = vda2.lib.vdn_vda_forward_opt(vda2.h, p(x["q"]), p(x["k"]), p(x["v"]), p(x["beta"]), p(x["gate"]), p(out2),
                                      w.B, w.T, w.F, w.H, w.d, ctypes.byref(opt), None)
    torch.cuda.synchronize()
    assert st == 0 and "scan_tc" in [n for (n, _, _) in vda2.kernel_times()]
    check(w, x, out2, **kw)
    # forcing it without the room is an error, and nothing runs
    vda3 = binding.Vda(w.d, w.dtype, flags=CHUNKWISE)
    vda3.lib.vdn_vda_set_workspace(vda3.h, ctypes.c_void_p(small.data_ptr()), small.numel())
    st = vda3.lib.vdn_vda_forward_opt(vda3.h, p(x["q"]), p(x["k"]), p(x["v"]), p(x["beta"]), p(x["gate"]), p(out2),
                                      w.B, w.T, w.F, w.H, w.d, ctypes.byref(opt), None)
    assert st == 3
    torch.cuda.synchronize()


@pytest.mark.parametrize("dtype,d", [("bf16", 128), ("f32", 64), ("f32", 128)])
def test_random_window_settings_on_every_scan_schedule(dtype, d):
    # seeded sweep over (T, chunk, radius, anchors, alpha?, s0?) on small frames: the bookkeeping of which state a
    # frame reads, where a chain may stop, and which chunks get composed, against the checker every time
    import random
    rnd = random.Random(20744)
    for trial in range(24):
        T = rnd.randint(1, 27)
        chunk = rnd.choice([1, 2, 3, 4, 5, 7])
        radius = rnd.choice([0, 0, 1, 1, 2])
        anchors = rnd.random() < 0.5
        use_alpha = rnd.random() < 0.6
        use_s0 = rnd.random() < 0.6
        flags = rnd.choice([0, binding.VDN_FLAG_SCAN_FRAMEWISE, CHUNKWISE])
        w = inputs.TINY.scaled(dtype=dtype, d=d, B=1, H=1, T=T, F=48, seed=1000 + trial)
        x = inputs.generate(w, "cuda")
        alpha, s0 = inputs.generate_recurrence_extras(w, "cuda")
        alpha = alpha if use_alpha else None
        s0 = s0 if use_s0 else None
        vda = binding.Vda(w.d, w.dtype, flags=flags)
        kw = dict(chunk=chunk, radius=radius, anchors=anchors)
        out = torch.full_like(x["q"], 9.0)
        vda.forward(x["q"], x["k"], x["v"], x["beta"], x["gate"], out=out, alpha=alpha, s0=s0, **kw)
        torch.cuda.synchronize()
        assert vda.status() == binding.VDN_OK, (trial, T, kw, flags)
        try:
            check(w, x, out, alpha, s0, **kw)
        except AssertionError as e:
            raise AssertionError(f"trial {trial}: T={T} {kw} alpha={use_alpha} s0={use_s0} flags={flags}: {e}")
        vda.close()


def test_chunk_composites_match_an_fp64_fold_of_the_same_frames():
    # Sec. 5, "Chunk-wise scans": S_out = S_in M + J per chunk.  The composites the scan leaves in the workspace (J in
    # fp32, M as three bf16 parts) against an fp64 fold of the chunk's frames from the GPU's own statistics and
    # inverses: isolates the arithmetic of the tensor-core scan (three-way bf16 splits of both fp32 factors, six
    # products, fp32 accumulation) at fp32 resolution -- the stored read states are bf16 and cannot show it.
    d = 128
    w = inputs.TINY.scaled(dtype="bf16", d=d, B=1, H=2, T=21, F=300, seed=3)
    x = inputs.generate(w, "cuda")
    vda = binding.Vda(w.d, w.dtype, flags=binding.VDN_FLAG_SCAN_CHUNKWISE)
    vda.forward(x["q"], x["k"], x["v"], x["beta"], x["gate"], chunk=5, radius=1)
    torch.cuda.synchronize()
    stats = vda.view(binding.VIEW_STATS, 1, w.T, w.F, w.H).double().cpu().numpy()[0]
    split = vda.view(binding.VIEW_INV_SPLIT, 1, w.T, w.F, w.H).double().cpu().numpy()[0]
    J = vda.view(binding.VIEW_COMP_J, 1, w.T, w.F, w.H).double().cpu().numpy()
    M = vda.view(binding.VIEW_COMP_M, 1, w.T, w.F, w.H).double().cpu().numpy()
    assert J.shape[:3] == (w.H, 2, 5) and M.shape[:4] == (w.H, 2, 5, 3)
    rel = lambda g, r: np.max(np.abs(g - r)) / np.max(np.abs(r))
    for h in range(w.H):
        for direction in (0, 1):
            for pos in range(2):                                   # the first two chunks each direction folds
                frames = range(5 * pos, 5 * pos + 5) if direction == 0 else range(w.T - 1 - 5 * pos, w.T - 2 - 5 * pos, -1) \
                    if pos == 0 else range(19 - 5 * (pos - 1), 14 - 5 * (pos - 1), -1)
                Z, Mm = np.zeros((d, d)), np.eye(d)
                for t in frames:
                    C = split[h, t].sum(0).T                       # the scan multiplies by the transpose of what is stored
                    Z = C @ (Z + stats[h, t, d:].T)
                    Mm = C @ Mm
                assert rel(J[h, direction, pos].T, Z) <= 3e-6      # measured 6e-7: about 1.3e-7 per product
                assert rel(M[h, direction, pos].sum(0), Mm) <= 6e-6   # measured 1.7e-6

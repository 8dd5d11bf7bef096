"""vdn_vda_scan_static: the frame scan for callers that must not allocate device memory.

Some users of the library run inside programs that claim all GPU memory up front and forbid (or cannot
afford) any later cudaMalloc; they cannot give vdn_vda_forward a workspace.  The entry point tested here
runs the fp32 scan + gather stage with its scratch held in an array inside the library image.  It must
give the very states the regular entry point leaves in its workspace -- and the states the fp64 checker
computes from the same inputs -- call after call (the scratch is shared and keeps the previous call's contents).  This file sorts last on purpose: a run that stops at the
first failure has then already run every other test.
"""
import ctypes

import numpy as np
import pytest
import torch

from oracle import vda_oracle as orc
from paper_2609_20744_b200 import binding, build, inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    binding.load_library()


def regular_path_states(w):
    """Run vdn_vda_forward on the plain-fp32 kernels and return its statistics, inverses and read states."""
    x = inputs.generate(w, "cuda")
    vda = binding.Vda(w.d, w.dtype, flags=binding.VDN_FLAG_FORCE_SIMT)
    vda.forward(x["q"], x["k"], x["v"], x["beta"], x["gate"])
    torch.cuda.synchronize()
    shp = (w.B, w.T, w.F, w.H)
    n = w.B * w.H
    stats = vda.view(binding.VIEW_STATS, *shp).reshape(n, w.T, 2 * w.d, w.d).clone()
    inv = vda.view(binding.VIEW_INV, *shp).reshape(n, w.T, w.d, w.d).clone()
    read = vda.view(binding.VIEW_READ, *shp).reshape(n, w.T, w.d, w.d).clone()
    return stats, inv, read, x


@pytest.mark.parametrize("kw", [dict(d=64, T=4, F=64, H=2), dict(d=128, T=7, F=90, H=3), dict(d=128, T=1, F=16, H=1)])
def test_static_scratch_scan_matches_regular_entry_point_twice_in_a_row(kw):
    w = inputs.TINY.scaled(**kw)
    stats, inv, want, x = regular_path_states(w)
    other = inputs.TINY.scaled(seed=11, **kw)
    stats2, inv2, want2, _ = regular_path_states(other)

    got = torch.full_like(want, float("nan"))
    got2 = torch.full_like(want2, float("nan"))
    binding.scan_static(stats, inv, got)          # a first call on this device may look up the array's address
    torch.cuda.synchronize()
    got.fill_(float("nan"))
    allocations_before = torch.cuda.memory_stats()["allocation.all.allocated"]   # count of allocator requests
    free_before, _ = torch.cuda.mem_get_info()    # what the driver itself reports: a cudaMalloc inside the library would show
    binding.scan_static(stats, inv, got)          # leaves its forward states in the shared scratch
    binding.scan_static(stats2, inv2, got2)       # other data: must not see the previous call's scratch
    binding.scan_static(stats, inv, got)          # and again with the first data
    torch.cuda.synchronize()
    # neither torch's allocator nor the CUDA runtime was asked for memory while the three calls ran
    assert torch.cuda.memory_stats()["allocation.all.allocated"] == allocations_before
    assert torch.cuda.mem_get_info()[0] == free_before
    # same kernel arithmetic as the regular path; the tests' f32 bar is 1e-4 of the slice maximum
    for g, wnt in ((got, want), (got2, want2)):
        assert torch.isfinite(g).all()
        scale = wnt.abs().amax().clamp_min(1e-30)
        assert float((g - wnt).abs().amax() / scale) <= 1e-4
        assert torch.equal(g, wnt)                                        # in fact bit-identical
    # and against the fp64 checker directly: slot t of the output is the transpose of P_{t-1} + R_{t+1} (Eq. A.4)
    n = 0
    for b in range(w.B):
        for h in range(w.H):
            q, k, v, beta, gate = inputs.head_slice(x, b, h)
            ref = orc.vda_slice(q, k, v, beta, gate, 1e-6, want=("P", "R"))
            for t in range(w.T):
                rd = np.zeros((w.d, w.d))
                if t > 0:
                    rd = rd + ref["P"][t - 1]
                if t + 1 < w.T:
                    rd = rd + ref["R"][t + 1]
                g = got[n, t].double().cpu().numpy().T
                assert np.max(np.abs(g - rd)) <= 1e-4 * max(np.max(np.abs(rd)), 1e-30)
            n += 1


def test_static_scratch_scan_rejects_shapes_beyond_its_limit():
    d, T = 128, 129                                                       # 129 frames x 64 KiB > 8 MiB
    stats = torch.zeros((1, T, 2 * d, d), device="cuda")
    inv = torch.zeros((1, T, d, d), device="cuda")
    read = torch.full((1, T, d, d), 3.0, device="cuda")
    with pytest.raises(binding.VdnError) as e:
        binding.scan_static(stats, inv, read)
    assert e.value.status == 3 and "VDN_SCAN_STATIC_MAX_BYTES" in str(e.value)
    torch.cuda.synchronize()
    assert torch.all(read == 3.0)                                         # nothing was enqueued
    lib = binding.load_library()
    st = lib.vdn_vda_scan_static(None, ctypes.c_void_p(inv.data_ptr()), ctypes.c_void_p(read.data_ptr()),
                                 1, 4, d, 0, None, None, 0)
    assert st == 1

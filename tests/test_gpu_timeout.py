"""A bounded device-side wait that runs out, made to happen without starving any real pipeline.

The tensor-core kernels wait on mbarriers for tiles and accumulators; every such wait gives up after a limit,
raises the CTA's abort flag, lets every role leave its loop, frees the CTA's tensor memory and records
VDN_ERR_TIMEOUT in the handle's status word.  vdn_vda_selftest_wait_expiry launches a stand-alone kernel that is
set up like those kernels and whose only wait is on a barrier nobody ever arrives at (no copy is bound to it), with
a limit of a millisecond.  The kernel must return, the status must say so, clearing it must work, and the handle
must be as good as new afterwards.
"""
import time

import pytest
import torch

from paper_2609_20744_b200 import binding, build, inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    binding.load_library()


def test_wait_expiry_sets_the_status_word_and_leaves_the_handle_usable():
    w = inputs.TINY.scaled(dtype="bf16", d=128, T=5, F=300, H=2)
    x = inputs.generate(w, "cuda")
    vda = binding.Vda(w.d, w.dtype)
    assert vda.uses_tensor_cores()
    before = vda.forward(x["q"], x["k"], x["v"], x["beta"], x["gate"]).clone()
    torch.cuda.synchronize()
    assert vda.status() == binding.VDN_OK and vda.selftest_marker() == 0

    t0 = time.perf_counter()
    vda.selftest_wait_expiry(limit_us=1000)
    torch.cuda.synchronize()                                   # returns: the kernel gave up by itself
    assert time.perf_counter() - t0 < 5.0
    # bit 0: the CTA reached its last instruction after giving up; bit 1: the warp that had waited for nothing was told
    # at the block-level barrier (the way threads of the pipeline kernels leave together)
    assert vda.selftest_marker() == 3
    assert vda.status() == binding.VDN_ERR_TIMEOUT
    assert vda.status() == binding.VDN_ERR_TIMEOUT             # sticky: reading clears nothing

    # a forward call does not clear it either (an error must not get lost between a call and the check) ...
    after = vda.forward(x["q"], x["k"], x["v"], x["beta"], x["gate"])
    torch.cuda.synchronize()
    assert vda.status() == binding.VDN_ERR_TIMEOUT
    # ... but the call itself is unaffected: tensor memory was freed, the context is intact
    assert torch.equal(after, before)

    assert vda.clear_status() == binding.VDN_ERR_TIMEOUT
    assert vda.status() == binding.VDN_OK
    again = vda.forward(x["q"], x["k"], x["v"], x["beta"], x["gate"])
    torch.cuda.synchronize()
    assert vda.status() == binding.VDN_OK
    assert torch.equal(again, before)


def test_wait_limit_is_a_property_of_the_handle():
    vda = binding.Vda(128, "bf16")
    vda.set_wait_limit_us(500_000)
    with pytest.raises(binding.VdnError):
        vda.set_wait_limit_us(0)
    with pytest.raises(binding.VdnError):
        vda.selftest_wait_expiry(limit_us=2_000_000)            # the self-test never waits longer than a second
    w = inputs.TINY.scaled(dtype="bf16", d=128, T=3, F=130, H=1)
    x = inputs.generate(w, "cuda")
    vda.forward(x["q"], x["k"], x["v"], x["beta"], x["gate"])
    torch.cuda.synchronize()
    assert vda.status() == binding.VDN_OK


def test_other_handles_do_not_see_the_timeout():
    a, b = binding.Vda(128, "bf16"), binding.Vda(128, "bf16")
    a.selftest_wait_expiry(limit_us=200)
    torch.cuda.synchronize()
    assert a.status() == binding.VDN_ERR_TIMEOUT and b.status() == binding.VDN_OK
    a.clear_status()

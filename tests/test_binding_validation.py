"""The Python binding refuses tensors whose dtype, shape, device or layout differ from what the C ABI will assume.

The library receives bare pointers and indexes them by the shape it is told, so a tensor of the wrong dtype or a
short gate vector would be read -- and `out` written -- past its end.  These checks run before any ctypes call;
here they are exercised without a GPU (host tensors stand for the host-buffer entry point, and a host tensor
handed to a device entry point is itself one of the refused cases).
"""
import pytest
import torch

from paper_2609_20744_b200 import binding

B, T, F, H, d = 2, 3, 5, 2, 64


def good(dtype=torch.bfloat16):
    return dict(q=torch.zeros(B, T, F, H, d, dtype=dtype), k=torch.zeros(B, T, F, H, d, dtype=dtype),
                v=torch.zeros(B, T, F, H, d, dtype=dtype), beta=torch.zeros(B, T, F, H), gate=torch.zeros(H))


def check(x, **kw):
    io = kw.pop("io", torch.bfloat16)
    return binding.validate_layer_args(io, d, 0, x["q"], x["k"], x["v"], x["beta"], x["gate"], on_cuda=False, **kw)


def test_matching_host_tensors_pass_and_give_the_shape():
    assert check(good()) == (B, T, F, H, d)
    assert check(good(torch.float32), io=torch.float32) == (B, T, F, H, d)


@pytest.mark.parametrize("name,bad", [
    ("q", lambda x: x["q"].float()),                                  # f32 tensor on a bf16 handle
    ("k", lambda x: x["k"][:, :, :-1].contiguous()),                  # one token short
    ("v", lambda x: x["v"].transpose(1, 2)),                          # not contiguous (and the wrong shape)
    ("beta", lambda x: x["beta"].bfloat16()),                         # a 16-bit write gate
    ("beta", lambda x: x["beta"][..., :1].contiguous()),              # one head only
    ("gate", lambda x: x["gate"][:1].contiguous()),                   # short gate vector
    ("gate", lambda x: x["gate"].double()),
])
def test_mismatched_tensor_is_refused(name, bad):
    x = good()
    x[name] = bad(x)
    with pytest.raises(ValueError, match=name):
        check(x)


def test_optional_tensors_are_checked_too():
    x = good()
    ok = dict(out=torch.zeros(B, T, F, H, d, dtype=torch.bfloat16), alpha=torch.zeros(B, T, H, d),
              s0=torch.zeros(B, H, d, d), gate_elem=torch.zeros(B, T, F, H, d, dtype=torch.bfloat16),
              norm_weight=torch.zeros(H, d))
    assert check(x, **ok) == (B, T, F, H, d)
    for name, bad in [("out", ok["out"].float()), ("out", ok["out"][:1].contiguous()), ("alpha", ok["alpha"].bfloat16()),
                      ("alpha", torch.zeros(B, T, H)), ("s0", torch.zeros(B, H, d)), ("gate_elem", ok["gate_elem"].float()),
                      ("norm_weight", torch.zeros(d))]:
        with pytest.raises(ValueError, match=name):
            check(x, **{**ok, name: bad})


def test_gate_may_only_be_missing_with_an_elementwise_gate():
    x = good()
    x["gate"] = None
    with pytest.raises(ValueError, match="gate"):
        check(x)
    assert check(x, gate_elem=torch.zeros(B, T, F, H, d, dtype=torch.bfloat16)) == (B, T, F, H, d)


def test_host_tensor_is_refused_by_a_device_entry_point_and_nothing_is_called():
    # on_cuda=True is what Vda.forward and Vda.prepare ask for; the check needs no GPU to say no
    x = good()
    with pytest.raises(ValueError, match="CUDA"):
        binding.validate_layer_args(torch.bfloat16, d, 0, x["q"], x["k"], x["v"], x["beta"], x["gate"])
    with pytest.raises(ValueError, match="shape"):
        binding.validate_layer_args(torch.bfloat16, d, 0, x["q"][0], x["k"], x["v"], x["beta"], x["gate"])

"""The seeded workload generator: shapes, distributions, determinism (CPU)."""
import numpy as np
import torch

from paper_2609_20744_b200 import inputs


def test_tiny_shapes_and_distributions():
    w = inputs.TINY
    x = inputs.generate(w)
    assert x["q"].shape == (1, 4, 64, 2, 64) and x["q"].dtype == torch.float32
    assert x["beta"].shape == (1, 4, 64, 2) and x["gate"].shape == (2,)
    assert torch.allclose(x["k"].norm(dim=-1), torch.ones(1, 4, 64, 2), atol=1e-5)
    assert torch.allclose(x["q"].norm(dim=-1), torch.ones(1, 4, 64, 2), atol=1e-5)
    assert float(x["beta"].min()) > 0 and float(x["beta"].max()) < 1
    assert float(x["gate"].min()) > 0 and float(x["gate"].max()) < 1
    assert abs(float(x["v"].mean())) < 0.05 and abs(float(x["v"].std()) - 1) < 0.05


def test_generation_is_deterministic_and_seed_dependent():
    w = inputs.TINY
    a, b = inputs.generate(w), inputs.generate(w)
    for n in a:
        assert torch.equal(a[n], b[n])
    c = inputs.generate(w.scaled(seed=9))
    assert not torch.equal(a["k"], c["k"])


def test_correlated_key_structure_of_768p_recipe():
    w = inputs.CLIP_768P.scaled(H=2, T=2, F=2000)
    x = inputs.generate(w)
    assert x["k"].dtype == torch.bfloat16
    k = x["k"][0, 0, :, 0, :].double().numpy()                # one frame, one head
    assert np.allclose(np.linalg.norm(k, axis=1), 1.0, atol=1e-2)   # bf16 rounding of unit vectors
    lam = np.linalg.eigvalsh(k.T @ k)
    # ~30% of 2000 keys sit near 8 shared directions: 8 dominant eigenvalues near 600/8, rest near 1400/128
    assert lam[-8] > 40 and lam[-9] < 25
    # beta = sigmoid(1.5 N(0,1)) is wider than sigmoid(N(0,1))
    assert float(x["beta"].std()) > 0.26
    # shared directions persist across frames of the same head
    k1 = x["k"][0, 1, :, 0, :].double().numpy()
    top0 = np.linalg.eigh(k.T @ k)[1][:, -8:]
    top1 = np.linalg.eigh(k1.T @ k1)[1][:, -8:]
    assert np.linalg.svd(top0.T @ top1, compute_uv=False).min() > 0.9


def test_head_slice_is_exact_copy():
    w = inputs.TINY.scaled(dtype="bf16")
    x = inputs.generate(w)
    q, k, v, beta, gate = inputs.head_slice(x, 0, 1)
    assert q.dtype == np.float64 and q.shape == (4, 64, 64)
    assert np.array_equal(k, x["k"][0, :, :, 1, :].double().numpy())
    assert gate == float(x["gate"][1])


def test_degenerate_recipes_do_what_they_say_and_leave_the_default_streams_alone():
    base = inputs.TINY.scaled(H=2, T=3, F=40, d=64)
    x0 = inputs.generate(base, "cpu")
    # repeated keys: one vector per (batch, frame, head)
    x = inputs.generate(base.scaled(key_repeat_frac=1.0), "cpu")
    k = x["k"]
    assert torch.equal(k, k[:, :, :1].expand_as(k))
    assert not torch.equal(k[0, 0, 0, 0], k[0, 1, 0, 0]) and not torch.equal(k[0, 0, 0, 0], k[0, 0, 0, 1])
    assert torch.allclose(k.norm(dim=-1), torch.ones(k.shape[:-1]), atol=1e-5)
    for n in ("q", "v", "beta", "gate"):
        assert torch.equal(x[n], x0[n])                       # the extra draws come after the default ones
    # partly repeated keys
    x = inputs.generate(base.scaled(key_repeat_frac=0.5, F=400), "cpu")
    k = x["k"][0, 0, :, 0]
    same = (k == k.mode(dim=0).values).all(dim=-1).float().mean()
    assert 0.35 < float(same) < 0.65
    # key norms
    x = inputs.generate(base.scaled(key_norm_lo=0.25, key_norm_hi=4.0, F=500), "cpu")
    n = x["k"].norm(dim=-1)
    assert float(n.min()) >= 0.25 * (1 - 1e-5) and float(n.max()) <= 4.0 * (1 + 1e-5) and float(n.std()) > 0.5
    # write gates
    x = inputs.generate(base.scaled(zero_beta_frames=(1,)), "cpu")
    assert torch.count_nonzero(x["beta"][:, 1]) == 0 and torch.equal(x["beta"][:, 0], x0["beta"][:, 0])
    x = inputs.generate(base.scaled(beta_const=0.3), "cpu")
    assert torch.all(x["beta"] == 0.3)

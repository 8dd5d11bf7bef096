"""Pins for the fp64 checker: what the paper and the mathematics fix, independent of the checker.

Every test here would fail for at least one plausible mistake in `oracle/vda_oracle.py`
(dropped term, wrong sign, transposed operand, off-by-one read index, inclusive window).
"""
import json
import os

import numpy as np
import pytest

from oracle import vda_oracle as orc
from tests.bruteforce import lstsq_frame_update, softmax_sees, vda_bruteforce, vda_bruteforce_windowed

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "worked_examples.json")


def rng(seed):
    return np.random.default_rng(seed)


def unit(x):
    return x / np.linalg.norm(x, axis=-1, keepdims=True)


def random_frame(r, U, dk, dv):
    K = unit(r.standard_normal((U, dk)))
    V = r.standard_normal((U, dv))
    beta = 1.0 / (1.0 + np.exp(-r.standard_normal(U)))
    return K, V, beta


# ---------------------------------------------------------------- Eq. 3b
def test_statistics_match_literal_token_sums():
    r = rng(1)
    K, V, beta = random_frame(r, 7, 5, 3)
    A, B = orc.frame_statistics(K, V, beta)
    A_ref = np.zeros((5, 5))
    B_ref = np.zeros((3, 5))
    for u in range(7):
        for i in range(5):
            for j in range(5):
                A_ref[i, j] += beta[u] * K[u, i] * K[u, j]
        for c in range(3):
            for j in range(5):
                B_ref[c, j] += beta[u] * V[u, c] * K[u, j]
    assert np.allclose(A, A_ref, atol=1e-14)
    assert np.allclose(B, B_ref, atol=1e-14)
    assert A.shape == (5, 5) and B.shape == (3, 5)          # d_k x d_k and d_v x d_k


def test_invariant_a_token_permutation_within_frame():
    r = rng(2)
    K, V, beta = random_frame(r, 33, 8, 8)
    S_prev = r.standard_normal((8, 8))
    alpha = r.uniform(0, 1, 8)
    A, B = orc.frame_statistics(K, V, beta)
    p = r.permutation(33)
    A2, B2 = orc.frame_statistics(K[p], V[p], beta[p])
    assert np.allclose(A, A2, atol=1e-13) and np.allclose(B, B2, atol=1e-13)
    S1 = orc.frame_update(S_prev, alpha, A, B)
    S2 = orc.frame_update(S_prev, alpha, A2, B2)
    assert np.allclose(S1, S2, atol=1e-13)


# ---------------------------------------------------------------- Eq. 4 / Eq. 5
@pytest.mark.parametrize("U,dk,dv", [(1, 4, 4), (3, 4, 6), (9, 6, 3), (40, 8, 8)])
def test_update_is_least_squares_minimiser_of_joint_objective(U, dk, dv):
    r = rng(10 + U)
    K, V, beta = random_frame(r, U, dk, dv)
    K = K * r.uniform(0.5, 2.0, (U, 1))                      # no unit-norm assumption
    S_prev = r.standard_normal((dv, dk))
    alpha = r.uniform(0, 1, dk)
    A, B = orc.frame_statistics(K, V, beta)
    S = orc.frame_update(S_prev, alpha, A, B)
    S_ls = lstsq_frame_update(S_prev * alpha[None, :], K, V, beta)
    assert np.allclose(S, S_ls, atol=1e-12)

    # objective value cannot be lowered by perturbing S (strict convexity)
    def J(Sx):
        Sb = S_prev * alpha[None, :]
        return 0.5 * np.sum((Sx - Sb) ** 2) + 0.5 * np.sum(beta * np.sum((K @ Sx.T - V) ** 2, axis=1))
    for _ in range(5):
        assert J(S + 1e-3 * r.standard_normal(S.shape)) > J(S)


def test_first_order_condition_and_affine_split():
    r = rng(3)
    K, V, beta = random_frame(r, 20, 6, 5)
    S_prev = r.standard_normal((5, 6))
    alpha = r.uniform(0, 1, 6)
    A, B = orc.frame_statistics(K, V, beta)
    S = orc.frame_update(S_prev, alpha, A, B)
    S_bar = S_prev * alpha[None, :]
    # S_t = S_bar + sum_u beta_u (v_u - S_t k_u) k_u^T      (Sec. A.3)
    rhs = S_bar.copy()
    for u in range(20):
        rhs += beta[u] * np.outer(V[u] - S @ K[u], K[u])
    assert np.allclose(S, rhs, atol=1e-13)
    # S_t = S_{t-1} M_t + J_t                                (Eq. A.1)
    assert np.allclose(S, S_prev @ orc.transition(A, alpha) + orc.injection(A, B), atol=1e-13)
    # C_t really is the inverse
    assert np.allclose(orc.resolve(A) @ (np.eye(6) + A), np.eye(6), atol=1e-13)


def test_token_space_woodbury_form():
    r = rng(4)
    K, V, beta = random_frame(r, 5, 9, 4)                    # fewer tokens than channels
    S_bar = r.standard_normal((4, 9))
    A, B = orc.frame_statistics(K, V, beta)
    S = orc.frame_update(S_bar, np.ones(9), A, B)
    resid = V - K @ S_bar.T                                  # U x d_v residuals at the entering state
    W = np.linalg.solve(np.diag(1.0 / beta) + K @ K.T, resid)
    assert np.allclose(S, S_bar + (K.T @ W).T, atol=1e-12)


def test_single_token_frame_is_the_token_delta_rule():
    # Eq. 2 with the implicit (joint) step: beta_eff = beta / (1 + beta |k|^2)
    r = rng(5)
    k = r.standard_normal(6)
    v = r.standard_normal(4)
    beta = 0.7
    alpha = r.uniform(0, 1, 6)
    S_prev = r.standard_normal((4, 6))
    A, B = orc.frame_statistics(k[None], v[None], np.array([beta]))
    S = orc.frame_update(S_prev, alpha, A, B)
    S_bar = S_prev * alpha[None, :]
    be = beta / (1.0 + beta * k @ k)
    assert np.allclose(S, S_bar + be * np.outer(v - S_bar @ k, k), atol=1e-13)


def test_small_beta_limit_is_the_additive_batch_update():
    # Eq. 3c: S_bar (I - A) + B, reached to first order in beta
    r = rng(6)
    K, V, _ = random_frame(r, 12, 5, 5)
    S_bar = r.standard_normal((5, 5))
    errs = []
    for scale in (1e-3, 1e-4):
        beta = scale * r.uniform(0.5, 1.0, 12)
        A, B = orc.frame_statistics(K, V, beta)
        S = orc.frame_update(S_bar, np.ones(5), A, B)
        errs.append(np.max(np.abs(S - (S_bar @ (np.eye(5) - A) + B))))
    assert errs[0] < 1e-4 and errs[1] < errs[0] * 2e-2        # O(beta^2)


def test_zero_write_gate_passes_decayed_state_through():
    r = rng(7)
    K, V, _ = random_frame(r, 6, 4, 4)
    S_prev = r.standard_normal((4, 4))
    alpha = r.uniform(0, 1, 4)
    A, B = orc.frame_statistics(K, V, np.zeros(6))
    assert np.array_equal(orc.frame_update(S_prev, alpha, A, B), S_prev * alpha[None, :])


# ---------------------------------------------------------------- Eq. 3a / 3c: the additive baseline
def test_additive_rule_is_the_literal_frozen_state_sum_with_scaled_keys():
    r = rng(40)
    U, dk, dv = 9, 5, 4
    K, V, beta = random_frame(r, U, dk, dv)
    S_prev = r.standard_normal((dv, dk))
    alpha = r.uniform(0, 1, dk)
    A, B = orc.frame_statistics(K, V, beta)
    S = orc.frame_update_additive(S_prev, alpha, A, B, U)
    S_bar = S_prev * alpha[None, :]
    want = S_bar.copy()                                          # Eq. 3a with k -> k / sqrt(U)
    for u in range(U):
        ks = K[u] / np.sqrt(U)
        want += beta[u] * np.outer(V[u] - S_bar @ ks, ks)
    assert np.allclose(S, want, atol=1e-13)
    # Eq. 3c written with the scaled statistics
    assert np.allclose(S, S_bar @ (np.eye(dk) - A / U) + B / np.sqrt(U), atol=1e-13)


def test_additive_rule_scaled_transition_is_non_expansive_for_unit_keys():
    r = rng(41)
    for U in (1, 7, 200):
        K = unit(r.standard_normal((U, 8)))
        if U > 1:
            K[: U // 2] = unit(K[0] + 0.01 * r.standard_normal((U // 2, 8)))      # aligned keys: the worst case
        beta = r.uniform(0, 1, U)
        A, _ = orc.frame_statistics(K, np.zeros((U, 8)), beta)
        assert np.linalg.norm(np.eye(8) - A / U, 2) <= 1.0 + 1e-12               # Sec. A.3
    # without the scale the factor I - A does leave [-1, 1] for aligned keys
    assert np.linalg.norm(np.eye(8) - A, 2) > 1.0


def test_additive_whole_layer_matches_literal_loops():
    r = rng(42)
    T, U, d = 4, 6, 5
    q, k, v, beta = random_slice(r, T, U, d, d)
    alpha = r.uniform(0.3, 1, (T, d))
    s0 = r.standard_normal((d, d))
    res = orc.vda_slice(q, k, v, beta, 0.7, 1e-6, alpha, s0, want=("P", "R", "O"), rule="additive")
    def fold(S, t):
        Sb = S * alpha[t][None, :]
        out = Sb.copy()
        for u in range(U):
            ks = k[t, u] / np.sqrt(U)
            out += beta[t, u] * np.outer(v[t, u] - Sb @ ks, ks)
        return out
    S = 0.5 * s0
    for t in range(T):
        S = fold(S, t)
        assert np.allclose(res["P"][t], S, atol=1e-12)
    S = 0.5 * s0
    for t in range(T - 1, -1, -1):
        S = fold(S, t)
        assert np.allclose(res["R"][t], S, atol=1e-12)
    t = 2
    want = (res["P"][t - 1] + res["R"][t + 1]) * alpha[t][None, :]
    assert np.allclose(res["O"][t], q[t] @ want.T, atol=1e-12)


# ---------------------------------------------------------------- golden worked examples
def golden():
    with open(GOLDEN) as f:
        return json.load(f)


@pytest.mark.parametrize("case", ["repeated_key", "orthonormal_keys"])
def test_golden_single_frame(case):
    g = golden()[case]
    A, B = orc.frame_statistics(np.array(g["k"], float), np.array(g["v"], float), np.array(g["beta"], float))
    S = orc.frame_update(np.array(g["S_bar"], float), np.ones(2), A, B)
    assert np.allclose(S, np.array(g["S_t"], float), atol=1e-14)


def test_repeated_key_closed_form_random():
    # Eq. A.3 on random data
    r = rng(8)
    d, U, beta = 7, 11, 0.37
    k = unit(r.standard_normal(d))
    V = r.standard_normal((U, d))
    S_bar = r.standard_normal((d, d))
    A, B = orc.frame_statistics(np.tile(k, (U, 1)), V, np.full(U, beta))
    S = orc.frame_update(S_bar, np.ones(d), A, B)
    want = (S_bar @ k) / (1 + U * beta) + (U * beta) / (1 + U * beta) * V.mean(axis=0)
    assert np.allclose(S @ k, want, atol=1e-13)


@pytest.mark.parametrize("case", ["two_frames_whole_layer", "three_frames_decay_text",
                                  "six_frames_chunk_window_anchors"])
def test_golden_whole_layer(case):
    g = golden()[case]
    arr = lambda n: np.array(g[n], float)
    res = orc.vda_slice(arr("q"), arr("k"), arr("v"), arr("beta"), g["gate"], g["eps"],
                        alpha=arr("alpha") if "alpha" in g else None,
                        s0=arr("s0") if "s0" in g else None, want=("P", "R", "O"),
                        chunk=g.get("chunk", 1), radius=g.get("radius", 0), anchors=g.get("anchors", False))
    assert np.allclose(res["P"], arr("P"), atol=1e-14)
    assert np.allclose(res["R"], arr("R"), atol=1e-14)
    if "O" in g:
        assert np.allclose(res["O"], arr("O"), atol=1e-14)
    assert np.allclose(res["out"], arr("out"), atol=1e-12)


# ---------------------------------------------------------------- Proposition 1
@pytest.mark.parametrize("seed", range(6))
def test_invariant_b_transition_is_non_expansive(seed):
    r = rng(100 + seed)
    d = 16
    U = [1, 4, 16, 64, 300, 1000][seed]
    K = r.standard_normal((U, d)) * r.uniform(0.1, 3.0)       # not unit norm on purpose
    if seed % 2:
        K[: U // 2] = K[0] + 0.01 * r.standard_normal((U // 2, d))   # strongly correlated writes
    beta = r.uniform(0, 1, U) * (10.0 if seed == 5 else 1.0)
    alpha = r.uniform(0, 1, d)
    A, _ = orc.frame_statistics(K, np.zeros((U, d)), beta)
    M = orc.transition(A, alpha)
    assert np.linalg.norm(M, 2) <= 1.0 + 1e-12
    ev = np.linalg.eigvalsh(orc.resolve(A))
    assert ev.min() > 0 and ev.max() <= 1 + 1e-12
    # the additive rule of Eq. 3c is expansive once lambda_max(A) > 2 (Sec. A.3)
    if np.linalg.eigvalsh(A).max() > 2.0:
        assert np.linalg.norm(np.eye(d) - A, 2) > 1.0


# ---------------------------------------------------------------- scans, gather, read-out
def random_slice(r, T, U, dk, dv):
    q = unit(r.standard_normal((T, U, dk)))
    k = unit(r.standard_normal((T, U, dk)))
    v = r.standard_normal((T, U, dv))
    beta = 1.0 / (1.0 + np.exp(-r.standard_normal((T, U))))
    return q, k, v, beta


def test_invariant_c_frame_reversal_swaps_directions():
    r = rng(20)
    T, U, d = 5, 9, 6
    q, k, v, beta = random_slice(r, T, U, d, d)
    alpha = r.uniform(0.3, 1, (T, d))
    s0 = r.standard_normal((d, d))
    a = orc.vda_slice(q, k, v, beta, 0.8, 1e-6, alpha, s0, want=("o_fwd", "o_bwd", "P", "R"))
    b = orc.vda_slice(q[::-1], k[::-1], v[::-1], beta[::-1], 0.8, 1e-6, alpha[::-1], s0,
                      want=("o_fwd", "o_bwd", "P", "R"))
    assert np.allclose(a["o_fwd"], b["o_bwd"][::-1], atol=1e-13)
    assert np.allclose(a["o_bwd"], b["o_fwd"][::-1], atol=1e-13)
    assert np.allclose(a["P"], b["R"][::-1], atol=1e-13)
    assert np.allclose(a["out"], b["out"][::-1], atol=1e-12)
    assert not np.allclose(a["o_fwd"], a["o_bwd"])            # the swap is not vacuous


def test_disjoint_regions_by_linearity_in_values():
    # Only frame j writes a value: forward read-outs see it for t > j, reverse ones for t < j,
    # frame j itself never does (each frame is counted at most once, Sec. 2.2).
    r = rng(21)
    T, U, d, j = 6, 5, 4, 2
    q, k, v, beta = random_slice(r, T, U, d, d)
    v0 = np.zeros_like(v)
    v0[j] = v[j]
    res = orc.vda_slice(q, k, v0, beta, 1.0, 1e-6, want=("o_fwd", "o_bwd"))
    for t in range(T):
        f = np.abs(res["o_fwd"][t]).max()
        b = np.abs(res["o_bwd"][t]).max()
        assert (f > 1e-8) == (t > j)
        assert (b > 1e-8) == (t < j)


def test_single_frame_clip_reads_nothing():
    r = rng(22)
    q, k, v, beta = random_slice(r, 1, 8, 4, 4)
    res = orc.vda_slice(q, k, v, beta, 0.9, 1e-6)
    assert np.array_equal(res["out"], np.zeros_like(res["out"]))


def test_text_state_is_counted_once():
    # Eq. 1b: with no video writes (beta = 0) and alpha = 1 every query reads exactly S_T q
    r = rng(23)
    T, U, d = 3, 4, 5
    q, k, v, _ = random_slice(r, T, U, d, d)
    s0 = r.standard_normal((d, d))
    res = orc.vda_slice(q, k, v, np.zeros((T, U)), 1.0, 0.0, None, s0, want=("O",))
    assert np.allclose(res["O"], q @ s0.T, atol=1e-13)


def test_rmsnorm_gate_identities():
    r = rng(24)
    O = r.standard_normal((3, 7, 16)) * r.uniform(0.01, 10, (3, 7, 1))
    eps, g = 1e-6, 0.37
    y = orc.rmsnorm_gate(O, g, eps)
    ms = np.mean(O * O, axis=-1)
    assert np.allclose(np.mean(y * y, axis=-1), g * g * ms / (ms + eps), rtol=1e-12)
    assert np.allclose(orc.rmsnorm_gate(5.0 * O, g, 0.0), orc.rmsnorm_gate(O, g, 0.0), atol=1e-13)
    assert np.array_equal(orc.rmsnorm_gate(np.zeros((2, 4)), g, eps), np.zeros((2, 4)))
    # norm is over channels only: one row must not influence another
    O2 = O.copy()
    O2[0, 0] *= 100.0
    assert np.array_equal(orc.rmsnorm_gate(O2, g, eps)[1:], y[1:])


def test_rotation_covariance():
    r = rng(25)
    T, U, d = 4, 6, 5
    q, k, v, beta = random_slice(r, T, U, d, d)
    Qk, _ = np.linalg.qr(r.standard_normal((d, d)))
    Qv, _ = np.linalg.qr(r.standard_normal((d, d)))
    a = orc.vda_slice(q, k, v, beta, 1.0, 1e-9)["out"]
    b = orc.vda_slice(q @ Qk, k @ Qk, v, beta, 1.0, 1e-9)["out"]
    c = orc.vda_slice(q, k, v @ Qv, beta, 1.0, 1e-9)["out"]
    assert np.allclose(a, b, atol=1e-12)
    assert np.allclose(a @ Qv, c, atol=1e-12)


@pytest.mark.parametrize("T,U,dk,dv,extras", [
    (1, 3, 4, 4, False), (2, 1, 4, 4, False), (3, 7, 4, 4, True),
    (5, 3, 8, 8, True), (4, 5, 6, 3, True), (2, 4, 3, 5, False)])
def test_invariant_d_bruteforce_agreement(T, U, dk, dv, extras):
    r = rng(1000 + 10 * T + U)
    q, k, v, beta = random_slice(r, T, U, dk, dv)
    alpha = r.uniform(0.2, 1, (T, dk)) if extras else None
    s0 = r.standard_normal((dv, dk)) if extras else None
    res = orc.vda_slice(q, k, v, beta, 0.6, 1e-6, alpha, s0, want=("o_fwd", "o_bwd"))
    out, of, ob = vda_bruteforce(q, k, v, beta, 0.6, 1e-6, alpha, s0)
    assert np.allclose(res["o_fwd"], of, atol=1e-12)
    assert np.allclose(res["o_bwd"], ob, atol=1e-12)
    assert np.allclose(res["out"], out, atol=1e-11)


# ---------------------------------------------------------------- chunk windows, anchors (Sec. 2.1, Sec. A.4)
@pytest.mark.parametrize("T,chunk,radius,anchors", [
    (6, 2, 0, True), (7, 2, 1, False), (11, 3, 1, True), (10, 5, 0, True), (9, 1, 1, False), (5, 1, 0, True),
    (4, 5, 1, True), (3, 1, 0, True), (2, 1, 0, True), (12, 2, 2, True), (6, 1, 0, False)])
def test_windowed_layer_matches_mask_driven_bruteforce(T, chunk, radius, anchors):
    r = rng(2000 + 100 * T + 10 * chunk + radius)
    U, dk, dv = 3, 4, 3
    q, k, v, beta = random_slice(r, T, U, dk, dv)
    alpha = r.uniform(0.2, 1, (T, dk))
    s0 = r.standard_normal((dv, dk))
    gate = r.uniform(0.1, 1, (T, U, dv))
    w = r.uniform(0.5, 2, dv)
    res = orc.vda_slice(q, k, v, beta, gate, 1e-6, alpha, s0, want=("o_fwd", "o_bwd"),
                        chunk=chunk, radius=radius, anchors=anchors, norm_weight=w)
    out, of, ob = vda_bruteforce_windowed(q, k, v, beta, gate, 1e-6, alpha, s0, chunk, radius, anchors, w)
    assert np.allclose(res["o_fwd"], of, atol=1e-12)
    assert np.allclose(res["o_bwd"], ob, atol=1e-12)
    assert np.allclose(res["out"], out, atol=1e-11)
    if anchors:
        assert np.array_equal(res["out"][0], np.zeros((U, dv)))
        assert np.array_equal(res["out"][T - 1], np.zeros((U, dv)))


def test_window_bounds_are_the_clipped_chunk_neighbourhood():
    for T, chunk, radius, anchors in [(12, 5, 1, True), (17, 5, 1, False), (9, 2, 0, True), (8, 3, 2, False)]:
        first, last = orc.interior_range(T, anchors)
        for t in range(first, last + 1):
            lo, hi = orc.local_window(t, T, chunk, radius, anchors)
            seen = [j for j in range(first, last + 1) if softmax_sees(t, j, T, chunk, radius, False)]
            assert (lo, hi) == (seen[0], seen[-1]) and seen == list(range(lo, hi + 1))
    # the 15-frame window of Sec. 2.1: chunk 5, radius 1, away from the ends of the clip
    assert orc.local_window(52, 102, 5, 1, True) == (45, 59)
    assert orc.local_window(3, 102, 5, 1, True) == (1, 9)
    assert orc.local_window(99, 102, 5, 1, True) == (90, 100)


def test_windowed_regions_are_disjoint_and_complete_by_linearity_in_values():
    # Only frame j writes a value.  Queries of frame t see it through the forward state iff j lies before t's
    # window, through the reverse state iff it lies after it, and not at all when Softmax sees it (inside the
    # window, or an anchor): no frame is counted twice and none is lost (Sec. 2.2).
    r = rng(2100)
    T, U, d, chunk, radius = 11, 3, 4, 2, 1
    q, k, v, beta = random_slice(r, T, U, d, d)
    alpha = r.uniform(0.5, 1, (T, d))
    for j in range(T):
        v0 = np.zeros_like(v)
        v0[j] = v[j]
        res = orc.vda_slice(q, k, v0, beta, 1.0, 1e-6, alpha, want=("o_fwd", "o_bwd"),
                            chunk=chunk, radius=radius, anchors=True)
        for t in range(T):
            f = np.abs(res["o_fwd"][t]).max() > 1e-9
            b = np.abs(res["o_bwd"][t]).max() > 1e-9
            linear = t not in (0, T - 1) and not softmax_sees(t, j, T, chunk, radius, True)
            assert f == (linear and j < t)
            assert b == (linear and j > t)


def test_window_of_one_frame_without_anchors_is_the_default_layer():
    r = rng(2200)
    q, k, v, beta = random_slice(r, 5, 4, 4, 4)
    alpha = r.uniform(0.2, 1, (5, 4))
    a = orc.vda_slice(q, k, v, beta, 0.5, 1e-6, alpha)["out"]
    b = orc.vda_slice(q, k, v, beta, 0.5, 1e-6, alpha, chunk=1, radius=0, anchors=False)["out"]
    assert np.array_equal(a, b)


def test_windowed_frame_reversal_swaps_directions():
    # chunk grids line up under reversal when T is a multiple of the chunk length
    r = rng(2300)
    T, U, d = 8, 3, 4
    q, k, v, beta = random_slice(r, T, U, d, d)
    alpha = r.uniform(0.3, 1, (T, d))
    s0 = r.standard_normal((d, d))
    kw = dict(want=("o_fwd", "o_bwd"), chunk=2, radius=1, anchors=True)
    a = orc.vda_slice(q, k, v, beta, 0.8, 1e-6, alpha, s0, **kw)
    b = orc.vda_slice(q[::-1], k[::-1], v[::-1], beta[::-1], 0.8, 1e-6, alpha[::-1], s0, **kw)
    assert np.allclose(a["o_fwd"], b["o_bwd"][::-1], atol=1e-13)
    assert np.allclose(a["out"], b["out"][::-1], atol=1e-12)


def test_elementwise_gate_and_norm_weight_literal():
    # Eq. 1c with a content-dependent gate (one value per token and channel) and a per-channel norm scale
    r = rng(2400)
    O = r.standard_normal((2, 3, 5))
    g = r.uniform(0, 1, (2, 3, 5))
    w = r.uniform(0.5, 2, 5)
    y = orc.rmsnorm_gate(O, g, 1e-3, w)
    for t in range(2):
        for u in range(3):
            ms = sum(O[t, u, c] ** 2 for c in range(5)) / 5
            for c in range(5):
                assert abs(y[t, u, c] - g[t, u, c] * w[c] * O[t, u, c] / np.sqrt(ms + 1e-3)) < 1e-14


def test_boundary_layout_wrapper_matches_slices():
    r = rng(30)
    B, T, U, H, d = 2, 3, 4, 3, 4
    q = unit(r.standard_normal((B, T, U, H, d)))
    k = unit(r.standard_normal((B, T, U, H, d)))
    v = r.standard_normal((B, T, U, H, d))
    beta = r.uniform(0, 1, (B, T, U, H))
    gate = r.uniform(0.1, 1, H)
    out = orc.vda_forward(q, k, v, beta, gate, 1e-6)
    for b in range(B):
        for h in range(H):
            want, _, _ = vda_bruteforce(q[b, :, :, h], k[b, :, :, h], v[b, :, :, h], beta[b, :, :, h],
                                        gate[h], 1e-6)
            assert np.allclose(out[b, :, :, h], want, atol=1e-11)


def test_slice_error_metric():
    want = np.array([0.0, 2.0, -4.0])
    assert orc.slice_error(want, want) == 0.0
    assert abs(orc.slice_error(want + np.array([0.04, 0, 0]), want) - 0.01) < 1e-15

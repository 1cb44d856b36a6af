"""Pins for the oracle's unit operations: closed forms, hand-computed values, special cases
and brute force -- chosen so that a dropped term, a wrong sign or index, or a transposed
operand in oracle/dbt_oracle.c fails at least one of them.  None of the expected values
comes from the oracle itself."""
import itertools
import math

import numpy as np
import pytest
import torch

import oracle


# ---- RMSNorm(v; g) = g * v / sqrt(mean(v^2) + eps)  (Eq. embeddings) --------------------

def test_rmsnorm_hand_value():
    # mean([9,16]) = 12.5 ; 3/sqrt(12.5), 4/sqrt(12.5)
    y = oracle.rmsnorm([3.0, 4.0], [1.0, 1.0], 0.0)
    np.testing.assert_allclose(y, [0.848528137, 1.131370850], rtol=1e-6)


def test_rmsnorm_gain_and_eps():
    # constant vector c: y = g * c / sqrt(c^2 + eps)
    y = oracle.rmsnorm([2.0] * 8, np.arange(1, 9), 5.0)
    np.testing.assert_allclose(y, np.arange(1, 9) * 2.0 / 3.0, rtol=1e-6)


def test_rmsnorm_scale_invariant_and_unit_rms():
    rng = np.random.default_rng(0)
    x = rng.standard_normal(64).astype(np.float32)
    y1 = oracle.rmsnorm(x, np.ones(64), 0.0)
    y2 = oracle.rmsnorm(7.5 * x, np.ones(64), 0.0)
    np.testing.assert_allclose(y1, y2, rtol=1e-6)
    assert abs(float(np.mean(y1.astype(np.float64) ** 2)) - 1.0) < 1e-6


# ---- linear: Y = X W^T with W stored [out, in] ------------------------------------------

def test_linear_matches_float64_matmul_fp32_and_orientation():
    rng = np.random.default_rng(1)
    W = torch.from_numpy(rng.standard_normal((5, 7)).astype(np.float32))
    X = rng.standard_normal((3, 7)).astype(np.float32)
    Y = oracle.linear(W, X)
    assert Y.shape == (3, 5)
    np.testing.assert_allclose(Y, X.astype(np.float64) @ W.numpy().astype(np.float64).T, rtol=1e-6, atol=1e-7)
    # a one-hot input picks out a column of W (catches a transposed operand)
    e = np.zeros((1, 7), dtype=np.float32)
    e[0, 2] = 1.0
    np.testing.assert_array_equal(oracle.linear(W, e)[0], W.numpy()[:, 2])


def test_linear_bf16_weights_are_widened_exactly():
    vals = torch.tensor([[1.0, -2.5, 0.15625, 3.0e-3]], dtype=torch.float32).to(torch.bfloat16)
    e = np.eye(4, dtype=np.float32)
    got = oracle.linear(vals.contiguous(), e)[:, 0]
    np.testing.assert_array_equal(got, vals.float().numpy()[0])


# ---- RoPE --------------------------------------------------------------------------------

def test_rope_identity_at_position_zero():
    x = np.random.default_rng(2).standard_normal(2 * 8).astype(np.float32)
    np.testing.assert_array_equal(oracle.rope(x, 2, 8, 0, 10000.0), x)


def test_rope_two_dim_rotation_hand_values():
    # head_dim 2: the single pair (0,1) turns by t radians; (1,0) -> (cos t, sin t)
    y = oracle.rope([1.0, 0.0], 1, 2, 1, 10000.0)
    np.testing.assert_allclose(y, [math.cos(1.0), math.sin(1.0)], rtol=1e-6)
    y = oracle.rope([0.0, 1.0], 1, 2, 2, 10000.0)
    np.testing.assert_allclose(y, [-math.sin(2.0), math.cos(2.0)], rtol=1e-6)


def test_rope_pairs_are_half_split_with_geometric_frequencies():
    # head_dim 4, base 10000: pair (0,2) turns by t, pair (1,3) by t / 100
    t = 50
    y = oracle.rope([1.0, 1.0, 0.0, 0.0], 1, 4, t, 10000.0)
    np.testing.assert_allclose(y, [math.cos(50.0), math.cos(0.5), math.sin(50.0), math.sin(0.5)], rtol=1e-5,
                               atol=1e-6)


def test_rope_preserves_norm_and_relative_position():
    rng = np.random.default_rng(3)
    q = rng.standard_normal(16).astype(np.float32)
    k = rng.standard_normal(16).astype(np.float32)
    assert abs(np.linalg.norm(oracle.rope(q, 1, 16, 37, 10000.0)) - np.linalg.norm(q)) < 1e-5
    d1 = float(oracle.rope(q, 1, 16, 9, 10000.0) @ oracle.rope(k, 1, 16, 4, 10000.0))
    d2 = float(oracle.rope(q, 1, 16, 109, 10000.0) @ oracle.rope(k, 1, 16, 104, 10000.0))
    assert abs(d1 - d2) < 1e-4


def test_rope_heads_are_rotated_independently():
    x = np.random.default_rng(4).standard_normal(3 * 8).astype(np.float32)
    y = oracle.rope(x, 3, 8, 11, 10000.0)
    for h in range(3):
        np.testing.assert_array_equal(y[h * 8:(h + 1) * 8], oracle.rope(x[h * 8:(h + 1) * 8], 1, 8, 11, 10000.0))


# ---- attention over cached keys ----------------------------------------------------------

def test_attend_single_key_returns_its_value():
    rng = np.random.default_rng(5)
    u, K, V = rng.standard_normal(8), rng.standard_normal((1, 8)), rng.standard_normal((1, 8))
    np.testing.assert_allclose(oracle.attend(u, K, V), V[0].astype(np.float32), rtol=1e-6)


def test_attend_scale_is_inverse_sqrt_head_dim():
    # u.k0 = ln(2) * sqrt(d_h), u.k1 = 0  ->  weights 2/3 and 1/3
    dh = 16
    u = np.zeros(dh)
    u[0] = 1.0
    K = np.zeros((2, dh))
    K[0, 0] = math.log(2.0) * math.sqrt(dh)
    V = np.zeros((2, dh))
    V[0, :] = 3.0
    V[1, :] = -3.0
    np.testing.assert_allclose(oracle.attend(u, K, V), np.full(dh, 1.0), rtol=1e-5)


def test_attend_equal_scores_average_values_and_sharp_score_selects():
    rng = np.random.default_rng(6)
    V = rng.standard_normal((5, 4))
    K = np.tile(rng.standard_normal((1, 4)), (5, 1))
    np.testing.assert_allclose(oracle.attend(rng.standard_normal(4), K, V), V.mean(0), rtol=1e-5, atol=1e-6)
    K2 = np.zeros((5, 4))
    K2[3, 1] = 500.0
    u = np.array([0.0, 1.0, 0.0, 0.0])
    np.testing.assert_allclose(oracle.attend(u, K2, V), V[3], rtol=1e-6, atol=1e-6)


def test_attend_matches_library_sdpa():
    rng = np.random.default_rng(7)
    u, K, V = rng.standard_normal(32), rng.standard_normal((19, 32)), rng.standard_normal((19, 32))
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.tensor(u)[None, None, None, :], torch.tensor(K)[None, None], torch.tensor(V)[None, None])
    np.testing.assert_allclose(oracle.attend(u, K, V), ref[0, 0, 0].numpy(), rtol=1e-5, atol=1e-6)


# ---- SwiGLU ------------------------------------------------------------------------------

def test_swiglu_hand_values():
    # silu(0) = 0 ; silu(1) = 1/(1+e^-1) = 0.7310585786 ; silu(-1) = -0.2689414214
    h = oracle.swiglu([0.0, 1.0, -1.0, 30.0], [5.0, 2.0, 2.0, 0.5])
    np.testing.assert_allclose(h, [0.0, 2 * 0.7310585786, -2 * 0.2689414214, 15.0], rtol=1e-6, atol=1e-7)


def test_swiglu_gate_and_up_are_not_swapped():
    h = oracle.swiglu([0.0], [3.0])  # silu(gate=0) * 3 = 0 ; swapped would give silu(3)*0 = 0 too
    assert h[0] == 0.0
    h = oracle.swiglu([3.0], [1.0])  # silu(3) = 2.857722
    np.testing.assert_allclose(h, [2.8577224], rtol=1e-6)


# ---- router (Eq. moe_layer; Section 4.3) -------------------------------------------------

def test_route_weights_are_softmax_restricted_to_selection():
    rng = np.random.default_rng(8)
    r = rng.standard_normal(16).astype(np.float32)
    idx, w = oracle.route(r, 4)
    order = np.argsort(-r.astype(np.float64), kind="stable")[:4]
    np.testing.assert_array_equal(idx, order)
    e = np.exp(r[idx].astype(np.float64))
    np.testing.assert_allclose(w, e / e.sum(), rtol=1e-6)
    assert abs(float(w.sum()) - 1.0) < 1e-6


def test_route_brute_force_tiny():
    rng = np.random.default_rng(9)
    for _ in range(20):
        r = rng.standard_normal(6).astype(np.float32)
        idx, _ = oracle.route(r, 3)
        best = max(itertools.combinations(range(6), 3), key=lambda s: sum(float(r[i]) for i in s))
        assert set(idx.tolist()) == set(best)


def test_route_ties_prefer_lower_index_and_full_fanout_is_softmax():
    idx, w = oracle.route([1.0, 2.0, 2.0, 0.0, 2.0], 2)
    np.testing.assert_array_equal(idx, [1, 2])
    np.testing.assert_allclose(w, [0.5, 0.5], rtol=1e-6)
    r = np.array([0.3, -1.0, 2.0], dtype=np.float32)
    idx, w = oracle.route(r, 3)
    full = np.exp(r.astype(np.float64)) / np.exp(r.astype(np.float64)).sum()
    np.testing.assert_allclose(w, full[idx], rtol=1e-6)


def test_route_replay_uses_given_set_with_own_probabilities():
    # w_2 = Normalize(softmax(r_2)[I_1])
    r2 = np.array([0.0, math.log(3.0), 5.0, 0.0], dtype=np.float32)
    idx, w = oracle.route(r2, 2, forced=[0, 1])
    np.testing.assert_array_equal(idx, [0, 1])
    np.testing.assert_allclose(w, [0.25, 0.75], rtol=1e-6)


# ---- readout (Eq. mixloss, Eq. alpha) ----------------------------------------------------

def test_readout_one_hot_primary_gives_alpha_one_and_mixture_p():
    z1 = np.full(10, -100.0)
    z1[4] = 100.0
    z2 = np.zeros(10)
    tok, alpha, mix = oracle.readout(z1, z2)
    assert tok == 4 and alpha == 1.0
    np.testing.assert_allclose(mix, np.eye(10)[4], atol=1e-7)


def test_readout_uniform_primary_clips_alpha_to_half():
    z2 = np.array([0.0, math.log(3.0), 0.0, 0.0])  # q = [1/6, 1/2, 1/6, 1/6]
    tok, alpha, mix = oracle.readout(np.zeros(4), z2)
    assert alpha == 0.5 and tok == 1
    np.testing.assert_allclose(mix, 0.5 * 0.25 + 0.5 * np.array([1 / 6, 1 / 2, 1 / 6, 1 / 6]), rtol=1e-6)


def test_readout_two_equal_peaks_alpha_exactly_half():
    z1 = np.array([50.0, 50.0, -50.0, -50.0])
    _, alpha, _ = oracle.readout(z1, np.zeros(4))
    assert alpha == 0.5


def test_readout_unclipped_alpha_is_collision_probability():
    # p = [0.9, 0.1] -> sum p^2 = 0.82 ; q = [0.2, 0.8] -> mix = [0.774, 0.226]
    z1 = np.log(np.array([0.9, 0.1]))
    z2 = np.log(np.array([0.2, 0.8]))
    tok, alpha, mix = oracle.readout(z1, z2)
    assert abs(alpha - 0.82) < 1e-6 and tok == 0
    np.testing.assert_allclose(mix, [0.82 * 0.9 + 0.18 * 0.2, 0.82 * 0.1 + 0.18 * 0.8], rtol=1e-6)


def test_readout_mixture_is_a_distribution_and_alpha_in_range():
    rng = np.random.default_rng(10)
    for scale in (0.1, 1.0, 10.0):
        z1, z2 = scale * rng.standard_normal(200), rng.standard_normal(200)
        tok, alpha, mix = oracle.readout(z1, z2)
        assert 0.5 <= alpha <= 1.0
        assert abs(float(mix.astype(np.float64).sum()) - 1.0) < 1e-5
        assert tok == int(np.argmax(mix))


def test_readout_tie_breaks_to_lowest_index():
    tok, _, _ = oracle.readout(np.array([1.0, 3.0, 3.0, 0.0]), np.array([1.0, 3.0, 3.0, 0.0]))
    assert tok == 1


def test_readout_is_shift_invariant():
    rng = np.random.default_rng(11)
    z1, z2 = rng.standard_normal(50), rng.standard_normal(50)
    _, a1, m1 = oracle.readout(z1, z2)
    _, a2, m2 = oracle.readout(z1 + 3.0, z2 - 7.0)
    assert abs(a1 - a2) < 1e-6
    np.testing.assert_allclose(m1, m2, rtol=1e-5)

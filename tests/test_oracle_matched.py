"""Pins for the oracle's compute-matched MoE allocation (Appendix B.3): the branch evaluates
no attention and no shared expert of its own; it receives g_A * A_1 and g_G * G(N_1)."""
import copy

import numpy as np
import pytest
import torch

import oracle
import ref_torch
from paper_2608_12385_b200.inputs import ModelConfig, make_tokens, make_weights
from test_oracle_model import run_incremental, small_dense


def matched_moe(**kw):
    base = dict(d_model=32, n_layers=2, n_q_heads=4, n_kv_heads=2, head_dim=8, d_ff=0, vocab=50,
                weight_dtype="fp32", n_experts=6, d_expert=16, n_shared_experts=1, k_primary=3, k_branch=1,
                compute_matched=1)
    base.update(kw)
    return ModelConfig(**base)


@pytest.mark.parametrize("cfg", [matched_moe(), matched_moe(k_primary=2, k_branch=2),
                                 matched_moe(k_primary=1, k_branch=3, n_shared_experts=2),
                                 matched_moe(n_shared_experts=0)])
def test_incremental_equals_full_recomputation_and_the_float64_restatement(cfg):
    w = make_weights(cfg, seed=2, matrix_std=0.3)
    tok = make_tokens(cfg, 2, 8, seed=3).numpy()
    z1_full, z2_full, k_full, v_full = oracle.full_forward(cfg, w, tok, want_kv=True)
    z1_ref, z2_ref, _, _ = ref_torch.forward(cfg, w, tok, branch=True)
    np.testing.assert_allclose(z1_full, z1_ref.numpy(), rtol=2e-4, atol=2e-5)
    np.testing.assert_allclose(z2_full, z2_ref.numpy(), rtol=2e-4, atol=2e-5)
    _, outs, m = run_incremental(cfg, w, tok, n_prefill=3, grouped=True)
    for i, o in enumerate(outs):
        t = 3 + i
        np.testing.assert_allclose(o["z1"], z1_full[:, t], rtol=1e-5, atol=1e-5)
        np.testing.assert_allclose(o["z2"], z2_full[:, t], rtol=1e-5, atol=1e-5)
        alpha_ref, mix_ref = ref_torch.mixture(z1_ref[:, t], z2_ref[:, t])
        np.testing.assert_allclose(o["alpha"], alpha_ref.numpy(), rtol=1e-5)
        np.testing.assert_allclose(o["mix"], mix_ref.numpy(), rtol=2e-4, atol=1e-7)
    np.testing.assert_allclose(m.k_cache[:, :2, :8], k_full, rtol=1e-6, atol=1e-6)


def test_unit_gates_same_embedding_and_equal_fanout_make_the_branch_equal_the_primary():
    """S_2^0 = S_1^0, A_2 = A_1, N_2 = N_1 so R_2 = R_1, and M_2 = R_1 + G(N_1) = M_1 at every layer."""
    cfg = matched_moe(k_primary=2, k_branch=2)
    w = make_weights(cfg, seed=10, matrix_std=0.3)
    w["embed_branch"] = w["embed_primary"].clone()
    for lw in w["layers"]:
        lw["gate_a"] = torch.ones_like(lw["gate_a"])
        lw["gate_g"] = torch.ones_like(lw["gate_g"])
    tok = make_tokens(cfg, 2, 6, seed=11).numpy()
    _, outs, _ = run_incremental(cfg, w, tok, n_prefill=2)
    for o in outs:
        np.testing.assert_array_equal(o["z2"], o["z1"])


def test_zero_gates_leave_a_branch_that_sees_only_its_own_token():
    """With g_A = g_G = 0 nothing of the context reaches the branch: its logits are a function of the
    current token alone, whatever the history and the position."""
    cfg = matched_moe()
    w = make_weights(cfg, seed=12, matrix_std=0.3)
    for lw in w["layers"]:
        lw["gate_a"] = torch.zeros_like(lw["gate_a"])
        lw["gate_g"] = torch.zeros_like(lw["gate_g"])
    tok = make_tokens(cfg, 2, 7, seed=13).numpy()
    tok[1, 5] = tok[0, 3]
    tok[1, 4] = (tok[0, 3] + 7) % cfg.vocab
    z2 = oracle.full_forward(cfg, w, tok)[1]
    np.testing.assert_allclose(z2[1, 5], z2[0, 3], rtol=1e-6, atol=1e-6)
    assert np.abs(z2[1, 4] - z2[0, 3]).max() > 1e-3
    # and it is the attention-free, routed-only stack of the float64 restatement on one token
    one = np.array([[tok[0, 3]]])
    z2_one = ref_torch.forward(cfg, w, one, branch=True)[1].numpy()
    np.testing.assert_allclose(z2[0, 3], z2_one[0, 0], rtol=2e-4, atol=2e-5)


def test_primary_path_is_the_default_models_and_the_couplings_are_not_applied():
    cfg = matched_moe()
    w = make_weights(cfg, seed=14, matrix_std=0.3)
    tok = make_tokens(cfg, 2, 6, seed=15).numpy()
    _, base, m0 = run_incremental(cfg, w, tok, n_prefill=2)
    _, dflt, m1 = run_incremental(cfg.replace(compute_matched=0), w, tok, n_prefill=2)
    for a, b in zip(base, dflt):
        np.testing.assert_array_equal(a["z1"], b["z1"])
        assert np.abs(a["z2"] - b["z2"]).max() > 1e-2
    np.testing.assert_array_equal(m0.k_cache, m1.k_cache)
    np.testing.assert_array_equal(m0.v_cache, m1.v_cache)
    w2 = copy.deepcopy(w)
    for lw in w2["layers"]:
        for name in ("coup_a", "coup_b", "coup_c"):
            lw[name] = lw[name] * 2.0 + 1.0
    _, pert, _ = run_incremental(cfg, w2, tok, n_prefill=2)
    for a, b in zip(base, pert):
        np.testing.assert_array_equal(a["z2"], b["z2"])


@pytest.mark.parametrize("name", ["gate_a", "gate_g"])
def test_each_gate_matters_and_never_reaches_the_primary_path(name):
    cfg = matched_moe()
    w = make_weights(cfg, seed=16, matrix_std=0.3)
    tok = make_tokens(cfg, 2, 6, seed=17).numpy()
    _, base, m0 = run_incremental(cfg, w, tok, n_prefill=2)
    w2 = copy.deepcopy(w)
    w2["layers"][0][name] = w2["layers"][0][name] * -1.5 + 0.3
    _, pert, m1 = run_incremental(cfg, w2, tok, n_prefill=2)
    np.testing.assert_array_equal(m0.k_cache, m1.k_cache)
    for a, b in zip(base, pert):
        np.testing.assert_array_equal(a["z1"], b["z1"])
        assert np.abs(a["z2"] - b["z2"]).max() > 1e-2


def test_last_layers_shared_expert_gate_enters_the_branch_logits_linearly():
    """Without a final norm z_2 = W (S-bar_2 + R_2 + g_G * G(N_1)): affine in the last layer's g_G, with the
    slope W diag(G(N_1)) that the restatement's primary shared expert gives."""
    cfg = matched_moe(final_norm=0)
    w = make_weights(cfg, seed=18, matrix_std=0.3)
    tok = make_tokens(cfg, 1, 5, seed=19).numpy()

    def z2_with(g):
        w2 = copy.deepcopy(w)
        w2["layers"][-1]["gate_g"] = g
        return oracle.full_forward(cfg, w2, tok)[1].astype(np.float64)

    g = w["layers"][-1]["gate_g"]
    z0, zg, z2g = z2_with(torch.zeros_like(g)), z2_with(g), z2_with(2 * g)
    np.testing.assert_allclose(z2g - zg, zg - z0, rtol=1e-3, atol=1e-4)
    e = torch.zeros_like(g)
    e[5] = 1.0
    col = z2_with(e) - z0  # = W[:, 5] * G(N_1)[5] at every position
    ratio = col[0, :, :] / w["lm_head"].double().numpy()[:, 5][None, :]
    np.testing.assert_allclose(ratio, np.repeat(ratio[:, :1], ratio.shape[1], 1), rtol=1e-3, atol=1e-5)


def test_dense_models_reject_the_variant():
    cfg = small_dense().replace(compute_matched=1)
    w = make_weights(small_dense(), seed=0)
    with pytest.raises(Exception):
        oracle.OracleModel(cfg, w, max_batch=1, max_seq=4)

"""Pins for the oracle's K > 2 form (Appendix C.1, "More decode branches"): every decode branch has its
own embedding table and same-position state, reads the primary cache, shares the coupling vectors with
the other branches, and the readout mixes p with the mean of the branch distributions.

A branch couples to the primary path only, never to another branch, so branch j of a K-path model must
be exactly the single branch of the main text's two-path model given table E_j: that reduces every K-path
result to the two-path oracle (pinned elsewhere) and to the library-built float64 restatement."""
import numpy as np
import pytest
import torch

import oracle
import ref_torch
from paper_2608_12385_b200.inputs import ModelConfig, make_tokens, make_weights


def small_dense(**kw):
    base = dict(d_model=32, n_layers=2, n_q_heads=4, n_kv_heads=2, head_dim=8, d_ff=48, vocab=50,
                weight_dtype="fp32", n_paths=3)
    base.update(kw)
    return ModelConfig(**base)


def small_moe(**kw):
    base = dict(d_model=32, n_layers=2, n_q_heads=4, n_kv_heads=2, head_dim=8, d_ff=0, vocab=50,
                weight_dtype="fp32", n_experts=6, d_expert=16, n_shared_experts=1, k_primary=2, k_branch=3,
                n_paths=3)
    base.update(kw)
    return ModelConfig(**base)


def two_path_view(cfg, w, j):
    """The two-path model whose single branch uses table E_j (j = 2..K) of the K-path weights."""
    w2 = dict(w)
    V = cfg.vocab
    w2["embed_branch"] = w["embed_branch"][(j - 2) * V:(j - 1) * V].contiguous()
    return cfg.replace(n_paths=2), w2


def run(cfg, w, tok, npre):
    B, T = tok.shape
    m = oracle.OracleModel(cfg, w, B, T)
    m.prefill(tok[:, :npre], want_logits=False)
    return [m.decode_step(tok[:, t], want_mix=True) for t in range(npre, T)], m


# ---- readout: mean of the branch distributions ---------------------------------------------------

def test_readout_multi_by_hand():
    """p = (0.9, 0.1): alpha = 0.82; q_2 = (0.5, 0.5), q_3 = (0.1, 0.9): qbar = (0.3, 0.7);
    mix = 0.82 p + 0.18 qbar = (0.792, 0.208)."""
    z1 = np.log(np.array([0.9, 0.1]))
    zb = np.log(np.array([[0.5, 0.5], [0.1, 0.9]]))
    tok, alpha, mix = oracle.readout_multi(z1, zb)
    assert tok == 0
    assert alpha == pytest.approx(0.82, abs=1e-6)
    np.testing.assert_allclose(mix, [0.792, 0.208], atol=1e-6)


def test_readout_multi_reduces_to_the_two_path_readout_and_to_float64_library_softmax():
    rng = np.random.default_rng(0)
    z1 = rng.normal(0, 3, 40).astype(np.float32)
    zb = rng.normal(0, 3, (3, 40)).astype(np.float32)
    t1, a1, m1 = oracle.readout(z1, zb[0])
    t2, a2, m2 = oracle.readout_multi(z1, zb[:1])
    assert t1 == t2 and a1 == a2
    np.testing.assert_array_equal(m1, m2)
    # identical branches: the mean is the branch itself
    t3, a3, m3 = oracle.readout_multi(z1, np.stack([zb[0]] * 3))
    assert t3 == t1 and a3 == a1
    np.testing.assert_allclose(m3, m1, rtol=1e-6, atol=1e-9)
    # library restatement; the order of the branches does not matter
    p = torch.softmax(torch.from_numpy(z1).double(), -1)
    qbar = torch.softmax(torch.from_numpy(zb).double(), -1).mean(0)
    alpha = float((p * p).sum().clamp(0.5, 1.0))
    want = alpha * p + (1 - alpha) * qbar
    tok, a, mix = oracle.readout_multi(z1, zb)
    tokp, ap, mixp = oracle.readout_multi(z1, zb[::-1].copy())
    assert a == pytest.approx(alpha, rel=1e-6) and ap == a and tok == int(want.argmax()) == tokp
    np.testing.assert_allclose(mix, want.numpy(), rtol=1e-5, atol=1e-9)
    np.testing.assert_allclose(mixp, mix, rtol=1e-6, atol=1e-9)
    assert float(mix.sum()) == pytest.approx(1.0, abs=1e-5)


# ---- model level ---------------------------------------------------------------------------------

@pytest.mark.parametrize("cfg", [small_dense(), small_dense(n_paths=4, n_kv_heads=1), small_moe(),
                                 small_moe(router_mode=1), small_moe(compute_matched=1)])
def test_each_branch_of_the_k_path_model_is_the_two_path_models_branch(cfg):
    """Branch j is bit for bit the branch of the two-path oracle built on E_j; the primary logits and
    the cache do not depend on how many branches run; the mixture is alpha p + (1-alpha) mean_j q_j."""
    w = make_weights(cfg, seed=3, matrix_std=0.3)
    tok = make_tokens(cfg, 2, 9, seed=4).numpy()
    outs, m = run(cfg, w, tok, 5)
    K = cfg.n_paths
    for j in range(2, K + 1):
        cfg2, w2 = two_path_view(cfg, w, j)
        outs2, m2 = run(cfg2, w2, tok, 5)
        for o, o2 in zip(outs, outs2):
            np.testing.assert_array_equal(o["z1"], o2["z1"])
            np.testing.assert_array_equal(o["z2"][j - 2], o2["z2"])
            np.testing.assert_array_equal(o["alpha"], o2["alpha"])
            if cfg.is_moe:
                np.testing.assert_array_equal(o["experts"][:, 0], o2["experts"][:, 0])
                np.testing.assert_array_equal(o["experts"][:, j - 1], o2["experts"][:, 1])
        np.testing.assert_array_equal(m.k_cache, m2.k_cache)
        np.testing.assert_array_equal(m.v_cache, m2.v_cache)
    for o in outs:
        for b in range(2):
            p = torch.softmax(torch.from_numpy(o["z1"][b]).double(), -1)
            qbar = torch.softmax(torch.from_numpy(o["z2"][:, b]).double(), -1).mean(0)
            a = float(o["alpha"][b])
            np.testing.assert_allclose(o["mix"][b], (a * p + (1 - a) * qbar).numpy(), rtol=1e-5, atol=1e-9)
            assert o["next"][b] == int(np.argmax(o["mix"][b]))


@pytest.mark.parametrize("cfg", [small_dense(), small_moe()])
def test_incremental_equals_full_recomputation_and_library_restatement(cfg):
    w = make_weights(cfg, seed=5, matrix_std=0.3)
    tok = make_tokens(cfg, 2, 8, seed=6).numpy()
    z1_full, z2_full, k_full, v_full = oracle.full_forward(cfg, w, tok, want_kv=True)
    assert z2_full.shape == (cfg.n_paths - 1, 2, 8, cfg.vocab)
    outs, m = run(cfg, w, tok, 3)
    for i, o in enumerate(outs):
        np.testing.assert_allclose(o["z1"], z1_full[:, 3 + i], rtol=1e-5, atol=1e-5)
        np.testing.assert_allclose(o["z2"], z2_full[:, :, 3 + i], rtol=1e-5, atol=1e-5)
    np.testing.assert_allclose(m.k_cache[:, :2, :8], k_full, rtol=1e-6, atol=1e-6)
    for j in range(2, cfg.n_paths + 1):
        cfg2, w2 = two_path_view(cfg, w, j)
        z1_ref, z2_ref, _, _ = ref_torch.forward(cfg2, w2, tok, branch=True)
        np.testing.assert_allclose(z1_full, z1_ref.numpy(), rtol=2e-4, atol=2e-5)
        np.testing.assert_allclose(z2_full[j - 2], z2_ref.numpy(), rtol=2e-4, atol=2e-5)


def test_identical_tables_give_identical_branches_and_the_two_path_mixture():
    cfg = small_dense(n_paths=3)
    w = make_weights(cfg, seed=7, matrix_std=0.3)
    V = cfg.vocab
    w["embed_branch"] = torch.cat([w["embed_branch"][:V], w["embed_branch"][:V]]).contiguous()
    tok = make_tokens(cfg, 2, 7, seed=8).numpy()
    outs, _ = run(cfg, w, tok, 4)
    cfg2, w2 = two_path_view(cfg, w, 2)
    outs2, _ = run(cfg2, w2, tok, 4)
    for o, o2 in zip(outs, outs2):
        np.testing.assert_array_equal(o["z2"][0], o["z2"][1])
        np.testing.assert_allclose(o["mix"], o2["mix"], rtol=1e-6, atol=1e-9)
        np.testing.assert_array_equal(o["next"], o2["next"])


def test_the_branches_differ_when_their_tables_differ_and_both_reach_the_mixture():
    cfg = small_dense(n_paths=3)
    w = make_weights(cfg, seed=9, matrix_std=0.3, lm_head_std=1.0)
    tok = make_tokens(cfg, 2, 7, seed=10).numpy()
    outs, _ = run(cfg, w, tok, 4)
    cfg2, w2 = two_path_view(cfg, w, 2)
    outs2, _ = run(cfg2, w2, tok, 4)
    assert np.abs(outs[-1]["z2"][0] - outs[-1]["z2"][1]).max() > 1e-2
    assert np.abs(outs[-1]["mix"] - outs2[-1]["mix"]).max() > 1e-4  # dropping branch 3 would show


def test_bad_path_counts_are_rejected():
    cfg = small_dense(n_paths=3)
    w = make_weights(cfg, seed=0)
    with pytest.raises(ValueError):
        oracle.OracleModel(cfg.replace(n_paths=1), {**w, "embed_branch": w["embed_branch"][:0]}, 1, 4)
    with pytest.raises(AssertionError):
        oracle.OracleModel(cfg.replace(n_paths=4), w, 1, 4)  # three tables needed, two given

"""Model-level pins for the oracle: the invariants the paper states (primary path unchanged
by the branch; prefill equals a standard causal LM; incremental decode equals the full
non-incremental two-path computation), reductions to an independent library-built
restatement (tests/ref_torch.py), and special cases of the coupling, GQA and MoE rules."""
import copy

import numpy as np
import pytest
import torch

import oracle
import ref_torch
from paper_2608_12385_b200.inputs import ModelConfig, make_tokens, make_weights, tiny_dense_fp32


def small_dense(**kw):
    base = dict(d_model=32, n_layers=2, n_q_heads=4, n_kv_heads=2, head_dim=8, d_ff=48, vocab=50,
                weight_dtype="fp32")
    base.update(kw)
    return ModelConfig(**base)


def small_moe(**kw):
    base = dict(d_model=32, n_layers=2, n_q_heads=4, n_kv_heads=2, head_dim=8, d_ff=0, vocab=50,
                weight_dtype="fp32", n_experts=6, d_expert=16, n_shared_experts=1, k_primary=2, k_branch=3)
    base.update(kw)
    return ModelConfig(**base)


def run_incremental(cfg, w, tokens, n_prefill, grouped=True, kv_round=False):
    """Prefill tokens[:, :n_prefill], then teacher-forced decode over the rest.
    Returns per-step dicts and the model (for cache inspection)."""
    B, T = tokens.shape
    m = oracle.OracleModel(cfg, w, max_batch=B, max_seq=T, kv_round_bf16=kv_round)
    pre = m.prefill(tokens[:, :n_prefill]) if n_prefill > 0 else None
    outs = [m.decode_step(tokens[:, t], grouped=grouped, want_mix=True) for t in range(n_prefill, T)]
    return pre, outs, m


# ---- I2: the primary path is a textbook causal LM ----------------------------------------

@pytest.mark.parametrize("cfg", [small_dense(), small_dense(n_kv_heads=4), small_dense(n_kv_heads=1),
                                 small_dense(final_norm=0), small_moe()])
def test_primary_path_equals_library_causal_lm(cfg):
    w = make_weights(cfg, seed=0, matrix_std=0.3)
    tok = make_tokens(cfg, 2, 9, seed=1).numpy()
    z1_ref, _, k_ref, v_ref = ref_torch.forward(cfg, w, tok, branch=False)
    pre, outs, m = run_incremental(cfg, w, tok, n_prefill=5, grouped=False)
    np.testing.assert_allclose(pre, z1_ref[:, 4].numpy(), rtol=2e-4, atol=2e-5)
    for i, o in enumerate(outs):
        np.testing.assert_allclose(o["z1"], z1_ref[:, 5 + i].numpy(), rtol=2e-4, atol=2e-5)
        assert "z2" not in o
        np.testing.assert_array_equal(o["next"], z1_ref[:, 5 + i].argmax(-1).numpy())
    np.testing.assert_allclose(m.k_cache[:, :2, :9], k_ref.numpy(), rtol=2e-4, atol=2e-5)
    np.testing.assert_allclose(m.v_cache[:, :2, :9], v_ref.numpy(), rtol=2e-4, atol=2e-5)


# ---- I3: incremental decode == full non-incremental two-path computation ------------------

@pytest.mark.parametrize("cfg", [small_dense(), small_moe(), small_moe(router_mode=1),
                                 small_moe(moe_b_coupling=0, n_shared_experts=0)])
def test_incremental_equals_full_recomputation(cfg):
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
    np.testing.assert_allclose(m.v_cache[:, :2, :8], v_full, rtol=1e-6, atol=1e-6)


def test_boundary_step_from_empty_cache():
    """Grouped decode from position 0 (no prefill at all) is the first row of the full pass."""
    cfg = small_dense()
    w = make_weights(cfg, seed=4, matrix_std=0.3)
    tok = make_tokens(cfg, 1, 4, seed=5).numpy()
    z1_full, z2_full = oracle.full_forward(cfg, w, tok)
    _, outs, _ = run_incremental(cfg, w, tok, n_prefill=0)
    for t, o in enumerate(outs):
        np.testing.assert_allclose(o["z2"], z2_full[:, t], rtol=1e-5, atol=1e-5)


# ---- I1 / I4: the primary path never reads the branch --------------------------------------

@pytest.mark.parametrize("cfg", [small_dense(), small_moe()])
def test_primary_logits_and_cache_identical_with_branch_on_or_off(cfg):
    w = make_weights(cfg, seed=6, matrix_std=0.3)
    tok = make_tokens(cfg, 3, 7, seed=7).numpy()
    _, on, m_on = run_incremental(cfg, w, tok, n_prefill=2, grouped=True)
    _, off, m_off = run_incremental(cfg, w, tok, n_prefill=2, grouped=False)
    for a, b in zip(on, off):
        np.testing.assert_array_equal(a["z1"], b["z1"])
    np.testing.assert_array_equal(m_on.k_cache, m_off.k_cache)
    np.testing.assert_array_equal(m_on.v_cache, m_off.v_cache)


def test_branch_side_perturbations_never_reach_the_cache_or_z1():
    cfg = small_dense()
    w = make_weights(cfg, seed=8, matrix_std=0.3)
    tok = make_tokens(cfg, 2, 6, seed=9).numpy()
    _, base, m0 = run_incremental(cfg, w, tok, n_prefill=2)
    k0, v0 = m0.k_cache.copy(), m0.v_cache.copy()
    w2 = copy.deepcopy(w)
    w2["embed_branch"] = w2["embed_branch"] * -3.0 + 0.1
    for lw in w2["layers"]:
        for name in ("coup_a", "coup_b", "coup_c"):
            lw[name] = lw[name] * 2.0 + 1.0
    _, pert, m1 = run_incremental(cfg, w2, tok, n_prefill=2)
    np.testing.assert_array_equal(m1.k_cache, k0)
    np.testing.assert_array_equal(m1.v_cache, v0)
    for a, b in zip(base, pert):
        np.testing.assert_array_equal(a["z1"], b["z1"])
        assert np.abs(a["z2"] - b["z2"]).max() > 1e-2


# ---- I5 / I6: coupling special cases -------------------------------------------------------

@pytest.mark.parametrize("cfg", [small_dense(), small_moe(k_branch=2)])
def test_same_embedding_and_zero_coupling_make_branch_equal_primary(cfg):
    w = make_weights(cfg, seed=10, matrix_std=0.3)
    w["embed_branch"] = w["embed_primary"].clone()
    for lw in w["layers"]:
        for name in ("coup_a", "coup_b", "coup_c"):
            lw[name] = torch.zeros_like(lw[name])
    tok = make_tokens(cfg, 2, 6, seed=11).numpy()
    _, outs, _ = run_incremental(cfg, w, tok, n_prefill=2)
    for o in outs:
        np.testing.assert_array_equal(o["z2"], o["z1"])
        p = torch.softmax(torch.tensor(o["z1"], dtype=torch.float64), -1).numpy()
        np.testing.assert_allclose(o["mix"], p, rtol=1e-5, atol=1e-9)
        np.testing.assert_array_equal(o["next"], p.argmax(-1))


@pytest.mark.parametrize("name", ["coup_a", "coup_b", "coup_c"])
def test_each_coupling_vector_matters(name):
    cfg = small_dense()
    w = make_weights(cfg, seed=12, matrix_std=0.3)
    tok = make_tokens(cfg, 1, 5, seed=13).numpy()
    _, base, _ = run_incremental(cfg, w, tok, n_prefill=2)
    w2 = copy.deepcopy(w)
    for lw in w2["layers"]:
        lw[name] = torch.zeros_like(lw[name])
    _, zeroed, _ = run_incremental(cfg, w2, tok, n_prefill=2)
    assert np.abs(base[-1]["z2"] - zeroed[-1]["z2"]).max() > 5e-2
    np.testing.assert_array_equal(base[-1]["z1"], zeroed[-1]["z1"])


def test_coupling_is_linear_in_each_vector_at_the_last_layer():
    """Q~_2 - Q_2 = a*Q_1 and M_2 - H_2 W_D = (b*H_1) W_D + c*M_1: in a one-layer model z_2
    before the final norm is affine in c, so (c=2v) - (c=v) == (c=v) - (c=0) after removing
    the norm (final_norm=0)."""
    cfg = small_dense(n_layers=1, final_norm=0)
    w = make_weights(cfg, seed=14, matrix_std=0.3)
    tok = make_tokens(cfg, 1, 3, seed=15).numpy()
    zs = []
    for s in (0.0, 1.0, 2.0):
        w2 = copy.deepcopy(w)
        w2["layers"][0]["coup_c"] = w["layers"][0]["coup_c"] * s
        zs.append(oracle.full_forward(cfg, w2, tok)[1].astype(np.float64))
    np.testing.assert_allclose(zs[2] - zs[1], zs[1] - zs[0], rtol=1e-3, atol=1e-5)
    assert np.abs(zs[1] - zs[0]).max() > 1e-2


# ---- I10: GQA head -> group map -------------------------------------------------------------

def test_gqa_equals_mha_with_repeated_kv_heads():
    cfg_g = small_dense(n_q_heads=4, n_kv_heads=2)
    cfg_m = small_dense(n_q_heads=4, n_kv_heads=4)
    w = make_weights(cfg_g, seed=16, matrix_std=0.3)
    wm = copy.deepcopy(w)
    dh = cfg_g.head_dim
    for lw in wm["layers"]:
        for name in ("wk", "wv"):
            heads = lw[name].view(cfg_g.n_kv_heads, dh, cfg_g.d_model)
            lw[name] = heads.repeat_interleave(2, dim=0).reshape(cfg_m.kv_dim, cfg_m.d_model).contiguous()
    tok = make_tokens(cfg_g, 2, 6, seed=17).numpy()
    zg = oracle.full_forward(cfg_g, w, tok)
    zm = oracle.full_forward(cfg_m, wm, tok)
    np.testing.assert_allclose(zg[0], zm[0], rtol=1e-6, atol=1e-6)
    np.testing.assert_allclose(zg[1], zm[1], rtol=1e-6, atol=1e-6)


# ---- I13: batch independence ------------------------------------------------------------------

def test_sequences_do_not_see_their_batch_mates():
    cfg = small_dense()
    w = make_weights(cfg, seed=18, matrix_std=0.3)
    tok = make_tokens(cfg, 3, 6, seed=19).numpy()
    _, all3, _ = run_incremental(cfg, w, tok, n_prefill=3)
    _, only1, _ = run_incremental(cfg, w, tok[1:2], n_prefill=3)
    for a, b in zip(all3, only1):
        np.testing.assert_array_equal(a["z1"][1], b["z1"][0])
        np.testing.assert_array_equal(a["z2"][1], b["z2"][0])


# ---- MoE special cases (I9) ---------------------------------------------------------------------

def test_moe_with_identical_experts_and_no_shared_expert_is_the_dense_mlp():
    cfg_moe = small_moe(n_shared_experts=0, d_expert=48, k_primary=2, k_branch=4)
    cfg_dense = small_dense(d_ff=48)
    w = make_weights(cfg_moe, seed=20, matrix_std=0.3)
    wd = copy.deepcopy(w)
    for lw_m, lw_d in zip(w["layers"], wd["layers"]):
        for e in range(1, cfg_moe.n_experts):
            lw_m["exp_gate"][e] = lw_m["exp_gate"][0]
            lw_m["exp_up"][e] = lw_m["exp_up"][0]
            lw_m["exp_down"][e] = lw_m["exp_down"][0]
        lw_d["w_gate"] = lw_m["exp_gate"][0].clone()
        lw_d["w_up"] = lw_m["exp_up"][0].clone()
        lw_d["w_down"] = lw_m["exp_down"][0].clone()
        lw_d["coup_b"] = torch.zeros(48)  # the MoE layer has no shared expert for b to act on
    tok = make_tokens(cfg_moe, 2, 5, seed=21).numpy()
    zm = oracle.full_forward(cfg_moe, w, tok)
    zd = oracle.full_forward(cfg_dense, wd, tok)
    np.testing.assert_allclose(zm[0], zd[0], rtol=1e-5, atol=1e-5)
    np.testing.assert_allclose(zm[1], zd[1], rtol=1e-5, atol=1e-5)


def test_router_replay_reuses_primary_expert_set():
    cfg = small_moe(router_mode=1)
    w = make_weights(cfg, seed=22, matrix_std=0.3)
    tok = make_tokens(cfg, 2, 5, seed=23).numpy()
    _, outs, _ = run_incremental(cfg, w, tok, n_prefill=2)
    for o in outs:
        ex = o["experts"]  # [L, 2, B, kmax]
        np.testing.assert_array_equal(ex[:, 0, :, :cfg.k_primary], ex[:, 1, :, :cfg.k_primary])
        assert (ex[:, 1, :, cfg.k_primary:] == -1).all()


def test_independent_routing_fanouts_and_forced_experts_roundtrip():
    cfg = small_moe()
    w = make_weights(cfg, seed=24, matrix_std=0.3)
    tok = make_tokens(cfg, 2, 4, seed=25).numpy()
    m = oracle.OracleModel(cfg, w, 2, 4)
    m.prefill(tok[:, :3], want_logits=False)
    o = m.decode_step(tok[:, 3])
    ex = o["experts"]
    assert (ex[:, 0, :, :cfg.k_primary] >= 0).all() and (ex[:, 0, :, cfg.k_primary:] == -1).all()
    assert (ex[:, 1, :, :cfg.k_branch] >= 0).all()
    for l in range(cfg.n_layers):
        for p, k in ((0, cfg.k_primary), (1, cfg.k_branch)):
            for b in range(2):
                assert len(set(ex[l, p, b, :k].tolist())) == k
    m2 = oracle.OracleModel(cfg, w, 2, 4)
    m2.prefill(tok[:, :3], want_logits=False)
    o2 = m2.decode_step(tok[:, 3], forced_experts=ex)
    np.testing.assert_array_equal(o["z1"], o2["z1"])
    np.testing.assert_array_equal(o["z2"], o2["z2"])


# ---- storage types --------------------------------------------------------------------------------

def test_bf16_weights_equal_their_fp32_widening():
    cfg16 = small_dense(weight_dtype="bf16")
    w16 = make_weights(cfg16, seed=26, matrix_std=0.3)
    cfg32 = small_dense(weight_dtype="fp32")
    w32 = copy.deepcopy(w16)
    for name in ("embed_primary", "embed_branch", "lm_head"):
        w32[name] = w16[name].float()
    for lw in w32["layers"]:
        for name in ("wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down"):
            lw[name] = lw[name].float()
    tok = make_tokens(cfg16, 2, 5, seed=27).numpy()
    a = oracle.full_forward(cfg16, w16, tok)
    b = oracle.full_forward(cfg32, w32, tok)
    np.testing.assert_array_equal(a[0], b[0])
    np.testing.assert_array_equal(a[1], b[1])


def test_kv_rounding_switch_only_rounds_the_cache():
    cfg = small_dense()
    w = make_weights(cfg, seed=28, matrix_std=0.3)
    tok = make_tokens(cfg, 1, 5, seed=29).numpy()
    _, a, ma = run_incremental(cfg, w, tok, n_prefill=2, kv_round=False)
    _, b, mb = run_incremental(cfg, w, tok, n_prefill=2, kv_round=True)
    # first cached position of layer 0 differs only by bf16 rounding of the same value
    k_exact = torch.tensor(ma.k_cache[0, 0, 0])
    np.testing.assert_array_equal(mb.k_cache[0, 0, 0], k_exact.to(torch.bfloat16).float().numpy())
    assert 0 < np.abs(a[-1]["z1"] - b[-1]["z1"]).max() < 0.1


def test_injected_cache_is_used_as_is():
    cfg = small_dense()
    w = make_weights(cfg, seed=30, matrix_std=0.3)
    tok = make_tokens(cfg, 2, 6, seed=31).numpy()
    _, _, k_full, v_full = oracle.full_forward(cfg, w, tok, want_kv=True)
    _, outs, _ = run_incremental(cfg, w, tok, n_prefill=5)
    m = oracle.OracleModel(cfg, w, 2, 6)
    m.inject_kv(k_full[:, :, :5], v_full[:, :, :5], 5)
    o = m.decode_step(tok[:, 5])
    np.testing.assert_allclose(o["z2"], outs[0]["z2"], rtol=1e-5, atol=1e-6)


def test_capacity_and_token_range_are_rejected():
    cfg = small_dense()
    w = make_weights(cfg, seed=32)
    m = oracle.OracleModel(cfg, w, 1, 2)
    m.decode_step([1])
    m.decode_step([2])
    with pytest.raises(RuntimeError):
        m.decode_step([3])
    m.reset()
    with pytest.raises(RuntimeError):
        m.decode_step([cfg.vocab])


def test_tiny_config_random_init_gives_alpha_half():
    """With N(0,0.02) weights the primary distribution is nearly flat, so the collision
    probability is far below 0.5 and alpha sits on its lower clip (Eq. alpha)."""
    cfg = tiny_dense_fp32().replace(n_layers=1)
    w = make_weights(cfg, seed=0)
    tok = make_tokens(cfg, 1, 3, seed=1).numpy()
    _, outs, _ = run_incremental(cfg, w, tok, n_prefill=2)
    assert outs[0]["alpha"][0] == 0.5


def test_recorded_router_logits_explain_the_chosen_experts():
    """orc_router_logits exposes r_i = N_i W_r of the last step: the experts the step chose are the
    brute-force top-k of those logits, the replayed branch reuses the primary's set, and the logits of
    the first layer's primary rows equal the library-built float64 restatement."""
    for cfg in (small_moe(), small_moe(router_mode=1)):
        w = make_weights(cfg, seed=2, matrix_std=0.3)
        tok = make_tokens(cfg, 3, 6, seed=3).numpy()
        m = oracle.OracleModel(cfg, w, 3, 6)
        m.prefill(tok[:, :4], want_logits=False)
        o = m.decode_step(tok[:, 4])
        r = m.router_logits(3)
        assert r.shape == (cfg.n_layers, 2, 3, cfg.n_experts)
        for l in range(cfg.n_layers):
            for b in range(3):
                top1 = set(np.argsort(-r[l, 0, b], kind="stable")[:cfg.k_primary].tolist())
                assert set(o["experts"][l, 0, b, :cfg.k_primary].tolist()) == top1
                if cfg.router_mode == 1:
                    assert set(o["experts"][l, 1, b, :cfg.k_primary].tolist()) == top1
                else:
                    top2 = set(np.argsort(-r[l, 1, b], kind="stable")[:cfg.k_branch].tolist())
                    assert set(o["experts"][l, 1, b, :cfg.k_branch].tolist()) == top2
        # layer 0, primary rows, position 4: RMSNorm(S-bar_1) W_r rebuilt from library routines
        import torch.nn.functional as F
        lw = w["layers"][0]
        tk = torch.as_tensor(tok[:, :5]).long()
        s1 = F.rms_norm(w["embed_primary"].double()[tk], (cfg.d_model,), w["embed_norm_g"].double(), cfg.rms_eps)
        n1 = F.rms_norm(s1, (cfg.d_model,), lw["attn_norm_g"].double(), cfg.rms_eps)
        q1 = ref_torch._rope_complex(n1 @ lw["wq"].double().T, cfg.n_q_heads, cfg.head_dim, cfg.rope_base)
        k1 = ref_torch._rope_complex(n1 @ lw["wk"].double().T, cfg.n_kv_heads, cfg.head_dim, cfg.rope_base)
        v1 = n1 @ lw["wv"].double().T
        sbar = s1 + ref_torch._attn(q1, k1, v1, cfg) @ lw["wo"].double().T
        m1 = F.rms_norm(sbar, (cfg.d_model,), lw["mlp_norm_g"].double(), cfg.rms_eps)
        want = (m1 @ lw["router"].double().T)[:, 4].numpy()
        np.testing.assert_allclose(r[0, 0], want, rtol=2e-4, atol=2e-5)

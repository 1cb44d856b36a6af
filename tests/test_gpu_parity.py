"""GPU parity: the CUDA library against the CPU oracle through the C ABI, element by element
on the same seeded inputs, plus the properties that must hold at any size."""
import numpy as np
import pytest
import torch

import oracle
from gpu_util import TOL, assert_logits_close, make_gpu_model, teacher_forced_compare
from paper_2608_12385_b200 import binding
from paper_2608_12385_b200.inputs import (ModelConfig, dense_1b, make_page_table, make_synthetic_kv, make_tokens,
                                          make_weights, moe_1b, tiny_dense_fp32)

pytestmark = pytest.mark.gpu


def small_bf16(**kw):
    base = dict(d_model=256, n_layers=3, n_q_heads=8, n_kv_heads=2, head_dim=64, d_ff=712, vocab=1000,
                weight_dtype="bf16")
    base.update(kw)
    return ModelConfig(**base)


def small_moe(**kw):
    base = dict(d_model=256, n_layers=2, n_q_heads=4, n_kv_heads=2, head_dim=64, d_ff=0, vocab=1000,
                weight_dtype="bf16", n_experts=8, d_expert=200, n_shared_experts=1, k_primary=2, k_branch=3)
    base.update(kw)
    return ModelConfig(**base)


# ---- end-to-end parity ---------------------------------------------------------------------------

def test_tiny_fp32_config_prefill_and_16_grouped_steps():
    """Tiny dense fp32 model, batch 2, prompt 64 (prefill 63 + boundary step), 16 grouped steps."""
    cfg = tiny_dense_fp32()
    w = make_weights(cfg, seed=0)
    tok = make_tokens(cfg, 2, 64 + 15, seed=1)
    teacher_forced_compare(cfg, w, tok, n_prefill=63, grouped=True)


def test_tiny_fp32_primary_only():
    cfg = tiny_dense_fp32()
    w = make_weights(cfg, seed=0)
    tok = make_tokens(cfg, 2, 40, seed=1)
    teacher_forced_compare(cfg, w, tok, n_prefill=33, grouped=False)


@pytest.mark.parametrize("cfg,B,T,npre", [
    (small_bf16(), 3, 40, 35),                                     # GQA 4 queries per KV head, ragged d_ff
    (small_bf16(n_q_heads=4, n_kv_heads=4, head_dim=64), 1, 20, 17),  # MHA, batch 1
    (small_bf16(n_q_heads=2, n_kv_heads=1, head_dim=128, d_model=128, vocab=777), 5, 50, 47),  # MQA, odd batch
    (small_bf16(final_norm=0, n_layers=1), 2, 18, 0),              # no prefill at all: decode from position 0
    (small_bf16(n_q_heads=8, n_kv_heads=1, head_dim=64), 3, 40, 35),   # 8 queries per KV head: 16-row attention tile
    (small_bf16(n_q_heads=8, n_kv_heads=1, head_dim=128, d_model=256), 2, 90, 70),  # the same at d_h 128, two tiles
])
def test_small_bf16_models(cfg, B, T, npre):
    w = make_weights(cfg, seed=5, matrix_std=0.05)
    tok = make_tokens(cfg, B, T, seed=6)
    teacher_forced_compare(cfg, w, tok, n_prefill=npre, grouped=True)


def test_prefill_longer_than_one_chunk_and_page_boundaries():
    """Prompt of 300 positions at batch 2 crosses the prefill chunking and 18 page boundaries."""
    cfg = small_bf16(n_layers=2)
    w = make_weights(cfg, seed=7, matrix_std=0.05)
    tok = make_tokens(cfg, 2, 306, seed=8)
    teacher_forced_compare(cfg, w, tok, n_prefill=300, grouped=True)


@pytest.mark.parametrize("cfg,B,n", [
    (small_bf16(n_layers=2), 2, 2100),                                    # three chunks of <= 1024 positions, 4 positions per query tile
    (small_bf16(n_layers=2), 3, 700),                                     # ragged chunks (682 + 18) and tail tiles
    (small_bf16(n_layers=1, n_q_heads=4, n_kv_heads=4), 1, 2500),         # MHA: 16 positions per tile, 2048 + 452
    (small_bf16(n_layers=1, n_q_heads=2, n_kv_heads=1, head_dim=128, d_model=128, vocab=777), 5, 1000),  # 8 per tile
    (small_bf16(n_layers=1, n_q_heads=8, n_kv_heads=1), 2, 333),          # 2 positions per tile
    (small_bf16(n_layers=1, n_q_heads=3, n_kv_heads=1), 2, 400),          # 3 heads per KV head: 5 positions per tile (the 16-row kernel)
])
def test_long_prompt_prefill_matches_the_oracle(cfg, B, n):
    """Section 4.4 item 1, prompt-wide prefill: prompts of up to 2500 positions go through in chunks of up to
    2048 rows (GEMMs over several row tiles per weight tile, vector kernels between them, causal attention
    with 16 / G consecutive positions per query tile and eight tiles per CTA).  Last-position logits and the
    whole cache against the oracle's position-by-position primary pass, then two grouped steps on top of the
    device's own cache."""
    w = make_weights(cfg, seed=51, matrix_std=0.05)
    tok = make_tokens(cfg, B, n + 2, seed=52)
    om = oracle.OracleModel(cfg, w, B, n + 2)
    gm = make_gpu_model(cfg, w, B, n + 2)
    want = om.prefill(tok[:, :n].numpy())
    got = gm.prefill(tok[:, :n].cuda().contiguous(), want_logits=True)
    assert_logits_close(got, want, "bf16", "prefill logits")
    k_dev, v_dev = gm.export_kv(B, n)
    np.testing.assert_allclose(k_dev.float().numpy(), om.k_cache[:, :B, :n], rtol=2.0 ** -8, atol=5e-3)
    np.testing.assert_allclose(v_dev.float().numpy(), om.v_cache[:, :B, :n], rtol=2.0 ** -8, atol=5e-3)
    for t in range(n, n + 2):
        o = om.decode_step(tok[:, t].numpy())
        g = gm.decode_full(tok[:, t].cuda().contiguous())
        assert_logits_close(g["z1"], o["z1"], "bf16", f"step {t} z1")
        assert_logits_close(g["z2"], o["z2"], "bf16", f"step {t} z2")
    assert gm.sync_status() == (0, 0)


@pytest.mark.parametrize("cfg", [small_bf16(n_layers=2), tiny_dense_fp32().replace(n_layers=2), small_moe(),
                                 small_bf16(n_layers=2, n_paths=3)])
def test_prefill_boundary_is_prefill_of_all_but_one_plus_the_grouped_step(cfg):
    """Section 4.4 items 1-2 in one call: the same bits as dbt_prefill over x_1..x_{S-1} followed by
    dbt_decode_step on x_S, the same cache, and (dense models) the oracle's values for that boundary."""
    w = make_weights(cfg, seed=61, matrix_std=0.05)
    B, S = 3, 37
    tok = make_tokens(cfg, B, S + 1, seed=62)
    wd = binding.weights_to_device(w)
    a, b = binding.Model(cfg, wd, B, S + 1), binding.Model(cfg, wd, B, S + 1)
    ga = a.prefill_boundary(tok[:, :S].cuda().contiguous())
    b.prefill(tok[:, :S - 1].cuda().contiguous())
    gb = b.decode_full(tok[:, S - 1].cuda().contiguous())
    for k in ("next", "z1", "z2", "alpha"):
        assert torch.equal(ga[k], gb[k]), k
    assert [a.seq_len(i) for i in range(B)] == [S] * B
    ka, va = a.export_kv(B, S)
    kb, vb = b.export_kv(B, S)
    assert torch.equal(ka.float(), kb.float()) and torch.equal(va.float(), vb.float())
    if not cfg.is_moe:
        om = oracle.OracleModel(cfg, w, B, S + 1)
        om.prefill(tok[:, :S - 1].numpy(), want_logits=False)
        o = om.decode_step(tok[:, S - 1].numpy())
        assert_logits_close(ga["z1"], o["z1"], cfg.weight_dtype, "boundary z1")
        assert_logits_close(ga["z2"], o["z2"], cfg.weight_dtype, "boundary z2")
    # and the next step continues from there on both handles alike
    ga2 = a.decode_full(tok[:, S].cuda().contiguous())
    gb2 = b.decode_full(tok[:, S].cuda().contiguous())
    assert torch.equal(ga2["z1"], gb2["z1"]) and torch.equal(ga2["z2"], gb2["z2"])


def test_prompt_chunks_through_the_16_row_attention_kernel(monkeypatch):
    """DBT_PROMPT_ATTN=tile: the earlier form of the prompt attention (one 16-row tile per CTA pass) still
    serves head ratios that do not divide 16, and computes the same prefill."""
    monkeypatch.setenv("DBT_PROMPT_ATTN", "tile")
    test_long_prompt_prefill_matches_the_oracle(small_bf16(n_layers=2), 3, 700)


def test_prompt_chunks_with_the_swiglu_as_a_kernel_of_its_own(monkeypatch):
    """DBT_PROMPT_FUSE_SWIGLU=0: the gate|up GEMM of a prompt chunk leaves fp32 partials and the vector SwiGLU
    kernel follows (the default applies it in the GEMM's epilogue)."""
    monkeypatch.setenv("DBT_PROMPT_FUSE_SWIGLU", "0")
    test_long_prompt_prefill_matches_the_oracle(small_bf16(n_layers=2), 3, 700)


def test_prefill_in_one_call_equals_prefill_in_pieces():
    """The cache does not depend on how the prompt is cut into calls: 1500 positions at once (one chunk, six
    row tiles) and as 700 + 800 give the same logits within tolerance and caches equal to bf16 rounding."""
    cfg = small_bf16(n_layers=2)
    w = make_weights(cfg, seed=53, matrix_std=0.05)
    tok = make_tokens(cfg, 1, 1500, seed=54).cuda()
    wd = binding.weights_to_device(w)
    a, b = binding.Model(cfg, wd, 1, 1500), binding.Model(cfg, wd, 1, 1500)
    za = a.prefill(tok.contiguous(), want_logits=True)
    b.prefill(tok[:, :700].contiguous())
    zb = b.prefill(tok[:, 700:].contiguous(), want_logits=True)
    assert_logits_close(za, zb.cpu().numpy(), "bf16", "one call vs two")
    ka, va = a.export_kv(1, 1500)
    kb, vb = b.export_kv(1, 1500)
    np.testing.assert_allclose(ka.float().numpy(), kb.float().numpy(), rtol=2.0 ** -7, atol=5e-3)
    np.testing.assert_allclose(va.float().numpy(), vb.float().numpy(), rtol=2.0 ** -7, atol=5e-3)


def test_1b_width_prompt_of_2100_positions_on_a_sampled_sequence():
    """The 1B model's width (two of its layers, to keep the oracle's 2100 positions within a minute): three
    sequences prefilled together on the device, sequence 1 checked against the oracle run on it alone."""
    cfg = dense_1b().replace(n_layers=2)
    w = make_weights(cfg, seed=0)
    B, n, pick = 3, 2100, 1
    tok = make_tokens(cfg, B, n + 1, seed=2)
    gm = make_gpu_model(cfg, w, B, n + 1)
    got = gm.prefill(tok[:, :n].cuda().contiguous(), want_logits=True)
    om = oracle.OracleModel(cfg, w, 1, n + 1)
    want = om.prefill(tok[pick:pick + 1, :n].numpy())
    assert_logits_close(got[pick:pick + 1], want, "bf16", "1B-width prefill logits")
    k_dev, v_dev = gm.export_kv(1, n, seq_ids=[pick])
    np.testing.assert_allclose(k_dev.float().numpy(), om.k_cache[:, :1, :n], rtol=2.0 ** -8, atol=5e-3)
    np.testing.assert_allclose(v_dev.float().numpy(), om.v_cache[:, :1, :n], rtol=2.0 ** -8, atol=5e-3)
    o = om.decode_step(tok[pick:pick + 1, n].numpy())
    g = gm.decode_full(tok[:, n].cuda().contiguous())
    assert_logits_close(g["z1"][pick:pick + 1], o["z1"], "bf16", "step after prefill z1")
    assert_logits_close(g["z2"][pick:pick + 1], o["z2"], "bf16", "step after prefill z2")


@pytest.mark.parametrize("ctx", [0, 1, 15, 16, 17, 63, 64, 65, 255, 256, 257, 2047, 4100, 8200])
def test_context_lengths_around_page_and_chunk_boundaries(ctx):
    """Synthetic cache of `ctx` positions, then two grouped steps."""
    cfg = small_bf16(n_layers=1)
    w = make_weights(cfg, seed=9, matrix_std=0.05)
    B = 2
    tok = make_tokens(cfg, B, 2, seed=10)
    om = oracle.OracleModel(cfg, w, B, ctx + 2)
    gm = make_gpu_model(cfg, w, B, ctx + 2)
    if ctx > 0:
        k, v = make_synthetic_kv(cfg, B, ctx, seed=11)
        om.inject_kv(k, v, ctx)
        gm.import_kv(k, v)
    for t in range(2):
        o = om.decode_step(tok[:, t].numpy())
        g = gm.decode_full(tok[:, t].cuda().contiguous())
        assert_logits_close(g["z1"], o["z1"], "bf16", f"ctx {ctx} step {t} z1")
        assert_logits_close(g["z2"], o["z2"], "bf16", f"ctx {ctx} step {t} z2")


def test_1b_shape_full_width_grouped_step_with_synthetic_cache():
    """The 1B configuration at full width and depth: batch 3, a 300-position synthetic cache
    (same bytes on both sides), two grouped steps and one primary-only step."""
    cfg = dense_1b()
    w = make_weights(cfg, seed=0)
    B, ctx = 3, 300
    tok = make_tokens(cfg, B, 3, seed=2)
    k, v = make_synthetic_kv(cfg, B, ctx, seed=3)
    om = oracle.OracleModel(cfg, w, B, ctx + 3)
    gm = make_gpu_model(cfg, w, B, ctx + 3)
    om.inject_kv(k, v, ctx)
    gm.import_kv(k, v)
    for t in range(2):
        o = om.decode_step(tok[:, t].numpy())
        g = gm.decode_full(tok[:, t].cuda().contiguous())
        assert_logits_close(g["z1"], o["z1"], "bf16", f"1B step {t} z1")
        assert_logits_close(g["z2"], o["z2"], "bf16", f"1B step {t} z2")
        assert (g["alpha"].cpu().numpy() == 0.5).all() and (o["alpha"] == 0.5).all()
    o = om.decode_step(tok[:, 2].numpy(), grouped=False)
    g = gm.decode_full(tok[:, 2].cuda().contiguous(), grouped=False)
    assert_logits_close(g["z1"], o["z1"], "bf16", "1B primary-only z1")


def test_1b_at_the_benchmarks_launch_configuration_on_sampled_sequences():
    """The configuration bench.py times -- dense 1B, batch 16, context 2048 -- with the same launch
    shapes (row tile 32, the attention split of 128 pairs of 33 stages).  The oracle cannot afford 16
    sequences at this size in a test, so two of them (0 and 11) carry a seeded cache that both sides
    receive; the other fourteen are filled on the device.  Sequences do not interact, so the sampled
    rows must match the oracle run on those two sequences alone."""
    cfg = dense_1b()
    w = make_weights(cfg, seed=0)
    B, ctx, pick = 16, 2048, [0, 11]
    tok = make_tokens(cfg, B, 2, seed=2)
    k, v = make_synthetic_kv(cfg, len(pick), ctx, seed=3)
    gm = make_gpu_model(cfg, w, B, ctx + 3)
    gen = torch.Generator(device=gm.device)
    gen.manual_seed(5)
    gm.kv_pool.normal_(0.0, 1.0, generator=gen)
    gm.import_kv(k, v, seq_ids=pick)
    gm.set_seq_lens([ctx] * B)
    om = oracle.OracleModel(cfg, w, len(pick), ctx + 3)
    om.inject_kv(k, v, ctx)
    for t in range(2):
        o = om.decode_step(tok[pick, t].numpy())
        g = gm.decode_full(tok[:, t].cuda().contiguous())
        assert_logits_close(g["z1"][pick], o["z1"], "bf16", f"bench config step {t} z1")
        assert_logits_close(g["z2"][pick], o["z2"], "bf16", f"bench config step {t} z2")
    o = om.decode_step(tok[pick, 1].numpy(), grouped=False)
    g = gm.decode_full(tok[:, 1].cuda().contiguous(), grouped=False)
    assert_logits_close(g["z1"][pick], o["z1"], "bf16", "bench config primary-only z1")
    assert gm.sync_status() == (0, 0)


@pytest.mark.parametrize("cfg,lens", [
    (small_bf16(n_layers=2), [0, 5, 17, 300, 64, 63]),                        # from an empty cache to 19 pages
    (small_bf16(n_layers=2, n_paths=3), [1, 1000, 16, 15, 129]),              # three paths
    (small_bf16(n_layers=1), [7 * i % 211 for i in range(40)]),               # 80 (sequence, KV head) pairs: the one-wave attention form
    (small_bf16(n_layers=1), [900 + 13 * i for i in range(40)]),              # the same with more stages per pair than its ring holds
    (small_moe(), [3, 90, 0, 31, 32, 33, 500]),
])
def test_sequences_of_different_lengths_in_one_batch(cfg, lens):
    """A serving batch is ragged: every sequence at its own position (its own RoPE angle, page count and share of
    the attention work split).  Each sequence gets a seeded cache of its own length through dbt_kv_import;
    sequences do not interact, so row b must match the oracle run on sequence b alone (dense models: two grouped
    steps and a primary-only one; the MoE model under the device's routing, checked as a valid top-k)."""
    B, steps = len(lens), 2
    w = make_weights(cfg, seed=41, matrix_std=0.05)
    tok = make_tokens(cfg, B, steps + 1, seed=42)
    T = max(lens) + steps + 2
    gm = make_gpu_model(cfg, w, B, T)
    oms = []
    for b, n in enumerate(lens):
        om = oracle.OracleModel(cfg, w, 1, T)
        if n:
            k, v = make_synthetic_kv(cfg, 1, n, seed=100 + b)
            gm.import_kv(k, v, seq_ids=[b])
            om.inject_kv(k, v, n)
        oms.append(om)
    gm.set_seq_lens(lens)
    for t in range(steps + 1):
        grouped = t < steps or cfg.is_moe  # (the MoE model: grouped steps only, the routing of every path is read back)
        g = gm.decode_full(tok[:, t].cuda().contiguous(), grouped=grouped)
        ex = gm.last_experts(B).numpy() if cfg.is_moe else None
        for b, om in enumerate(oms):
            forced = np.ascontiguousarray(ex[:, :, b:b + 1]) if cfg.is_moe else None
            o = om.decode_step(tok[b:b + 1, t].numpy(), grouped=grouped, forced_experts=forced)
            if cfg.is_moe:
                assert_routing_is_a_valid_topk(cfg, forced, om.router_logits(1), f"seq {b} step {t}")
            assert_logits_close(g["z1"][b:b + 1], o["z1"], cfg.weight_dtype, f"seq {b} (length {lens[b] + t}) z1")
            if grouped:
                z2 = g["z2"][:, b:b + 1] if cfg.n_paths > 2 else g["z2"][b:b + 1]
                assert_logits_close(z2, o["z2"], cfg.weight_dtype, f"seq {b} (length {lens[b] + t}) z2")
    assert [gm.seq_len(b) for b in range(B)] == [n + steps + 1 for n in lens]
    assert gm.sync_status() == (0, 0)


@pytest.mark.parametrize("cfg,B", [(small_bf16(n_layers=1), 128), (small_bf16(n_layers=1), 77),
                                   (small_bf16(n_layers=1, n_paths=3), 85)])
def test_large_batches_up_to_256_stacked_rows(cfg, B):
    """The widest decode tiles: 256 stacked rows (128 sequences x 2 paths), an odd 154, and 255 rows over three
    paths; prefill of 20 positions (a chunk of more than 2048 rows is cut), three grouped steps."""
    w = make_weights(cfg, seed=43, matrix_std=0.05)
    tok = make_tokens(cfg, B, 23, seed=44)
    teacher_forced_compare(cfg, w, tok, n_prefill=20, grouped=True)


def test_1b_width_three_paths_at_batch_16_on_sampled_sequences():
    """Appendix C.1 at the benchmark's batch and the 1B model's width (four of its layers): three residual paths,
    i.e. 48 stacked rows in 64-row GEMM tiles, six query rows per KV head in the one-wave attention form (128
    pairs of different lengths: sequence b holds 100 + 40 b positions), a block per branch in the kernels between
    the GEMMs, two branch distributions in the readout.  Sequences 3 and 14 against the oracle run on each alone."""
    cfg = dense_1b().replace(n_layers=4, n_paths=3)
    w = make_weights(cfg, seed=0)
    B, pick = 16, [3, 14]
    lens = [100 + 40 * b for b in range(B)]
    tok = make_tokens(cfg, B, 2, seed=2)
    gm = make_gpu_model(cfg, w, B, max(lens) + 3)
    gen = torch.Generator(device=gm.device)
    gen.manual_seed(5)
    gm.kv_pool.normal_(0.0, 1.0, generator=gen)
    oms = {}
    for b in pick:
        k, v = make_synthetic_kv(cfg, 1, lens[b], seed=3 + b)
        gm.import_kv(k, v, seq_ids=[b])
        oms[b] = oracle.OracleModel(cfg, w, 1, lens[b] + 3)
        oms[b].inject_kv(k, v, lens[b])
    gm.set_seq_lens(lens)
    for t in range(2):
        g = gm.decode_full(tok[:, t].cuda().contiguous())
        for b in pick:
            o = oms[b].decode_step(tok[b:b + 1, t].numpy())
            assert_logits_close(g["z1"][b:b + 1], o["z1"], "bf16", f"K=3 seq {b} step {t} z1")
            for j in range(2):
                assert_logits_close(g["z2"][j][b:b + 1], o["z2"][j], "bf16", f"K=3 seq {b} step {t} branch {j + 2}")
            np.testing.assert_allclose(g["alpha"][b:b + 1].cpu().numpy(), o["alpha"], rtol=1e-3)
    assert gm.sync_status() == (0, 0)


def test_8b_width_prompt_pass_with_two_weight_tiles_per_cta():
    """The prompt pass at the 8B shape's width (one layer; d 4096, 32 query / 8 KV heads of 128, F 14336): two
    sequences of 520 positions are one chunk of 1040 rows = five row tiles, where every GEMM of the layer takes
    two weight tiles per CTA (the Q|K|V launch across its three weight matrices), and the prompt attention
    kernel runs four heads per KV head.  Last-position logits and the cache against the oracle, then a grouped
    step on the device's cache."""
    from paper_2608_12385_b200.inputs import dense_8b
    cfg = dense_8b().replace(n_layers=1)
    w = make_weights(cfg, seed=0)
    B, n = 2, 520
    tok = make_tokens(cfg, B, n + 1, seed=2)
    om = oracle.OracleModel(cfg, w, B, n + 1)
    gm = make_gpu_model(cfg, w, B, n + 1)
    want = om.prefill(tok[:, :n].numpy())
    got = gm.prefill(tok[:, :n].cuda().contiguous(), want_logits=True)
    assert_logits_close(got, want, "bf16", "8B-width prefill logits")
    k_dev, v_dev = gm.export_kv(B, n)
    np.testing.assert_allclose(k_dev.float().numpy(), om.k_cache[:, :B, :n], rtol=2.0 ** -8, atol=5e-3)
    np.testing.assert_allclose(v_dev.float().numpy(), om.v_cache[:, :B, :n], rtol=2.0 ** -8, atol=5e-3)
    o = om.decode_step(tok[:, n].numpy())
    g = gm.decode_full(tok[:, n].cuda().contiguous())
    assert_logits_close(g["z1"], o["z1"], "bf16", "step after prefill z1")
    assert_logits_close(g["z2"], o["z2"], "bf16", "step after prefill z2")
    assert gm.sync_status() == (0, 0)


# ---- readout off the clip of alpha (Eq. alpha, Eq. mixloss) ---------------------------------------------------

@pytest.mark.parametrize("cfg,matrix_std", [(small_bf16(), 0.05), (tiny_dense_fp32(), 0.02), (small_bf16(n_paths=3), 0.05)])
def test_readout_with_alpha_between_the_clips_and_at_one(cfg, matrix_std):
    """Random-init models have sum p^2 ~ 1e-3, so alpha sits on its lower clip and the mixture is symmetric
    in p and q.  An output matrix drawn with standard deviation 2.0 makes p peaked: over these 6 sequences x 4
    steps alpha lands strictly between the clips for some rows, at 1.0 for others, and argmax p != argmax q
    everywhere, so a readout that swapped p and q, used sum q^2, or mis-folded a chunk would fail here.
    The logits and their rounding errors scale with the output matrix, so the absolute bar scales by the same
    factor f; d(alpha)/dz_j = 2 p_j (p_j - alpha), hence |d alpha| <= max|dz_1|.  The readout kernels alone are
    then checked tightly: the oracle's readout of the DEVICE's own logits must reproduce the device's alpha
    and, where the mixture's top two are apart, its token."""
    dt = cfg.weight_dtype
    head_std = 2.0
    f = head_std / matrix_std
    w = make_weights(cfg, seed=41, matrix_std=matrix_std, lm_head_std=head_std)
    B, T, npre = 6, 12, 8
    tok = make_tokens(cfg, B, T, seed=42)
    om = oracle.OracleModel(cfg, w, B, T)
    gm = make_gpu_model(cfg, w, B, T)
    om.prefill(tok[:, :npre].numpy(), want_logits=False)
    gm.prefill(tok[:, :npre].cuda().contiguous())
    alphas, swapped_would_differ = [], 0
    for t in range(npre, T):
        o = om.decode_step(tok[:, t].numpy(), want_mix=True)
        g = gm.decode_full(tok[:, t].cuda().contiguous())
        z1, z2 = g["z1"].cpu().numpy(), g["z2"].cpu().numpy()
        errs = []
        for name, got in (("z1", z1), ("z2", z2)):
            d = np.abs(got.astype(np.float64) - o[name])
            rel = np.linalg.norm(got.astype(np.float64) - o[name]) / np.linalg.norm(o[name])
            assert d.max() <= TOL[dt]["max_abs"] * f and rel <= TOL[dt]["rel_l2"], (name, t, d.max(), rel)
            errs.append(d.max())
        a_dev = g["alpha"].cpu().numpy()
        np.testing.assert_allclose(a_dev, o["alpha"], rtol=1e-3, atol=errs[0])
        nxt = g["next"].cpu().numpy()
        zb = z2 if z2.ndim == 3 else z2[None]  # [branches, B, V]
        for b in range(B):
            tok_o, a_o, mix_o = oracle.readout_multi(z1[b], np.ascontiguousarray(zb[:, b]))
            assert a_dev[b] == pytest.approx(a_o, rel=2e-5), (t, b, a_dev[b], a_o)
            top = np.sort(mix_o)[-2:]
            if top[1] - top[0] > 1e-4 * top[1]:
                assert nxt[b] == tok_o, (t, b, nxt[b], tok_o)
            # what a p <-> q swap would have produced
            _, a_sw, _ = oracle.readout(zb[0, b], z1[b])
            swapped_would_differ += int(abs(a_sw - a_o) > 1e-3)
        assert (o["z1"].argmax(-1) != o["z2"].argmax(-1)).all()  # (every branch, when there are several)
        alphas.append(o["alpha"])
    alphas = np.stack(alphas)
    assert ((alphas > 0.5) & (alphas < 1.0)).sum() >= 5 and (alphas == 1.0).sum() >= 1, alphas
    assert swapped_would_differ >= 5
    assert gm.sync_status() == (0, 0)


# ---- properties that hold at any size ---------------------------------------------------------------

def _run_steps(gm, tok_dev, n_prefill, grouped):
    if n_prefill:
        gm.prefill(tok_dev[:, :n_prefill].contiguous())
    outs = [gm.decode_full(tok_dev[:, t].contiguous(), grouped=grouped) for t in range(n_prefill, tok_dev.shape[1])]
    torch.cuda.synchronize()
    return outs


@pytest.mark.parametrize("cfg", [tiny_dense_fp32().replace(n_layers=2), small_bf16(), small_moe(),
                                 small_moe(compute_matched=1), small_bf16(n_paths=3), small_moe(n_paths=4),
                                 tiny_dense_fp32().replace(n_layers=2, n_paths=3)])
def test_kv_cache_bit_identical_grouped_vs_primary_only(cfg):
    """The primary path never reads the branch: the cache written by grouped decode and by
    primary-only decode is the same bits, and so are the primary logits."""
    w = make_weights(cfg, seed=12, matrix_std=0.05)
    B, T, npre = 3, 30, 20
    tok = make_tokens(cfg, B, T, seed=13).cuda()
    wd = binding.weights_to_device(w)
    a = binding.Model(cfg, wd, B, T)
    b = binding.Model(cfg, wd, B, T)
    oa = _run_steps(a, tok, npre, True)
    ob = _run_steps(b, tok, npre, False)
    for x, y in zip(oa, ob):
        assert torch.equal(x["z1"], y["z1"])
    ka, va = a.export_kv(B, T)
    kb, vb = b.export_kv(B, T)
    assert torch.equal(ka.view(torch.int16 if cfg.weight_dtype == "bf16" else torch.int32),
                       kb.view(torch.int16 if cfg.weight_dtype == "bf16" else torch.int32))
    assert torch.equal(va.view(torch.int16 if cfg.weight_dtype == "bf16" else torch.int32),
                       vb.view(torch.int16 if cfg.weight_dtype == "bf16" else torch.int32))
    assert ka.float().abs().sum() > 0


def test_moe_kv_cache_bit_identical_at_a_batch_with_row_tiled_expert_gemms():
    """34 sequences: 68 stacked rows grouped, 34 primary-only; the per-expert GEMMs use the same row tile in
    both modes, and the cache and the primary logits are the same bits."""
    cfg = small_moe(k_primary=2, k_branch=2)
    w = make_weights(cfg, seed=14, matrix_std=0.05)
    B, T, npre = 34, 12, 8
    tok = make_tokens(cfg, B, T, seed=15).cuda()
    wd = binding.weights_to_device(w)
    a = binding.Model(cfg, wd, B, T)
    b = binding.Model(cfg, wd, B, T)
    oa = _run_steps(a, tok, npre, True)
    ob = _run_steps(b, tok, npre, False)
    for x, y in zip(oa, ob):
        assert torch.equal(x["z1"], y["z1"])
    ka, va = a.export_kv(B, T)
    kb, vb = b.export_kv(B, T)
    assert torch.equal(ka.view(torch.int16), kb.view(torch.int16))
    assert torch.equal(va.view(torch.int16), vb.view(torch.int16))


def test_moe_kv_bit_identical_at_full_width_where_the_resident_cta_count_changes_with_the_tile():
    """One layer at the MoE model's width (d 2048, experts of 1408) and 34 sequences: the grouped step's 68
    stacked rows need a row tile of 128 (one GEMM CTA per SM), the 34 primary-only rows alone would fit a tile
    of 64 (two per SM) and a split-K search over twice the slots picks other factors for the shared expert
    (11 vs 6 and 11 vs 8).  Both modes therefore size their tiles from the batch, not from the rows present,
    and the primary logits and the cache come out bit-identical."""
    cfg = moe_1b(k_branch=2).replace(n_layers=1, vocab=2048)
    w = make_weights(cfg, seed=16)
    B, T, npre = 34, 6, 4
    tok = make_tokens(cfg, B, T, seed=17).cuda()
    wd = binding.weights_to_device(w)
    a = binding.Model(cfg, wd, B, T)
    b = binding.Model(cfg, wd, B, T)
    oa = _run_steps(a, tok, npre, True)
    ob = _run_steps(b, tok, npre, False)
    for x, y in zip(oa, ob):
        assert torch.equal(x["z1"], y["z1"])
    ka, va = a.export_kv(B, T)
    kb, vb = b.export_kv(B, T)
    assert torch.equal(ka.view(torch.int16), kb.view(torch.int16))
    assert torch.equal(va.view(torch.int16), vb.view(torch.int16))


def test_kv_export_import_round_trip_through_a_shuffled_page_table():
    """dbt_kv_export returns what dbt_kv_import stored, in logical order, whatever the page table; importing
    into a subset of the sequences leaves the others' lengths and contents alone; bad requests are refused."""
    cfg = small_bf16(n_layers=2)
    w = make_weights(cfg, seed=14, matrix_std=0.05)
    B, T = 3, 45
    gm = make_gpu_model(cfg, w, B, 64, num_pages=20)
    gm.set_page_table(make_page_table(B, 4, 20, seed=16))
    k, v = make_synthetic_kv(cfg, B, T, seed=3)
    gm.import_kv(k, v)
    assert [gm.seq_len(b) for b in range(B)] == [T] * B
    k2, v2 = gm.export_kv(B, T)
    assert torch.equal(k2.view(torch.int16), k.view(torch.int16)) and torch.equal(v2.view(torch.int16), v.view(torch.int16))
    # positions live where the page table says
    view = gm.kv_view()
    pt = gm.page_table
    for (l, b, t) in [(0, 0, 0), (1, 2, 17), (1, 1, 44)]:
        page, slot = int(pt[b, t // 16]), t % 16
        got = view[l, 0, page, :, slot, :].reshape(-1).cpu()
        assert torch.equal(got.view(torch.int16), k[l, b, t].view(torch.int16))
    # a subset, shorter: only sequence 2 changes
    k3, v3 = make_synthetic_kv(cfg, 1, 10, seed=5)
    gm.import_kv(k3, v3, seq_ids=[2])
    assert [gm.seq_len(b) for b in range(B)] == [T, T, 10]
    k4, _ = gm.export_kv(2, T)
    assert torch.equal(k4.view(torch.int16), k[:, :2].contiguous().view(torch.int16))
    k5, _ = gm.export_kv(1, 10, seq_ids=[2])
    assert torch.equal(k5.view(torch.int16), k3.view(torch.int16))
    with pytest.raises(binding.DbtError) as e:
        gm.export_kv(1, 11, seq_ids=[2])  # longer than the sequence
    assert e.value.status == 4
    with pytest.raises(binding.DbtError) as e:
        gm.import_kv(*make_synthetic_kv(cfg, 1, 65, seed=6))  # beyond four pages
    assert e.value.status == 3
    assert gm.sync_status() == (0, 0)


def test_page_table_permutation_does_not_change_results():
    cfg = small_bf16(n_layers=2)
    w = make_weights(cfg, seed=14, matrix_std=0.05)
    B, T, npre = 3, 60, 50
    tok = make_tokens(cfg, B, T, seed=15).cuda()
    wd = binding.weights_to_device(w)
    a = binding.Model(cfg, wd, B, T)
    b = binding.Model(cfg, wd, B, T, num_pages=64)
    pt = make_page_table(B, (T + 15) // 16, 64, seed=16)
    b.set_page_table(pt)
    oa = _run_steps(a, tok, npre, True)
    ob = _run_steps(b, tok, npre, True)
    for x, y in zip(oa, ob):
        assert torch.equal(x["z1"], y["z1"]) and torch.equal(x["z2"], y["z2"]) and torch.equal(x["next"], y["next"])
    ka, _ = a.export_kv(B, T)
    kb, _ = b.export_kv(B, T)
    assert torch.equal(ka.float(), kb.float())


def test_sequences_do_not_depend_on_batch_mates_and_runs_are_deterministic():
    cfg = small_bf16(n_layers=2)
    w = make_weights(cfg, seed=17, matrix_std=0.05)
    T, npre = 40, 33
    tok = make_tokens(cfg, 4, T, seed=18).cuda()
    wd = binding.weights_to_device(w)
    full = _run_steps(binding.Model(cfg, wd, 4, T), tok, npre, True)
    again = _run_steps(binding.Model(cfg, wd, 4, T), tok, npre, True)
    solo = _run_steps(binding.Model(cfg, wd, 4, T), tok[2:3].contiguous(), npre, True)
    for x, y, z in zip(full, again, solo):
        assert torch.equal(x["z1"], y["z1"]) and torch.equal(x["z2"], y["z2"])
        # a different batch size may pick a different split of the KV range: compare within tolerance
        assert_logits_close(z["z1"][0], x["z1"][2].cpu().numpy(), "bf16")
        assert_logits_close(z["z2"][0], x["z2"][2].cpu().numpy(), "bf16")


def test_host_buffer_entry_points_match_device_entry_points():
    cfg = small_bf16(n_layers=2)
    w = make_weights(cfg, seed=19, matrix_std=0.05)
    B = 3
    tok = make_tokens(cfg, B, 12, seed=20)
    wd = binding.weights_to_device(w)
    a, b = binding.Model(cfg, wd, B, 32), binding.Model(cfg, wd, B, 32)
    a.prefill(tok[:, :8].cuda().contiguous())
    b.prefill(tok[:, :8].cuda().contiguous())
    cur_dev = tok[:, 8].cuda().contiguous()
    cur_host = tok[:, 8].clone().pin_memory()
    nxt_host = torch.empty(B, dtype=torch.int32).pin_memory()
    alpha_host = torch.empty(B, dtype=torch.float32).pin_memory()
    for i in range(4):  # free-running greedy decode, next tokens fed back
        grouped = i % 2 == 0
        out = a.decode_full(cur_dev, grouped=grouped)
        if grouped:
            b.decode_step_host(cur_host, nxt_host, alpha_host)
            assert torch.equal(alpha_host, out["alpha"].cpu())
        else:
            b.decode_step_primary_only_host(cur_host, nxt_host)
        assert torch.equal(nxt_host, out["next"].cpu())
        cur_dev = out["next"].clone()
        cur_host.copy_(nxt_host)
    assert a.seq_len(0) == b.seq_len(0) == 12
    assert a.launch_count() > 0


# ---- MoE ----------------------------------------------------------------------------------------------

ROUTER_EPS = {"bf16": 1e-2, "fp32": 1e-4}  # router logits are O(1); half the bar on model logits


def assert_routing_is_a_valid_topk(cfg, ex, rlog, what=""):
    """ex [L, K, B, kmax]: the device's expert ids; rlog [L, K, B, E]: the oracle's router logits for the same
    rows (computed under the device's choice in the earlier layers).  Eq. moe_layer fixes the selected set
    only up to rounding at near-ties, so what must hold is: k distinct experts per row, none of them below
    an unselected expert by more than the logit tolerance (softmax is monotone, so logits order as the
    probabilities do), the unused slots -1, and under router replay (Section 4.3) the branch's set is the
    primary's."""
    eps = ROUTER_EPS[cfg.weight_dtype]
    L, K, B, _ = ex.shape
    assert K == cfg.n_paths
    replay = cfg.router_mode == 1
    for l in range(L):
        for p in range(K):
            k = cfg.k_primary if (p == 0 or replay) else cfg.k_branch
            for b in range(B):
                chosen = ex[l, p, b, :k]
                assert (ex[l, p, b, k:] == -1).all(), f"{what} layer {l} path {p} row {b}: unused slots"
                assert ((chosen >= 0) & (chosen < cfg.n_experts)).all() and len(set(chosen.tolist())) == k, \
                    f"{what} layer {l} path {p} row {b}: {chosen}"
                if p >= 1 and replay:
                    assert chosen.tolist() == ex[l, 0, b, :k].tolist(), f"{what} layer {l} row {b}: replay set"
                    continue
                r = rlog[l, p, b]
                rest = np.delete(r, chosen)
                if rest.size:
                    assert r[chosen].min() >= rest.max() - eps, \
                        f"{what} layer {l} path {p} row {b}: chose {chosen} with logits {r[chosen]}, left {rest.max()}"


def _moe_compare(cfg, B, T, npre, matrix_std=0.05):
    w = make_weights(cfg, seed=21, matrix_std=matrix_std)
    tok = make_tokens(cfg, B, T, seed=22)
    om = oracle.OracleModel(cfg, w, B, T)
    gm = make_gpu_model(cfg, w, B, T)
    z1_full, _, k_full, v_full = oracle.full_forward(cfg, w, tok[:, :npre].numpy(), want_kv=True)
    om.inject_kv(k_full, v_full, npre)
    # the decode steps below start from the oracle's cache on both sides and impose the device's routing
    # on the oracle; the prefill itself is compared in test_moe_prefill_matches_the_oracle
    gm.import_kv(torch.from_numpy(k_full), torch.from_numpy(v_full))
    for t in range(npre, T):
        g = gm.decode_full(tok[:, t].cuda().contiguous())
        ex = gm.last_experts(B).numpy()
        o = om.decode_step(tok[:, t].numpy(), forced_experts=ex)
        assert_routing_is_a_valid_topk(cfg, ex, om.router_logits(B), f"step {t}")
        assert_logits_close(g["z1"], o["z1"], cfg.weight_dtype, f"moe step {t} z1")
        assert_logits_close(g["z2"], o["z2"], cfg.weight_dtype, f"moe step {t} z2")
        union = gm.last_expert_union()
        for l in range(cfg.n_layers):
            assert union[l] == len(set(ex[l][ex[l] >= 0].tolist()))
    assert gm.sync_status() == (0, 0)


@pytest.mark.parametrize("cfg", [small_moe(), small_moe(router_mode=1), small_moe(n_shared_experts=0, k_branch=8),
                                 small_moe(moe_b_coupling=0, k_primary=1, k_branch=1)])
def test_moe_decode_matches_oracle_under_the_devices_routing(cfg):
    """Router near-ties are decided by rounding, so the device's expert choice is read back, checked
    row by row against the oracle's router logits (a valid top-k up to the logit tolerance), and imposed
    on the oracle; everything else is compared element by element."""
    _moe_compare(cfg, B=3, T=14, npre=10)


@pytest.mark.parametrize("rowtile", ["auto", "32", "16", "0"])
def test_moe_at_batch_40(monkeypatch, rowtile):
    """40 sequences: 80 stacked rows over 8 experts, so every expert's list is longer than a row tile of 16
    or 32 and the per-expert GEMMs walk several row tiles per expert (0: one tile of 128 rows)."""
    if rowtile != "auto":
        monkeypatch.setenv("DBT_MOE_ROWTILE", rowtile)
    _moe_compare(small_moe(k_primary=2, k_branch=2), B=40, T=7, npre=5)


def test_moe_1b_shape_two_layers():
    cfg = moe_1b(k_branch=4).replace(n_layers=2)
    _moe_compare(cfg, B=2, T=8, npre=6, matrix_std=0.02)


@pytest.mark.parametrize("cfg", [small_moe(), small_moe(weight_dtype="fp32"), small_moe(compute_matched=1)])
def test_moe_prefill_matches_the_oracle(cfg):
    """dbt_prefill of an MoE model (Section 4.4 item 1: the primary path alone, fan-out k_1) against the
    oracle's position-by-position primary pass: last-position logits and every cached K and V.  The router
    matrix is scaled by 8 so that the k_1-th and (k_1+1)-th logits of every prompt row are far apart
    (checked below on the oracle's logits): the selected sets are then unique and both sides must agree."""
    w = make_weights(cfg, seed=79, matrix_std=0.05)
    for lw in w["layers"]:
        lw["router"] = (lw["router"].float() * 8).to(cfg.torch_dtype)
    B, n = 3, 40
    tok = make_tokens(cfg, B, n + 2, seed=179)
    om = oracle.OracleModel(cfg, w, B, n + 2)
    margin = np.inf
    for t in range(n):  # the oracle's prefill is this loop (orc_prefill walks the prompt the same way)
        o = om.decode_step(tok[:, t].numpy(), grouped=False)
        r = -np.sort(-om.router_logits(B)[:, 0], axis=-1)
        margin = min(margin, float((r[..., cfg.k_primary - 1] - r[..., cfg.k_primary]).min()))
    # device router logits at this scale are good to ~8e-3 (8 x the error on unit-scale logits)
    assert margin > 0.03, f"router logits not separated: {margin}"
    gm = make_gpu_model(cfg, w, B, n + 2)
    got = gm.prefill(tok[:, :n].cuda().contiguous(), want_logits=True)
    assert_logits_close(got, o["z1"], cfg.weight_dtype, "moe prefill logits")
    k_dev, v_dev = gm.export_kv(B, n)
    # the device stores K and V in the model's type: bf16 rounding (2^-9 relative) on top of the logit-level error
    rtol, atol = (2.0 ** -8, 5e-3) if cfg.weight_dtype == "bf16" else (1e-4, 1e-5)
    np.testing.assert_allclose(k_dev.float().numpy(), om.k_cache[:, :B, :n], rtol=rtol, atol=atol)
    np.testing.assert_allclose(v_dev.float().numpy(), om.v_cache[:, :B, :n], rtol=rtol, atol=atol)
    assert float(k_dev.float().abs().max()) > 0.1
    # and the caches are interchangeable: a grouped step on top of the device's own prefill
    o2 = om.decode_step(tok[:, n].numpy())
    g2 = gm.decode_full(tok[:, n].cuda().contiguous())
    ex = gm.last_experts(B).numpy()
    assert_routing_is_a_valid_topk(cfg, ex, om.router_logits(B), "step after prefill")
    if (np.sort(ex, -1) == np.sort(o2["experts"], -1)).all():
        assert_logits_close(g2["z1"], o2["z1"], cfg.weight_dtype, "step after moe prefill z1")
        assert_logits_close(g2["z2"], o2["z2"], cfg.weight_dtype, "step after moe prefill z2")
    assert gm.sync_status() == (0, 0)


@pytest.mark.parametrize("cfg,B,n,std", [(small_moe(), 3, 100, 0.05), (small_moe(), 1, 700, 0.05),
                                         (moe_1b(k_branch=2).replace(n_layers=2), 1, 300, 0.02)])
def test_moe_prompt_chunks_of_more_than_one_row_tile_match_the_oracle(cfg, B, n, std):
    """The MoE model's prompt pass in chunks of more than 256 rows (row-tiled GEMMs, the prompt attention kernel,
    64-row tiles with two weight tiles per CTA in the per-expert GEMMs, the shared-memory-atomic sort, the vector
    combine) against the oracle's position-by-position primary pass.  With hundreds of prompt rows some router
    near-ties are unavoidable, and there the selected set is not unique (Eq. moe_layer fixes it up to rounding):
    a row whose k_1-th and (k_1+1)-th oracle logits are closer than the margin in some layer is left out of the
    cache comparison (its own entries may legitimately differ; its influence on other rows goes through
    attention and stays far below the tolerance); every other position must match in every layer."""
    w = make_weights(cfg, seed=83, matrix_std=std)
    for lw in w["layers"]:
        lw["router"] = (lw["router"].float() * 8).to(cfg.torch_dtype)
    tok = make_tokens(cfg, B, n + 1, seed=183)
    om = oracle.OracleModel(cfg, w, B, n + 1)
    near = np.zeros((B, n), dtype=bool)
    for t in range(n):
        o = om.decode_step(tok[:, t].numpy(), grouped=False)
        r = -np.sort(-om.router_logits(B)[:, 0], axis=-1)                      # [L, B, E]
        near[:, t] = ((r[..., cfg.k_primary - 1] - r[..., cfg.k_primary]) < 0.03).any(axis=0)
    assert near.mean() < 0.2, "too many near-ties for the test to say anything"
    gm = make_gpu_model(cfg, w, B, n + 1)
    got = gm.prefill(tok[:, :n].cuda().contiguous(), want_logits=True)
    k_dev, v_dev = gm.export_kv(B, n)
    keep = ~near
    assert keep.sum() > 0.8 * B * n
    np.testing.assert_allclose(k_dev.float().numpy()[:, keep], om.k_cache[:, :B, :n][:, keep], rtol=2.0 ** -7, atol=1e-2)
    np.testing.assert_allclose(v_dev.float().numpy()[:, keep], om.v_cache[:, :B, :n][:, keep], rtol=2.0 ** -7, atol=1e-2)
    last_ok = keep[:, n - 1]
    if last_ok.any():
        assert_logits_close(got[torch.from_numpy(last_ok)], o["z1"][last_ok], cfg.weight_dtype, "moe long-prompt logits")
    assert gm.sync_status() == (0, 0)


@pytest.mark.parametrize("matched", [0, 1])
def test_moe_1b_at_the_benchmarks_launch_configuration_on_sampled_sequences(matched):
    """The MoE configuration bench.py times -- 64 experts x 1408 + 1 shared, 16 layers, batch 8, context
    4096, top-2 primary + top-2 branch -- with the same launch shapes (row tile 16, 32 attention pairs of 9
    segments, the shared expert beside the routed chain).  Two sequences (0 and 5) carry a seeded cache that
    both sides receive; the oracle runs them alone under the experts the device chose for them."""
    cfg = moe_1b(k_branch=2).replace(compute_matched=matched)
    w = make_weights(cfg, seed=0)
    B, ctx, pick = 8, 4096, [0, 5]
    tok = make_tokens(cfg, B, 2, seed=2)
    k, v = make_synthetic_kv(cfg, len(pick), ctx, seed=3)
    gm = make_gpu_model(cfg, w, B, ctx + 3)
    gen = torch.Generator(device=gm.device)
    gen.manual_seed(5)
    gm.kv_pool.normal_(0.0, 1.0, generator=gen)
    gm.import_kv(k, v, seq_ids=pick)
    gm.set_seq_lens([ctx] * B)
    om = oracle.OracleModel(cfg, w, len(pick), ctx + 3)
    om.inject_kv(k, v, ctx)
    for t in range(2):
        g = gm.decode_full(tok[:, t].cuda().contiguous())
        ex = gm.last_experts(B).numpy()[:, :, pick]
        o = om.decode_step(tok[pick, t].numpy(), forced_experts=np.ascontiguousarray(ex))
        assert_routing_is_a_valid_topk(cfg, np.ascontiguousarray(ex), om.router_logits(len(pick)), f"step {t}")
        assert_logits_close(g["z1"][pick], o["z1"], "bf16", f"moe bench config step {t} z1")
        assert_logits_close(g["z2"][pick], o["z2"], "bf16", f"moe bench config step {t} z2")
    assert gm.sync_status() == (0, 0)


# ---- more decode branches (Appendix C.1) ----------------------------------------------------------------------

@pytest.mark.parametrize("cfg,B,T,npre", [
    (small_bf16(n_paths=3), 3, 40, 35),                                        # 3 paths x 4 queries per KV head: 12 of 16 rows
    (small_bf16(n_paths=4, n_q_heads=4, n_kv_heads=4), 2, 24, 20),             # MHA, 4 paths
    (small_bf16(n_paths=8, n_q_heads=2, n_kv_heads=1, head_dim=128, d_model=128, vocab=777), 5, 50, 47),  # 8 paths, 16 rows
    (tiny_dense_fp32().replace(n_paths=3), 2, 30, 25),                         # the fp32 kernels
    (small_bf16(n_paths=3, n_q_heads=8, n_kv_heads=2), 33, 20, 18),            # 99 stacked rows: row tile 128
])
def test_more_decode_branches_dense(cfg, B, T, npre):
    """K > 2: every branch's logits, alpha and the token of alpha p + (1-alpha) mean_j q_j against the oracle."""
    w = make_weights(cfg, seed=5, matrix_std=0.05 if cfg.weight_dtype == "bf16" else 0.02)
    tok = make_tokens(cfg, B, T, seed=6)
    teacher_forced_compare(cfg, w, tok, n_prefill=npre, grouped=True)


@pytest.mark.parametrize("cfg", [small_moe(n_paths=3), small_moe(n_paths=3, router_mode=1),
                                 small_moe(n_paths=4, compute_matched=1), small_moe(n_paths=3, weight_dtype="fp32")])
def test_more_decode_branches_moe(cfg):
    """Every branch routes for itself (fan-out k_2; router replay: the primary's set), checked row by row."""
    _moe_compare(cfg, B=3, T=14, npre=10)


def test_identical_branch_tables_give_identical_branch_logits_on_the_device():
    cfg = small_bf16(n_paths=3)
    w = make_weights(cfg, seed=5, matrix_std=0.05)
    V = cfg.vocab
    w["embed_branch"] = torch.cat([w["embed_branch"][:V], w["embed_branch"][:V]]).contiguous()
    tok = make_tokens(cfg, 3, 24, seed=6).cuda()
    gm = make_gpu_model(cfg, w, 3, 24)
    for o in _run_steps(gm, tok, 20, True):
        assert torch.equal(o["z2"][0], o["z2"][1]) and float(o["z2"].abs().max()) > 0


def test_too_many_query_rows_over_all_paths_are_rejected():
    cfg = small_bf16(n_paths=5)  # 5 paths x 4 queries per KV head > 16
    w = make_weights(cfg, seed=0)
    with pytest.raises(binding.DbtError) as e:
        make_gpu_model(cfg, w, 1, 16)
    assert e.value.status == 2


# ---- compute-matched MoE allocation (Appendix B.3) ---------------------------------------------------------

@pytest.mark.parametrize("cfg", [small_moe(compute_matched=1, k_primary=3, k_branch=1),
                                 small_moe(compute_matched=1, k_primary=2, k_branch=2, n_shared_experts=2),
                                 small_moe(compute_matched=1, k_primary=1, k_branch=3, n_shared_experts=0),
                                 small_moe(compute_matched=1, router_mode=1),
                                 small_moe(compute_matched=1, n_q_heads=8, n_kv_heads=1, head_dim=128, d_model=384),
                                 small_moe(compute_matched=1, weight_dtype="fp32")])
def test_compute_matched_moe_decode_matches_oracle(cfg):
    """The branch evaluates neither attention nor the shared expert: A_2 = g_A * A_1 and
    M_2 = R_2(N_2; k_2) + g_G * G(N_1), compared element by element under the device's routing."""
    _moe_compare(cfg, B=3, T=14, npre=10)


@pytest.mark.parametrize("knob,value", [("DBT_FORCE_PATH", "simt"), ("DBT_ATTN", "simt"), ("DBT_MOE", "simt"),
                                        ("DBT_FUSE_QKV", "0"), ("DBT_GRAPH", "0"), ("DBT_MOE_OVERLAP", "0")])
def test_compute_matched_moe_on_the_alternative_chains(monkeypatch, knob, value):
    monkeypatch.setenv(knob, value)
    _moe_compare(small_moe(compute_matched=1, k_primary=2, k_branch=2), B=5, T=13, npre=9)


@pytest.mark.parametrize("knob,value", [("DBT_MOE_OVERLAP", "0"), ("DBT_GRAPH", "0"), ("DBT_MOE", "simt"),
                                        ("DBT_FUSE_QKV", "0"), ("DBT_ATTN", "simt"), ("DBT_MOE_PERSIST", "0"),
                                        ("DBT_MOE_PERSIST", "1"), ("DBT_MOE_FUSE_SWIGLU", "0")])
def test_moe_on_the_alternative_chains(monkeypatch, knob, value):
    """The shared expert on the main stream instead of beside the routed chain, direct launches instead
    of graph replay, the CUDA-core expert kernels, the separate Q|K|V epilogue kernel, the CUDA-core
    attention kernel, the per-expert GEMMs as one CTA per unit / as persistent CTAs (the default takes the
    persistent form up to 16 stacked rows)."""
    monkeypatch.setenv(knob, value)
    _moe_compare(small_moe(), B=5, T=13, npre=9)


@pytest.mark.parametrize("cfg,B", [(small_moe(), 5), (small_moe(k_branch=8, n_shared_experts=0), 3),
                                   (moe_1b(k_branch=2).replace(n_layers=2), 12), (small_moe(n_paths=3), 20)])
def test_persistent_per_expert_gemm_gives_the_same_bits(monkeypatch, cfg, B):
    """Both forms of the per-expert GEMM launch add the same products in the same order: logits, expert choice
    and cache are the same bits (row tiles of 16 and of 32 rows, several row tiles per expert at batch 20 x 3
    paths, grouped and primary-only steps)."""
    w = make_weights(cfg, seed=71, matrix_std=0.02 if cfg.d_model > 1000 else 0.05)
    T, npre = 9, 6
    tok = make_tokens(cfg, B, T, seed=72).cuda()
    wd = binding.weights_to_device(w)
    runs = {}
    for value in ("0", "1"):
        monkeypatch.setenv("DBT_MOE_PERSIST", value)
        for grouped in (True, False):
            gm = binding.Model(cfg, wd, B, T)
            outs = _run_steps(gm, tok, npre, grouped)
            runs[value, grouped] = (outs, gm.export_kv(B, T), gm.last_experts(B))
            assert gm.sync_status() == (0, 0)
    for grouped in (True, False):
        (oa, kva, ea), (ob, kvb, eb) = runs["0", grouped], runs["1", grouped]
        for x, y in zip(oa, ob):
            assert torch.equal(x["z1"], y["z1"])
            if grouped:
                assert torch.equal(x["z2"], y["z2"])
        assert torch.equal(kva[0].float(), kvb[0].float()) and torch.equal(kva[1].float(), kvb[1].float())
        assert torch.equal(ea, eb)


def test_compute_matched_moe_1b_shape_two_layers():
    cfg = moe_1b(k_branch=2).replace(n_layers=2, compute_matched=1)
    _moe_compare(cfg, B=2, T=8, npre=6, matrix_std=0.02)


def test_compute_matched_unit_gates_same_embedding_equal_fanout_give_identical_paths():
    """S_2^0 = S_1^0, A_2 = A_1, R_2 = R_1 and M_2 = R_1 + G(N_1): the two paths' logits are the same bits,
    at the full MoE width and batch 16."""
    cfg = moe_1b(k_branch=2).replace(n_layers=2, compute_matched=1)
    w = make_weights(cfg, seed=31)
    w["embed_branch"] = w["embed_primary"].clone()
    for lw in w["layers"]:
        lw["gate_a"] = torch.ones_like(lw["gate_a"])
        lw["gate_g"] = torch.ones_like(lw["gate_g"])
    B, T, npre = 16, 40, 37
    tok = make_tokens(cfg, B, T, seed=32).cuda()
    gm = make_gpu_model(cfg, w, B, T)
    for o in _run_steps(gm, tok, npre, True):
        assert torch.equal(o["z1"], o["z2"])
        assert float(o["z1"].abs().max()) > 0


def test_compute_matched_is_rejected_for_dense_models():
    cfg = small_bf16(n_layers=1)
    w = make_weights(cfg, seed=0)
    with pytest.raises(binding.DbtError):
        make_gpu_model(cfg.replace(compute_matched=1), w, 1, 16)


# ---- error paths (host-detected, and device-detected without any fault) ---------------------------------

def test_capacity_and_argument_errors():
    cfg = small_bf16(n_layers=1)
    w = make_weights(cfg, seed=23, matrix_std=0.05)
    gm = make_gpu_model(cfg, w, 2, 20)
    tok = make_tokens(cfg, 2, 21, seed=24).cuda()
    with pytest.raises(binding.DbtError) as e:
        gm.prefill(tok.contiguous())
    assert e.value.status == 3
    gm.prefill(tok[:, :20].contiguous())
    with pytest.raises(binding.DbtError) as e:
        gm.decode_step(tok[:, 20].contiguous())
    assert e.value.status == 3
    gm.reset()
    with pytest.raises(binding.DbtError) as e:
        gm.decode_step(make_tokens(cfg, 3, 1).cuda().view(-1))
    assert e.value.status == 3
    with pytest.raises(binding.DbtError):
        gm.set_page_table(torch.tensor([[0, 0], [1, 2]]))


def test_out_of_range_token_is_reported_not_faulted():
    cfg = small_bf16(n_layers=1)
    w = make_weights(cfg, seed=25, matrix_std=0.05)
    gm = make_gpu_model(cfg, w, 2, 8)
    bad = torch.tensor([3, cfg.vocab + 5], dtype=torch.int32).cuda()
    gm.decode_step(bad)
    status, detail = gm.sync_status()
    assert status == 1 and detail == cfg.vocab + 5
    gm.reset()
    gm.decode_step(torch.tensor([3, 4], dtype=torch.int32).cuda())
    assert gm.sync_status() == (0, 0)


def test_fresh_models_give_bitwise_identical_results():
    """Three handles built one after another run the same prefill and grouped steps: every logit
    is bit-identical (kernels overlap through programmatic dependent launch; a read issued
    before its producer finished would show up here as run-to-run noise)."""
    cfg = small_bf16(n_q_heads=2, n_kv_heads=1, head_dim=128, d_model=128, vocab=777)
    w = make_weights(cfg, seed=5, matrix_std=0.05)
    B, T, npre = 5, 50, 47
    tok = make_tokens(cfg, B, T, seed=6).cuda()
    wd = binding.weights_to_device(w)
    runs = []
    for _ in range(3):
        gm = binding.Model(cfg, wd, B, T)
        runs.append(_run_steps(gm, tok, npre, True))
    for other in runs[1:]:
        for x, y in zip(runs[0], other):
            assert torch.equal(x["z1"], y["z1"]) and torch.equal(x["z2"], y["z2"])


@pytest.mark.parametrize("knob,value", [("DBT_READOUT", "row"), ("DBT_FUSE_QKV", "0"), ("DBT_EVICT_FIRST", "0"),
                                        ("DBT_GRAPH", "0"), ("DBT_PDL", "0"), ("DBT_ATTN", "simt"),
                                        ("DBT_FORCE_PATH", "simt")])
def test_alternative_kernel_chains_match_oracle(monkeypatch, knob, value):
    """The fallbacks of the dense chain -- the one-CTA-per-row readout (vocabularies beyond the chunked
    kernel's reach), a separate Q|K|V epilogue kernel (the one prefill uses), no L2 eviction hints, direct
    launches instead of graph replay, no programmatic dependent launch, the CUDA-core attention and GEMM
    kernels (what fp32 models run on) -- compute the same step."""
    monkeypatch.setenv(knob, value)
    cfg = small_bf16()
    w = make_weights(cfg, seed=5, matrix_std=0.05)
    tok = make_tokens(cfg, 3, 40, seed=6)
    teacher_forced_compare(cfg, w, tok, n_prefill=35, grouped=True)
    teacher_forced_compare(cfg, w, tok, n_prefill=35, grouped=False)


def test_8b_shape_two_layers_paged_with_shuffled_pages():
    """The 8B-shaped configuration at full width (d 4096, 32 query / 8 KV heads, F 14336, vocab
    128256) with two layers: batch 2, a 100-position synthetic cache scattered over a shuffled
    page table, two grouped steps."""
    from paper_2608_12385_b200.inputs import dense_8b
    cfg = dense_8b().replace(n_layers=2)
    w = make_weights(cfg, seed=0)
    B, ctx = 2, 100
    tok = make_tokens(cfg, B, 2, seed=2)
    k, v = make_synthetic_kv(cfg, B, ctx, seed=3)
    om = oracle.OracleModel(cfg, w, B, ctx + 2)
    gm = make_gpu_model(cfg, w, B, ctx + 2, num_pages=40)
    pt = make_page_table(B, (ctx + 2 + 15) // 16, 40, seed=4)
    gm.set_page_table(pt)
    om.inject_kv(k, v, ctx)
    gm.import_kv(k, v)
    for t in range(2):
        o = om.decode_step(tok[:, t].numpy())
        g = gm.decode_full(tok[:, t].cuda().contiguous())
        assert_logits_close(g["z1"], o["z1"], "bf16", f"8B-shape step {t} z1")
        assert_logits_close(g["z2"], o["z2"], "bf16", f"8B-shape step {t} z2")

"""Seeded synthetic inputs: model shapes, random-init weights, token streams, KV fills.

This module is the one piece shared by the CPU oracle's tests and the CUDA path's tests
and benchmark.  It holds no arithmetic of the method -- only shapes, seeds and draws from
torch's CPU generator -- so both sides see byte-identical inputs.  Tensors are torch CPU
tensors (fp32, or bf16 produced by round-to-nearest-even from the fp32 draw).

Shapes follow the paper's experimental families (LLaMA-style dense with RMSNorm, RoPE,
gated MLP and GQA; Qwen-style MoE with routed and shared experts); trained weights and
real prompts are replaced by N(0, 0.02) matrices and uniform random token ids.
"""
from __future__ import annotations

import dataclasses
from dataclasses import dataclass

import torch


@dataclass
class ModelConfig:
    d_model: int
    n_layers: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    d_ff: int
    vocab: int
    weight_dtype: str = "bf16"  # "fp32" | "bf16"; the KV cache uses the same storage type
    rope_base: float = 10000.0
    rms_eps: float = 1e-5
    final_norm: int = 1
    n_experts: int = 0
    d_expert: int = 0
    n_shared_experts: int = 0
    k_primary: int = 0
    k_branch: int = 0
    router_mode: int = 0  # 0 independent routing, 1 router replay
    moe_b_coupling: int = 1
    compute_matched: int = 0  # 1: compute-matched MoE allocation (Appendix B.3): A_2 = g_A*A_1, shared expert gated
    n_paths: int = 2  # K of Appendix C.1: the primary path plus K-1 decode branches (own embedding table each)
    page_size: int = 16

    @property
    def q_dim(self) -> int:
        return self.n_q_heads * self.head_dim

    @property
    def kv_dim(self) -> int:
        return self.n_kv_heads * self.head_dim

    @property
    def is_moe(self) -> bool:
        return self.n_experts > 0

    @property
    def kmax(self) -> int:
        return max(self.k_primary, self.k_branch, 1)

    @property
    def torch_dtype(self) -> torch.dtype:
        return torch.float32 if self.weight_dtype == "fp32" else torch.bfloat16

    @property
    def elem_bytes(self) -> int:
        return 4 if self.weight_dtype == "fp32" else 2

    def replace(self, **kw) -> "ModelConfig":
        return dataclasses.replace(self, **kw)

    def matrix_bytes_dense_step(self) -> int:
        """Bytes of the shared matrices one dense decode step must read once each."""
        per_layer = (self.q_dim + 2 * self.kv_dim) * self.d_model + self.d_model * self.q_dim
        per_layer += 3 * self.d_ff * self.d_model if not self.is_moe else 0
        return (self.n_layers * per_layer + self.vocab * self.d_model) * self.elem_bytes

    def matrix_bytes_moe_step(self, experts_loaded_per_layer) -> int:
        """Bytes of the matrices one MoE decode step must read once each: attention projections,
        router, shared expert, output matrix, and the routed experts actually selected
        (`experts_loaded_per_layer`: the size of the union over all rows of both paths)."""
        attn = (self.q_dim + 2 * self.kv_dim) * self.d_model + self.d_model * self.q_dim
        router = self.n_experts * self.d_model
        shared = 3 * self.n_shared_experts * self.d_expert * self.d_model
        expert = 3 * self.d_expert * self.d_model
        total = self.n_layers * (attn + router + shared) + self.vocab * self.d_model
        total += expert * int(sum(experts_loaded_per_layer))
        return total * self.elem_bytes

    def kv_bytes_per_token(self) -> int:
        return 2 * self.kv_dim * self.n_layers * self.elem_bytes


# The workload family of the grouped-decode study.
def tiny_dense_fp32() -> ModelConfig:
    return ModelConfig(d_model=256, n_layers=4, n_q_heads=4, n_kv_heads=4, head_dim=64, d_ff=704,
                       vocab=4096, weight_dtype="fp32")


def dense_1b() -> ModelConfig:
    return ModelConfig(d_model=2048, n_layers=16, n_q_heads=16, n_kv_heads=8, head_dim=128, d_ff=5632,
                       vocab=32000, weight_dtype="bf16")


def dense_8b() -> ModelConfig:
    return ModelConfig(d_model=4096, n_layers=32, n_q_heads=32, n_kv_heads=8, head_dim=128, d_ff=14336,
                       vocab=128256, weight_dtype="bf16")


def moe_1b(k_branch: int = 2) -> ModelConfig:
    return ModelConfig(d_model=2048, n_layers=16, n_q_heads=16, n_kv_heads=4, head_dim=128, d_ff=0,
                       vocab=32000, weight_dtype="bf16", n_experts=64, d_expert=1408,
                       n_shared_experts=1, k_primary=2, k_branch=k_branch)


PRESETS = {"tiny": tiny_dense_fp32, "1b": dense_1b, "8b": dense_8b, "moe": moe_1b}

LAYER_MATRICES_DENSE = ("wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down")
LAYER_MATRICES_MOE = ("wq", "wk", "wv", "wo", "router", "exp_gate", "exp_up", "exp_down",
                      "sh_gate", "sh_up", "sh_down")
LAYER_VECTORS = ("attn_norm_g", "coup_a", "mlp_norm_g", "coup_b", "coup_c", "gate_a", "gate_g")


def _normal(gen: torch.Generator, shape, std: float, dtype: torch.dtype, mean: float = 0.0) -> torch.Tensor:
    t = torch.empty(shape, dtype=torch.float32)
    t.normal_(mean, std, generator=gen)
    return t.to(dtype).contiguous()


def make_weights(cfg: ModelConfig, seed: int = 0, coupling_std: float = 0.5,
                 matrix_std: float = 0.02, lm_head_std: float | None = None) -> dict:
    """Random-init weights: matrices and embeddings N(0, matrix_std), router N(0, 1/d)
    (router logits come out near N(0,1)), norm gains 1 + N(0, 0.02), coupling vectors
    N(0, coupling_std).  Couplings are O(1) on purpose: a dropped coupling then moves the
    branch logits by far more than any parity tolerance."""
    gen = torch.Generator(device="cpu")
    gen.manual_seed(seed)
    wd = cfg.torch_dtype
    d, qd, kvd = cfg.d_model, cfg.q_dim, cfg.kv_dim
    w: dict = {
        "embed_primary": _normal(gen, (cfg.vocab, d), matrix_std, wd),
        # E_2 .. E_K, one table per decode branch, stacked [(K-1) * V, d]
        "embed_branch": _normal(gen, ((cfg.n_paths - 1) * cfg.vocab, d), matrix_std, wd),
        "embed_norm_g": _normal(gen, (d,), 0.02, torch.float32, 1.0),
        "final_norm_g": _normal(gen, (d,), 0.02, torch.float32, 1.0),
        "lm_head": _normal(gen, (cfg.vocab, d), lm_head_std if lm_head_std is not None else matrix_std, wd),
        "layers": [],
    }
    for _ in range(cfg.n_layers):
        lw = {
            "attn_norm_g": _normal(gen, (d,), 0.02, torch.float32, 1.0),
            "wq": _normal(gen, (qd, d), matrix_std, wd),
            "wk": _normal(gen, (kvd, d), matrix_std, wd),
            "wv": _normal(gen, (kvd, d), matrix_std, wd),
            "wo": _normal(gen, (d, qd), matrix_std, wd),
            "coup_a": _normal(gen, (qd,), coupling_std, torch.float32),
            "mlp_norm_g": _normal(gen, (d,), 0.02, torch.float32, 1.0),
            "coup_c": _normal(gen, (d,), coupling_std, torch.float32),
        }
        if cfg.is_moe:
            E, Fe, Fs = cfg.n_experts, cfg.d_expert, cfg.n_shared_experts * cfg.d_expert
            lw["router"] = _normal(gen, (E, d), 1.0 / d ** 0.5, wd)
            lw["exp_gate"] = _normal(gen, (E, Fe, d), matrix_std, wd)
            lw["exp_up"] = _normal(gen, (E, Fe, d), matrix_std, wd)
            lw["exp_down"] = _normal(gen, (E, d, Fe), matrix_std, wd)
            if Fs > 0:
                lw["sh_gate"] = _normal(gen, (Fs, d), matrix_std, wd)
                lw["sh_up"] = _normal(gen, (Fs, d), matrix_std, wd)
                lw["sh_down"] = _normal(gen, (d, Fs), matrix_std, wd)
            lw["coup_b"] = _normal(gen, (max(Fs, 1),), coupling_std, torch.float32)
            if cfg.compute_matched:  # g_A, g_G: trained from one; spread so that a dropped gate shows
                lw["gate_a"] = _normal(gen, (d,), coupling_std, torch.float32, 1.0)
                lw["gate_g"] = _normal(gen, (d,), coupling_std, torch.float32, 1.0)
        else:
            F = cfg.d_ff
            lw["w_gate"] = _normal(gen, (F, d), matrix_std, wd)
            lw["w_up"] = _normal(gen, (F, d), matrix_std, wd)
            lw["w_down"] = _normal(gen, (d, F), matrix_std, wd)
            lw["coup_b"] = _normal(gen, (F,), coupling_std, torch.float32)
        w["layers"].append(lw)
    return w


def make_tokens(cfg: ModelConfig, batch: int, length: int, seed: int = 1) -> torch.Tensor:
    """Uniform random token ids, int32 [batch, length]."""
    gen = torch.Generator(device="cpu")
    gen.manual_seed(seed)
    return torch.randint(0, cfg.vocab, (batch, length), generator=gen, dtype=torch.int32)


def make_synthetic_kv(cfg: ModelConfig, batch: int, length: int, seed: int = 3,
                      k_std: float = 1.0, v_std: float = 0.9) -> tuple[torch.Tensor, torch.Tensor]:
    """Stand-in cache contents for timing and long-context parity where a real prefill is
    too slow for the CPU oracle: K and V ~ N(0, std) in the model's storage type, shape
    [n_layers, batch, length, kv_dim].  Both sides receive the same bytes."""
    gen = torch.Generator(device="cpu")
    gen.manual_seed(seed)
    shape = (cfg.n_layers, batch, length, cfg.kv_dim)
    k = _normal(gen, shape, k_std, cfg.torch_dtype)
    v = _normal(gen, shape, v_std, cfg.torch_dtype)
    return k, v


def make_page_table(batch: int, pages_per_seq: int, num_pages: int, seed: int = 4,
                    shuffle: bool = True) -> torch.Tensor:
    """int32 [batch, pages_per_seq]: distinct physical pages, a seeded random permutation of
    the pool when shuffle is set (pages deliberately non-contiguous), identity otherwise."""
    need = batch * pages_per_seq
    if need > num_pages:
        raise ValueError("page pool too small")
    if shuffle:
        gen = torch.Generator(device="cpu")
        gen.manual_seed(seed)
        perm = torch.randperm(num_pages, generator=gen)[:need]
    else:
        perm = torch.arange(need)
    return perm.to(torch.int32).reshape(batch, pages_per_seq).contiguous()

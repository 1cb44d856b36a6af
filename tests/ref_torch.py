"""Independent float64 restatement of the two-path forward pass from PyTorch library routines.

Used only to pin the C oracle (it shares no code with it and none with the CUDA path):
whole sequences at once, batched, built from F.rms_norm, F.scaled_dot_product_attention,
F.silu, torch.softmax and torch.topk; RoPE is done as a complex multiplication.  With the
branch ignored this is a textbook LLaMA-style causal LM, which is what the paper says the
primary path must be (Section 4.1: primary attention is exactly causal self-attention;
Section 4.4: prefill is identical to the one-flow Transformer).
"""
from __future__ import annotations

import torch
import torch.nn.functional as F


def _w(t):
    return t.to(torch.float64)


def _rope_complex(x, n_heads, head_dim, base):
    """x [B,T,n_heads*head_dim]; pair (i, i+half) treated as one complex number."""
    B, T, _ = x.shape
    half = head_dim // 2
    x = x.view(B, T, n_heads, head_dim)
    z = torch.complex(x[..., :half], x[..., half:])
    inv_freq = base ** (-torch.arange(half, dtype=torch.float64) * 2.0 / head_dim)
    ang = torch.arange(T, dtype=torch.float64)[:, None] * inv_freq[None, :]
    rot = torch.polar(torch.ones_like(ang), ang)  # e^{i t theta_i}
    z = z * rot[None, :, None, :]
    return torch.cat([z.real, z.imag], dim=-1).reshape(B, T, n_heads * head_dim)


def _attn(q, k, v, cfg):
    """q [B,T,q_dim], k/v [B,T,kv_dim] -> [B,T,q_dim]; library causal SDPA with GQA by
    repeating each KV head for its contiguous group of query heads."""
    B, T, _ = q.shape
    G = cfg.n_q_heads // cfg.n_kv_heads
    qh = q.view(B, T, cfg.n_q_heads, cfg.head_dim).transpose(1, 2)
    kh = k.view(B, T, cfg.n_kv_heads, cfg.head_dim).transpose(1, 2).repeat_interleave(G, dim=1)
    vh = v.view(B, T, cfg.n_kv_heads, cfg.head_dim).transpose(1, 2).repeat_interleave(G, dim=1)
    o = F.scaled_dot_product_attention(qh, kh, vh, is_causal=True)
    return o.transpose(1, 2).reshape(B, T, cfg.q_dim)


def _norm(x, g, eps):
    return F.rms_norm(x, (x.shape[-1],), _w(g), eps)


def _swiglu_hidden(m, wg, wu):
    return F.silu(m @ _w(wg).T) * (m @ _w(wu).T)


def _moe_routed(m, lw, cfg, k, idx_override=None):
    """Sum of renormalised top-k experts.  m [B,T,d].  Returns (out, idx)."""
    probs = torch.softmax(m @ _w(lw["router"]).T, dim=-1)
    if idx_override is None:
        _, idx = torch.topk(probs, k, dim=-1)
    else:
        idx = idx_override
    sel = torch.gather(probs, -1, idx)
    wts = sel / sel.sum(-1, keepdim=True)
    out = torch.zeros_like(m)
    Bn, Tn, _ = m.shape
    for b in range(Bn):
        for t in range(Tn):
            for j in range(idx.shape[-1]):
                e = int(idx[b, t, j])
                h = _swiglu_hidden(m[b, t], lw["exp_gate"][e], lw["exp_up"][e])
                out[b, t] += wts[b, t, j] * (h @ _w(lw["exp_down"][e]).T)
    return out, idx


def forward(cfg, w, tokens, branch: bool = True):
    """tokens int [B,T] -> (z1 [B,T,V], z2 or None, K [L,B,T,kv], V [L,B,T,kv])."""
    tok = torch.as_tensor(tokens).long()
    eps = cfg.rms_eps
    s1 = _norm(_w(w["embed_primary"])[tok], w["embed_norm_g"], eps)
    s2 = _norm(_w(w["embed_branch"])[tok], w["embed_norm_g"], eps) if branch else None
    ks, vs = [], []
    for lw in w["layers"]:
        n1 = _norm(s1, lw["attn_norm_g"], eps)
        q1 = _rope_complex(n1 @ _w(lw["wq"]).T, cfg.n_q_heads, cfg.head_dim, cfg.rope_base)
        k1 = _rope_complex(n1 @ _w(lw["wk"]).T, cfg.n_kv_heads, cfg.head_dim, cfg.rope_base)
        v1 = n1 @ _w(lw["wv"]).T
        ks.append(k1)
        vs.append(v1)
        a1 = _attn(q1, k1, v1, cfg) @ _w(lw["wo"]).T
        s1 = s1 + a1
        matched = bool(getattr(cfg, "compute_matched", 0))
        if branch and matched:  # Appendix B.3: a gated copy of the primary attention update
            s2 = s2 + _w(lw["gate_a"]) * a1
        elif branch:
            n2 = _norm(s2, lw["attn_norm_g"], eps)
            q2 = _rope_complex(n2 @ _w(lw["wq"]).T, cfg.n_q_heads, cfg.head_dim, cfg.rope_base)
            q2 = q2 + _w(lw["coup_a"]) * q1
            s2 = s2 + _attn(q2, k1, v1, cfg) @ _w(lw["wo"]).T
        m1 = _norm(s1, lw["mlp_norm_g"], eps)
        m2 = _norm(s2, lw["mlp_norm_g"], eps) if branch else None
        if cfg.n_experts == 0:
            h1 = _swiglu_hidden(m1, lw["w_gate"], lw["w_up"])
            M1 = h1 @ _w(lw["w_down"]).T
            s1 = s1 + M1
            if branch:
                h2 = _swiglu_hidden(m2, lw["w_gate"], lw["w_up"]) + _w(lw["coup_b"]) * h1
                s2 = s2 + h2 @ _w(lw["w_down"]).T + _w(lw["coup_c"]) * M1
        else:
            M1, idx1 = _moe_routed(m1, lw, cfg, cfg.k_primary)
            hs1 = None
            shared1 = torch.zeros_like(M1)
            if cfg.n_shared_experts > 0:
                hs1 = _swiglu_hidden(m1, lw["sh_gate"], lw["sh_up"])
                shared1 = hs1 @ _w(lw["sh_down"]).T
                M1 = M1 + shared1
            s1 = s1 + M1
            if branch and matched:  # Appendix B.3: own routed experts + gated primary shared expert
                M2, _ = _moe_routed(m2, lw, cfg, cfg.k_branch)
                s2 = s2 + M2 + _w(lw["gate_g"]) * shared1
            elif branch:
                if cfg.router_mode == 1:
                    M2, _ = _moe_routed(m2, lw, cfg, cfg.k_primary, idx_override=idx1)
                else:
                    M2, _ = _moe_routed(m2, lw, cfg, cfg.k_branch)
                if cfg.n_shared_experts > 0:
                    hs2 = _swiglu_hidden(m2, lw["sh_gate"], lw["sh_up"])
                    if cfg.moe_b_coupling:
                        hs2 = hs2 + _w(lw["coup_b"]) * hs1
                    M2 = M2 + hs2 @ _w(lw["sh_down"]).T
                s2 = s2 + M2 + _w(lw["coup_c"]) * M1
    f1 = _norm(s1, w["final_norm_g"], eps) if cfg.final_norm else s1
    z1 = f1 @ _w(w["lm_head"]).T
    z2 = None
    if branch:
        f2 = _norm(s2, w["final_norm_g"], eps) if cfg.final_norm else s2
        z2 = f2 @ _w(w["lm_head"]).T
    return z1, z2, torch.stack(ks), torch.stack(vs)


def mixture(z1, z2):
    p = torch.softmax(z1, -1)
    q = torch.softmax(z2, -1)
    alpha = (p * p).sum(-1).clamp(0.5, 1.0)
    return alpha, alpha[..., None] * p + (1 - alpha[..., None]) * q

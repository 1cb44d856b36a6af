"""ctypes binding of the CPU oracle (oracle/dbt_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by tests/, the smoke check and the benchmark's CPU
baseline leg.  Nothing here touches CUDA, and the CUDA package never imports this module.
Weights are passed as a dict of torch CPU tensors (fp32 or bf16) whose storage the oracle
borrows; the wrapper keeps them alive.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
import threading

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "dbt_oracle.c")
_HDR = os.path.join(_HERE, "dbt_oracle.h")
_LIB = os.path.join(_HERE, "libdbt_oracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (plain C, OpenMP on outer loops)."""
    with _lock:
        stale = (not os.path.exists(_LIB)
                 or os.path.getmtime(_LIB) < max(os.path.getmtime(_SRC), os.path.getmtime(_HDR)))
        if force or stale:
            tmp = _LIB + f".tmp{os.getpid()}"
            subprocess.run(["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"],
                           check=True)
            os.replace(tmp, _LIB)
    return _LIB


class OrcConfig(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("d_model", "n_layers", "n_q_heads", "n_kv_heads", "head_dim",
                                         "d_ff", "vocab", "weight_dtype", "kv_round_bf16")]
    _fields_ += [("rope_base", C.c_float), ("rms_eps", C.c_float)]
    _fields_ += [(n, C.c_int32) for n in ("final_norm", "n_experts", "d_expert", "n_shared_experts",
                                         "k_primary", "k_branch", "router_mode", "moe_b_coupling",
                                         "compute_matched", "n_paths", "max_batch", "max_seq")]


_LAYER_FIELDS = ("attn_norm_g", "wq", "wk", "wv", "wo", "coup_a", "mlp_norm_g", "w_gate", "w_up", "w_down",
                 "coup_b", "coup_c", "router", "exp_gate", "exp_up", "exp_down", "sh_gate", "sh_up", "sh_down",
                 "gate_a", "gate_g")


class OrcLayer(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in _LAYER_FIELDS]


class OrcWeights(C.Structure):
    _fields_ = [("embed_primary", C.c_void_p), ("embed_branch", C.c_void_p), ("embed_norm_g", C.c_void_p),
                ("final_norm_g", C.c_void_p), ("lm_head", C.c_void_p), ("layers", C.POINTER(OrcLayer))]


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        vp, i32p, fp = C.c_void_p, C.POINTER(C.c_int32), C.POINTER(C.c_float)
        L.orc_create.restype = vp
        L.orc_create.argtypes = [C.POINTER(OrcConfig), C.POINTER(OrcWeights)]
        L.orc_destroy.argtypes = [vp]
        L.orc_reset.argtypes = [vp]
        L.orc_seq_len.argtypes = [vp, C.c_int]
        L.orc_seq_len.restype = C.c_int
        L.orc_k_cache.argtypes = [vp]
        L.orc_k_cache.restype = vp
        L.orc_v_cache.argtypes = [vp]
        L.orc_v_cache.restype = vp
        L.orc_set_seq_len.argtypes = [vp, C.c_int, C.c_int]
        L.orc_router_logits.argtypes = [vp]
        L.orc_router_logits.restype = vp
        L.orc_prefill.argtypes = [vp, vp, C.c_int, C.c_int, vp]
        L.orc_decode_step.argtypes = [vp, vp, C.c_int, C.c_int, vp, vp, vp, vp, vp, vp, vp]
        L.orc_full_forward.argtypes = [C.POINTER(OrcConfig), C.POINTER(OrcWeights), vp, C.c_int, C.c_int,
                                       vp, vp, vp, vp]
        L.orc_rmsnorm.argtypes = [vp, vp, C.c_int, C.c_float, vp]
        L.orc_linear.argtypes = [vp, C.c_int, C.c_int, C.c_int, vp, C.c_int, vp]
        L.orc_rope.argtypes = [vp, C.c_int, C.c_int, C.c_int, C.c_float]
        L.orc_attend.argtypes = [vp, vp, vp, C.c_int, C.c_int, C.c_int, vp]
        L.orc_swiglu.argtypes = [vp, vp, C.c_int, vp]
        L.orc_route.argtypes = [vp, C.c_int, C.c_int, vp, vp, vp]
        L.orc_readout.argtypes = [vp, vp, C.c_int, vp, vp]
        L.orc_readout.restype = C.c_int
        L.orc_readout_multi.argtypes = [vp, vp, C.c_int, C.c_int, vp, vp]
        L.orc_readout_multi.restype = C.c_int
        L.orc_set_threads.argtypes = [C.c_int]
        L.orc_get_threads.restype = C.c_int
        _lib = L
    return _lib


def _ptr(t):
    if t is None:
        return None
    if isinstance(t, np.ndarray):
        assert t.flags["C_CONTIGUOUS"]
        return t.ctypes.data
    assert t.is_contiguous() and t.device.type == "cpu"
    return t.data_ptr()


def _cfg_struct(cfg, max_batch: int, max_seq: int, kv_round_bf16: bool = False) -> OrcConfig:
    return OrcConfig(d_model=cfg.d_model, n_layers=cfg.n_layers, n_q_heads=cfg.n_q_heads,
                     n_kv_heads=cfg.n_kv_heads, head_dim=cfg.head_dim, d_ff=cfg.d_ff, vocab=cfg.vocab,
                     weight_dtype=0 if cfg.weight_dtype == "fp32" else 1, kv_round_bf16=int(kv_round_bf16),
                     rope_base=cfg.rope_base, rms_eps=cfg.rms_eps, final_norm=cfg.final_norm,
                     n_experts=cfg.n_experts, d_expert=cfg.d_expert, n_shared_experts=cfg.n_shared_experts,
                     k_primary=cfg.k_primary, k_branch=cfg.k_branch, router_mode=cfg.router_mode,
                     moe_b_coupling=cfg.moe_b_coupling, compute_matched=cfg.compute_matched,
                     n_paths=getattr(cfg, "n_paths", 2), max_batch=max_batch, max_seq=max_seq)


def _weights_struct(cfg, w: dict):
    want = torch.float32 if cfg.weight_dtype == "fp32" else torch.bfloat16
    vec = {"attn_norm_g", "coup_a", "mlp_norm_g", "coup_b", "coup_c", "gate_a", "gate_g"}
    layers = (OrcLayer * cfg.n_layers)()
    for l, lw in enumerate(w["layers"]):
        for name in _LAYER_FIELDS:
            t = lw.get(name)
            if t is not None:
                assert t.dtype == (torch.float32 if name in vec else want), name
            setattr(layers[l], name, _ptr(t))
    for name in ("embed_primary", "embed_branch", "lm_head"):
        assert w[name].dtype == want, name
    nb = getattr(cfg, "n_paths", 2) - 1  # one embedding table per decode branch, stacked [K-1][V][d]
    assert w["embed_branch"].numel() == nb * cfg.vocab * cfg.d_model, "embed_branch must hold K-1 tables"
    ws = OrcWeights(embed_primary=_ptr(w["embed_primary"]), embed_branch=_ptr(w["embed_branch"]),
                    embed_norm_g=_ptr(w["embed_norm_g"]), final_norm_g=_ptr(w["final_norm_g"]),
                    lm_head=_ptr(w["lm_head"]), layers=layers)
    return ws, layers


class OracleModel:
    """Incremental two-path model with an fp32 KV cache [L, max_batch, max_seq, kv_dim]."""

    def __init__(self, cfg, weights: dict, max_batch: int, max_seq: int, kv_round_bf16: bool = False):
        self.cfg, self.weights = cfg, weights  # keeps the tensors alive
        self.max_batch, self.max_seq = max_batch, max_seq
        self._c = _cfg_struct(cfg, max_batch, max_seq, kv_round_bf16)
        self._w, self._layers = _weights_struct(cfg, weights)
        self._h = lib().orc_create(C.byref(self._c), C.byref(self._w))
        if not self._h:
            raise ValueError("orc_create rejected the configuration")

    def close(self):
        if self._h:
            lib().orc_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def reset(self):
        lib().orc_reset(self._h)

    def seq_len(self, b: int) -> int:
        return lib().orc_seq_len(self._h, b)

    def _cache(self, which: str) -> np.ndarray:
        p = lib().orc_k_cache(self._h) if which == "k" else lib().orc_v_cache(self._h)
        shape = (self.cfg.n_layers, self.max_batch, self.max_seq, self.cfg.kv_dim)
        n = int(np.prod(shape))
        return np.ctypeslib.as_array(C.cast(p, C.POINTER(C.c_float)), shape=(n,)).reshape(shape)

    @property
    def k_cache(self) -> np.ndarray:
        return self._cache("k")

    @property
    def v_cache(self) -> np.ndarray:
        return self._cache("v")

    def inject_kv(self, k, v, length: int):
        """Load cache contents [L, B, length, kv_dim] (torch or numpy, any float type)."""
        k = k.float().numpy() if isinstance(k, torch.Tensor) else np.asarray(k, dtype=np.float32)
        v = v.float().numpy() if isinstance(v, torch.Tensor) else np.asarray(v, dtype=np.float32)
        B = k.shape[1]
        self.k_cache[:, :B, :length] = k
        self.v_cache[:, :B, :length] = v
        for b in range(B):
            lib().orc_set_seq_len(self._h, b, length)

    def router_logits(self, batch: int) -> np.ndarray:
        """MoE: router logits of the last step, [L, K, batch, E] (a copy)."""
        p = lib().orc_router_logits(self._h)
        assert p, "not an MoE model"
        K = getattr(self.cfg, "n_paths", 2)
        shape = (self.cfg.n_layers, K, self.max_batch, self.cfg.n_experts)
        n = int(np.prod(shape))
        a = np.ctypeslib.as_array(C.cast(p, C.POINTER(C.c_float)), shape=(n,)).reshape(shape)
        return a[:, :, :batch].copy()

    def prefill(self, tokens, want_logits: bool = True):
        tok = np.ascontiguousarray(np.asarray(tokens, dtype=np.int32))
        B, n = tok.shape
        out = np.empty((B, self.cfg.vocab), dtype=np.float32) if want_logits else None
        rc = lib().orc_prefill(self._h, _ptr(tok), B, n, _ptr(out))
        if rc != 0:
            raise RuntimeError("orc_prefill failed")
        return out

    def decode_step(self, tokens, grouped: bool = True, forced_experts=None, want_mix: bool = False):
        tok = np.ascontiguousarray(np.asarray(tokens, dtype=np.int32).reshape(-1))
        B, V, cfg = tok.shape[0], self.cfg.vocab, self.cfg
        K = getattr(cfg, "n_paths", 2)
        out = {"next": np.empty(B, dtype=np.int32), "z1": np.empty((B, V), dtype=np.float32)}
        if grouped:  # one decode branch: z2 [B, V]; more (Appendix C.1): [K-1, B, V]
            out["z2"] = np.empty((B, V) if K == 2 else (K - 1, B, V), dtype=np.float32)
            out["alpha"] = np.empty(B, dtype=np.float32)
            if want_mix:
                out["mix"] = np.empty((B, V), dtype=np.float32)
        if cfg.is_moe:
            out["experts"] = np.full((cfg.n_layers, K, B, cfg.kmax), -1, dtype=np.int32)
        forced = None
        if forced_experts is not None:
            forced = np.ascontiguousarray(np.asarray(forced_experts, dtype=np.int32))
            assert forced.shape == (cfg.n_layers, K, B, cfg.kmax)
        rc = lib().orc_decode_step(self._h, _ptr(tok), B, int(grouped), _ptr(forced), _ptr(out.get("experts")),
                                   _ptr(out["next"]), _ptr(out["z1"]), _ptr(out.get("z2")),
                                   _ptr(out.get("alpha")), _ptr(out.get("mix")))
        if rc != 0:
            raise RuntimeError("orc_decode_step failed")
        return out


def full_forward(cfg, weights: dict, tokens, want_kv: bool = False):
    """Non-incremental forward of every path: returns z1 [B,T,V], z2 [B,T,V] (one decode branch)
    or [K-1,B,T,V] (more), and K,V [L,B,T,kv_dim] on request."""
    tok = np.ascontiguousarray(np.asarray(tokens, dtype=np.int32))
    B, T = tok.shape
    c = _cfg_struct(cfg, B, T)
    ws, layers = _weights_struct(cfg, weights)
    K = getattr(cfg, "n_paths", 2)
    z1 = np.empty((B, T, cfg.vocab), dtype=np.float32)
    z2 = np.empty((B, T, cfg.vocab) if K == 2 else (K - 1, B, T, cfg.vocab), dtype=np.float32)
    k = np.empty((cfg.n_layers, B, T, cfg.kv_dim), dtype=np.float32) if want_kv else None
    v = np.empty((cfg.n_layers, B, T, cfg.kv_dim), dtype=np.float32) if want_kv else None
    rc = lib().orc_full_forward(C.byref(c), C.byref(ws), _ptr(tok), B, T, _ptr(z1), _ptr(z2), _ptr(k), _ptr(v))
    if rc != 0:
        raise RuntimeError("orc_full_forward failed")
    return (z1, z2, k, v) if want_kv else (z1, z2)


# ---- unit operations ---------------------------------------------------------------------

def _f32(a):
    return np.ascontiguousarray(np.asarray(a, dtype=np.float32))


def rmsnorm(x, g, eps):
    x, g = _f32(x), _f32(g)
    y = np.empty_like(x)
    lib().orc_rmsnorm(_ptr(x), _ptr(g), x.shape[-1], eps, _ptr(y))
    return y


def linear(W: torch.Tensor, X):
    """Y[r, i] = sum_k W[i, k] X[r, k]; W a torch fp32/bf16 matrix."""
    X = _f32(X)
    R, n_in = X.shape
    n_out = W.shape[0]
    assert W.shape[1] == n_in and W.is_contiguous()
    Y = np.empty((R, n_out), dtype=np.float32)
    lib().orc_linear(W.data_ptr(), 0 if W.dtype == torch.float32 else 1, n_out, n_in, _ptr(X), R, _ptr(Y))
    return Y


def rope(x, n_heads, head_dim, t, base):
    y = _f32(x).copy()
    lib().orc_rope(_ptr(y), n_heads, head_dim, t, base)
    return y


def attend(u, K, V):
    """One query head u [d_h] against K, V [n_keys, d_h]."""
    u, K, V = _f32(u), _f32(K), _f32(V)
    o = np.empty_like(u)
    lib().orc_attend(_ptr(u), _ptr(K), _ptr(V), K.shape[0], K.shape[1], u.shape[0], _ptr(o))
    return o


def swiglu(g, u):
    g, u = _f32(g), _f32(u)
    h = np.empty_like(g)
    lib().orc_swiglu(_ptr(g), _ptr(u), g.size, _ptr(h))
    return h


def route(logits, k, forced=None):
    logits = _f32(logits)
    idx = np.empty(k, dtype=np.int32)
    wts = np.empty(k, dtype=np.float32)
    f = None if forced is None else np.ascontiguousarray(np.asarray(forced, dtype=np.int32))
    lib().orc_route(_ptr(logits), logits.shape[0], k, _ptr(f), _ptr(idx), _ptr(wts))
    return idx, wts


def readout(z1, z2, want_mix=True):
    z1, z2 = _f32(z1), _f32(z2)
    alpha = np.empty(1, dtype=np.float32)
    mix = np.empty_like(z1) if want_mix else None
    tok = lib().orc_readout(_ptr(z1), _ptr(z2), z1.shape[0], _ptr(alpha), _ptr(mix))
    return tok, float(alpha[0]), mix


def readout_multi(z1, zb, want_mix=True):
    """zb [nb, V]: the logits of nb decode branches (Appendix C.1)."""
    z1, zb = _f32(z1), _f32(zb)
    alpha = np.empty(1, dtype=np.float32)
    mix = np.empty_like(z1) if want_mix else None
    tok = lib().orc_readout_multi(_ptr(z1), _ptr(zb), zb.shape[0], z1.shape[0], _ptr(alpha), _ptr(mix))
    return tok, float(alpha[0]), mix


def set_threads(n: int):
    lib().orc_set_threads(n)


def get_threads() -> int:
    return lib().orc_get_threads()

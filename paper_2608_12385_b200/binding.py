"""Thin ctypes binding over the C ABI of include/dbt.h (argument marshalling only).

PyTorch supplies device memory and the CUDA stream; every step of the path runs inside
libdbt_b200.so.  Loading fails loudly when the library has not been built
(`python -m paper_2608_12385_b200.build`): there is no fallback.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

from .inputs import ModelConfig

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libdbt_b200.so")

DBT_OK = 0
STATUS_NAMES = {0: "DBT_OK", 1: "DBT_ERR_INVALID_ARG", 2: "DBT_ERR_UNSUPPORTED", 3: "DBT_ERR_CAPACITY",
                4: "DBT_ERR_STATE", 5: "DBT_ERR_CUDA", 6: "DBT_ERR_DEVICE", 7: "DBT_ERR_TIMEOUT"}

EXPORTS = ["dbt_query_sizes", "dbt_create", "dbt_destroy", "dbt_set_page_table", "dbt_reset", "dbt_set_seq_lens",
           "dbt_seq_len", "dbt_prefill", "dbt_decode_step", "dbt_decode_step_primary_only", "dbt_decode_step_host",
           "dbt_decode_step_primary_only_host", "dbt_last_experts", "dbt_last_expert_union", "dbt_sync_status",
           "dbt_launch_count", "dbt_last_error", "dbt_version", "dbt_profile_begin", "dbt_profile_end", "dbt_op_gemm_tc",
           "dbt_op_gemm_tc_static", "dbt_kv_export", "dbt_kv_import", "dbt_prefill_boundary"]


class DbtError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"{STATUS_NAMES.get(status, status)}: {message}")
        self.status = status


class DbtConfig(C.Structure):
    _fields_ = [("struct_size", C.c_uint32)]
    _fields_ += [(n, C.c_int32) for n in ("d_model", "n_layers", "n_q_heads", "n_kv_heads", "head_dim", "d_ff",
                                         "vocab", "weight_dtype")]
    _fields_ += [("rope_base", C.c_float), ("rms_eps", C.c_float)]
    _fields_ += [(n, C.c_int32) for n in ("final_norm", "n_experts", "d_expert", "n_shared_experts", "k_primary",
                                         "k_branch", "router_mode", "moe_b_coupling", "compute_matched", "n_paths", "max_batch", "max_seq",
                                         "page_size", "num_pages")]


LAYER_FIELDS = ("attn_norm_g", "wq", "wk", "wv", "wo", "coup_a", "mlp_norm_g", "w_gate", "w_up", "w_down", "coup_b",
                "coup_c", "router", "exp_gate", "exp_up", "exp_down", "sh_gate", "sh_up", "sh_down", "gate_a", "gate_g")


class DbtLayerWeights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in LAYER_FIELDS]


class DbtProfileEntry(C.Structure):
    _fields_ = [("name", C.c_char * 32), ("launches", C.c_int64), ("total_ms", C.c_double), ("bytes", C.c_double)]


class DbtWeights(C.Structure):
    _fields_ = [("embed_primary", C.c_void_p), ("embed_branch", C.c_void_p), ("embed_norm_g", C.c_void_p),
                ("final_norm_g", C.c_void_p), ("lm_head", C.c_void_p), ("layers", C.POINTER(DbtLayerWeights))]


_lib = None


def load_library():
    """dlopen libdbt_b200.so and declare the signatures.  Raises if it is not built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2608_12385_b200.build` "
                           "(there is no CPU or PyTorch fallback)")
    L = C.CDLL(LIB_PATH)
    vp, i32, i32p = C.c_void_p, C.c_int32, C.POINTER(C.c_int32)
    L.dbt_query_sizes.argtypes = [C.POINTER(DbtConfig), C.POINTER(C.c_size_t), C.POINTER(C.c_size_t)]
    L.dbt_create.argtypes = [C.POINTER(DbtConfig), C.POINTER(DbtWeights), vp, vp, vp, C.POINTER(vp)]
    L.dbt_destroy.argtypes = [vp]
    L.dbt_destroy.restype = None
    L.dbt_set_page_table.argtypes = [vp, vp, i32, i32]
    L.dbt_reset.argtypes = [vp]
    L.dbt_set_seq_lens.argtypes = [vp, vp, i32]
    L.dbt_seq_len.argtypes = [vp, i32]
    L.dbt_seq_len.restype = i32
    L.dbt_prefill.argtypes = [vp, vp, i32, i32, vp]
    L.dbt_decode_step.argtypes = [vp, vp, i32, vp, vp, vp, vp]
    L.dbt_prefill_boundary.argtypes = [vp, vp, i32, i32, vp, vp, vp, vp]
    L.dbt_decode_step_primary_only.argtypes = [vp, vp, i32, vp, vp]
    L.dbt_decode_step_host.argtypes = [vp, vp, i32, vp, vp]
    L.dbt_decode_step_primary_only_host.argtypes = [vp, vp, i32, vp]
    L.dbt_last_experts.argtypes = [vp, C.POINTER(vp), i32p]
    L.dbt_last_expert_union.argtypes = [vp, vp]
    L.dbt_sync_status.argtypes = [vp, i32p, i32p]
    L.dbt_kv_export.argtypes = [vp, vp, i32, i32, vp, vp]
    L.dbt_kv_import.argtypes = [vp, vp, i32, i32, vp, vp]
    L.dbt_op_gemm_tc.argtypes = [vp, vp, i32, i32, i32, i32, vp, vp, C.c_size_t, vp, vp, i32p]
    L.dbt_op_gemm_tc_static.argtypes = [vp, vp, i32, i32, i32, i32, vp, vp, vp, i32p]
    L.dbt_profile_begin.argtypes = [vp]
    L.dbt_profile_end.argtypes = [vp, C.POINTER(DbtProfileEntry), i32, i32p]
    L.dbt_launch_count.argtypes = [vp]
    L.dbt_launch_count.restype = C.c_int64
    L.dbt_last_error.argtypes = [vp]
    L.dbt_last_error.restype = C.c_char_p
    L.dbt_version.restype = C.c_char_p
    for name in EXPORTS:
        if name not in ("dbt_destroy", "dbt_seq_len", "dbt_launch_count", "dbt_last_error", "dbt_version"):
            getattr(L, name).restype = C.c_int
    _lib = L
    return L


def make_config_struct(cfg: ModelConfig, max_batch: int, max_seq: int, num_pages: int) -> DbtConfig:
    return DbtConfig(struct_size=C.sizeof(DbtConfig), d_model=cfg.d_model, n_layers=cfg.n_layers,
                     n_q_heads=cfg.n_q_heads, n_kv_heads=cfg.n_kv_heads, head_dim=cfg.head_dim, d_ff=cfg.d_ff,
                     vocab=cfg.vocab, weight_dtype=0 if cfg.weight_dtype == "fp32" else 1, rope_base=cfg.rope_base,
                     rms_eps=cfg.rms_eps, final_norm=cfg.final_norm, n_experts=cfg.n_experts, d_expert=cfg.d_expert,
                     n_shared_experts=cfg.n_shared_experts, k_primary=cfg.k_primary, k_branch=cfg.k_branch,
                     router_mode=cfg.router_mode, moe_b_coupling=cfg.moe_b_coupling,
                     compute_matched=cfg.compute_matched, n_paths=cfg.n_paths, max_batch=max_batch,
                     max_seq=max_seq, page_size=cfg.page_size, num_pages=num_pages)


def query_sizes(cfg: ModelConfig, max_batch: int, max_seq: int, num_pages: int) -> tuple[int, int]:
    L = load_library()
    c = make_config_struct(cfg, max_batch, max_seq, num_pages)
    kv, ws = C.c_size_t(0), C.c_size_t(0)
    st = L.dbt_query_sizes(C.byref(c), C.byref(kv), C.byref(ws))
    if st != DBT_OK:
        raise DbtError(st, L.dbt_last_error(None).decode())
    return kv.value, ws.value


def op_gemm_tc(W: torch.Tensor, X: torch.Tensor, force_split: int = 0, scratch: torch.Tensor | None = None):
    """Y = X W^T on the tensor cores.  W bf16 [n_out, K], X bf16 [R, K] on the GPU.
    Returns (Y fp32 [R, n_out], split used)."""
    L = load_library()
    assert W.dtype == torch.bfloat16 and X.dtype == torch.bfloat16 and W.is_cuda and X.is_cuda
    n_out, K = W.shape
    R = X.shape[0]
    Y = torch.empty(R, n_out, dtype=torch.float32, device=W.device)
    if scratch is None:
        scratch = torch.empty(max(force_split, 16) * 256 * n_out if R > 128 else max(force_split, 16) * 128 * n_out,
                              dtype=torch.float32, device=W.device)
    status = torch.zeros(2, dtype=torch.int32, device=W.device)
    used = C.c_int32(0)
    st = L.dbt_op_gemm_tc(W.data_ptr(), X.data_ptr(), n_out, K, R, force_split, Y.data_ptr(), scratch.data_ptr(),
                          scratch.numel(), status.data_ptr(), torch.cuda.current_stream().cuda_stream, C.byref(used))
    if st != DBT_OK:
        raise DbtError(st, L.dbt_last_error(None).decode())
    torch.cuda.synchronize()
    code = status.cpu().tolist()
    if code[0] != 0:  # 3: a bounded device wait ran out (the codes of dbt_sync_status)
        raise DbtError(7 if code[0] == 3 else 6, f"device status {code}")
    return Y, used.value


def op_gemm_tc_static(W: torch.Tensor, X: torch.Tensor, force_split: int = 0, Y: torch.Tensor | None = None,
                      status: torch.Tensor | None = None):
    """Y = X W^T through the entry point that allocates no device memory: its split-K workspace
    is a fixed 8 MiB array inside the library.  Pass Y and status to make the call itself
    allocation-free on the Python side too.  Returns (Y, split used)."""
    L = load_library()
    assert W.dtype == torch.bfloat16 and X.dtype == torch.bfloat16 and W.is_cuda and X.is_cuda
    n_out, K = W.shape
    R = X.shape[0]
    if Y is None:
        Y = torch.empty(R, n_out, dtype=torch.float32, device=W.device)
    if status is None:
        status = torch.zeros(2, dtype=torch.int32, device=W.device)
    used = C.c_int32(0)
    st = L.dbt_op_gemm_tc_static(W.data_ptr(), X.data_ptr(), n_out, K, R, force_split, Y.data_ptr(), status.data_ptr(),
                                 torch.cuda.current_stream().cuda_stream, C.byref(used))
    if st != DBT_OK:
        raise DbtError(st, L.dbt_last_error(None).decode())
    torch.cuda.synchronize()
    code = status.cpu().tolist()
    if code[0] != 0:  # 3: a bounded device wait ran out (the codes of dbt_sync_status)
        raise DbtError(7 if code[0] == 3 else 6, f"device status {code}")
    return Y, used.value


def weights_to_device(weights: dict, device="cuda") -> dict:
    out = {k: v.to(device) for k, v in weights.items() if k != "layers"}
    out["layers"] = [{k: v.to(device) for k, v in lw.items()} for lw in weights["layers"]]
    return out


def _p(t):
    return None if t is None else t.data_ptr()


class Model:
    """A Decode-Branch model handle: owns (as torch tensors) the KV pool and the workspace
    the library borrows, and keeps the device weights alive."""

    def __init__(self, cfg: ModelConfig, weights_dev: dict, max_batch: int, max_seq: int,
                 num_pages: int | None = None, stream: torch.cuda.Stream | None = None):
        self.L = load_library()
        self.cfg, self.weights = cfg, weights_dev
        self.max_batch, self.max_seq = max_batch, max_seq
        self.pages_per_seq_max = (max_seq + cfg.page_size - 1) // cfg.page_size
        self.num_pages = num_pages if num_pages is not None else max_batch * self.pages_per_seq_max
        self.device = weights_dev["lm_head"].device
        self.stream = stream
        self._c = make_config_struct(cfg, max_batch, max_seq, self.num_pages)
        kv_bytes, ws_bytes = query_sizes(cfg, max_batch, max_seq, self.num_pages)
        self.kv_pool = torch.zeros(kv_bytes // cfg.elem_bytes, dtype=cfg.torch_dtype, device=self.device)
        self.workspace = torch.zeros(ws_bytes, dtype=torch.uint8, device=self.device)
        layers = (DbtLayerWeights * cfg.n_layers)()
        for l, lw in enumerate(weights_dev["layers"]):
            for name in LAYER_FIELDS:
                t = lw.get(name)
                if t is not None:
                    assert t.is_cuda and t.is_contiguous(), name
                setattr(layers[l], name, _p(t))
        self._layers = layers
        self._w = DbtWeights(embed_primary=_p(weights_dev["embed_primary"]), embed_branch=_p(weights_dev["embed_branch"]),
                             embed_norm_g=_p(weights_dev["embed_norm_g"]), final_norm_g=_p(weights_dev["final_norm_g"]),
                             lm_head=_p(weights_dev["lm_head"]), layers=layers)
        h = C.c_void_p(None)
        torch.cuda.synchronize(self.device)
        st = self.L.dbt_create(C.byref(self._c), C.byref(self._w), self.kv_pool.data_ptr(), self.workspace.data_ptr(),
                               stream.cuda_stream if stream is not None else None, C.byref(h))
        if st != DBT_OK:
            raise DbtError(st, self.L.dbt_last_error(None).decode())
        self._h = h
        self.page_table = self.default_page_table(max_batch)

    # -- plumbing -------------------------------------------------------------------------
    def _check(self, st: int):
        if st != DBT_OK:
            raise DbtError(st, self.L.dbt_last_error(self._h).decode())

    def close(self):
        if getattr(self, "_h", None):
            torch.cuda.synchronize(self.device)
            self.L.dbt_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def kv_view(self) -> torch.Tensor:
        """The pool as [n_layers, 2, num_pages, n_kv_heads, page_size, head_dim]."""
        c = self.cfg
        return self.kv_pool.view(c.n_layers, 2, self.num_pages, c.n_kv_heads, c.page_size, c.head_dim)

    # -- state ----------------------------------------------------------------------------
    def reset(self):
        self._check(self.L.dbt_reset(self._h))

    def set_page_table(self, table: torch.Tensor):
        t = table.to(torch.int32).cpu().contiguous()
        self._check(self.L.dbt_set_page_table(self._h, t.data_ptr(), t.shape[0], t.shape[1]))
        self.page_table = t

    def set_seq_lens(self, lens):
        t = torch.as_tensor(lens, dtype=torch.int32).cpu().contiguous()
        self._check(self.L.dbt_set_seq_lens(self._h, t.data_ptr(), t.shape[0]))

    def seq_len(self, b: int) -> int:
        return self.L.dbt_seq_len(self._h, b)

    def default_page_table(self, batch: int) -> torch.Tensor:
        pps = min(self.pages_per_seq_max, self.num_pages // self.max_batch) \
            if self.max_batch * self.pages_per_seq_max > self.num_pages else self.pages_per_seq_max
        return (torch.arange(batch, dtype=torch.int32)[:, None] * pps + torch.arange(pps, dtype=torch.int32)[None, :])

    # -- the four calls of the problem statement -------------------------------------------
    def prefill(self, tokens_dev: torch.Tensor, want_logits: bool = False):
        assert tokens_dev.dtype == torch.int32 and tokens_dev.is_cuda and tokens_dev.is_contiguous()
        B, n = tokens_dev.shape
        out = torch.empty(B, self.cfg.vocab, dtype=torch.float32, device=self.device) if want_logits else None
        self._check(self.L.dbt_prefill(self._h, tokens_dev.data_ptr(), B, n, _p(out)))
        return out

    def prefill_boundary(self, tokens_dev: torch.Tensor) -> dict:
        """The whole prompt [B, S] and the boundary evaluation at its last token (Section 4.4 items 1-2)."""
        assert tokens_dev.dtype == torch.int32 and tokens_dev.is_cuda and tokens_dev.is_contiguous()
        B, S = tokens_dev.shape
        V, K = self.cfg.vocab, self.cfg.n_paths
        out = {"next": torch.empty(B, dtype=torch.int32, device=self.device),
               "z1": torch.empty(B, V, dtype=torch.float32, device=self.device),
               "z2": torch.empty((B, V) if K == 2 else (K - 1, B, V), dtype=torch.float32, device=self.device),
               "alpha": torch.empty(B, dtype=torch.float32, device=self.device)}
        self._check(self.L.dbt_prefill_boundary(self._h, tokens_dev.data_ptr(), B, S, _p(out["next"]), _p(out["z1"]),
                                                _p(out["z2"]), _p(out["alpha"])))
        return out

    def decode_step(self, tokens_dev: torch.Tensor, next_dev: torch.Tensor | None = None, z1=None, z2=None,
                    alpha=None):
        B = tokens_dev.shape[0]
        self._check(self.L.dbt_decode_step(self._h, tokens_dev.data_ptr(), B, _p(next_dev), _p(z1), _p(z2), _p(alpha)))

    def decode_step_primary_only(self, tokens_dev: torch.Tensor, next_dev: torch.Tensor | None = None, z1=None):
        B = tokens_dev.shape[0]
        self._check(self.L.dbt_decode_step_primary_only(self._h, tokens_dev.data_ptr(), B, _p(next_dev), _p(z1)))

    def decode_step_host(self, tokens_host: torch.Tensor, next_host: torch.Tensor, alpha_host=None):
        self._check(self.L.dbt_decode_step_host(self._h, tokens_host.data_ptr(), tokens_host.shape[0],
                                                next_host.data_ptr(), _p(alpha_host)))

    def decode_step_primary_only_host(self, tokens_host: torch.Tensor, next_host: torch.Tensor):
        self._check(self.L.dbt_decode_step_primary_only_host(self._h, tokens_host.data_ptr(), tokens_host.shape[0],
                                                             next_host.data_ptr()))

    def decode_full(self, tokens_dev: torch.Tensor, grouped: bool = True) -> dict:
        """One step returning every output (test convenience).  The library replays a step as
        a CUDA graph keyed by its buffer addresses, so the buffers are kept and reused; the
        returned tensors are copies."""
        B, V = tokens_dev.shape[0], self.cfg.vocab
        cache = self.__dict__.setdefault("_full_bufs", {})
        buf = cache.get(B)
        if buf is None:
            buf = {"tok": torch.empty(B, dtype=torch.int32, device=self.device),
                   "next": torch.empty(B, dtype=torch.int32, device=self.device),
                   "z1": torch.empty(B, V, dtype=torch.float32, device=self.device),
                   "z2": torch.empty((B, V) if self.cfg.n_paths == 2 else (self.cfg.n_paths - 1, B, V),
                                     dtype=torch.float32, device=self.device),
                   "alpha": torch.empty(B, dtype=torch.float32, device=self.device)}
            cache[B] = buf
        buf["tok"].copy_(tokens_dev)
        if grouped:
            self.decode_step(buf["tok"], buf["next"], buf["z1"], buf["z2"], buf["alpha"])
            return {k: buf[k].clone() for k in ("next", "z1", "z2", "alpha")}
        self.decode_step_primary_only(buf["tok"], buf["next"], buf["z1"])
        return {k: buf[k].clone() for k in ("next", "z1")}

    # -- diagnostics ----------------------------------------------------------------------
    def last_experts(self, batch: int) -> torch.Tensor:
        """[n_layers, n_paths, batch, kmax] expert ids used by the last decode step."""
        ptr, km = C.c_void_p(None), C.c_int32(0)
        self._check(self.L.dbt_last_experts(self._h, C.byref(ptr), C.byref(km)))
        n = self.cfg.n_layers * self.cfg.n_paths * self.max_batch * km.value
        torch.cuda.synchronize(self.device)
        host = torch.empty(n, dtype=torch.int32)
        # the ids live inside the workspace tensor: locate them by address
        off = ptr.value - self.workspace.data_ptr()
        host.copy_(self.workspace[off:off + 4 * n].view(torch.int32).cpu())
        return host.view(self.cfg.n_layers, self.cfg.n_paths, self.max_batch, km.value)[:, :, :batch].contiguous()

    def last_expert_union(self) -> list[int]:
        buf = (C.c_int32 * self.cfg.n_layers)()
        self._check(self.L.dbt_last_expert_union(self._h, buf))
        return list(buf)

    def sync_status(self) -> tuple[int, int]:
        s, d = C.c_int32(0), C.c_int32(0)
        st = self.L.dbt_sync_status(self._h, C.byref(s), C.byref(d))
        if st not in (DBT_OK, 6, 7):
            self._check(st)
        return s.value, d.value

    def profile_begin(self):
        self._check(self.L.dbt_profile_begin(self._h))

    def profile_end(self) -> list[dict]:
        buf = (DbtProfileEntry * 64)()
        n = C.c_int32(0)
        self._check(self.L.dbt_profile_end(self._h, buf, 64, C.byref(n)))
        return [dict(name=buf[i].name.decode(), launches=buf[i].launches, total_ms=buf[i].total_ms,
                     bytes=buf[i].bytes) for i in range(n.value)]

    def launch_count(self) -> int:
        return self.L.dbt_launch_count(self._h)

    # -- the cache through the C ABI (dbt_kv_export / dbt_kv_import) ---------------------------
    def export_kv(self, batch: int, length: int, seq_ids=None):
        """K, V [n_layers, batch, length, kv_dim] of sequences `seq_ids` (default 0..batch-1) as CPU
        tensors of the model's storage type."""
        c = self.cfg
        k = torch.empty(c.n_layers, batch, length, c.kv_dim, dtype=c.torch_dtype)
        v = torch.empty_like(k)
        ids = None if seq_ids is None else torch.as_tensor(seq_ids, dtype=torch.int32).contiguous()
        assert ids is None or ids.numel() == batch
        self._check(self.L.dbt_kv_export(self._h, _p(ids), batch, length, k.data_ptr(), v.data_ptr()))
        return k, v

    def import_kv(self, k: torch.Tensor, v: torch.Tensor, seq_ids=None):
        """Load K, V [n_layers, B, T, kv_dim] (any float type; converted to the model's) into sequences
        `seq_ids` (default 0..B-1) and set their lengths to T."""
        c = self.cfg
        k = k.to("cpu", c.torch_dtype).contiguous()
        v = v.to("cpu", c.torch_dtype).contiguous()
        assert k.shape == v.shape and k.shape[0] == c.n_layers and k.shape[3] == c.kv_dim
        ids = None if seq_ids is None else torch.as_tensor(seq_ids, dtype=torch.int32).contiguous()
        assert ids is None or ids.numel() == k.shape[1]
        self._check(self.L.dbt_kv_import(self._h, _p(ids), k.shape[1], k.shape[2], k.data_ptr(), v.data_ptr()))

    # -- direct pool access for the benchmark's synthetic fills (the pool is the caller's memory) --
    def write_kv(self, k: torch.Tensor, v: torch.Tensor, page_table: torch.Tensor | None = None):
        """Scatter contiguous K, V [L, B, T, kv_dim] into the paged pool and set the lengths."""
        B, T = k.shape[1], k.shape[2]
        pt = page_table if page_table is not None else self.page_table
        scatter_kv(self.kv_view(), k.to(self.device, self.cfg.torch_dtype), v.to(self.device, self.cfg.torch_dtype),
                   pt.to(self.device), self.cfg)
        self.set_seq_lens([T] * B)


def _page_slot(pt: torch.Tensor, T: int, page_size: int):
    pos = torch.arange(T, device=pt.device)
    pages = pt.long()[:, pos // page_size]                       # [B, T] physical page of each position
    slots = (pos % page_size)[None, :].expand(pt.shape[0], T)    # [B, T]
    return pages, slots


def scatter_kv(view: torch.Tensor, k: torch.Tensor, v: torch.Tensor, pt: torch.Tensor, cfg: ModelConfig):
    """view [L, 2, P, n_kv, page, dh]  <-  k, v [L, B, T, kv_dim] through page table pt [B, pages]."""
    Lyr, B, T, _ = k.shape
    pages, slots = _page_slot(pt[:B], T, cfg.page_size)
    for which, src in ((0, k), (1, v)):
        s = src.view(Lyr, B, T, cfg.n_kv_heads, cfg.head_dim).permute(1, 2, 0, 3, 4)  # [B, T, L, n_kv, dh]
        sub = view[:, which]                                                          # [L, P, n_kv, page, dh]
        sub[:, pages, :, slots, :] = s  # the two index tensors broadcast to [B, T] and move to the front

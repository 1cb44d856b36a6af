#!/usr/bin/env python
"""Benchmark of the grouped decode step (Decode-Branch Transformer) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                    [--model 1b|8b|moe|tiny] [--batch B] [--ctx S] [--kv prefill|synthetic]

One "step" is one grouped decode step (primary + branch rows through the shared matrices and
one pass over the primary KV cache) for a batch of B sequences.  The default workload is the
1B dense bf16 model at batch 16 with a 2048-token prompt.  Rank 0 prints one JSON line.
With N > 1 (torchrun) every rank runs an independent replica on its own GPU: the step has no
exchange between sequences, so there is no collective on the data path.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2608_12385_b200 import replicas  # noqa: E402
from paper_2608_12385_b200.inputs import PRESETS, make_synthetic_kv, make_tokens, make_weights  # noqa: E402

# ncu DRAM traffic / algorithmic bytes per launch (captures summarised under profiles/): attention 140.8 MB
# read+written for 134.6 MB of visible K/V (the rest is the Q|K|V partials it consumes and its output); the GEMMs
# read their weights once (46.47 MB for 46.14 MB of gate|up weights).
NCU_TRAFFIC_OVER_ALGORITHMIC = {"attention": 141.9 / 134.45, "gemm_gateup": 1.007, "gemm_down": 1.034, "gemm_qkv": 1.02,
                                "gemm_o": 1.04}
METRIC = "grouped_decode_tokens_per_s"
UNIT = "tokens/s"


def load_peaks() -> dict:
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", 1400.0)),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def prefill_flops(cfg, B: int, n: int) -> float:
    """Useful FLOPs of a primary-only prefill of n positions for B sequences: every layer matrix once per token
    (2 FLOP per weight; MoE: k_primary routed experts + the shared ones) plus causal attention
    (Q K^T and P V over n (n + 1) / 2 query-key pairs per head)."""
    per_layer = (cfg.q_dim + 2 * cfg.kv_dim) * cfg.d_model + cfg.d_model * cfg.q_dim
    if cfg.is_moe:
        per_layer += 3 * cfg.d_expert * cfg.d_model * (cfg.k_primary + cfg.n_shared_experts) + cfg.n_experts * cfg.d_model
    else:
        per_layer += 3 * cfg.d_ff * cfg.d_model
    gemm = 2.0 * per_layer * cfg.n_layers * B * n
    attn = 4.0 * cfg.q_dim * cfg.n_layers * B * (n * (n + 1) / 2.0)
    return gemm + attn


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples taken while the timed region runs."""
    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index: int):
        self.proc, self.path = None, None
        try:
            uuid = str(torch.cuda.get_device_properties(device_index).uuid)
            if not uuid.startswith("GPU-"):
                uuid = "GPU-" + uuid
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={uuid}", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self) -> dict:
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        rows = []
        try:
            with open(self.path) as f:
                for line in f:
                    parts = [x.strip() for x in line.split(",")]
                    if len(parts) == 7 and parts[0].replace(".", "").isdigit():
                        rows.append(parts)
            os.unlink(self.path)
        except Exception:
            pass
        if rows:
            sm = sorted(float(r[0]) for r in rows)
            out["sm_mhz"] = sm[len(sm) // 2]
            out["sm_max_mhz"] = float(rows[0][1])
            out["power_w_max"] = max(float(r[2]) for r in rows if r[2].replace(".", "").isdigit())
            names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
            out["reasons"] = [n for i, n in enumerate(names) if any(r[3 + i] == "Active" for r in rows)]
            out["samples"] = len(rows)
        return out


def step_bytes(cfg, B: int, ctx_keys_first: int, steps: int, union=None) -> float:
    """Algorithmic bytes of one step, averaged over `steps` steps whose first reads
    ctx_keys_first keys per sequence: every shared matrix once + every visible K/V once.
    MoE: `union` = routed experts loaded per layer (realised, read back from the device)."""
    avg_keys = ctx_keys_first + (steps - 1) / 2.0
    mats = cfg.matrix_bytes_moe_step(union) if cfg.is_moe else cfg.matrix_bytes_dense_step()
    return mats + B * avg_keys * cfg.kv_bytes_per_token()


def bench_config(args):
    cfg = PRESETS[args.model]()
    if cfg.is_moe:
        cfg = cfg.replace(k_branch=args.k_branch, router_mode=args.router_mode, compute_matched=args.compute_matched)
        if args.k_primary:
            cfg = cfg.replace(k_primary=args.k_primary)
    if args.paths != 2:  # more decode branches (Appendix C.1)
        cfg = cfg.replace(n_paths=args.paths)
    if args.layers:  # profiler captures of one kernel: fewer layers, less device memory to save and restore
        cfg = cfg.replace(n_layers=args.layers)
    return cfg


def workload_name(cfg, args) -> str:
    if not cfg.is_moe:
        return (f"dense-{args.model}" + (f" (cut to {cfg.n_layers} layers)" if args.layers else "")
                + (f" with {cfg.n_paths - 1} decode branches" if cfg.n_paths != 2 else ""))
    kind = "compute-matched " if cfg.compute_matched else ""
    cut = f", cut to {cfg.n_layers} layers" if args.layers else ""
    return f"{kind}moe-{args.model} (top-{cfg.k_primary} primary, top-{cfg.k_branch} branch{cut})"


def run_ours(args) -> dict | None:
    from paper_2608_12385_b200 import binding, build

    rank, local_rank, world = replicas.init()
    torch.cuda.set_device(local_rank)
    dev = f"cuda:{local_rank}"
    build.build()
    cfg = bench_config(args)
    B, S, K, W = args.batch, args.ctx, args.steps, args.warmup
    t0 = time.time()
    w = make_weights(cfg, seed=0)
    wd = binding.weights_to_device(w, dev)
    max_seq = S + max(K, 8) + W + 8
    stream = torch.cuda.current_stream()
    m = binding.Model(cfg, wd, B, max_seq, stream=stream)
    prompt = make_tokens(cfg, B, S, seed=1 + rank)
    kv_mode = args.kv
    t_prefill = None
    if kv_mode == "prefill":
        tp = time.time()
        m.prefill(prompt[:, : S - 1].to(dev).contiguous())
        torch.cuda.synchronize()
        t_prefill = time.time() - tp
    elif 2 * cfg.n_layers * B * (S - 1) * cfg.kv_dim * (2 if cfg.weight_dtype == "bf16" else 4) <= 8e9:
        k, v = make_synthetic_kv(cfg, B, S - 1, seed=3 + rank)
        m.write_kv(k, v)
        del k, v
    else:
        # caches beyond a few GB are not drawn on the host: the pool is filled in place, layer by layer, from a seeded
        # device generator with the same distributions (K ~ N(0, 1), V ~ N(0, 0.9)); timing does not depend on the values
        gen = torch.Generator(device=dev)
        gen.manual_seed(3 + rank)
        view = m.kv_view()  # [L, 2, pages, n_kv, page, d_h]
        for layer in range(view.shape[0]):
            view[layer, 0].normal_(0.0, 1.0, generator=gen)
            view[layer, 1].normal_(0.0, 0.9, generator=gen)
        m.set_seq_lens([S - 1] * B)
        kv_mode = "synthetic (drawn on the device)"
    setup_s = time.time() - t0
    first = prompt[:, S - 1].to(dev).contiguous()
    tok_a = torch.empty(B, dtype=torch.int32, device=dev)
    tok_b = torch.empty(B, dtype=torch.int32, device=dev)

    def timed(grouped: bool, steps: int, warmup: int, sample_clocks: bool, min_total_ms: float = 500.0, max_regions: int = 200):
        """Regions of exactly `steps` steps (every region restarts from the prompt's end, after `warmup` untimed
        steps), each bracketed by barrier + synchronize and timed with CUDA events on the launching stream;
        repeated until at least min_total_ms of device time has been timed, so that the clock sampler sees the
        GPU under load for several samples whatever `steps` is.  Returns the MEDIAN region."""
        step = m.decode_step if grouped else m.decode_step_primary_only
        sampler = ClockSampler(local_rank) if sample_clocks else None
        regions, launches = [], 0
        while True:
            m.set_seq_lens([S - 1] * B)
            tok_a.copy_(first)
            cur, nxt = tok_a, tok_b
            for _ in range(warmup):
                step(cur, nxt)
                cur, nxt = nxt, cur
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            replicas.barrier()
            torch.cuda.synchronize()
            launches0 = m.launch_count()
            e0.record(stream)
            for _ in range(steps):
                step(cur, nxt)
                cur, nxt = nxt, cur
            e1.record(stream)
            torch.cuda.synchronize()
            replicas.barrier()
            regions.append(e0.elapsed_time(e1))
            launches = m.launch_count() - launches0
            # every rank must leave the loop in the same round: decide on rank-uniform data
            done = replicas.all_agree(sum(regions) >= min_total_ms or len(regions) >= max_regions, dev)
            if done:
                break
        clocks = sampler.stop() if sampler else None
        regions.sort()
        return regions[len(regions) // 2], launches, clocks, len(regions)

    ms_po, _, _, _ = timed(False, K, W, False, min_total_ms=0.4 * args.min_timed_ms)
    po_union_m = m.last_expert_union() if cfg.is_moe else None
    ms_total, launches, clocks, n_regions = timed(True, K, W, True, min_total_ms=args.min_timed_ms)
    value, ms_max = replicas.aggregate_throughput(B * K, ms_total, dev)
    ms_step = ms_max / K
    union = po_union = None
    if cfg.is_moe:  # the routed experts actually loaded by the last grouped step, per layer
        union = m.last_expert_union()
    bytes_step = step_bytes(cfg, B, S + W, K, union)

    # per-kernel device time, on the launching stream, for the roofline of the dominant kernel
    m.set_seq_lens([S - 1] * B)
    tok_a.copy_(first)
    for _ in range(2):
        m.decode_step(tok_a, tok_b)
    m.profile_begin()
    nprof = min(K, 8)
    for _ in range(nprof):
        m.decode_step(tok_a, tok_b)
    prof = sorted(m.profile_end(), key=lambda r: -r["total_ms"])
    prof_total = sum(r["total_ms"] for r in prof)
    peaks = load_peaks()
    dom = next((r for r in prof if r["bytes"] > 0), prof[0])
    # DRAM traffic per launch of the dominant kernel: the ncu capture of the default workload
    # (dram__bytes_read.sum + dram__bytes_write.sum over the launch's algorithmic bytes), scaled to
    # this launch by its algorithmic bytes -- every kernel here reads its operands exactly once, so
    # traffic grows in proportion.  Kernels without a capture report null.
    ncu_ratio = NCU_TRAFFIC_OVER_ALGORITHMIC.get(dom["name"])
    dom_traffic = ncu_ratio * dom["bytes"] / max(dom["launches"], 1) if ncu_ratio else None
    dom_gbs = dom["bytes"] / (dom["total_ms"] * 1e-3) / 1e9 if dom["total_ms"] > 0 else 0.0

    # end to end through the host-buffer entry point: H2D of the step's tokens, D2H of its result
    m.set_seq_lens([S - 1] * B)
    th = first.cpu().pin_memory()
    nh = torch.empty(B, dtype=torch.int32).pin_memory()
    ah = torch.empty(B, dtype=torch.float32).pin_memory()
    for _ in range(W):
        m.decode_step_host(th, nh, ah)
        th.copy_(nh)
    replicas.barrier()
    torch.cuda.synchronize()
    te = time.perf_counter()
    for _ in range(K):
        m.decode_step_host(th, nh, ah)
        th.copy_(nh)
    torch.cuda.synchronize()
    e2e_ms = (time.perf_counter() - te) * 1e3
    e2e_value, _ = replicas.aggregate_throughput(B * K, e2e_ms, dev)
    status = m.sync_status()

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu = cpu_baseline(cfg, w, S, steps=4, warm=1)
        one = cpu_baseline(cfg, w, S, steps=1, warm=1, threads=1)
        cpu["one_thread"] = {"value": one["value"], "ms_per_step": one["ms_per_step"]}
    if rank != 0:
        return None
    hbm = peaks["hbm_gbs"]
    achieved_step_gbs = bytes_step / (ms_step * 1e-3) / 1e9
    return {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16" if cfg.weight_dtype == "bf16" else "f32", "data": "synthetic",
        "config": {"workload": f"{workload_name(cfg, args)} bf16 grouped decode, batch {B}/GPU, prompt {S}, "
                               f"{K} steps (paged KV, 16-token pages)",
                   "batch_per_gpu": B, "prompt": S, "kv_population": kv_mode,
                   "l2_policy": "inputs larger than L2 (weights + KV >= 1.7 GB per step vs 126 MB)",
                   "replicas": world, "device_status": status[0],
                   "timed_regions": n_regions, "region_reported": "median of the K-step regions"},
        "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": 4 * B, "d2h_bytes_per_step": 8 * B,
                "ms_per_step": e2e_ms / K},
        "gpu_launches": launches,
        "roofline": {"bound": "hbm", "kernel": dom["name"], "achieved": dom_gbs, "peak": hbm, "unit": "GB/s",
                     "frac": dom_gbs / hbm, "peak_source": peaks["source"], "traffic": dom_traffic,
                     "traffic_source": "ncu capture of dense-1b batch 16 context 2048, scaled by algorithmic bytes" if dom_traffic else None,
                     "kernel_share_of_step": dom["total_ms"] / prof_total if prof_total else None,
                     "kernel_avg_us": 1e3 * dom["total_ms"] / max(dom["launches"], 1),
                     "kernel_bytes_per_launch": dom["bytes"] / max(dom["launches"], 1)},
        "step_roofline": {"algorithmic_bytes_per_step": bytes_step, "achieved_gbs": achieved_step_gbs,
                          "frac_of_measured_copy": achieved_step_gbs / hbm, "frac_of_8tbs_nominal": achieved_step_gbs / 8000.0},
        "primary_only": {"ms_per_step": ms_po / K, "grouped_over_primary_only": (ms_total / K) / (ms_po / K),
                         "experts_loaded_per_layer": po_union_m},
        "moe": None if not cfg.is_moe else {"k_primary": cfg.k_primary, "k_branch": cfg.k_branch,
                                            "router_mode": cfg.router_mode, "compute_matched": cfg.compute_matched,
                                            "experts_loaded_per_layer": union,
                                            "mean_union": sum(union) / len(union)},
        "kernels": [{"name": r["name"], "launches_per_step": r["launches"] / nprof,
                     "us_per_step": 1e3 * r["total_ms"] / nprof,
                     "gbs": (r["bytes"] / (r["total_ms"] * 1e-3) / 1e9) if r["bytes"] > 0 and r["total_ms"] > 0 else None}
                    for r in prof],
        "cpu_baseline": cpu, "setup_s": setup_s, "prefill_s": t_prefill,
        "prefill": None if t_prefill is None else {
            "tokens": B * (S - 1), "tokens_per_s": B * (S - 1) / t_prefill,
            "useful_tflops": prefill_flops(cfg, B, S - 1) / t_prefill / 1e12,
            "frac_of_bf16_sustained": prefill_flops(cfg, B, S - 1) / t_prefill / 1e12 / peaks["bf16_tflops_sustained"],
            "bound": "tensor", "note": "primary path only (Section 4.4 item 1); wall clock of one dbt_prefill call "
                                       "including its launches; activations as two bf16 planes double the tensor work"},
    }


def cpu_baseline(cfg, w, S: int, steps: int, batch: int = 1, warm: int = 0, threads: int = 0) -> dict:
    """The oracle as it stands, timed on this machine's host cores on a bounded sample of the
    workload: `batch` sequence(s) with an S-1 position synthetic cache, `warm` untimed and `steps`
    timed grouped steps (threads: 0 = all cores)."""
    import oracle

    all_threads = oracle.get_threads()
    if threads:
        oracle.set_threads(threads)

    k, v = make_synthetic_kv(cfg, batch, S - 1, seed=3)
    om = oracle.OracleModel(cfg, w, batch, S + steps + warm + 1)
    om.inject_kv(k, v, S - 1)
    tok = make_tokens(cfg, batch, steps + warm, seed=2).numpy()
    for i in range(warm):
        om.decode_step(tok[:, i])
    t0 = time.perf_counter()
    for i in range(steps):
        om.decode_step(tok[:, warm + i])
    dt = time.perf_counter() - t0
    used = oracle.get_threads()
    if threads:
        oracle.set_threads(all_threads)
    return {"value": batch * steps / dt, "unit": UNIT, "cores": used, "kind": "oracle",
            "sample": f"{steps} grouped steps (after {warm} warm) of {batch} sequence(s) at context {S} "
                      f"(synthetic cache), full model",
            "ms_per_step": 1e3 * dt / steps}


def run_reference(args) -> dict | None:
    """The reference arm: the CPU oracle on the same model and context, one sequence per step."""
    rank, _, world = replicas.env_rank()
    if rank != 0:
        return None
    cfg = bench_config(args)
    w = make_weights(cfg, seed=0)
    S, K, W = args.ctx, args.steps, min(args.warmup, 1)
    K = min(K, args.reference_max_steps)
    base = cpu_baseline(cfg, w, S, steps=K, batch=1, warm=W)
    return {
        "impl": "reference", "metric": METRIC, "value": base["value"], "unit": UNIT, "n_gpus": world, "steps": K,
        "warmup": W, "ms_per_step": base["ms_per_step"], "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32 storage, f64 accumulate", "data": "synthetic",
        "config": {"workload": f"{workload_name(cfg, args)} grouped decode, CPU oracle, 1 sequence per step (bounded sample of "
                               f"batch {args.batch}), context {S}"},
        "cpu_baseline": {"value": base["value"], "unit": UNIT, "kind": "oracle", "cores": base["cores"],
                         "sample": base["sample"]},
        "e2e": {"value": base["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=128)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--model", default="1b", choices=sorted(PRESETS))
    ap.add_argument("--batch", type=int, default=16)
    ap.add_argument("--ctx", type=int, default=2048)
    ap.add_argument("--kv", default="prefill", choices=["prefill", "synthetic"])
    ap.add_argument("--k-branch", type=int, default=2, help="MoE: branch top-k")
    ap.add_argument("--k-primary", type=int, default=0, help="MoE: primary top-k (0: the preset's)")
    ap.add_argument("--router-mode", type=int, default=0, help="MoE: 0 independent routing, 1 router replay")
    ap.add_argument("--compute-matched", type=int, default=0,
                    help="MoE: 1 = compute-matched allocation (attention and shared expert on the primary path only)")
    ap.add_argument("--paths", type=int, default=2, help="residual paths K: the primary plus K-1 decode branches (Appendix C.1)")
    ap.add_argument("--layers", type=int, default=0, help="cut the model to this many layers (profiler captures only)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--min-timed-ms", type=float, default=500.0,
                    help="repeat the K-step timed region until this much device time has been timed (0: one region; "
                         "profiler captures)")
    ap.add_argument("--reference-max-steps", type=int, default=128)
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    out = run_reference(args) if args.impl == "reference" else run_ours(args)
    if out is not None:
        print(json.dumps(out), flush=True)
    replicas.shutdown()


if __name__ == "__main__":
    main()

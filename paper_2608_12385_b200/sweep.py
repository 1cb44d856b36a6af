"""Batch x context sweep of the grouped decode step on one GPU.

    python -m paper_2608_12385_b200.sweep --model 1b --out sweep_1b.json

For every (batch, context) cell: grouped and primary-only step time (CUDA events around a run of
graph-replayed steps), algorithmic bytes (shared matrices once + visible K/V once), achieved
GB/s against the measured copy peak and the 8 TB/s nominal figure, and the grouped /
primary-only ratio.  With --tiers the small cells are also run through the CUDA-core GEMV
path (DBT_FORCE_PATH=simt) to show where the tensor-core tier takes over.  The cache is filled
on the device with seeded N(0,1) values (timing does not depend on the values); cells whose
cache would exceed --kv-cap-gb are recorded as skipped, not run.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import time

import torch

from . import binding, build
from .inputs import PRESETS, make_tokens, make_weights


def time_steps(m: binding.Model, B: int, ctx: int, steps: int, warmup: int, grouped: bool) -> float:
    dev = m.device
    m.set_seq_lens([ctx - 1] * B)
    a = make_tokens(m.cfg, B, 1, seed=5).to(dev).view(-1).contiguous()
    b = torch.empty_like(a)
    step = m.decode_step if grouped else m.decode_step_primary_only
    cur, nxt = a, b
    for _ in range(warmup):
        step(cur, nxt)
        cur, nxt = nxt, cur
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(steps):
        step(cur, nxt)
        cur, nxt = nxt, cur
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / steps


def run_cell(cfg, wd, B: int, ctx: int, steps: int, warmup: int, force_path: str | None) -> dict:
    if force_path:
        os.environ["DBT_FORCE_PATH"] = force_path
    else:
        os.environ.pop("DBT_FORCE_PATH", None)
    m = binding.Model(cfg, wd, B, ctx + steps + warmup + 8)
    gen = torch.Generator(device=m.device)
    gen.manual_seed(3)
    m.kv_pool.normal_(0.0, 1.0, generator=gen)
    ms_g = time_steps(m, B, ctx, steps, warmup, True)
    ms_p = time_steps(m, B, ctx, steps, warmup, False)
    status = m.sync_status()
    m.close()
    del m
    torch.cuda.empty_cache()
    avg_keys = ctx + warmup + (steps - 1) / 2.0
    bytes_step = cfg.matrix_bytes_dense_step() + B * avg_keys * cfg.kv_bytes_per_token()
    return {"batch": B, "ctx": ctx, "path": force_path or "tensor-core", "ms_grouped": ms_g, "ms_primary_only": ms_p,
            "grouped_over_primary_only": ms_g / ms_p, "tokens_per_s": B / (ms_g * 1e-3), "bytes_per_step": bytes_step,
            "gbs": bytes_step / (ms_g * 1e-3) / 1e9, "device_status": status[0]}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--model", default="1b", choices=sorted(PRESETS))
    ap.add_argument("--batches", default="1,2,4,8,16,32,64,128")
    ap.add_argument("--contexts", default="1024,4096,16384,65536")
    ap.add_argument("--steps", type=int, default=32)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--kv-cap-gb", type=float, default=100.0)
    ap.add_argument("--tiers", action="store_true", help="also run small cells through the CUDA-core GEMV path")
    ap.add_argument("--peak-gbs", type=float, default=None)
    ap.add_argument("--out", default="sweep.json")
    args = ap.parse_args()
    build.build()
    cfg = PRESETS[args.model]()
    if cfg.is_moe:
        raise SystemExit("the sweep times dense models")
    peak = args.peak_gbs
    if peak is None:
        path = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "MEASURED_PEAKS.json")
        peak = json.load(open(path))["hbm_gbs"] if os.path.exists(path) else 6650.0
    t0 = time.time()
    wd = binding.weights_to_device(make_weights(cfg, seed=0))
    rows = []
    for ctx in [int(x) for x in args.contexts.split(",")]:
        for B in [int(x) for x in args.batches.split(",")]:
            kv_gb = B * (ctx + 64) * cfg.kv_bytes_per_token() / 1e9
            if kv_gb > args.kv_cap_gb:
                rows.append({"batch": B, "ctx": ctx, "skipped": f"cache {kv_gb:.0f} GB exceeds the {args.kv_cap_gb:.0f} GB cap"})
                continue
            paths = [None] + (["simt"] if args.tiers and B <= 8 and ctx <= 4096 else [])
            for fp in paths:
                r = run_cell(cfg, wd, B, ctx, args.steps, args.warmup, fp)
                r["frac_of_measured_copy"] = r["gbs"] / peak
                r["frac_of_8tbs"] = r["gbs"] / 8000.0
                rows.append(r)
                print(json.dumps(r), file=sys.stderr, flush=True)
    os.environ.pop("DBT_FORCE_PATH", None)
    out = {"model": args.model, "peak_gbs": peak, "steps": args.steps, "warmup": args.warmup, "wall_s": time.time() - t0,
           "rows": rows}
    os.makedirs(os.path.dirname(os.path.abspath(args.out)), exist_ok=True)
    with open(args.out, "w") as f:
        json.dump(out, f, indent=1)
    print(json.dumps({"cells": len(rows), "out": args.out, "wall_s": out["wall_s"]}))


if __name__ == "__main__":
    main()

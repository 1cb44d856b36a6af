"""In-graph timeline of a grouped decode step: when each kernel of the captured step starts, when its
dependency wait returns and when it ends, in device time (%globaltimer), read from one replay of the
step's CUDA graph.

    python -m paper_2608_12385_b200.timeline [--model 1b|8b|moe] [--batch B] [--ctx S] [--layers L]
                                             [--primary-only] [--out FILE.json]

The figures that per-launch CUDA events give serialise the graph (every kernel is timed alone, launch
included); this tool shows the step as it runs: kernels overlap through programmatic dependent launch, so a
kernel's "resident" time starts before its predecessor ends and what matters is the distance between
consecutive dependency-wait returns.  It builds an instrumented copy of the library
(libdbt_b200_timeline.so, -DDBT_TIMELINE: block 0 of every kernel stores three timestamps and up to four
marks; stores only, a few nanoseconds) next to the normal one and loads that copy in this process only.

Columns, per kernel of one layer in the middle of the model, in microseconds relative to the layer's first
kernel: entry (block 0 resident), wait (its griddepcontrol.wait returned: the predecessor's results are
visible), end (block 0 done), then wait-to-wait = the kernel's share of the critical path.
"""
from __future__ import annotations

import argparse
import ctypes as C
import json
import os
import subprocess
import sys

import torch

from . import binding, build
from .inputs import PRESETS, make_tokens, make_weights

TL_LIB = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libdbt_b200_timeline.so")


def build_instrumented() -> str:
    src_time = build._newest_source_mtime()
    if os.path.exists(TL_LIB) and os.path.getmtime(TL_LIB) >= src_time:
        return TL_LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    tmp = TL_LIB + f".tmp{os.getpid()}"
    cmd = [nvcc, *build.NVCC_FLAGS, "-DDBT_TIMELINE", "-o", tmp,
           *[os.path.join(build.CSRC, s) for s in build.SOURCES], "-lcuda"]
    subprocess.run(cmd, check=True)
    os.replace(tmp, TL_LIB)
    return TL_LIB


def read_records(L, max_records: int = 16384):
    buf = (C.c_ulonglong * (8 * max_records))()
    L.dbt_debug_timeline.argtypes = [C.c_void_p, C.c_int]
    L.dbt_debug_timeline.restype = C.c_int
    n = L.dbt_debug_timeline(buf, max_records)
    recs = []
    for i in range(max(n, 0)):
        r = buf[8 * i: 8 * i + 8]
        tag = bytes((r[0] >> (8 * k)) & 0xFF for k in range(8)).rstrip(b"\0").decode(errors="replace")
        recs.append({"name": tag, "entry": r[1], "wait": r[2] or r[1], "end": r[3], "marks": list(r[4:8])})
    recs.sort(key=lambda x: x["wait"])
    return recs


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--model", default="1b", choices=sorted(PRESETS))
    ap.add_argument("--batch", type=int, default=16)
    ap.add_argument("--ctx", type=int, default=2048)
    ap.add_argument("--layers", type=int, default=0)
    ap.add_argument("--paths", type=int, default=2, help="residual paths K (the primary plus K-1 decode branches)")
    ap.add_argument("--primary-only", action="store_true")
    ap.add_argument("--out", default="")
    args = ap.parse_args()
    binding.LIB_PATH = build_instrumented()  # this process loads the instrumented copy
    L = binding.load_library()
    cfg = PRESETS[args.model]()
    if args.layers:
        cfg = cfg.replace(n_layers=args.layers)
    if args.paths != 2:
        cfg = cfg.replace(n_paths=args.paths)
    w = make_weights(cfg, seed=0)
    B, S = args.batch, args.ctx
    m = binding.Model(cfg, binding.weights_to_device(w), B, S + 64)
    m.kv_pool.normal_()
    m.set_seq_lens([S - 1] * B)
    tok = make_tokens(cfg, B, 1).cuda().view(-1).contiguous()
    nxt = torch.empty_like(tok)
    step = m.decode_step_primary_only if args.primary_only else m.decode_step
    for _ in range(6):
        step(tok, nxt)
    torch.cuda.synchronize()
    read_records(L)  # drop the warm-up records
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    step(tok, nxt)
    e1.record()
    torch.cuda.synchronize()
    recs = read_records(L)
    t0 = recs[0]["wait"]
    step_us = (max(r["end"] for r in recs) - t0) / 1e3
    print(f"{args.model} batch {B} ctx {S}: one step = {e0.elapsed_time(e1) * 1e3:.1f} us by events, "
          f"{step_us:.1f} us first wait to last end, {len(recs)} records")
    # one layer in the middle: from the Q|K|V GEMM before an attention record to the one before the next
    names = [r["name"] for r in recs]
    att = [i for i, n in enumerate(names) if n == "attentio"]
    k = len(att) // 2
    lo = att[k] - 1
    hi = att[k + 1] - 1 if k + 1 < len(att) else len(recs) - 1
    layer = recs[lo: hi + 1]
    base = layer[0]["wait"]
    print(f"{'kernel':12s} {'entry':>8s} {'wait':>8s} {'end':>8s} {'wait->wait':>10s}  marks (us after wait)")
    rows = []
    for i, r in enumerate(layer[:-1]):
        nxt_wait = layer[i + 1]["wait"]
        marks = [round((x - r["wait"]) / 1e3, 2) for x in r["marks"] if x]
        row = {"name": r["name"], "entry": (r["entry"] - base) / 1e3, "wait": (r["wait"] - base) / 1e3,
               "end": (r["end"] - base) / 1e3, "crit": (nxt_wait - r["wait"]) / 1e3, "marks": marks}
        rows.append(row)
        print(f"{row['name']:12s} {row['entry']:8.2f} {row['wait']:8.2f} {row['end']:8.2f} {row['crit']:10.2f}  {marks}")
    print(f"layer total {sum(r['crit'] for r in rows):.2f} us")
    # whole-step shares by kernel name (wait -> next wait)
    share: dict[str, float] = {}
    for i, r in enumerate(recs[:-1]):
        share[r["name"]] = share.get(r["name"], 0.0) + (recs[i + 1]["wait"] - r["wait"]) / 1e3
    print("critical-path share per kernel family (us per step):",
          {k: round(v, 1) for k, v in sorted(share.items(), key=lambda kv: -kv[1])})
    if args.out:
        with open(args.out, "w") as f:
            json.dump({"config": vars(args), "step_us": step_us, "layer": rows, "share": share, "names": names[:40]}, f)


if __name__ == "__main__":
    main()

"""Writes tests/golden/oracle_small_dense.json by calling only oracle/ (never the CUDA path).

The paper prints no worked numeric example of the forward pass, so this fixture is not a
paper value: it freezes the oracle's own output on one small seeded model so that a later
edit to the oracle's arithmetic shows up as a diff that its commit message has to justify.
Run from the repo root:  python tests/golden/make_golden.py
"""
import json
import os
import sys

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.dirname(os.path.dirname(HERE)))

import oracle  # noqa: E402
from paper_2608_12385_b200.inputs import ModelConfig, make_tokens, make_weights  # noqa: E402

CASES = {
    "dense": dict(d_model=32, n_layers=2, n_q_heads=4, n_kv_heads=2, head_dim=8, d_ff=48, vocab=50,
                  weight_dtype="fp32"),
    "moe": dict(d_model=32, n_layers=2, n_q_heads=4, n_kv_heads=2, head_dim=8, d_ff=0, vocab=50,
                weight_dtype="fp32", n_experts=6, d_expert=16, n_shared_experts=1, k_primary=2, k_branch=3),
}


def compute(case: str) -> dict:
    cfg = ModelConfig(**CASES[case])
    w = make_weights(cfg, seed=100, matrix_std=0.3)
    tok = make_tokens(cfg, 2, 6, seed=101).numpy()
    m = oracle.OracleModel(cfg, w, 2, 6)
    m.prefill(tok[:, :4], want_logits=False)
    m.decode_step(tok[:, 4])
    o = m.decode_step(tok[:, 5])
    return {"z1_head": o["z1"][:, :6].astype(float).round(6).tolist(),
            "z2_head": o["z2"][:, :6].astype(float).round(6).tolist(),
            "alpha": o["alpha"].astype(float).round(6).tolist(),
            "next": o["next"].tolist()}


if __name__ == "__main__":
    out = {case: compute(case) for case in CASES}
    with open(os.path.join(HERE, "oracle_small_dense.json"), "w") as f:
        json.dump({"source": "oracle/dbt_oracle.c via tests/golden/make_golden.py (no paper value exists)",
                   "cases": out}, f, indent=1)
    print(json.dumps(out)[:400])

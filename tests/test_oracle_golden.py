"""Regression fixture: the oracle's frozen output on one small seeded model (see
tests/golden/make_golden.py -- written by the oracle only; the paper prints no example)."""
import importlib.util
import json
import os

import numpy as np
import pytest

HERE = os.path.dirname(os.path.abspath(__file__))


@pytest.mark.parametrize("case", ["dense", "moe"])
def test_oracle_matches_frozen_fixture(case):
    spec = importlib.util.spec_from_file_location("make_golden", os.path.join(HERE, "golden", "make_golden.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    with open(os.path.join(HERE, "golden", "oracle_small_dense.json")) as f:
        want = json.load(f)["cases"][case]
    got = mod.compute(case)
    np.testing.assert_allclose(got["z1_head"], want["z1_head"], atol=2e-6)
    np.testing.assert_allclose(got["z2_head"], want["z2_head"], atol=2e-6)
    np.testing.assert_allclose(got["alpha"], want["alpha"], atol=2e-6)
    assert got["next"] == want["next"]

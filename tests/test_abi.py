"""CPU-side checks of the C-ABI library: it builds, loads, exports every symbol that
include/dbt.h declares, and its host-side argument validation works without a GPU."""
import ctypes as C
import os
import re

import pytest

from paper_2608_12385_b200 import binding, build
from paper_2608_12385_b200.inputs import dense_1b, moe_1b, tiny_dense_fp32

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.load_library()


def declared_symbols():
    names = set()
    for fn in os.listdir(os.path.join(ROOT, "include")):
        if fn.endswith(".h"):
            text = open(os.path.join(ROOT, "include", fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names |= set(re.findall(r"\b(dbt_[a-z0-9_]+)\s*\(", text))
    return names


def test_every_declared_symbol_is_exported(lib):
    names = declared_symbols()
    assert {"dbt_create", "dbt_prefill", "dbt_decode_step", "dbt_decode_step_primary_only"} <= names
    for name in names:
        assert hasattr(lib, name), f"{name} declared in include/ but not exported"
    assert set(binding.EXPORTS) <= names


def test_version_string(lib):
    assert b"sm_100a" in lib.dbt_version()


def test_query_sizes_matches_pool_layout(lib):
    cfg = dense_1b()
    kv, ws = binding.query_sizes(cfg, max_batch=4, max_seq=256, num_pages=64)
    assert kv == cfg.n_layers * 2 * 64 * cfg.n_kv_heads * 16 * cfg.head_dim * 2
    assert ws > 0 and ws % 256 == 0
    kv32, _ = binding.query_sizes(tiny_dense_fp32(), max_batch=2, max_seq=80, num_pages=10)
    assert kv32 == 4 * 2 * 10 * 4 * 16 * 64 * 4


@pytest.mark.parametrize("mutate,status", [
    (dict(head_dim=96), 2), (dict(page_size=32), 2), (dict(n_kv_heads=3), 2), (dict(d_model=0), 1),
    (dict(n_q_heads=32, n_kv_heads=2), 2), (dict(weight_dtype="fp32", d_ff=100), 2),
])
def test_unsupported_configs_are_rejected_on_the_host(lib, mutate, status):
    cfg = dense_1b().replace(**mutate)
    with pytest.raises(binding.DbtError) as e:
        binding.query_sizes(cfg, 1, 64, 8)
    assert e.value.status == status


def test_moe_topk_larger_than_expert_count_is_rejected(lib):
    with pytest.raises(binding.DbtError):
        binding.query_sizes(moe_1b().replace(k_branch=65), 1, 64, 8)


def test_create_rejects_bad_struct_size_and_null_pointers(lib):
    c = binding.make_config_struct(dense_1b(), 1, 64, 8)
    h = C.c_void_p(None)
    w = binding.DbtWeights()
    assert lib.dbt_create(C.byref(c), C.byref(w), None, None, None, C.byref(h)) == 1
    assert h.value is None
    c.struct_size = 4
    assert lib.dbt_create(C.byref(c), C.byref(w), None, None, None, C.byref(h)) == 1
    assert b"struct_size" in lib.dbt_last_error(None)


def test_null_handle_calls_do_not_crash(lib):
    assert lib.dbt_reset(None) == 1
    assert lib.dbt_seq_len(None, 0) == -1
    assert lib.dbt_launch_count(None) == 0
    lib.dbt_destroy(None)


def _c_layout(header: str, structs: dict) -> dict:
    """sizeof and field offsets as the C compiler sees them (gcc on the header itself)."""
    import subprocess
    import tempfile
    lines = [f'#include "{header}"', "#include <stdio.h>", "#include <stddef.h>", "int main(void) {"]
    for sname, fields in structs.items():
        lines.append(f'printf("{sname} %zu\\n", sizeof({sname}));')
        for f in fields:
            lines.append(f'printf("{sname}.{f} %zu\\n", offsetof({sname}, {f}));')
    lines += ["return 0;", "}"]
    with tempfile.TemporaryDirectory() as td:
        src, exe = os.path.join(td, "layout.c"), os.path.join(td, "layout")
        open(src, "w").write("\n".join(lines))
        subprocess.run(["gcc", "-I", os.path.dirname(header), "-o", exe, src], check=True)
        out = subprocess.run([exe], check=True, capture_output=True, text=True).stdout
    return {k: int(v) for k, v in (line.split() for line in out.splitlines())}


def _ctypes_layout(name: str, struct) -> dict:
    d = {name: C.sizeof(struct)}
    for f, _ in struct._fields_:
        d[f"{name}.{f}"] = getattr(struct, f).offset
    return d


def test_binding_structs_have_the_headers_layout():
    """The ctypes mirrors of dbt_config / dbt_layer_weights / dbt_weights follow include/dbt.h field by field."""
    pairs = {"dbt_config": binding.DbtConfig, "dbt_layer_weights": binding.DbtLayerWeights, "dbt_weights": binding.DbtWeights}
    want = _c_layout(os.path.join(ROOT, "include", "dbt.h"), {n: [f for f, _ in s._fields_] for n, s in pairs.items()})
    for n, s in pairs.items():
        for k, v in _ctypes_layout(n, s).items():
            assert want[k] == v, k


def test_oracle_wrapper_structs_have_the_oracle_headers_layout():
    import oracle
    pairs = {"orc_config": oracle.OrcConfig, "orc_layer_weights": oracle.OrcLayer, "orc_weights": oracle.OrcWeights}
    want = _c_layout(os.path.join(ROOT, "oracle", "dbt_oracle.h"), {n: [f for f, _ in s._fields_] for n, s in pairs.items()})
    for n, s in pairs.items():
        for k, v in _ctypes_layout(n, s).items():
            assert want[k] == v, k


def test_compute_matched_needs_an_moe_model(lib):
    with pytest.raises(binding.DbtError) as e:
        binding.query_sizes(dense_1b().replace(compute_matched=1), 1, 64, 8)
    assert e.value.status == 2
    kv, ws = binding.query_sizes(moe_1b().replace(compute_matched=1), 2, 64, 16)
    assert kv > 0 and ws > 0

"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every
declared symbol, sizes workspaces correctly and rejects bad arguments before any
CUDA call."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def pkg():
    import __graft_entry__

    __graft_entry__.build()
    import paper_2306_14048_b200 as p

    return p


def _declared_functions():
    names = []
    for fn in os.listdir(os.path.join(ROOT, "include")):
        if fn.endswith(".h"):
            text = open(os.path.join(ROOT, "include", fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names += re.findall(r"\b(h2o_[a-z0-9_]+)\s*\(", text)
    return sorted(set(names))


def test_library_exports_every_declared_symbol(pkg):
    declared = _declared_functions()
    assert "h2o_cache_create" in declared and "h2o_decode_step" in declared and "h2o_prefill_select" in declared
    assert "h2o_decode_chunk" in declared
    raw = ctypes.CDLL(pkg.binding.LIB_PATH)
    for name in declared:
        assert hasattr(raw, name), "missing export: " + name
    assert set(pkg.EXPORTED) <= set(declared)


def test_workspace_arithmetic(pkg):
    cfg, keep = pkg.make_config(8, 32, 128, "bf16", [205] * 8, [205] * 8)
    slots = 8 * 32 * 412  # every unit's slot range is padded to a multiple of 4
    nbytes = pkg.h2o_cache_workspace_bytes(cfg)
    payload = slots * (2 * 128 * 2 + 8 + 4)
    assert payload <= nbytes <= payload + 64 * 1024  # K, V, acc (f64), pos (i32) + small tables
    cfg32, keep32 = pkg.make_config(1, 4, 64, "f32", [32], [32])
    assert pkg.h2o_cache_workspace_bytes(cfg32) >= 4 * 64 * (2 * 64 * 4 + 12)
    assert pkg.h2o_prefill_scratch_bytes(cfg, 16384) >= 16384 * 32 * 16
    assert pkg.h2o_prefill_scratch_bytes(cfg, 0) == 0


def test_full_cache_bytes_match_the_papers_example(pkg):
    """Section 1: a 30B model, batch 128, sequence length 1024 -> 180 GB of KV cache.  With a budget equal to the
    sequence length the library's K/V slots are that cache; its scores and positions add 12 bytes per slot."""
    vals = {}
    for line in open(os.path.join(ROOT, "tests", "golden", "kv_cache_size.txt")):
        if line.strip() and not line.startswith("#"):
            k, v = line.split()
            vals[k] = int(v)
    b, h, d, n = vals["batch"], vals["n_heads"], vals["head_dim"], vals["seq_len"]
    cfg, keep = pkg.make_config(b, h, d, "bf16", [n // 2] * b, [n // 2] * b)
    per_layer = pkg.h2o_cache_workspace_bytes(cfg)
    slots = b * h * n
    kv = 2 * slots * d * vals["bytes_per_element"]
    assert abs(kv * vals["model_layers"] / 1e9 - vals["kv_cache_gb"]) < 1.0  # 180.4 GB
    assert kv + slots * 12 <= per_layer <= kv + slots * 12 + slots * 4 + (b * h + 1024) * (d + 4) * 4 + (1 << 20)
    import bench

    one_unit_step = bench.decode_bytes_per_unit_step(n, d, vals["bytes_per_element"])
    assert one_unit_step == 2 * n * d * 2 + 20 * n + 6 * d * 2  # the decode step reads that cache once


@pytest.mark.parametrize("kw", [
    dict(head_dim=96), dict(dtype=7), dict(batch=0), dict(n_heads=0), dict(heavy=[-1]), dict(heavy=[0], recent=[0]),
    dict(recent=[1 << 20]),
])
def test_invalid_configs_are_rejected_on_the_host(pkg, kw):
    args = dict(batch=1, n_heads=2, head_dim=64, dtype="f32", heavy=[4], recent=[4])
    args.update(kw)
    cfg, keep = pkg.make_config(args["batch"], args["n_heads"], args["head_dim"], args["dtype"], args["heavy"], args["recent"])
    assert pkg.h2o_cache_workspace_bytes(cfg) == 0
    handle = ctypes.c_void_p()
    rc = pkg.lib.h2o_cache_create(ctypes.byref(handle), ctypes.byref(cfg), 256, 1 << 30)
    assert rc in (pkg.H2O_ERR_INVALID_ARG, pkg.H2O_ERR_UNSUPPORTED)
    assert handle.value is None


def test_create_argument_checks_and_no_fallback(pkg):
    import torch

    cfg, keep = pkg.make_config(1, 2, 64, "f32", [4], [4])
    need = pkg.h2o_cache_workspace_bytes(cfg)
    handle = ctypes.c_void_p()
    assert pkg.lib.h2o_cache_create(None, ctypes.byref(cfg), 256, need) == pkg.H2O_ERR_INVALID_ARG
    assert pkg.lib.h2o_cache_create(ctypes.byref(handle), ctypes.byref(cfg), None, need) == pkg.H2O_ERR_INVALID_ARG
    assert pkg.lib.h2o_cache_create(ctypes.byref(handle), ctypes.byref(cfg), 256, need - 1) == pkg.H2O_ERR_WORKSPACE
    assert pkg.lib.h2o_cache_create(ctypes.byref(handle), ctypes.byref(cfg), 8, need) == pkg.H2O_ERR_WORKSPACE
    if not torch.cuda.is_available():
        # no device: the library reports it instead of computing anything on the CPU
        assert pkg.lib.h2o_cache_create(ctypes.byref(handle), ctypes.byref(cfg), 256, need) == pkg.H2O_ERR_CUDA
        assert handle.value is None
    assert pkg.lib.h2o_cache_destroy(None) == 0
    for code in range(-7, 1):
        assert pkg.lib.h2o_strerror(code)
    assert pkg.lib.h2o_decode_step(None, None, None, None, None, None, None) == pkg.H2O_ERR_INVALID_ARG
    assert pkg.lib.h2o_decode_chunk(None, None, None, None, 4, None, None, None) == pkg.H2O_ERR_INVALID_ARG
    assert pkg.lib.h2o_cache_set_chunk_path(None, 0) == pkg.H2O_ERR_INVALID_ARG
    assert pkg.lib.h2o_cache_set_score_mode(None, 0) == pkg.H2O_ERR_INVALID_ARG
    assert pkg.lib.h2o_cache_fscore(None, 0, None, None) == pkg.H2O_ERR_INVALID_ARG
    assert pkg.lib.h2o_cache_set_mask(None, 1, 4, 2) == pkg.H2O_ERR_INVALID_ARG
    assert pkg.lib.h2o_cache_set_topk(None, 4) == pkg.H2O_ERR_INVALID_ARG
    assert pkg.lib.h2o_prefill_select(None, None, None, None, None, None, None, 0, None) == pkg.H2O_ERR_INVALID_ARG


def test_product_package_does_not_touch_the_oracle():
    """The CUDA package and the oracle share no code and never import each other."""
    pat = re.compile(r"(import\s+oracle|from\s+oracle|h2o_oracle|oracle/)")
    for dirpath, _, files in os.walk(os.path.join(ROOT, "paper_2306_14048_b200")):
        for fn in files:
            if fn.endswith((".py", ".cu", ".cuh", ".h")):
                assert not pat.search(open(os.path.join(dirpath, fn)).read()), fn
    for fn in os.listdir(os.path.join(ROOT, "oracle")):
        if fn.endswith((".py", ".c", ".h")):
            assert "paper_2306_14048_b200" not in open(os.path.join(ROOT, "oracle", fn)).read(), fn

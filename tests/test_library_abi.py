"""The C-ABI library builds for sm_100a, loads without a GPU and exports every entry point that
include/sentinel.h declares (no compute calls here)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def built():
    from paper_2603_03592_b200 import _build
    return _build.build()


def declared_entry_points():
    text = open(os.path.join(ROOT, "include", "sentinel.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(sentinel_[a-z_]+)\s*\(", text)))


def test_header_declares_the_named_calls():
    names = declared_entry_points()
    for must in ("sentinel_verifier_create", "sentinel_verify", "sentinel_update_reference", "sentinel_destroy"):
        assert must in names


def test_library_exports_every_declared_symbol(built):
    lib = ctypes.CDLL(built)
    for name in declared_entry_points():
        assert hasattr(lib, name), name


def test_checked_build_exports_the_same_symbols():
    """The second target (the same sources with bounds checks compiled in) builds and loads too."""
    from paper_2603_03592_b200 import _build
    lib = ctypes.CDLL(_build.build_checked())
    for name in declared_entry_points():
        assert hasattr(lib, name), name


def test_binding_mirrors_the_header(built):
    from paper_2603_03592_b200 import binding
    assert sorted(binding.EXPORTS) == declared_entry_points()
    binding.lib()
    for name in binding.EXPORTS:
        if name in ("sentinel_default_config", "sentinel_distance", "sentinel_distance_noalloc",
                    "sentinel_sliced_wasserstein", "sentinel_bounds_violations"):
            assert hasattr(binding, name)
        elif name not in ("sentinel_verifier_create", "sentinel_last_error"):
            assert hasattr(binding.Verifier, name), name


def test_default_config_matches_the_paper_table(built):
    """Host-only call: the library's defaults against the golden copy of the paper's table."""
    from paper_2603_03592_b200 import binding
    cfg = binding.sentinel_default_config()
    want = {}
    with open(os.path.join(ROOT, "tests", "golden", "hyperparams_table.txt")) as fh:
        for line in fh:
            if line.startswith("#") or not line.strip():
                continue
            tok = line.split()
            want[tok[0]] = tuple(float(v) for v in tok[1:])
    for key, field in [("beta", "beta"), ("k0", "k0"), ("alpha", "alpha"), ("n_max", "n_max"),
                       ("gamma_g", "gamma_grow"), ("gamma_s", "gamma_shrink"),
                       ("lambda", "lambda_min"), ("eps", "iqr_eps")]:
        assert tuple(getattr(cfg, field)) == want[key]
    assert cfg.ban_violations == want["c"][0] and cfg.forgiveness_steps == want["t_forgiveness"][0]
    assert cfg.window_steps == want["l"][0] and cfg.severe_mult == want["severe_mult"][0]
    assert cfg.metric_mask == 15 and cfg.shrink_ratio == 0.5 and cfg.n_workers == 1   # every metric of M may flag


def test_host_side_argument_checks_need_no_gpu(built):
    from paper_2603_03592_b200 import binding
    L = binding.lib()
    assert L.sentinel_default_config(None) == binding.ERR_INVALID_ARG
    assert L.sentinel_verifier_create(None, None) == binding.ERR_INVALID_ARG
    assert L.sentinel_destroy(None) == binding.ERR_INVALID_ARG
    assert L.sentinel_state_bytes(None) == 0
    assert b"NULL" in L.sentinel_last_error(None)
    cfg = binding.sentinel_default_config(B=65, T=4, d=16)
    h = ctypes.c_void_p()
    assert L.sentinel_verifier_create(ctypes.byref(cfg), ctypes.byref(h)) == binding.ERR_UNSUPPORTED
    assert not h.value
    cfg = binding.sentinel_default_config(B=2, T=0, d=16)
    assert L.sentinel_verifier_create(ctypes.byref(cfg), ctypes.byref(h)) == binding.ERR_INVALID_ARG
    # calls that take a handle refuse NULL before anything else
    assert L.sentinel_num_metrics(None) == 0
    assert L.sentinel_set_directions(None, None, 8, None) == binding.ERR_INVALID_ARG
    assert L.sentinel_skip_tainted(None, 0, None) == binding.ERR_INVALID_ARG
    assert L.sentinel_verify(None, None, 0, 1, 1, 8, None, None, None) == binding.ERR_INVALID_ARG
    assert L.sentinel_verify_replicas(None, None, 0, 1, 1, 8, None, None, None) == binding.ERR_INVALID_ARG
    assert L.sentinel_verify_replicas_tainted(None, None, 0, 1, 1, 1, 8, None, None, None) == binding.ERR_INVALID_ARG
    assert L.sentinel_verify_strided(None, None, 0, 1, 1, 8, 9, None, None, None) == binding.ERR_INVALID_ARG
    assert L.sentinel_replace_if_flagged(None, None, 0, 1, 1, 8, 0, None, None) == binding.ERR_INVALID_ARG
    assert L.sentinel_import_state(None, None, 0, None) == binding.ERR_INVALID_ARG
    # stateless calls check their pointers and shapes on the host
    assert L.sentinel_distance(None, None, 1, 1, 8, 0, None, None, None) == binding.ERR_INVALID_ARG
    assert L.sentinel_sliced_wasserstein(None, None, None, 8, 1, 1, 8, 0, None, None) == binding.ERR_INVALID_ARG
    assert L.sentinel_distance_noalloc(None, None, 1, 1, 8, 0, None, None, None) == binding.ERR_INVALID_ARG
    # configuration ranges
    for bad in (dict(n_workers=17), dict(ema_bf16=2), dict(ref_over_batch=3), dict(window_steps=0),
                dict(ref_over_batch=1, ref_over_tokens=2)):
        cfg = binding.sentinel_default_config(B=2, T=4, d=16, **bad)
        assert L.sentinel_verifier_create(ctypes.byref(cfg), ctypes.byref(h)) == binding.ERR_INVALID_ARG, bad
    # combinations of variants that are not built
    for bad in (dict(ref_over_tokens=1, n_workers=2), dict(ref_over_batch=1, n_workers=2), dict(ema_bf16=1, ref_over_batch=1),
                dict(ref_over_batch=1, ref_over_tokens=1, ema_bf16=1)):
        cfg = binding.sentinel_default_config(B=2, T=4, d=16, **bad)
        assert L.sentinel_verifier_create(ctypes.byref(cfg), ctypes.byref(h)) == binding.ERR_UNSUPPORTED, bad
    with pytest.raises(TypeError):
        binding.sentinel_default_config(B=2, T=4, d=16, no_such_field=1)


def test_product_path_does_not_touch_the_oracle():
    """Nothing under the package imports, reads or links the oracle."""
    pkg = os.path.join(ROOT, "paper_2603_03592_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in text.lower(), os.path.join(dirpath, f)

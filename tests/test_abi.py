"""The C-ABI library loads and exports every symbol include/csat.h declares (no GPU needed)."""
import ctypes as C
import os
import re

import pytest

from paper_2507_02957_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "csat.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(csat_[a-z0-9_]+)\s*\(", text)))


def test_header_declares_the_named_entry_points():
    syms = declared_symbols()
    for must in ("csat_create", "csat_forward", "csat_destroy"):
        assert must in syms


def test_library_builds_loads_and_exports_every_declared_symbol():
    path = build.build_library()
    assert os.path.exists(path)
    lib = C.CDLL(path)
    for s in declared_symbols():
        assert hasattr(lib, s), f"libcsat.so lacks {s}"
    # the binding lists exactly the declared entry points
    assert sorted(binding.SIGNATURES) == declared_symbols()


def test_host_only_calls_need_no_gpu():
    lib = binding.load()
    assert lib.csat_version() >= 100
    assert lib.csat_destroy(None) == binding.CSAT_OK            # NULL is a no-op
    assert lib.csat_set_i64(None, binding.CSAT_T, 3) == 1       # CSAT_ERR_INVALID_ARG
    assert lib.csat_set_f64(None, binding.CSAT_LAMBDA, 0.1) == 1
    assert lib.csat_forward(None, None, None, None, None, None) == 1
    assert lib.csat_workspace_bytes(None) == 0
    # bad shapes are refused before any device work
    for args in ((0, 1, 64, 1), (64, 65, 64, 1), (64, 64, 0, 1), (64, 64, 64, 0), (64, 64, 60, 1), (64, 64, 512, 1)):
        assert not lib.csat_create(*args, 0)
        assert b"csat_create" in lib.csat_last_error(None)


def test_binding_refuses_to_run_without_cuda():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    with pytest.raises(RuntimeError):
        binding.Csat(64, 64, 64, 1)

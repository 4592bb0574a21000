"""The C-ABI library loads without a GPU and exports every entry point the header declares."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    import importlib.util
    spec = importlib.util.spec_from_file_location("windq_build", os.path.join(ROOT, "paper_2605_26660_b200", "_build.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    return ctypes.CDLL(mod.build())


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "windq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(windq_[a-z_]+)\s*\(", text)))


def test_header_declares_the_five_calls():
    names = declared_symbols()
    for want in ("windq_act_stats", "windq_unit_features", "windq_fit_eval", "windq_apply_plan", "windq_effective_bits",
                 "windq_create", "windq_destroy", "windq_last_error"):
        assert want in names


def test_library_exports_every_declared_symbol(lib):
    for name in declared_symbols():
        assert hasattr(lib, name), name


def test_null_context_is_rejected_without_a_gpu(lib):
    lib.windq_last_error.restype = ctypes.c_char_p
    lib.windq_last_error.argtypes = [ctypes.c_void_p]
    vp = ctypes.c_void_p
    st = lib.windq_act_stats(vp(), vp(), ctypes.c_int64(1), ctypes.c_int64(8), ctypes.c_int64(8), vp(), vp())
    assert st == 1  # WINDQ_ERR_NULL
    assert b"ctx is NULL" in lib.windq_last_error(vp())
    assert lib.windq_create(vp(), 0) == 1
    lib.windq_scratch_bytes_fit_eval.restype = ctypes.c_int64
    lib.windq_scratch_bytes_fit_eval.argtypes = [ctypes.c_int64, ctypes.c_int64, ctypes.c_int]
    assert lib.windq_scratch_bytes_fit_eval(4096, 4096, 128) == 16 + 32 * 512 * 8 * 8
    assert lib.windq_scratch_bytes_fit_eval(4096, 4096, 100) == 0

"""CPU-side checks of the product: the C-ABI library builds, loads and exports every symbol the
header declares; argument validation that needs no GPU; the binding fails loudly without it."""
import ctypes
import os
import re

import pytest

from paper_2605_08840_b200 import binding as rk
from paper_2605_08840_b200 import build as rk_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    rk_build.build()
    return rk.load_library()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "restkv.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(restkv_[a-z_]+)\s*\(", text)))


def test_header_and_binding_agree_on_the_exports():
    assert declared_symbols() == sorted(rk.EXPORTS)


def test_library_exports_every_declared_symbol(lib):
    for name in declared_symbols():
        assert hasattr(lib, name), name


def test_error_strings(lib):
    for code in range(6):
        assert rk.error_string(code) not in ("", "unknown status")
    assert rk.error_string(99) == "unknown status"


def test_workspace_bytes_validates_without_a_gpu(lib):
    ok = rk.make_shape(1, 32, 8, 128, 131072, 32)
    n = lib.restkv_workspace_bytes(ctypes.byref(ok), 2048)
    assert n > 0 and n % 256 == 0
    assert lib.restkv_workspace_bytes_adaptive(ctypes.byref(ok), 2048) > n
    for bad in (rk.make_shape(1, 7, 2, 128, 100, 32),          # heads not divisible
                rk.make_shape(1, 8, 2, 128, 100, 32, causal_tail=3),
                rk.make_shape(1, 8, 2, 128, 32, 32, causal_tail=32),   # no scored rows left
                rk.make_shape(0, 8, 2, 128, 100, 32),
                rk.make_shape(1, 8, 2, 20, 100, 32),
                rk.make_shape(1, 8, 2, 128, 100, 32, dtype=5)):
        assert lib.restkv_workspace_bytes(ctypes.byref(bad), 16) == 0
    assert lib.restkv_workspace_bytes(None, 16) == 0


def test_null_handle_is_rejected(lib):
    assert lib.restkv_destroy(None) == rk.ERR_INVALID_ARG
    assert lib.restkv_poll_status(None, None) == rk.ERR_INVALID_ARG
    assert lib.restkv_launch_count(None) == 0
    shape = rk.make_shape(1, 8, 2, 64, 100, 32)
    pool = rk.fixed_pool(7)
    assert lib.restkv_score(None, ctypes.byref(shape), None, None, None, 0.9, ctypes.byref(pool), None, None, None,
                            0, None) == rk.ERR_INVALID_ARG


def test_no_silent_fallback_when_the_library_is_missing(monkeypatch, tmp_path):
    monkeypatch.setattr(rk, "_lib", None)
    monkeypatch.setattr(rk, "LIB_PATH", str(tmp_path / "missing.so"))
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        rk.load_library()


def test_product_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_2605_08840_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in src.lower() or f == "inputs.py", f
    for f in os.listdir(os.path.join(ROOT, "oracle")):
        if f.endswith((".py", ".c")):
            src = open(os.path.join(ROOT, "oracle", f)).read()
            assert "paper_2605_08840_b200" not in src and "librestkv.so" not in src, f

"""The C-ABI library loads and exports every function include/celty.h declares (no GPU needed)."""
import ctypes
import os
import re

import numpy as np
import pytest

from conftest import ROOT
from paper_2608_01536_b200 import build, celty


@pytest.fixture(scope="module")
def lib():
    build.build()
    return celty.load()


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "celty.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(celty_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported_and_bound(lib):
    names = _declared_functions()
    assert "celty_encode" in names and "celty_spmspv" in names and len(names) >= 14
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(celty.SIGNATURES) == names


def test_header_is_plain_c(tmp_path):
    src = tmp_path / "t.c"
    src.write_text('#include "celty.h"\nint main(void){ celty_encode_opts o = {4, CELTY_LAYOUT_COLUMN, 0, 0}; return o.slabs_per_block; }\n')
    import subprocess
    subprocess.check_call(["gcc", "-std=c99", "-Wall", "-Werror", "-I", os.path.join(ROOT, "include"), "-c", str(src),
                           "-o", str(tmp_path / "t.o")])


def test_argument_errors(lib):
    W = np.ones((4, 4), np.float16)
    with pytest.raises(celty.CeltyError) as e:
        celty.Matrix(W, layout=celty.LAYOUT_COLUMN, tile_rows=16)
    assert e.value.status == -1
    with pytest.raises(celty.CeltyError):
        celty.Matrix(W, layout=7)
    with pytest.raises(celty.CeltyError):
        celty.Matrix(W, layout=celty.LAYOUT_LANE_TILE, tile_rows=241)
    with pytest.raises(celty.CeltyError):
        celty.Matrix(W, layout=celty.LAYOUT_LANE_TILE, slabs_per_block=16)
    with pytest.raises(celty.CeltyError):
        celty.Matrix(W, layout=celty.LAYOUT_COLUMN, slabs_per_block=1)
    h = ctypes.c_void_p()
    tall = np.zeros((49153, 1), np.float16)                      # one row more than the library takes
    assert lib.celty_encode(tall.ctypes.data_as(ctypes.c_void_p), 1, None, 49153, 1, None, ctypes.byref(h)) == -1
    assert lib.celty_encode(None, 4, None, 4, 4, None, ctypes.byref(h)) == -1
    assert lib.celty_encode(W.ctypes.data_as(ctypes.c_void_p), 4, None, 0, 4, None, ctypes.byref(h)) == -1
    assert lib.celty_encode(W.ctypes.data_as(ctypes.c_void_p), 2, None, 4, 4, None, ctypes.byref(h)) == -1
    m = celty.Matrix(W)
    # not bound to device memory yet
    assert lib.celty_spmspv(m._h, ctypes.c_void_p(16), 0.0, ctypes.c_void_p(16), None) == -4
    assert lib.celty_spmspv(m._h, ctypes.c_void_p(16), -1.0, ctypes.c_void_p(16), None) == -1
    assert lib.celty_spmspv(m._h, ctypes.c_void_p(16), float("nan"), ctypes.c_void_p(16), None) == -1
    assert lib.celty_spmspv(m._h, ctypes.c_void_p(8), 0.0, ctypes.c_void_p(16), None) == -1
    assert lib.celty_last_status(m._h, None) == -4
    assert lib.celty_compact(ctypes.c_void_p(16), 0, 0.0, ctypes.c_void_p(16), ctypes.c_void_p(16), ctypes.c_void_p(16), None) == -1
    assert lib.celty_strerror(-5) == b"a bounded wait inside a kernel ran out"
    lib.celty_destroy(None)


def test_missing_library_fails_loudly(monkeypatch):
    monkeypatch.setattr(celty, "_lib", None)
    monkeypatch.setattr(celty, "LIB_PATH", "/nonexistent/libcelty.so")
    with pytest.raises(RuntimeError, match="no CPU or PyTorch fallback"):
        celty.load()

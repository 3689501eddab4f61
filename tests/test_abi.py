"""The C-ABI library loads and exports every symbol include/cstr.h declares;
argument validation that happens before any CUDA call returns error codes."""
import ctypes
import os
import re

import numpy as np
import pytest

from helpers import ROOT

from paper_2407_08103_b200 import build, cstr


@pytest.fixture(scope="module")
def lib():
    build.build_library()
    return cstr.lib()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "cstr.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(cstr_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_functions()
    assert len(names) >= 15
    for name in names:
        assert hasattr(lib, name), name
    assert sorted(cstr.EXPORTS) == [n for n in names if n in cstr.EXPORTS]
    assert set(names) == set(cstr.EXPORTS)


def test_header_compiles_as_plain_c(tmp_path):
    src = tmp_path / "t.c"
    src.write_text('#include "cstr.h"\nint main(void) { return CSTR_OK; }\n')
    import subprocess
    subprocess.run(["gcc", "-std=c99", "-Wall", "-Werror", "-I", os.path.join(ROOT, "include"),
                    "-c", str(src), "-o", str(tmp_path / "t.o")], check=True)


def test_null_and_range_errors(lib):
    out = ctypes.c_void_p()
    assert lib.cstr_load_dfa(None, None, 1, 0, ctypes.byref(out)) == -1
    trans = np.full((2, 256), -1, dtype=np.int32)
    acc = np.zeros(2, dtype=np.uint8)
    tp, ap = trans.ctypes.data_as(ctypes.c_void_p), acc.ctypes.data_as(ctypes.c_void_p)
    assert lib.cstr_load_dfa(tp, ap, 0, 0, ctypes.byref(out)) == -2
    assert lib.cstr_load_dfa(tp, ap, 2, 2, ctypes.byref(out)) == -2
    trans[1, 7] = 2
    assert lib.cstr_load_dfa(tp, ap, 2, 0, ctypes.byref(out)) == -3
    assert b"state 1 byte 7" in lib.cstr_last_error()
    trans[1, 7] = -2
    assert lib.cstr_load_dfa(tp, ap, 2, 0, ctypes.byref(out)) == -3

    off = np.array([0, 2, 1], dtype=np.int64)
    by = np.zeros(4, dtype=np.uint8)
    op, bp = off.ctypes.data_as(ctypes.c_void_p), by.ctypes.data_as(ctypes.c_void_p)
    assert lib.cstr_load_vocab(bp, op, 2, ctypes.byref(out)) == -4
    off[:] = [1, 2, 3]
    assert lib.cstr_load_vocab(bp, op, 2, ctypes.byref(out)) == -4
    assert lib.cstr_load_vocab(bp, op, 0, ctypes.byref(out)) == -2
    assert lib.cstr_load_vocab(bp, None, 2, ctypes.byref(out)) == -1
    assert lib.cstr_table_create(None, 4, ctypes.byref(out)) == -1
    assert lib.cstr_table_build(None, None, -1, None) == -1
    assert lib.cstr_workspace_create(0, ctypes.byref(out)) == -2
    assert lib.cstr_step(None, 1, None, None, 0, 0, None, None, None, None, None, 1, None, None) == -1
    assert lib.cstr_step_status(None, None, None, None) == -1
    assert lib.cstr_step_host(None, 1, None, None, 0, 0, None, None, None, None, None, None, None,
                              None, None, 1, None, None) == -1
    assert lib.cstr_table_info(None, None, None, None, None) == -1
    # push-down entry points: validation that precedes every CUDA call
    z = np.zeros(2, dtype=np.int32)
    zp = z.ctypes.data_as(ctypes.c_void_p)
    assert lib.cstr_load_pda(None, None, None, None, None, None, None, 0, None, 1, 0, 0,
                             ctypes.byref(out)) == -1
    assert lib.cstr_load_pda(zp, zp, zp, zp, zp, zp, zp, 0, ap, 0, 0, 0, ctypes.byref(out)) == -2
    assert lib.cstr_load_pda(zp, zp, zp, zp, zp, zp, zp, 0, ap, 1, 255, 0, ctypes.byref(out)) == -10
    assert lib.cstr_load_pda(zp, zp, zp, zp, zp, zp, zp, 0, ap, 2, 1, 2, ctypes.byref(out)) == -2
    bad_byte = np.array([300], dtype=np.int32)
    assert lib.cstr_load_pda(zp, bad_byte.ctypes.data_as(ctypes.c_void_p), zp, zp, zp, zp, zp, 1,
                             ap, 2, 1, 0, ctypes.byref(out)) == -10
    assert b"no epsilon input" in lib.cstr_last_error()
    assert lib.cstr_build_pda_table(None, None, -1, None, ctypes.byref(out)) == -1
    assert lib.cstr_pda_table_info(None, None, None, None, None, None) == -1
    assert lib.cstr_pda_table_rebuild(None, -1, None) == -1
    assert lib.cstr_pda_table_download(None, 0, 0, None, None, None) == -1
    assert lib.cstr_pda_workspace_create(None, 4, ctypes.byref(out)) == -1
    assert lib.cstr_pda_step(None, None, 0, 0, None, None, None, None, 4, None, None, None, 1,
                             None, None) == -1
    assert lib.cstr_pda_step_status(None, None, None, None, None) == -1
    assert lib.cstr_pda_step_history(None, None, 0, 0, None, None, None, None, None, None, None, 4,
                                     None, None, None, 1, None, None) == -1
    assert lib.cstr_pda_accept_draft(None, None, None, None, None, 1, 1, 4, None, None, None, None,
                                     None, None) == -1
    # free functions accept NULL
    lib.cstr_free_pda(None)
    lib.cstr_free_pda_table(None)
    lib.cstr_free_pda_workspace(None)
    lib.cstr_free_dfa(None)
    lib.cstr_free_vocab(None)
    lib.cstr_free_table(None)
    lib.cstr_free_workspace(None)


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(cstr, "_lib", None)
    monkeypatch.setattr(cstr, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(RuntimeError, match="no fallback"):
        cstr.lib()

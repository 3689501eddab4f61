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


def test_checking_build_exports_the_release_symbols_and_the_debug_ones(lib):
    # libcstr_check.so: same entry points, plus those of include/cstr_debug.h, which the
    # release library must not have
    check = ctypes.CDLL(build.build_library(check=True))
    text = open(os.path.join(ROOT, "include", "cstr_debug.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    debug = sorted(set(re.findall(r"\b(cstr_[a-z_0-9]+)\s*\(", text)))
    assert debug == sorted(cstr.DEBUG_EXPORTS)
    for name in declared_functions() + debug:
        assert hasattr(check, name), name
    for name in debug:
        assert not hasattr(lib, name), name


def test_header_compiles_as_plain_c(tmp_path):
    src = tmp_path / "t.c"
    src.write_text('#include "cstr.h"\n#include "cstr_debug.h"\nint main(void) { return CSTR_OK; }\n')
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
    assert lib.cstr_table_build_dense(None, None, -1, None) == -1
    assert lib.cstr_workspace_create(0, ctypes.byref(out)) == -2
    assert lib.cstr_step(None, 1, None, None, 0, 0, None, None, None, None, None, 1, None, None) == -1
    assert lib.cstr_step_status(None, None, None, None) == -1
    assert lib.cstr_step_host(None, 1, None, None, 0, 0, None, None, None, None, None, None, None,
                              None, None, None, 1, None, None) == -1
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


@pytest.mark.parametrize("entry", ["cstr_step", "cstr_step_static", "cstr_step_history"])
def test_step_wrappers_reject_bad_row_tensors_before_any_launch(monkeypatch, entry):
    # a short or wrongly typed per-row tensor would be an out-of-bounds device write; the
    # binding must refuse it without reaching the library (lib() is made to fail here)
    import torch

    def no_library():
        raise AssertionError("the library was reached")
    monkeypatch.setattr(cstr, "lib", no_library)
    B, V = 4, 8
    logits = torch.zeros(B, V)
    good = dict(states=torch.zeros(B, dtype=torch.int32), tokens_out=torch.zeros(B, dtype=torch.int32),
                masked_out=torch.zeros(B, V), accept_out=torch.zeros(B, dtype=torch.uint8),
                row_table=torch.zeros(B, dtype=torch.int32), noise=torch.zeros(B, V))

    def call(**over):
        a = dict(good)
        a.update(over)
        table = cstr.Table(None)
        if entry == "cstr_step_static":
            cstr.cstr_step_static([table], logits, a["states"], a["tokens_out"], a["masked_out"],
                                  noise=a["noise"], row_table=a["row_table"], accept_out=a["accept_out"])
        elif entry == "cstr_step":
            cstr.cstr_step([table], logits, a["states"], a["tokens_out"], a["masked_out"], None,
                           noise=a["noise"], row_table=a["row_table"], accept_out=a["accept_out"])
        else:
            cstr.cstr_step_history([table], logits, a["states"], a["states"].clone(), a["tokens_out"],
                                   a["masked_out"], None, noise=a["noise"], row_table=a["row_table"],
                                   accept_out=a["accept_out"])

    with pytest.raises(ValueError, match="tokens_out"):
        call(tokens_out=torch.zeros(B - 1, dtype=torch.int32))
    with pytest.raises(ValueError, match="states"):
        call(states=torch.zeros(B, dtype=torch.int64))
    with pytest.raises(ValueError, match="accept_out"):
        call(accept_out=torch.zeros(B, dtype=torch.int32))
    with pytest.raises(ValueError, match="row_table"):
        call(row_table=torch.zeros(2 * B, dtype=torch.int32)[::2])
    with pytest.raises(TypeError, match="masked_out"):
        call(masked_out=torch.zeros(B, V, dtype=torch.bfloat16))
    with pytest.raises(TypeError, match="noise"):
        call(noise=torch.zeros(B, V, dtype=torch.float64))
    with pytest.raises(ValueError, match="masked_out"):
        call(masked_out=torch.zeros(B, V + 1))
    # well-formed arguments that live on the CPU are refused too (last check, still before the library)
    with pytest.raises(ValueError, match="CUDA tensor"):
        call()

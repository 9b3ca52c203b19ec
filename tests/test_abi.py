"""The C-ABI library builds, loads without a GPU and exports every symbol laser.h declares."""
import ctypes
import os
import re

from helpers import ensure_built

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    lib = ctypes.CDLL(ensure_built())
    header = open(os.path.join(ROOT, "include", "laser.h")).read()
    code = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = sorted(set(re.findall(r"\b(laser_[a-z_0-9]+)\s*\(", code)))
    assert len(declared) >= 20 and "laser_generate" in declared and "laser_verify_step" in declared
    for name in declared:
        assert hasattr(lib, name), name
    lib.laser_version.restype = ctypes.c_char_p
    assert b"sm_100a" in lib.laser_version()


def test_binding_structs_match_header_and_names():
    ensure_built()
    from paper_2408_05676_b200 import binding as L
    assert ctypes.sizeof(L.ModelCfg) == 13 * 4
    assert ctypes.sizeof(L.Params) == 13 * 4
    assert ctypes.sizeof(L.Weights) == 12 * 8
    assert ctypes.sizeof(L.Stats) == 6 * 8 + 5 * 4 + 4
    header = open(os.path.join(ROOT, "include", "laser.h")).read()
    for name in L.EXPORTS:
        assert name in header
        short = name[len("laser_"):]
        assert hasattr(L.lib, name)
        if short not in ("last_error", "pool_free", "pool_info", "model_free", "kv_free"):
            assert hasattr(L, short), short


def test_argument_errors_are_reported_without_a_gpu():
    ensure_built()
    from paper_2408_05676_b200 import binding as L
    p = L.make_params(K=8)
    st = L.lib.laser_draft(None, None, None, None, 4, ctypes.byref(p), None, None, None, None)
    assert st == -1 and b"null" in L.lib.laser_last_error()
    st = L.lib.laser_accept_commit(None, None, None, None, None, 1, 10, ctypes.byref(p), None, None, None, None)
    assert st == -1
    st = L.lib.laser_verify_accept(None, None, None, None, None, 1, ctypes.byref(p), 1, None, None, None, None, None)
    assert st == -1 and b"null" in L.lib.laser_last_error()

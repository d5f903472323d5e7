"""The C-ABI library loads without a GPU and exports every symbol include/pkv.h declares."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    src = open(os.path.join(ROOT, "include", "pkv.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(pkv_[a-z_0-9]+)\s*\(", src)))


def test_library_builds_loads_and_exports_every_declared_symbol():
    from paper_2609_39329_b200 import build
    path = build.build()
    lib = ctypes.CDLL(path)
    names = declared_functions()
    assert {"pkv_build_patch", "pkv_merge", "pkv_create", "pkv_destroy", "pkv_build_stack"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n


def test_binding_structs_match_header_sizes_and_strerror():
    from paper_2609_39329_b200 import binding as B
    L = B.lib()
    assert ctypes.sizeof(B.pkv_dims) == 44 and ctypes.sizeof(B.pkv_stats) == 7 * 8 + 8 + 48
    assert L.pkv_strerror(0) == b"ok"
    assert b"ascending" in L.pkv_strerror(-3)
    # workspace sizing needs no device; bad dims give 0
    d = B.make_dims(256, 4, 2, 64, 256, 1024, 64, 128, "fp32", 1e4, 1e-5)
    o = B.pkv_opts(B.ENGINE_SIMT, 0, None, 0, 0)
    assert L.pkv_workspace_bytes(ctypes.byref(d), ctypes.byref(o)) > 0
    d.hd = 96
    assert L.pkv_workspace_bytes(ctypes.byref(d), ctypes.byref(o)) == 0
    assert L.pkv_merge(None, 0, None, 0, None) == -1

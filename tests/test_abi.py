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
    # RTLD_NOW: every symbol the library itself refers to must resolve at load time (lazy binding would hide an
    # internal function that lost its definition until the first call on a GPU machine)
    lib = ctypes.CDLL(path, mode=os.RTLD_NOW)
    names = declared_functions()
    assert {"pkv_build_patch", "pkv_merge", "pkv_create", "pkv_destroy", "pkv_build_stack"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n


def test_binding_structs_match_header_sizes_and_strerror():
    from paper_2609_39329_b200 import binding as B
    L = B.lib()
    assert ctypes.sizeof(B.pkv_dims) == 44 and ctypes.sizeof(B.pkv_stats) == 7 * 8 + 8 + 48 + 2 * 8 + 2 * 4
    assert L.pkv_strerror(0) == b"ok"
    assert b"ascending" in L.pkv_strerror(-3)
    # workspace sizing needs no device; bad dims give 0
    d = B.make_dims(256, 4, 2, 64, 256, 1024, 64, 128, "fp32", 1e4, 1e-5)
    o = B.pkv_opts(B.ENGINE_SIMT, 0, None, 0, 0)
    assert L.pkv_workspace_bytes(ctypes.byref(d), ctypes.byref(o)) > 0
    d.hd = 96
    assert L.pkv_workspace_bytes(ctypes.byref(d), ctypes.byref(o)) == 0
    assert L.pkv_merge(None, 0, None, 0, None) == -1


def test_workspace_of_every_benchmark_config_fits_one_gpu_beside_its_inputs():
    """Host arithmetic only: the context's workspace plus the tensors one block keeps resident (weights,
    full cache, kept indices, states, patch) stays far below 180 GB for all five configs, for both engines
    and both solvers, and grows with the reference-token capacity."""
    from paper_2609_39329_b200 import binding as B
    from paper_2609_39329_b200 import inputs as gen
    L = B.lib()
    L.pkv_workspace_bytes.restype = ctypes.c_size_t
    for cid in range(1, 6):
        cfg = gen.benchmark_config(cid)
        eb = 4 if cfg.dtype == "fp32" else 2
        resident = eb * (cfg.d * (2 * cfg.Dq + 2 * cfg.Dkv) + 3 * cfg.d * cfg.F) + eb * 2 * cfg.Hkv * cfg.L * cfg.hd \
            + 4 * cfg.Hkv * cfg.budget + 4 * (4 * cfg.N * cfg.d + cfg.d * cfg.F)
        sizes = {}
        for engine in (B.ENGINE_AUTO, B.ENGINE_SIMT):
            for solver in (B.SOLVER_PRIMAL, B.SOLVER_DUAL):
                if solver == B.SOLVER_DUAL and (engine == B.ENGINE_SIMT or cfg.dtype == "fp32"):
                    continue
                d = B.dims_from_config(cfg)
                o = B.pkv_opts(engine, 0, None, 0, solver)
                ws = L.pkv_workspace_bytes(ctypes.byref(d), ctypes.byref(o))
                assert ws > 0, (cid, engine, solver)
                assert ws % 256 == 0
                assert ws + resident < 40e9, (cid, engine, solver, ws)
                sizes[(engine, solver)] = ws
                d2 = B.dims_from_config(cfg, N_max=2 * cfg.N)
                assert L.pkv_workspace_bytes(ctypes.byref(d2), ctypes.byref(o)) > ws
        if cfg.dtype == "bf16":
            assert sizes[(B.ENGINE_AUTO, B.SOLVER_PRIMAL)] > sizes[(B.ENGINE_SIMT, B.SOLVER_PRIMAL)]

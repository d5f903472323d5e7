"""ctypes marshalling over the C ABI of libpkv.so (see include/pkv.h).

Argument marshalling only: every step of the path runs in the library's CUDA kernels.  torch
is used for device memory and streams.  If the library is missing the import of a symbol
raises — there is no CPU or eager fallback.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, List, Optional, Sequence

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libpkv.so")

PKV_BF16, PKV_FP32 = 0, 1
LAMBDA_PAPER, LAMBDA_ABSOLUTE, LAMBDA_TRACE_MEAN = 0, 1, 2
ENGINE_AUTO, ENGINE_SIMT = 0, 1
SOLVER_PRIMAL, SOLVER_DUAL = 0, 1

ERRORS = {0: "PKV_OK", -1: "PKV_ERR_INVALID_ARG", -2: "PKV_ERR_UNSUPPORTED", -3: "PKV_ERR_BAD_INDEX",
          -4: "PKV_ERR_NOT_PD", -5: "PKV_ERR_DEGENERATE", -6: "PKV_ERR_NONFINITE", -7: "PKV_ERR_TIMEOUT",
          -8: "PKV_ERR_CUDA", -9: "PKV_ERR_NOMEM"}


class PkvError(RuntimeError):
    def __init__(self, code: int, msg: str, info=None):
        super().__init__("%s (%d): %s" % (ERRORS.get(code, "?"), code, msg))
        self.code = code
        self.info = info


class pkv_dims(C.Structure):
    _fields_ = [("d", C.c_int32), ("Hq", C.c_int32), ("Hkv", C.c_int32), ("hd", C.c_int32), ("F", C.c_int32),
                ("L", C.c_int32), ("N_max", C.c_int32), ("b_max", C.c_int32), ("dtype", C.c_int32),
                ("rope_theta", C.c_float), ("eps", C.c_float)]


class pkv_opts(C.Structure):
    _fields_ = [("engine", C.c_int32), ("kv_split", C.c_int32), ("workspace", C.c_void_p),
                ("workspace_bytes", C.c_size_t), ("solver", C.c_int32), ("reserve_sms", C.c_int32)]


class pkv_block_weights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in
                ("g_attn", "Wq", "Wk", "Wv", "Wo", "g_mlp", "Wgate", "Wup", "Wdown")]


class pkv_kv(C.Structure):
    _fields_ = [("K", C.c_void_p), ("V", C.c_void_p)]


class pkv_kv_compressed(C.Structure):
    _fields_ = [("head_off", C.POINTER(C.c_int32)), ("idx", C.c_void_p), ("Kc", C.c_void_p),
                ("Vc", C.c_void_p), ("bias", C.c_void_p), ("k_scale", C.c_void_p), ("v_scale", C.c_void_p),
                ("qbits", C.c_int32), ("qgroup", C.c_int32)]


class pkv_ref(C.Structure):
    _fields_ = [("xF", C.c_void_p), ("xC", C.c_void_p), ("N", C.c_int32), ("n_chunks", C.c_int32),
                ("chunk_off", C.POINTER(C.c_int32)), ("pos0", C.c_int32)]


class pkv_ref_next(C.Structure):
    _fields_ = [("xF_next", C.c_void_p), ("xC_next", C.c_void_p)]


class pkv_stats(C.Structure):
    _fields_ = [("lambda_eff", C.c_double), ("trace", C.c_double), ("fro2", C.c_double),
                ("target_fro2", C.c_double), ("resid_fro2", C.c_double), ("dW_fro2", C.c_double),
                ("min_pivot", C.c_double), ("err_info", C.c_int32 * 2), ("stage_ms", C.c_float * 12),
                ("cond_lower_bound", C.c_double), ("cond_upper_bound", C.c_double), ("cond_warning", C.c_int32),
                ("reserved", C.c_int32)]

    def as_dict(self) -> Dict[str, object]:
        return {"lambda_eff": self.lambda_eff, "trace": self.trace, "fro2": self.fro2,
                "target_fro2": self.target_fro2, "resid_fro2": self.resid_fro2, "dW_fro2": self.dW_fro2,
                "min_pivot": self.min_pivot, "err_info": (self.err_info[0], self.err_info[1]),
                "stage_ms": [float(x) for x in self.stage_ms], "cond_lower_bound": self.cond_lower_bound,
                "cond_upper_bound": self.cond_upper_bound, "cond_warning": int(self.cond_warning)}


_lib = None


def lib() -> C.CDLL:
    """Loads libpkv.so (built in-tree by paper_2609_39329_b200.build); raises if it is missing."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise FileNotFoundError("libpkv.so not built: run `python -m paper_2609_39329_b200.build`")
    L = C.CDLL(LIB_PATH)
    P = C.POINTER
    L.pkv_workspace_bytes.restype = C.c_size_t
    L.pkv_workspace_bytes.argtypes = [P(pkv_dims), P(pkv_opts)]
    L.pkv_create.restype = C.c_int
    L.pkv_create.argtypes = [P(C.c_void_p), P(pkv_dims), P(pkv_opts), C.c_void_p]
    L.pkv_destroy.restype = None
    L.pkv_destroy.argtypes = [C.c_void_p]
    L.pkv_build_patch.restype = C.c_int
    L.pkv_build_patch.argtypes = [C.c_void_p, P(pkv_block_weights), P(pkv_kv), P(pkv_kv_compressed), P(pkv_ref),
                                  C.c_float, C.c_int, C.c_void_p, P(pkv_ref_next), P(pkv_stats)]
    L.pkv_stream_begin.restype = C.c_int
    L.pkv_stream_begin.argtypes = [C.c_void_p, C.c_float, C.c_int]
    L.pkv_stream_add.restype = C.c_int
    L.pkv_stream_add.argtypes = [C.c_void_p, P(pkv_block_weights), P(pkv_kv), P(pkv_kv_compressed), P(pkv_ref), C.c_void_p]
    L.pkv_stream_finish.restype = C.c_int
    L.pkv_stream_finish.argtypes = [C.c_void_p, C.c_void_p, P(pkv_stats)]
    L.pkv_stream_propagate.restype = C.c_int
    L.pkv_stream_propagate.argtypes = [C.c_void_p, P(pkv_block_weights), P(pkv_kv), P(pkv_kv_compressed), P(pkv_ref),
                                       C.c_void_p, C.c_void_p]
    L.pkv_merge.restype = C.c_int
    L.pkv_merge.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_int64, C.c_void_p]
    L.pkv_build_stack.restype = C.c_int
    L.pkv_build_stack.argtypes = [C.c_void_p, C.c_int, C.c_int, P(pkv_block_weights), P(pkv_kv),
                                  P(pkv_kv_compressed), P(pkv_ref), C.c_float, C.c_int, P(C.c_void_p),
                                  P(pkv_ref_next), P(pkv_stats)]
    L.pkv_teacher_cache_bytes.restype = C.c_size_t
    L.pkv_teacher_cache_bytes.argtypes = [P(pkv_dims), C.c_int, C.c_int]
    L.pkv_build_stack_sweep.restype = C.c_int
    L.pkv_build_stack_sweep.argtypes = [C.c_void_p, C.c_int, P(pkv_block_weights), P(pkv_kv), P(pkv_kv_compressed),
                                        P(pkv_ref), C.c_int, P(C.c_float), C.c_int, P(C.c_void_p), C.c_void_p,
                                        C.c_size_t, P(pkv_stats)]
    L.pkv_gather_kept.restype = C.c_int
    L.pkv_gather_kept.argtypes = [C.c_void_p, P(pkv_kv), P(C.c_int32), C.c_void_p, C.c_void_p, C.c_void_p,
                                  P(C.c_int32), P(C.c_int32)]
    L.pkv_dequant_cache.restype = C.c_int
    L.pkv_dequant_cache.argtypes = [C.c_void_p, P(pkv_kv_compressed), C.c_void_p, C.c_void_p]
    L.pkv_attention.restype = C.c_int
    L.pkv_attention.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, P(pkv_kv), P(pkv_kv_compressed),
                                C.c_int32, C.c_int32, P(C.c_int32), C.c_void_p, C.c_void_p, C.c_void_p]
    L.pkv_gram.restype = C.c_int
    L.pkv_gram.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_int]
    L.pkv_gram_noalloc.restype = C.c_int
    L.pkv_gram_noalloc.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p,
                                   C.c_int, C.c_void_p]
    L.pkv_low_rank_scratch_bytes.restype = C.c_size_t
    L.pkv_low_rank_scratch_bytes.argtypes = [P(pkv_dims), C.c_int]
    L.pkv_low_rank.restype = C.c_int
    L.pkv_low_rank.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_void_p, C.c_size_t,
                               C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
    L.pkv_ridge_solve.restype = C.c_int
    L.pkv_ridge_solve.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_float, C.c_int, C.c_void_p, P(pkv_stats)]
    L.pkv_ridge_solve_refined.restype = C.c_int
    L.pkv_ridge_solve_refined.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_float, C.c_int, C.c_int32, C.c_void_p,
                                          P(pkv_stats)]
    L.pkv_fp32_product.restype = C.c_int
    L.pkv_fp32_product.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_float,
                                   C.c_void_p, C.c_int, C.c_int, C.c_int]
    L.pkv_selftest_bounded_wait.restype = C.c_int
    L.pkv_selftest_bounded_wait.argtypes = [C.c_void_p, P(C.c_int32)]
    L.pkv_set_timing.restype = C.c_int
    L.pkv_set_timing.argtypes = [C.c_void_p, C.c_int]
    L.pkv_launch_count.restype = C.c_int64
    L.pkv_launch_count.argtypes = [C.c_void_p]
    L.pkv_set_refinement.restype = C.c_int
    L.pkv_set_refinement.argtypes = [C.c_void_p, C.c_int]
    L.pkv_set_stack_schedule.restype = C.c_int
    L.pkv_set_stack_schedule.argtypes = [C.c_void_p, C.c_int]
    L.pkv_measure_fma_peak.restype = C.c_int
    L.pkv_measure_fma_peak.argtypes = [C.c_void_p, P(C.c_double)]
    L.pkv_teacher_sm_count.restype = C.c_int
    L.pkv_teacher_sm_count.argtypes = [C.c_void_p]
    for f in ("pkv_strerror", "pkv_stage_name"):
        getattr(L, f).restype = C.c_char_p
        getattr(L, f).argtypes = [C.c_int]
    L.pkv_last_cuda_error.restype = C.c_char_p
    L.pkv_last_cuda_error.argtypes = [C.c_void_p]
    _lib = L
    return L


def _i32(a: Sequence[int]):
    arr = (C.c_int32 * len(a))(*[int(v) for v in a])
    return arr


def _ptr(t) -> int:
    return 0 if t is None else int(t.data_ptr())


def make_dims(d, Hq, Hkv, hd, F, L, N_max, b_max, dtype, rope_theta, eps) -> pkv_dims:
    return pkv_dims(d, Hq, Hkv, hd, F, L, N_max, b_max, PKV_BF16 if dtype in ("bf16", PKV_BF16) else PKV_FP32,
                    float(rope_theta), float(eps))


def dims_from_config(cfg, N_max: Optional[int] = None, b_max: Optional[int] = None) -> pkv_dims:
    return make_dims(cfg.d, cfg.Hq, cfg.Hkv, cfg.hd, cfg.F, cfg.L, N_max or cfg.N,
                     cfg.budget if b_max is None else b_max, cfg.dtype, cfg.rope_theta, cfg.eps)


class PkvContext:
    """Owns one pkv_ctx.  Tensors passed in must live on the context's CUDA device."""

    def __init__(self, dims: pkv_dims, engine: int = ENGINE_AUTO, kv_split: int = 0, stream=None,
                 solver: int = SOLVER_PRIMAL, workspace=None, reserve_sms: int = 0):
        import torch
        self.torch = torch
        self.dims = dims
        self.L = lib()
        self.stream = stream
        self.workspace = workspace      # optional caller-owned uint8 CUDA tensor (kept alive with the context)
        self.opts = pkv_opts(engine, kv_split, _ptr(workspace) if workspace is not None else None,
                             int(workspace.numel()) if workspace is not None else 0, solver, reserve_sms)
        h = C.c_void_p()
        sp = C.c_void_p(stream.cuda_stream) if stream is not None else C.c_void_p(torch.cuda.current_stream().cuda_stream)
        rc = self.L.pkv_create(C.byref(h), C.byref(dims), C.byref(self.opts), sp)
        if rc != 0:
            raise PkvError(rc, self.L.pkv_strerror(rc).decode())
        self.h = h
        self.wdtype = torch.bfloat16 if dims.dtype == PKV_BF16 else torch.float32

    def close(self):
        if getattr(self, "h", None):
            self.L.pkv_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- helpers ----
    def _raise(self, rc: int, info=None):
        msg = self.L.pkv_strerror(rc).decode()
        if rc == -8:
            msg += " [" + self.L.pkv_last_cuda_error(self.h).decode() + "]"
        raise PkvError(rc, msg, info)

    def workspace_bytes(self) -> int:
        return int(self.L.pkv_workspace_bytes(C.byref(self.dims), C.byref(self.opts)))

    def launch_count(self) -> int:
        return int(self.L.pkv_launch_count(self.h))

    def set_stack_schedule(self, sequential: bool):
        self.L.pkv_set_stack_schedule(self.h, 1 if sequential else 0)

    def measure_fma_peak(self) -> float:
        """pkv_measure_fma_peak: fp32 FMA TFLOP/s of the device (CUDA-event timed FMA kernel)."""
        v = C.c_double(0.0)
        rc = self.L.pkv_measure_fma_peak(self.h, C.byref(v))
        if rc != 0:
            self._raise(rc)
        return float(v.value)

    def teacher_sm_count(self) -> int:
        return int(self.L.pkv_teacher_sm_count(self.h))

    def selftest_bounded_wait(self):
        """pkv_selftest_bounded_wait: returns (code, site)."""
        site = C.c_int32(0)
        rc = self.L.pkv_selftest_bounded_wait(self.h, C.byref(site))
        return int(rc), int(site.value)

    def set_refinement(self, steps):
        """Corrections of iterative refinement after every ridge solve of this context (0 = off)."""
        rc = self.L.pkv_set_refinement(self.h, int(steps))
        if rc != 0:
            self._raise(rc, {})

    def set_timing(self, on):
        """False/0: off; True/1: every stage (stacked schedule); 2: the solve's interval only, default schedule."""
        self.L.pkv_set_timing(self.h, 2 if on == 2 else (1 if on else 0))

    def stage_names(self) -> List[str]:
        return [self.L.pkv_stage_name(i).decode() for i in range(9)]

    @staticmethod
    def weights_struct(w: Dict[str, "object"]) -> pkv_block_weights:
        return pkv_block_weights(*[_ptr(w[n]) for n in
                                   ("g_attn", "Wq", "Wk", "Wv", "Wo", "g_mlp", "Wgate", "Wup", "Wdown")])

    @staticmethod
    def compressed_struct(head_off, idx=None, Kc=None, Vc=None, bias=None, quant=None):
        """quant: None or dict(k_scale, v_scale, bits, group) when Kc/Vc hold integer codes."""
        ho = _i32(head_off)
        q = quant or {}
        s = pkv_kv_compressed(C.cast(ho, C.POINTER(C.c_int32)), _ptr(idx), _ptr(Kc), _ptr(Vc), _ptr(bias),
                              _ptr(q.get("k_scale")), _ptr(q.get("v_scale")), int(q.get("bits", 0)), int(q.get("group", 0)))
        s._keep = ho
        return s

    # ---- the path ----
    def build_patch(self, w, K, V, head_off, idx, xF, xC, chunk_off, pos0, lam, mode=LAMBDA_PAPER,
                    want_next=True, Kc=None, Vc=None, bias=None, dW=None, quant=None):
        """pkv_build_patch.  Returns dict(dW, xF_next, xC_next, stats)."""
        torch = self.torch
        N = int(xF.shape[0])
        d, F = self.dims.d, self.dims.F
        if dW is None:
            dW = torch.empty((d, F), dtype=torch.float32, device=xF.device)
        ws = self.weights_struct(w)
        kv = pkv_kv(_ptr(K), _ptr(V))
        cb = self.compressed_struct(head_off, idx, Kc, Vc, bias, quant)
        co = _i32(chunk_off)
        ref = pkv_ref(_ptr(xF), _ptr(xC), N, len(chunk_off) - 1, C.cast(co, C.POINTER(C.c_int32)), int(pos0))
        st = pkv_stats()
        nx, xFn, xCn = None, None, None
        if want_next:
            xFn = torch.empty((N, d), dtype=torch.float32, device=xF.device)
            xCn = torch.empty((N, d), dtype=torch.float32, device=xF.device)
            nx = pkv_ref_next(_ptr(xFn), _ptr(xCn))
        rc = self.L.pkv_build_patch(self.h, C.byref(ws), C.byref(kv), C.byref(cb), C.byref(ref), float(lam),
                                    int(mode), _ptr(dW), C.byref(nx) if nx is not None else None, C.byref(st))
        if rc != 0:
            self._raise(rc, st.as_dict())
        return {"dW": dW, "xF_next": xFn, "xC_next": xCn, "stats": st.as_dict()}

    # ---- streamed reference sets ----
    def stream_begin(self, lam, mode=LAMBDA_PAPER):
        rc = self.L.pkv_stream_begin(self.h, float(lam), int(mode))
        if rc != 0:
            self._raise(rc)

    def _ref(self, xF, xC, chunk_off, pos0):
        co = _i32(chunk_off)
        ref = pkv_ref(_ptr(xF), _ptr(xC), int(xC.shape[0]), len(chunk_off) - 1, C.cast(co, C.POINTER(C.c_int32)), int(pos0))
        ref._keep = co
        return ref

    def stream_add(self, w, K, V, head_off, idx, xF, xC, chunk_off, pos0, want_next=False, Kc=None, Vc=None, bias=None,
                   quant=None):
        """pkv_stream_add; returns the teacher's next states of these tokens if asked."""
        ws = self.weights_struct(w)
        kv = pkv_kv(_ptr(K), _ptr(V))
        cb = self.compressed_struct(head_off, idx, Kc, Vc, bias, quant)
        ref = self._ref(xF, xC, chunk_off, pos0)
        xFn = self.torch.empty_like(xF) if want_next else None
        rc = self.L.pkv_stream_add(self.h, C.byref(ws), C.byref(kv), C.byref(cb), C.byref(ref), _ptr(xFn))
        if rc != 0:
            self._raise(rc)
        return xFn

    def stream_finish(self):
        dW = self.torch.empty((self.dims.d, self.dims.F), dtype=self.torch.float32, device="cuda")
        st = pkv_stats()
        rc = self.L.pkv_stream_finish(self.h, _ptr(dW), C.byref(st))
        if rc != 0:
            self._raise(rc, st.as_dict())
        return dW, st.as_dict()

    def stream_propagate(self, w, K, V, head_off, idx, xC, chunk_off, pos0, dW, Kc=None, Vc=None, bias=None, quant=None):
        ws = self.weights_struct(w)
        kv = pkv_kv(_ptr(K), _ptr(V))
        cb = self.compressed_struct(head_off, idx, Kc, Vc, bias, quant)
        ref = self._ref(xC, xC, chunk_off, pos0)
        out = self.torch.empty_like(xC)
        rc = self.L.pkv_stream_propagate(self.h, C.byref(ws), C.byref(kv), C.byref(cb), C.byref(ref), _ptr(dW), _ptr(out))
        if rc != 0:
            self._raise(rc)
        return out

    def merge(self, W, dW):
        """pkv_merge: W <- W + dW in place (W bf16 or fp32, dW fp32)."""
        torch = self.torch
        dt = PKV_BF16 if W.dtype == torch.bfloat16 else PKV_FP32
        sp = C.c_void_p(self.stream.cuda_stream) if self.stream is not None else C.c_void_p(
            torch.cuda.current_stream().cuda_stream)
        rc = self.L.pkv_merge(_ptr(W), dt, _ptr(dW), int(W.numel()), sp)
        if rc != 0:
            self._raise(rc)
        return W

    def build_stack(self, layers, xF0, xC0, chunk_off, pos0, lam, mode=LAMBDA_PAPER, first_layer=0,
                    want_final=True):
        """pkv_build_stack over a list of dict(w, K, V, head_off, idx).  Returns dWs, final states, stats."""
        torch = self.torch
        n = len(layers)
        N = int(xF0.shape[0])
        d, F = self.dims.d, self.dims.F
        W = (pkv_block_weights * n)(*[self.weights_struct(l["w"]) for l in layers])
        KV = (pkv_kv * n)(*[pkv_kv(_ptr(l["K"]), _ptr(l["V"])) for l in layers])
        cbs = [self.compressed_struct(l["head_off"], l.get("idx"), l.get("Kc"), l.get("Vc"), l.get("bias"), l.get("quant"))
               for l in layers]
        CB = (pkv_kv_compressed * n)(*cbs)
        co = _i32(chunk_off)
        ref = pkv_ref(_ptr(xF0), _ptr(xC0), N, len(chunk_off) - 1, C.cast(co, C.POINTER(C.c_int32)), int(pos0))
        dWs = [torch.empty((d, F), dtype=torch.float32, device=xF0.device) for _ in range(n)]
        DW = (C.c_void_p * n)(*[_ptr(t) for t in dWs])
        ST = (pkv_stats * n)()
        xFn = xCn = fin = None
        if want_final:
            xFn = torch.empty((N, d), dtype=torch.float32, device=xF0.device)
            xCn = torch.empty((N, d), dtype=torch.float32, device=xF0.device)
            fin = pkv_ref_next(_ptr(xFn), _ptr(xCn))
        rc = self.L.pkv_build_stack(self.h, n, first_layer, W, KV, CB, C.byref(ref), float(lam), int(mode), DW,
                                    C.byref(fin) if fin is not None else None, ST)
        if rc != 0:
            self._raise(rc)
        return {"dW": dWs, "xF_final": xFn, "xC_final": xCn, "stats": [s.as_dict() for s in ST]}

    def build_stack_sweep(self, layers, xF0, xC0, chunk_off, pos0, lams, mode=LAMBDA_PAPER, cache=None):
        """pkv_build_stack_sweep: every block's patch for each ridge coefficient in `lams`, the teacher run once.
        Returns dict(dW = [per lambda][per layer], stats likewise).  `cache`: optional uint8 CUDA tensor of at
        least pkv_teacher_cache_bytes (allocated here otherwise)."""
        torch = self.torch
        n, nl = len(layers), len(lams)
        N = int(xF0.shape[0])
        d, F = self.dims.d, self.dims.F
        need = int(self.L.pkv_teacher_cache_bytes(C.byref(self.dims), n, N))
        if cache is None:
            cache = torch.empty(need, dtype=torch.uint8, device=xF0.device)
        W = (pkv_block_weights * n)(*[self.weights_struct(l["w"]) for l in layers])
        KV = (pkv_kv * n)(*[pkv_kv(_ptr(l["K"]), _ptr(l["V"])) for l in layers])
        cbs = [self.compressed_struct(l["head_off"], l.get("idx"), l.get("Kc"), l.get("Vc"), l.get("bias"), l.get("quant"))
               for l in layers]
        CB = (pkv_kv_compressed * n)(*cbs)
        co = _i32(chunk_off)
        ref = pkv_ref(_ptr(xF0), _ptr(xC0), N, len(chunk_off) - 1, C.cast(co, C.POINTER(C.c_int32)), int(pos0))
        dWs = [[torch.empty((d, F), dtype=torch.float32, device=xF0.device) for _ in range(n)] for _ in range(nl)]
        DW = (C.c_void_p * (n * nl))(*[_ptr(t) for row in dWs for t in row])
        ST = (pkv_stats * (n * nl))()
        LAM = (C.c_float * nl)(*[float(v) for v in lams])
        rc = self.L.pkv_build_stack_sweep(self.h, n, W, KV, CB, C.byref(ref), nl, LAM, int(mode), DW, _ptr(cache),
                                          int(cache.numel()), ST)
        if rc != 0:
            self._raise(rc)
        return {"dW": dWs, "stats": [[ST[j * n + l].as_dict() for l in range(n)] for j in range(nl)], "cache": cache}

    # ---- single stages ----
    def gather_kept(self, K, V, head_off, idx):
        torch = self.torch
        total = int(head_off[-1])
        hd = self.dims.hd
        Kc = torch.zeros((max(total, 1), hd), dtype=K.dtype, device=K.device)
        Vc = torch.zeros((max(total, 1), hd), dtype=K.dtype, device=K.device)
        kv = pkv_kv(_ptr(K), _ptr(V))
        ho = _i32(head_off)
        bh, bp = C.c_int32(0), C.c_int32(0)
        rc = self.L.pkv_gather_kept(self.h, C.byref(kv), ho, _ptr(idx), _ptr(Kc), _ptr(Vc), C.byref(bh), C.byref(bp))
        if rc != 0:
            self._raise(rc, (bh.value, bp.value))
        return Kc[:total], Vc[:total]

    def dequant_cache(self, head_off, Kq, Vq, quant):
        """pkv_dequant_cache: decoded K', V' [rows][hd] of the context's cache dtype."""
        torch = self.torch
        total = int(head_off[-1])
        Kc = torch.zeros((max(total, 1), self.dims.hd), dtype=self.wdtype, device=Kq.device)
        Vc = torch.zeros_like(Kc)
        cb = self.compressed_struct(head_off, None, Kq, Vq, None, quant)
        rc = self.L.pkv_dequant_cache(self.h, C.byref(cb), _ptr(Kc), _ptr(Vc))
        if rc != 0:
            self._raise(rc)
        return Kc[:total], Vc[:total]

    def attention(self, q, k_new, v_new, K, V, head_off, idx, chunk_off, Kc=None, Vc=None, bias=None, quant=None):
        torch = self.torch
        N = int(q.shape[1])
        Dq = self.dims.Hq * self.dims.hd
        outs = [torch.empty((N, Dq), dtype=torch.float32, device=q.device) for _ in range(3)]
        kv = pkv_kv(_ptr(K), _ptr(V))
        cb = self.compressed_struct(head_off, idx, Kc, Vc, bias, quant)
        co = _i32(chunk_off)
        rc = self.L.pkv_attention(self.h, _ptr(q), _ptr(k_new), _ptr(v_new), C.byref(kv), C.byref(cb), N,
                                  len(chunk_off) - 1, co, _ptr(outs[0]), _ptr(outs[1]), _ptr(outs[2]))
        if rc != 0:
            self._raise(rc)
        return outs

    def gram(self, X, R, S_H=None, S_T=None, accumulate=False):
        torch = self.torch
        F, d = self.dims.F, self.dims.d
        if S_H is None:
            S_H = torch.zeros((F, F), dtype=torch.float32, device=X.device)
            S_T = torch.zeros((d, F), dtype=torch.float32, device=X.device)
        rc = self.L.pkv_gram(self.h, _ptr(X), _ptr(R), int(X.shape[0]), _ptr(S_H), _ptr(S_T), 1 if accumulate else 0)
        if rc != 0:
            self._raise(rc)
        return S_H, S_T

    def fp32_product(self, A, Bm, alpha=1.0, C_out=None, accumulate=False, passes=6, accumulators=4):
        """pkv_fp32_product: C (+)= alpha * A Bm^T through the split-bf16 tensor-core product of the solve."""
        torch = self.torch
        M, K = int(A.shape[0]), int(A.shape[1])
        N = int(Bm.shape[0])
        if C_out is None:
            C_out = torch.zeros((M, N), dtype=torch.float32, device=A.device)
        rc = self.L.pkv_fp32_product(self.h, _ptr(A), _ptr(Bm), M, N, K, float(alpha), _ptr(C_out),
                                     1 if accumulate else 0, int(passes), int(accumulators))
        if rc != 0:
            self._raise(rc)
        return C_out

    def low_rank(self, dW, S_H, r, iterations=0, want_expanded=True):
        """pkv_low_rank: returns dict(U [d][r], Br [r][F], dW_r [d][F] or None, ritz [r + 8])."""
        torch = self.torch
        d, F = self.dims.d, self.dims.F
        need = int(self.L.pkv_low_rank_scratch_bytes(C.byref(self.dims), int(r)))
        scratch = torch.empty(need, dtype=torch.uint8, device=dW.device)
        U = torch.empty((d, r), dtype=torch.float32, device=dW.device)
        Br = torch.empty((r, F), dtype=torch.float32, device=dW.device)
        dWr = torch.empty((d, F), dtype=torch.float32, device=dW.device) if want_expanded else None
        ritz = torch.empty(r + 8, dtype=torch.float32, device=dW.device)
        rc = self.L.pkv_low_rank(self.h, _ptr(dW), _ptr(S_H), int(r), int(iterations), _ptr(scratch), need, _ptr(U),
                                 _ptr(Br), _ptr(dWr), _ptr(ritz))
        if rc != 0:
            self._raise(rc)
        return {"U": U, "Br": Br, "dW_r": dWr, "ritz": ritz}

    def ridge_solve(self, S_H, S_T, lam, mode=LAMBDA_PAPER, refine_steps=0):
        torch = self.torch
        dW = torch.empty((self.dims.d, self.dims.F), dtype=torch.float32, device=S_H.device)
        st = pkv_stats()
        if refine_steps:
            rc = self.L.pkv_ridge_solve_refined(self.h, _ptr(S_H), _ptr(S_T), float(lam), int(mode), int(refine_steps),
                                                _ptr(dW), C.byref(st))
        else:
            rc = self.L.pkv_ridge_solve(self.h, _ptr(S_H), _ptr(S_T), float(lam), int(mode), _ptr(dW), C.byref(st))
        if rc != 0:
            self._raise(rc, st.as_dict())
        return dW, st.as_dict()


def gram_noalloc(X, R, S_H=None, S_T=None, accumulate=False, stream=None):
    """pkv_gram_noalloc: the Eq. 9 statistics without a context and without any device allocation by the
    library (the output tensors are the caller's).  For hosts that cannot call cudaMalloc at this point;
    sizes are limited (n <= 512, F, d <= 1024) and concurrent calls must be serialised by the caller."""
    import torch
    n, F = int(X.shape[0]), int(X.shape[1])
    d = int(R.shape[1])
    if S_H is None:
        S_H = torch.zeros((F, F), dtype=torch.float32, device=X.device)
        S_T = torch.zeros((d, F), dtype=torch.float32, device=X.device)
    sp = C.c_void_p(stream.cuda_stream if stream is not None else torch.cuda.current_stream().cuda_stream)
    rc = lib().pkv_gram_noalloc(_ptr(X), _ptr(R), n, F, d, _ptr(S_H), _ptr(S_T), 1 if accumulate else 0, sp)
    if rc != 0:
        raise PkvError(rc, lib().pkv_strerror(rc).decode())
    return S_H, S_T


def to_device(arrays: Dict[str, np.ndarray], dtype: str, device="cuda"):
    """Uploads generator arrays: weights/caches in the config dtype, norm gains in fp32."""
    import torch
    out = {}
    wd = torch.bfloat16 if dtype == "bf16" else torch.float32
    for k, v in arrays.items():
        t = torch.from_numpy(np.ascontiguousarray(v, dtype=np.float32))
        out[k] = t.to(device=device, dtype=torch.float32 if k.startswith("g_") else wd).contiguous()
    return out

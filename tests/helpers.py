"""Shared harness for the parity tests: one problem -> oracle result and CUDA result."""
import numpy as np

from oracle import pkv_oracle as orc
from paper_2609_39329_b200 import inputs as gen


def oracle_prefill(ctx_hidden, w, cfg):
    """Cache of the fp32 tiny config from context hidden states; observation queries = the
    rotated queries of the last n_obs context rows."""
    K, V, q = orc.prefill_kv(ctx_hidden, w, cfg)
    return K.astype(np.float32), V.astype(np.float32), q[-cfg.n_obs:].astype(np.float32)


def make_problem(cfg, layer=0, per_head_budget=None):
    """Layer tensors + reference states for a config (numpy, dtype-representable values)."""
    lay = gen.gen_layer(cfg, layer, prefill=oracle_prefill if cfg.dtype == "fp32" else None)
    if per_head_budget is not None:
        lay["kept"] = gen.select_kept(gen.scaled_config(cfg, kept_rule="random"), layer,
                                      per_head_budget=per_head_budget)
    ctx = gen.gen_context_hidden(cfg) if cfg.dtype == "fp32" else None
    lay["x0"] = gen.gen_reference(cfg, ctx)
    return lay


def run_oracle(cfg, lay, xF, xC, chunk_off, lam0, mode=orc.LAMBDA_PAPER, keep=False):
    return orc.build_patch(lay["weights"], lay["K"], lay["V"], lay["kept"], xF, xC, chunk_off, cfg.L, lam0, cfg,
                           mode=mode, keep_intermediates=keep)


def rel_fro(a, b):
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300))


def attn_max_rel(a, ref, Hq, hd):
    """max over heads of max|a - ref| / max|ref| (per head)."""
    a = np.asarray(a, dtype=np.float64).reshape(-1, Hq, hd)
    r = np.asarray(ref, dtype=np.float64).reshape(-1, Hq, hd)
    err = np.abs(a - r).max(axis=(0, 2))
    scale = np.abs(r).max(axis=(0, 2))
    return float((err / np.maximum(scale, 1e-300)).max())

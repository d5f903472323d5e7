"""Seeded synthetic workloads for PatchKV patch construction.

This module only *draws numbers*: it holds none of the method's arithmetic (no norm, no
projection, no RoPE, no ridge algebra).  Both the CPU checker used by the tests and the CUDA
library receive the arrays produced here, so that the two are compared on identical inputs.

Recipe (per config, per layer; every tensor has its own counter-keyed stream
``SeedSequence([seed, config id, layer, tensor id])`` so tensors can be generated in any
order and layer by layer):

* weight matrices ~ N(0, 0.02), norm gains = 1, rounded (RNE) to the config dtype before
  anybody sees them; layout ``[out][in]`` row-major (the paper writes the MLP output
  projection as ``W in R^{d x d_ff}``);
* bf16 configs: cached keys and values ~ N(0,1) with 4 outlier channels (ids drawn per
  layer, shared by all KV heads, K and V) multiplied by 10, rounded to bf16, layout
  ``[Hkv][L][hd]``;
* fp32 tiny config: the generator provides context hidden states ~ N(0,1) x per-channel
  U(0.5,2); the harness turns them into a cache with a prefill helper it supplies;
* reference tokens: ``N`` rows ~ N(0,1) x per-channel U(0.5,2), fp32 (tiny config: the last
  ``N`` context rows);
* kept-index sets (the compressed cache of an eviction compressor): ascending int32 per KV
  head, chosen by the rule of the config (recent window + top-k by summed attention
  probability of observation queries, uniform random subset, or recent window only).  The
  selection is the *compressor's* job and sits off the measured path; ties go to the lower
  index.

The evaluation suites the paper measures on are not reproduced here: these tensors only
share the shapes (model geometry, context length, cache budget) of those workloads.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Callable, Dict, List, Optional

import numpy as np

# tensor ids for the counter-keyed streams
_T = {name: i for i, name in enumerate(
    ["Wq", "Wk", "Wv", "Wo", "Wgate", "Wup", "Wdown", "K", "V", "outlier", "ref", "ref_scale",
     "ctx", "ctx_scale", "q_obs", "kept", "misc"])}


@dataclass(frozen=True)
class PkvConfig:
    """Shape and recipe of one synthetic workload."""
    name: str
    cfg_id: int
    dtype: str            # "fp32" | "bf16": storage type of weights and caches
    d: int                # hidden size
    Hq: int               # query heads
    Hkv: int              # key/value heads
    hd: int               # head dim
    F: int                # MLP intermediate width (the five benchmark configs use F = d)
    L: int                # context length = rows of the full cache
    N: int                # reference tokens per context
    n_layers: int
    lam0: float           # ridge coefficient (lambda_0 of the adaptive scaling)
    rope_theta: float
    eps: float
    kept_rule: str        # "window_topk" | "random" | "window"
    window: int           # recent rows always kept
    budget: int           # kept rows per KV head (window included)
    n_obs: int = 32       # observation queries used for scoring
    seed: int = 0
    lam_sweep: tuple = ()

    @property
    def Dq(self) -> int:
        return self.Hq * self.hd

    @property
    def Dkv(self) -> int:
        return self.Hkv * self.hd

    @property
    def g(self) -> int:
        return self.Hq // self.Hkv


def benchmark_config(i: int) -> PkvConfig:
    """The five benchmark workloads, numbered 1..5."""
    if i == 1:
        return PkvConfig("tiny-fp32", 1, "fp32", 256, 4, 2, 64, 256, 1024, 64, 1, 1e-2, 1e4, 1e-5,
                         "window_topk", 64, 128, n_obs=64)
    if i == 2:
        return PkvConfig("llama3-8b-1layer-L32k", 2, "bf16", 4096, 32, 8, 128, 4096, 32768, 512, 1,
                         1e-1, 5e5, 1e-5, "window_topk", 32, 3276)
    if i == 3:
        return PkvConfig("llama3-8b-32layer-L128k", 3, "bf16", 4096, 32, 8, 128, 4096, 131072, 1024,
                         32, 1e-1, 5e5, 1e-5, "window_topk", 1024, 3932)
    if i == 4:
        return PkvConfig("qwen2.5-7b-28layer-L170k", 4, "bf16", 3584, 28, 4, 128, 3584, 170000, 2048,
                         28, 1e-1, 1e6, 1e-6, "random", 0, 1700, lam_sweep=(1e-3, 1e-1, 10.0))
    if i == 5:
        return PkvConfig("mistral-nemo-12b-40layer-L64k", 5, "bf16", 5120, 32, 8, 128, 5120, 65536,
                         4096, 40, 1e-1, 1e6, 1e-5, "window", 2048, 2048)
    raise ValueError("benchmark configs are numbered 1..5")


def scaled_config(base: PkvConfig, **kw) -> PkvConfig:
    """A copy of ``base`` with some fields replaced (reduced-size parity cases)."""
    return replace(base, **kw)


# ----------------------------------------------------------------------------------------
# number formats
# ----------------------------------------------------------------------------------------

def round_to_bf16(a: np.ndarray) -> np.ndarray:
    """Round fp32 values to the nearest bf16 (ties to even); result stays in an fp32 array."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32)
    r = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) & np.uint32(0xFFFF0000)
    return r.view(np.float32)


def bf16_bits(a: np.ndarray) -> np.ndarray:
    """Upper 16 bits of bf16-representable fp32 values (uint16, same shape)."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    return (a.view(np.uint32) >> np.uint32(16)).astype(np.uint16)


def _to_dtype(a: np.ndarray, dtype: str) -> np.ndarray:
    a = np.ascontiguousarray(a, dtype=np.float32)
    return round_to_bf16(a) if dtype == "bf16" else a


def _rng(cfg: PkvConfig, layer: int, tensor: str) -> np.random.Generator:
    return np.random.default_rng(np.random.SeedSequence([cfg.seed, cfg.cfg_id, layer, _T[tensor]]))


# ----------------------------------------------------------------------------------------
# tensors
# ----------------------------------------------------------------------------------------

def gen_weights(cfg: PkvConfig, layer: int) -> Dict[str, np.ndarray]:
    """Block weights, ``[out][in]`` row-major fp32 arrays holding dtype-representable values."""
    shapes = {"Wq": (cfg.Dq, cfg.d), "Wk": (cfg.Dkv, cfg.d), "Wv": (cfg.Dkv, cfg.d),
              "Wo": (cfg.d, cfg.Dq), "Wgate": (cfg.F, cfg.d), "Wup": (cfg.F, cfg.d),
              "Wdown": (cfg.d, cfg.F)}
    w = {}
    for name, shp in shapes.items():
        r = _rng(cfg, layer, name)
        w[name] = _to_dtype(r.standard_normal(shp, dtype=np.float32) * np.float32(0.02), cfg.dtype)
    w["g_attn"] = np.ones(cfg.d, dtype=np.float32)
    w["g_mlp"] = np.ones(cfg.d, dtype=np.float32)
    return w


def gen_cache(cfg: PkvConfig, layer: int) -> Dict[str, np.ndarray]:
    """Synthetic full cache ``K, V [Hkv][L][hd]`` (bf16 configs)."""
    out_ch = _rng(cfg, layer, "outlier").choice(cfg.hd, size=4, replace=False)
    kv = {}
    for name in ("K", "V"):
        r = _rng(cfg, layer, name)
        a = r.standard_normal((cfg.Hkv, cfg.L, cfg.hd), dtype=np.float32)
        a[:, :, out_ch] *= np.float32(10.0)
        kv[name] = _to_dtype(a, cfg.dtype)
    kv["outlier_channels"] = np.sort(out_ch).astype(np.int32)
    return kv


def gen_context_hidden(cfg: PkvConfig) -> np.ndarray:
    """Context hidden states ``[L][d]`` ~ N(0,1) x per-channel U(0.5,2) (tiny fp32 config)."""
    scale = _rng(cfg, 0, "ctx_scale").uniform(0.5, 2.0, size=cfg.d).astype(np.float32)
    x = _rng(cfg, 0, "ctx").standard_normal((cfg.L, cfg.d), dtype=np.float32)
    return np.ascontiguousarray(x * scale[None, :], dtype=np.float32)


def gen_reference(cfg: PkvConfig, ctx_hidden: Optional[np.ndarray] = None) -> np.ndarray:
    """Reference-token hidden states entering block 1, ``[N][d]`` fp32."""
    if ctx_hidden is not None:
        return np.ascontiguousarray(ctx_hidden[-cfg.N:], dtype=np.float32)
    scale = _rng(cfg, 0, "ref_scale").uniform(0.5, 2.0, size=cfg.d).astype(np.float32)
    x = _rng(cfg, 0, "ref").standard_normal((cfg.N, cfg.d), dtype=np.float32)
    return np.ascontiguousarray(x * scale[None, :], dtype=np.float32)


def gen_obs_queries(cfg: PkvConfig, layer: int) -> np.ndarray:
    """Observation-window queries used only to *score* cache rows, ``[n_obs][Hq][hd]`` fp32."""
    return _rng(cfg, layer, "q_obs").standard_normal((cfg.n_obs, cfg.Hq, cfg.hd), dtype=np.float32)


# ----------------------------------------------------------------------------------------
# kept-index sets (stand-ins for an eviction compressor; off the measured path)
# ----------------------------------------------------------------------------------------

def _topk_lower_index_wins(score: np.ndarray, k: int) -> np.ndarray:
    """Indices of the k largest scores; equal scores go to the lower index."""
    if k <= 0:
        return np.zeros(0, dtype=np.int64)
    order = np.lexsort((np.arange(score.size), -score))   # by -score, then by index
    return order[:k]


def select_kept(cfg: PkvConfig, layer: int, K: Optional[np.ndarray] = None,
                q_obs: Optional[np.ndarray] = None,
                per_head_budget: Optional[List[int]] = None) -> List[np.ndarray]:
    """Kept rows per KV head, ascending int32.

    window_topk: the last ``window`` rows plus the highest-scoring of the rest, the score of a
        row being its attention probability (softmax over all L rows of q.k/sqrt(hd)) summed
        over the observation queries and over the query heads of the KV head's group.
    random:      a uniform random subset, seeded per (layer, head).
    window:      the last ``budget`` rows.
    """
    L = cfg.L
    budgets = per_head_budget if per_head_budget is not None else [cfg.budget] * cfg.Hkv
    kept: List[np.ndarray] = []
    for h in range(cfg.Hkv):
        b = int(min(budgets[h], L))
        if cfg.kept_rule == "window":
            idx = np.arange(L - b, L)
        elif cfg.kept_rule == "random":
            r = np.random.default_rng(np.random.SeedSequence([cfg.seed, cfg.cfg_id, layer, _T["kept"], h]))
            idx = np.sort(r.choice(L, size=b, replace=False))
        elif cfg.kept_rule == "window_topk":
            if K is None or q_obs is None:
                raise ValueError("window_topk needs the cache keys and observation queries")
            win = min(cfg.window, b)
            qh = q_obs[:, h * cfg.g:(h + 1) * cfg.g, :].reshape(-1, cfg.hd).astype(np.float64)
            logits = qh @ K[h].astype(np.float64).T / np.sqrt(cfg.hd)
            logits -= logits.max(axis=1, keepdims=True)
            p = np.exp(logits)
            p /= p.sum(axis=1, keepdims=True)
            score = p.sum(axis=0)
            top = _topk_lower_index_wins(score[:L - win], b - win)
            idx = np.sort(np.concatenate([top, np.arange(L - win, L)]))
        else:
            raise ValueError(cfg.kept_rule)
        kept.append(np.ascontiguousarray(idx, dtype=np.int32))
    return kept


def kept_to_csr(kept: List[np.ndarray]):
    """(head_off int32 [Hkv+1], idx int32 [sum b_h]) from a per-head list."""
    off = np.zeros(len(kept) + 1, dtype=np.int32)
    for h, k in enumerate(kept):
        off[h + 1] = off[h] + len(k)
    idx = np.concatenate(kept).astype(np.int32) if off[-1] > 0 else np.zeros(0, dtype=np.int32)
    return off, idx


def gen_layer(cfg: PkvConfig, layer: int,
              prefill: Optional[Callable] = None) -> Dict[str, object]:
    """Everything one block needs: weights, full cache, kept sets.

    For the fp32 tiny config the cache comes from context hidden states through ``prefill``
    (a callable ``(ctx_hidden, weights, cfg) -> (K, V, q_obs)`` supplied by the harness).
    """
    w = gen_weights(cfg, layer)
    if cfg.dtype == "fp32":
        if prefill is None:
            raise ValueError("the fp32 tiny config needs a prefill helper")
        K, V, q_obs = prefill(gen_context_hidden(cfg), w, cfg)
        kv = {"K": np.ascontiguousarray(K, dtype=np.float32), "V": np.ascontiguousarray(V, dtype=np.float32)}
    else:
        kv = gen_cache(cfg, layer)
        q_obs = gen_obs_queries(cfg, layer) if cfg.kept_rule == "window_topk" else None
    kept = select_kept(cfg, layer, kv["K"], q_obs)
    return {"weights": w, "K": kv["K"], "V": kv["V"], "kept": kept}


def quantize_rows(x: np.ndarray, bits: int, group: int):
    """A storage-side quantiser for compact caches (the compressor's job, off the measured path): symmetric,
    one fp32 scale per `group` consecutive elements of a row, signed codes of `bits` bits (8: int8 array
    [rows][hd]; 4: uint8 array [rows][hd/2], even element in the low nibble, two's complement).
    Returns (codes, scales fp32 [rows][hd/group])."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    rows, hd = x.shape
    qmax = 127 if bits == 8 else 7
    g = x.reshape(rows, hd // group, group)
    amax = np.abs(g).max(axis=2)
    scales = np.where(amax > 0, amax / qmax, 1.0).astype(np.float32)
    q = np.clip(np.rint(g / scales[:, :, None]), -qmax, qmax).astype(np.int32).reshape(rows, hd)
    if bits == 8:
        return q.astype(np.int8), scales
    u = (q & 15).astype(np.uint8)
    return (u[:, 0::2] | (u[:, 1::2] << 4)).astype(np.uint8), scales

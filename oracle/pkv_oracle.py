"""CPU oracle for PatchKV patch construction — TEST INFRASTRUCTURE, not the product.

A plain, slow, fp64 numpy statement of what one block of the method computes, written from
the paper's definitions (Sec. 2.2 Eq. 4-8, Sec. 2.3 Eq. 9, Algorithm 1).  It shares no code
with the CUDA library and is imported only by the tests, the smoke check and the benchmark's
CPU-baseline leg.  Library primitives (matmul, LAPACK Cholesky, triangular solve) serve as
single steps; there is no blocking, fusion or reordering beyond what the definitions state.

Conventions fixed here because the paper leaves the backbone unspecified (each listed in the
design notes as a reading):
  * weights are ``[out][in]``; the patched matrix is the MLP down projection
    ``W in R^{d x F}`` and the patch ``dW`` has the same shape (Sec. 2.2);
  * ``z`` is the residual stream after the attention sub-layer, ``z = x + a Wo^T``, so that
    ``W h + z`` is literally the block output of Eq. 4;
  * RMSNorm with gain, SiLU-gated MLP, no biases;
  * rotary embedding on half-split pairs ``(c, c + hd/2)``, angle ``pos * theta^(-2c/hd)``;
    cached keys arrive already rotated; chunk token ``i`` of a chunk starting at ``s`` sits
    at position ``pos0 + (i - s)`` in both streams;
  * a reference token attends to every row of the cache it is given and causally to the
    tokens of its own chunk; nothing crosses chunks (Sec. 2.3, chunked query encoding).

Pins: tests/test_oracle_pins.py checks every function below against closed forms, brute
force on tiny inputs, textbook routines that take another route (QR least squares on the
augmented system, the dual N x N form, eigenvalues) and the invariants Eq. 4-9 imply.
The RoPE / norm conventions and the input generators are our own definitions: nothing in
the paper pins them ("parity unpinned" for those conventions only).
``dequantize_cache`` states the storage format of quantised compact caches (ours: the paper names INT8 / INT4
only); it is pinned on hand-written bytes and closed-form products.
"""
from __future__ import annotations

from typing import Dict, List, Optional, Sequence

import numpy as np
import scipy.linalg

LAMBDA_PAPER = 0      # lambda = lambda0 * ||S_H||_F^2 / tr(S_H)   (Eq. 7)
LAMBDA_ABSOLUTE = 1   # lambda = lambda0                            (Eq. 6 as written)
LAMBDA_TRACE_MEAN = 2 # lambda = lambda0 * tr(S_H) / F              (ridge-scale ablation)


def f64(a) -> np.ndarray:
    return np.asarray(a, dtype=np.float64)


# ----------------------------------------------------------------------------------------
# backbone pieces (Algorithm 1, "forward block l")
# ----------------------------------------------------------------------------------------

def rmsnorm(x: np.ndarray, gain: np.ndarray, eps: float) -> np.ndarray:
    """u = x * gain / sqrt(mean(x^2) + eps), row by row."""
    x = f64(x)
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return x * f64(gain) / np.sqrt(ms + eps)


def rope(t: np.ndarray, pos: np.ndarray, theta: float) -> np.ndarray:
    """Rotate ``t [n][H][hd]`` at integer positions ``pos [n]`` (half-split pairs)."""
    t = f64(t)
    if theta == 0:
        return t.copy()
    n, H, hd = t.shape
    half = hd // 2
    inv = theta ** (-2.0 * np.arange(half, dtype=np.float64) / hd)
    ang = f64(pos)[:, None] * inv[None, :]
    c, s = np.cos(ang)[:, None, :], np.sin(ang)[:, None, :]
    lo, hi = t[..., :half], t[..., half:]
    return np.concatenate([lo * c - hi * s, hi * c + lo * s], axis=-1)


def silu(t: np.ndarray) -> np.ndarray:
    return t / (1.0 + np.exp(-t))


def prefill_kv(ctx_hidden, w: Dict[str, np.ndarray], dims) -> tuple:
    """Keys/values of context rows at positions 0..L-1 (Algorithm 1, "Prefill full cache";
    one block only, used by the harness to build the tiny config's cache).
    Returns K, V ``[Hkv][L][hd]`` and the rotated queries of those rows ``[L][Hq][hd]``."""
    L = ctx_hidden.shape[0]
    u = rmsnorm(ctx_hidden, w["g_attn"], dims.eps)
    pos = np.arange(L)
    q = rope((u @ f64(w["Wq"]).T).reshape(L, dims.Hq, dims.hd), pos, dims.rope_theta)
    k = rope((u @ f64(w["Wk"]).T).reshape(L, dims.Hkv, dims.hd), pos, dims.rope_theta)
    v = (u @ f64(w["Wv"]).T).reshape(L, dims.Hkv, dims.hd)
    return k.transpose(1, 0, 2).copy(), v.transpose(1, 0, 2).copy(), q


def attention(q: np.ndarray, k_new: np.ndarray, v_new: np.ndarray,
              K_cache: Sequence[np.ndarray], V_cache: Sequence[np.ndarray],
              chunk_off: Sequence[int], key_bias: Optional[Sequence[np.ndarray]] = None) -> np.ndarray:
    """Cached attention of the reference tokens (Sec. 2.2: forward passes over q with a cache).

    q      [n][Hq][hd]   rotated queries
    k_new  [n][Hkv][hd]  rotated keys of the reference tokens, v_new their values
    K_cache[h] [rows_h][hd], V_cache[h] likewise — the cache of KV head h (rows may differ)
    Token i of chunk [s, e) sees every cache row of its KV head and chunk tokens s..i.
    Returns a [n][Hq*hd].
    """
    q, k_new, v_new = f64(q), f64(k_new), f64(v_new)
    n, Hq, hd = q.shape
    Hkv = k_new.shape[1]
    g = Hq // Hkv
    out = np.zeros((n, Hq, hd))
    scale = 1.0 / np.sqrt(hd)
    for c in range(len(chunk_off) - 1):
        s, e = int(chunk_off[c]), int(chunk_off[c + 1])
        m = e - s
        causal = np.tril(np.ones((m, m), dtype=bool))
        for h in range(Hq):
            kh = h // g
            Kc, Vc = f64(K_cache[kh]), f64(V_cache[kh])
            rows = Kc.shape[0]
            logit_cache = (q[s:e, h, :] @ Kc.T) * scale if rows else np.zeros((m, 0))
            if key_bias is not None and rows:
                logit_cache = logit_cache + f64(key_bias[kh])[None, :]
            logit_new = (q[s:e, h, :] @ k_new[s:e, kh, :].T) * scale
            logit_new = np.where(causal, logit_new, -np.inf)
            logits = np.concatenate([logit_cache, logit_new], axis=1)
            logits = logits - logits.max(axis=1, keepdims=True)
            p = np.exp(logits)
            p = p / p.sum(axis=1, keepdims=True)
            vals = np.concatenate([Vc, v_new[s:e, kh, :]], axis=0) if rows else v_new[s:e, kh, :]
            out[s:e, h, :] = p @ vals
    return out.reshape(n, Hq * hd)


def block_forward(x: np.ndarray, w: Dict[str, np.ndarray], K_cache, V_cache, chunk_off, pos0: int,
                  dims, key_bias=None) -> Dict[str, np.ndarray]:
    """One transformer block on the reference tokens with a given cache (Algorithm 1,
    teacher / student forward).  Returns attention output ``a``, residual term ``z``,
    post-activation MLP features ``h`` and the rotated ``q``."""
    x = f64(x)
    n = x.shape[0]
    pos = np.zeros(n, dtype=np.int64)
    for c in range(len(chunk_off) - 1):
        s, e = int(chunk_off[c]), int(chunk_off[c + 1])
        pos[s:e] = pos0 + np.arange(e - s)
    u1 = rmsnorm(x, w["g_attn"], dims.eps)
    q = rope((u1 @ f64(w["Wq"]).T).reshape(n, dims.Hq, dims.hd), pos, dims.rope_theta)
    k = rope((u1 @ f64(w["Wk"]).T).reshape(n, dims.Hkv, dims.hd), pos, dims.rope_theta)
    v = (u1 @ f64(w["Wv"]).T).reshape(n, dims.Hkv, dims.hd)
    a = attention(q, k, v, K_cache, V_cache, chunk_off, key_bias)
    z = x + a @ f64(w["Wo"]).T
    u2 = rmsnorm(z, w["g_mlp"], dims.eps)
    h = silu(u2 @ f64(w["Wgate"]).T) * (u2 @ f64(w["Wup"]).T)
    return {"a": a, "z": z, "h": h, "q": q, "k": k, "v": v}


# ----------------------------------------------------------------------------------------
# the regression (Eq. 5-9)
# ----------------------------------------------------------------------------------------

def targets(Wdown: np.ndarray, hF, zF, hC, zC) -> np.ndarray:
    """t_i = W (h_i - h'_i) + (z_i - z'_i), stacked as rows of T [N][d] (Eq. 5)."""
    return (f64(hF) - f64(hC)) @ f64(Wdown).T + (f64(zF) - f64(zC))


def sufficient_statistics(H: np.ndarray, T: np.ndarray, chunk_off: Optional[Sequence[int]] = None):
    """S_H = H'^T H' [F][F], S_T = T^T H' [d][F] as running sums over chunks (Eq. 9)."""
    H, T = f64(H), f64(T)
    if chunk_off is None:
        chunk_off = [0, H.shape[0]]
    S_H = np.zeros((H.shape[1], H.shape[1]))
    S_T = np.zeros((T.shape[1], H.shape[1]))
    for c in range(len(chunk_off) - 1):
        s, e = int(chunk_off[c]), int(chunk_off[c + 1])
        S_H += H[s:e].T @ H[s:e]
        S_T += T[s:e].T @ H[s:e]
    return S_H, S_T


def ridge_lambda(S_H: np.ndarray, lam0: float, mode: int = LAMBDA_PAPER) -> float:
    """Adaptive ridge scaling lambda = lambda0 ||S_H||_F^2 / tr(S_H) (Eq. 7), or the variants."""
    S_H = f64(S_H)
    if mode == LAMBDA_ABSOLUTE:
        return float(lam0)
    tr = float(np.trace(S_H))
    if not tr > 0.0:
        raise ZeroDivisionError("tr(S_H) = 0: adaptive ridge scale undefined")
    if mode == LAMBDA_TRACE_MEAN:
        return float(lam0) * tr / S_H.shape[0]
    return float(lam0) * float(np.sum(S_H * S_H)) / tr


def ridge_solve(S_H: np.ndarray, S_T: np.ndarray, lam: float) -> np.ndarray:
    """dW = S_T (S_H + lambda I)^{-1}  [d][F]  (Eq. 8 / Algorithm 1), by Cholesky."""
    if not (lam > 0.0 and np.isfinite(lam)):
        raise ValueError("lambda must be positive and finite")
    G = f64(S_H) + lam * np.eye(S_H.shape[0])
    Lc = np.linalg.cholesky(G)                                   # G = Lc Lc^T
    Y = scipy.linalg.solve_triangular(Lc, f64(S_T).T, lower=True)      # Lc Y = S_T^T
    X = scipy.linalg.solve_triangular(Lc.T, Y, lower=False)            # Lc^T X = Y
    return np.ascontiguousarray(X.T)


def low_rank_patch(dW: np.ndarray, S_H: np.ndarray, r: int):
    """Rank-r patch (appendix, low-rank weight patches): with M = dW S_H dW^T  [d][d] and U_r its r
    leading eigenvectors, dW_r = U_r (U_r^T dW).  Returns (U_r [d][r], B_r = U_r^T dW [r][F],
    dW_r [d][F], all eigenvalues of M in descending order).  Storage of the factored form is
    (d + F) r numbers.  Eigenvector signs are arbitrary; dW_r is unique when the r-th and (r+1)-th
    eigenvalues differ."""
    dW = f64(dW)
    d = dW.shape[0]
    if not (0 <= r <= d):
        raise ValueError("rank must lie in [0, d]")
    M = dW @ f64(S_H) @ dW.T
    M = 0.5 * (M + M.T)
    evals, evecs = np.linalg.eigh(M)                            # ascending
    order = np.argsort(evals)[::-1]
    evals, evecs = evals[order], evecs[:, order]
    U = np.ascontiguousarray(evecs[:, :r])
    B = U.T @ dW
    return U, B, U @ B, evals


def round_bf16(a: np.ndarray) -> np.ndarray:
    """fp32 -> nearest bf16, ties to even, returned as fp32."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32).astype(np.uint64)
    r = ((u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000).astype(np.uint32)
    return r.view(np.float32)


def merge(W: np.ndarray, dW: np.ndarray, dtype: str) -> np.ndarray:
    """W <- W + dW (Algorithm 1, Merge): the sum is taken in fp32 and stored in W's type."""
    s = np.asarray(W, dtype=np.float32) + np.asarray(dW, dtype=np.float32)
    return round_bf16(s) if dtype == "bf16" else s


# ----------------------------------------------------------------------------------------
# index handling (compressed cache of an eviction compressor)
# ----------------------------------------------------------------------------------------

def check_kept(kept: Sequence[np.ndarray], L: int) -> Optional[tuple]:
    """First offending (head, position) of a kept-index set, or None if every head's list is
    strictly ascending inside [0, L)."""
    for h, idx in enumerate(kept):
        prev = -1
        for i, v in enumerate(np.asarray(idx).tolist()):
            if v < 0 or v >= L or v <= prev:
                return (h, i)
            prev = v
    return None


def gather_cache(K: np.ndarray, V: np.ndarray, kept: Sequence[np.ndarray]):
    """K'[h][i] = K[h][kept[h][i]] and the same for V — an eviction compressor's cache."""
    return [np.asarray(K[h])[np.asarray(kept[h], dtype=np.int64)] for h in range(len(kept))], \
           [np.asarray(V[h])[np.asarray(kept[h], dtype=np.int64)] for h in range(len(kept))]


def dequantize_cache(codes: np.ndarray, scales: np.ndarray, bits: int, group: int, dtype: str) -> np.ndarray:
    """Decode of a quantised compact cache (appendix, quantised caches: the patch is built against the cache
    the student will really read).  codes: int8 [rows][hd] for 8 bits; uint8 [rows][hd/2] for 4 bits with element
    2j in the low nibble of byte j and element 2j+1 in the high nibble, 4-bit two's complement.  scales: fp32
    [rows][hd/group].  An element is scale * code, the product taken in fp32 and stored in the cache's element
    type (rounded to bf16 for bf16 caches).  Returns fp32 values [rows][hd]."""
    scales = np.asarray(scales, dtype=np.float32)
    if bits == 8:
        q = np.asarray(codes).astype(np.int8).astype(np.int32)
    elif bits == 4:
        b = np.asarray(codes).astype(np.uint8).astype(np.int32)
        lo, hi = b & 15, b >> 4
        q = np.stack([lo, hi], axis=-1).reshape(b.shape[0], -1)
        q = np.where(q >= 8, q - 16, q)
    else:
        raise ValueError("bits must be 8 or 4")
    hd = q.shape[1]
    s = np.repeat(scales, group, axis=1)[:, :hd]
    x = (s * q.astype(np.float32)).astype(np.float32)           # fp32 product
    return round_bf16(x) if dtype == "bf16" else x


# ----------------------------------------------------------------------------------------
# one block of Algorithm 1
# ----------------------------------------------------------------------------------------

def build_patch(w: Dict[str, np.ndarray], K: np.ndarray, V: np.ndarray,
                kept: Optional[Sequence[np.ndarray]], xF: np.ndarray, xC: np.ndarray,
                chunk_off: Sequence[int], pos0: int, lam0: float, dims,
                mode: int = LAMBDA_PAPER, compressed: Optional[tuple] = None,
                keep_intermediates: bool = False) -> Dict[str, object]:
    """Teacher and student forward of one block, targets, statistics, ridge patch, next states.

    ``kept`` lists the cache rows the student keeps per KV head; alternatively
    ``compressed = (K'[h], V'[h], bias[h] or None)`` gives an explicit compact cache.
    Returns dW [d][F], xF_next, xC_next [N][d] and the scalars of the solve.
    """
    Kf = [np.asarray(K[h]) for h in range(dims.Hkv)]
    Vf = [np.asarray(V[h]) for h in range(dims.Hkv)]
    bias = None
    if compressed is not None:
        Kc, Vc = compressed[0], compressed[1]
        bias = compressed[2] if len(compressed) > 2 else None
    else:
        bad = check_kept(kept, K.shape[1])
        if bad is not None:
            raise IndexError("kept-index set invalid at (head, position) = %r" % (bad,))
        Kc, Vc = gather_cache(K, V, kept)
    tea = block_forward(xF, w, Kf, Vf, chunk_off, pos0, dims)            # Alg. 1: teacher forward
    stu = block_forward(xC, w, Kc, Vc, chunk_off, pos0, dims, bias)      # Alg. 1: student forward
    T = targets(w["Wdown"], tea["h"], tea["z"], stu["h"], stu["z"])      # Eq. 5
    H = stu["h"]
    S_H, S_T = sufficient_statistics(H, T, chunk_off)                     # Eq. 9
    lam = ridge_lambda(S_H, lam0, mode)                                   # Eq. 7
    dW = ridge_solve(S_H, S_T, lam)                                       # Eq. 8
    Wd = f64(w["Wdown"])
    xF_next = tea["z"] + tea["h"] @ Wd.T                                  # teacher never patched
    xC_next = stu["z"] + H @ (Wd + dW).T                                  # patched student block
    res = T - H @ dW.T
    out = {
        "dW": dW, "xF_next": xF_next, "xC_next": xC_next,
        "lam": lam, "tr": float(np.trace(S_H)), "fro2": float(np.sum(S_H * S_H)),
        "T_fro2": float(np.sum(T * T)), "res_fro2": float(np.sum(res * res)),
        "dW_fro": float(np.sqrt(np.sum(dW * dW))),
        "aF": tea["a"], "aC": stu["a"],
    }
    if keep_intermediates:
        out.update({"tea": tea, "stu": stu, "T": T, "H": H, "S_H": S_H, "S_T": S_T})
    return out

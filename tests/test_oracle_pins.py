"""Pins for the CPU oracle: each part is checked against something other than itself —
brute force on tiny inputs, closed forms, textbook routines that take another route, and the
invariants the paper's equations imply (Eq. 4-9, Algorithm 1)."""
import math

import numpy as np
import pytest

from oracle import pkv_oracle as orc
from paper_2609_39329_b200 import inputs as gen


def tiny_cfg(**kw):
    base = gen.benchmark_config(2)
    d = dict(d=32, Hq=4, Hkv=2, hd=8, F=24, L=40, N=12, window=4, budget=10, n_obs=4,
             rope_theta=1e4, name="pin")
    d.update(kw)
    return gen.scaled_config(base, **d)


def tiny_problem(cfg, seed=0, scale_w=0.3):
    r = np.random.default_rng(seed)
    w = {k: r.standard_normal(s) * scale_w for k, s in {
        "Wq": (cfg.Dq, cfg.d), "Wk": (cfg.Dkv, cfg.d), "Wv": (cfg.Dkv, cfg.d), "Wo": (cfg.d, cfg.Dq),
        "Wgate": (cfg.F, cfg.d), "Wup": (cfg.F, cfg.d), "Wdown": (cfg.d, cfg.F)}.items()}
    w["g_attn"] = 1.0 + 0.1 * r.standard_normal(cfg.d)
    w["g_mlp"] = 1.0 + 0.1 * r.standard_normal(cfg.d)
    K = r.standard_normal((cfg.Hkv, cfg.L, cfg.hd))
    V = r.standard_normal((cfg.Hkv, cfg.L, cfg.hd))
    x = r.standard_normal((cfg.N, cfg.d))
    kept = [np.sort(r.choice(cfg.L, size=cfg.budget, replace=False)).astype(np.int32) for _ in range(cfg.Hkv)]
    return w, K, V, x, kept


# ------------------------------------------------------------------ attention ----------

def brute_attention(q, k_new, v_new, K_cache, V_cache, chunk_off):
    """Literal per-element coding: one query row at a time, python loops, explicit key list."""
    n, Hq, hd = q.shape
    g = Hq // k_new.shape[1]
    out = np.zeros((n, Hq, hd))
    for c in range(len(chunk_off) - 1):
        s, e = chunk_off[c], chunk_off[c + 1]
        for i in range(s, e):
            for h in range(Hq):
                kh = h // g
                keys = [K_cache[kh][r] for r in range(len(K_cache[kh]))] + [k_new[j, kh] for j in range(s, i + 1)]
                vals = [V_cache[kh][r] for r in range(len(V_cache[kh]))] + [v_new[j, kh] for j in range(s, i + 1)]
                lg = [sum(q[i, h, t] * kk[t] for t in range(hd)) / math.sqrt(hd) for kk in keys]
                mx = max(lg)
                ex = [math.exp(v - mx) for v in lg]
                den = sum(ex)
                for t in range(hd):
                    out[i, h, t] = sum(ex[r] * vals[r][t] for r in range(len(keys))) / den
    return out.reshape(n, Hq * hd)


def rand_attn_inputs(seed=1, n=7, Hq=4, Hkv=2, hd=6, rows=(9, 5)):
    r = np.random.default_rng(seed)
    q = r.standard_normal((n, Hq, hd))
    k = r.standard_normal((n, Hkv, hd))
    v = r.standard_normal((n, Hkv, hd))
    Kc = [r.standard_normal((rows[h], hd)) for h in range(Hkv)]
    Vc = [r.standard_normal((rows[h], hd)) for h in range(Hkv)]
    return q, k, v, Kc, Vc


def test_attention_matches_brute_force_with_chunks_and_ragged_heads():
    q, k, v, Kc, Vc = rand_attn_inputs()
    for chunks in ([0, 7], [0, 3, 7], [0, 1, 2, 7]):
        a = orc.attention(q, k, v, Kc, Vc, chunks)
        b = brute_attention(q, k, v, Kc, Vc, chunks)
        np.testing.assert_allclose(a, b, rtol=1e-12, atol=1e-13)


def test_attention_equal_keys_gives_mean_of_visible_values():
    q, k, v, Kc, Vc = rand_attn_inputs(rows=(6, 6))
    one = np.ones(q.shape[2])
    Kc = [np.tile(one, (6, 1)) for _ in range(2)]
    k = np.tile(one, (q.shape[0], 2, 1))
    a = orc.attention(q, k, v, Kc, Vc, [0, q.shape[0]]).reshape(q.shape)
    for i in range(q.shape[0]):
        for h in range(q.shape[1]):
            kh = h // 2
            want = (Vc[kh].sum(0) + v[:i + 1, kh].sum(0)) / (6 + i + 1)
            np.testing.assert_allclose(a[i, h], want, rtol=1e-12)


def test_attention_dominant_key_returns_its_value():
    q, k, v, Kc, Vc = rand_attn_inputs()
    Kc[0][3] = 1e4 * q[2, 0] / np.linalg.norm(q[2, 0])      # aligned with query (token 2, head 0)
    a = orc.attention(q, k, v, Kc, Vc, [0, 7]).reshape(q.shape)
    np.testing.assert_allclose(a[2, 0], Vc[0][3], atol=1e-9)


def test_attention_invariant_to_cache_permutation_and_logit_shift():
    q, k, v, Kc, Vc = rand_attn_inputs()
    a = orc.attention(q, k, v, Kc, Vc, [0, 4, 7])
    perm = [np.random.default_rng(5).permutation(len(K)) for K in Kc]
    b = orc.attention(q, k, v, [K[p] for K, p in zip(Kc, perm)], [V[p] for V, p in zip(Vc, perm)], [0, 4, 7])
    np.testing.assert_allclose(a, b, rtol=1e-12, atol=1e-13)
    # a constant added to every logit of a head: the same bias on every cached key and an
    # extra key coordinate paired with a constant query coordinate for the chunk keys
    hd = q.shape[2]
    q2 = np.concatenate([q, np.ones(q.shape[:2] + (1,))], axis=2) * math.sqrt((hd + 1) / hd)
    k2 = np.concatenate([k, 3.0 * np.ones(k.shape[:2] + (1,))], axis=2)
    Kc2 = [np.concatenate([K, 3.0 * np.ones((len(K), 1))], axis=1) for K in Kc]
    v2 = np.concatenate([v, np.zeros(v.shape[:2] + (1,))], axis=2)
    Vc2 = [np.concatenate([V, np.zeros((len(V), 1))], axis=1) for V in Vc]
    c = orc.attention(q2, k2, v2, Kc2, Vc2, [0, 4, 7]).reshape(q.shape[0], q.shape[1], hd + 1)[..., :hd]
    np.testing.assert_allclose(a, c.reshape(a.shape), rtol=1e-11, atol=1e-12)


def test_attention_split_key_sets_merge_back():
    """Softmax partials (m, l, O) over disjoint key subsets recombine to the whole."""
    q, k, v, Kc, Vc = rand_attn_inputs(rows=(11, 11))
    whole = orc.attention(q, k, v, Kc, Vc, [0, 7]).reshape(q.shape)
    hd = q.shape[2]
    for i in (0, 3, 6):
        for h in range(q.shape[1]):
            kh = h // 2
            keys = np.concatenate([Kc[kh], k[:i + 1, kh]])
            vals = np.concatenate([Vc[kh], v[:i + 1, kh]])
            parts = np.array_split(np.arange(len(keys)), 3)
            ms, ls, Os = [], [], []
            for p in parts:
                lg = keys[p] @ q[i, h] / math.sqrt(hd)
                m = lg.max()
                e = np.exp(lg - m)
                ms.append(m); ls.append(e.sum()); Os.append(e @ vals[p])
            M = max(ms)
            num = sum(np.exp(m - M) * O for m, O in zip(ms, Os))
            den = sum(np.exp(m - M) * l for m, l in zip(ms, ls))
            np.testing.assert_allclose(whole[i, h], num / den, rtol=1e-12)


def test_gqa_equals_mha_with_replicated_kv_heads():
    q, k, v, Kc, Vc = rand_attn_inputs(rows=(9, 9))
    a = orc.attention(q, k, v, Kc, Vc, [0, 7])
    rep = lambda t: np.repeat(t, 2, axis=1)
    b = orc.attention(q, rep(k), rep(v), [Kc[0], Kc[0], Kc[1], Kc[1]], [Vc[0], Vc[0], Vc[1], Vc[1]], [0, 7])
    np.testing.assert_allclose(a, b, rtol=1e-12, atol=1e-13)


def test_kept_gather_equals_full_cache_with_evicted_rows_masked():
    q, k, v, Kc, Vc = rand_attn_inputs(rows=(9, 9))
    kept = [np.array([0, 2, 3, 8]), np.array([1, 4, 5, 6, 7])]
    Kg, Vg = orc.gather_cache(np.stack(Kc), np.stack(Vc), kept)
    a = orc.attention(q, k, v, Kg, Vg, [0, 7])
    bias = [np.where(np.isin(np.arange(9), kk), 0.0, -np.inf) for kk in kept]
    b = orc.attention(q, k, v, Kc, Vc, [0, 7], key_bias=bias)
    np.testing.assert_allclose(a, b, rtol=1e-12, atol=1e-13)


def test_empty_cache_and_first_token_sees_only_itself():
    q, k, v, _, _ = rand_attn_inputs()
    empty = [np.zeros((0, q.shape[2]))] * 2
    a = orc.attention(q, k, v, empty, empty, [0, 3, 7]).reshape(q.shape)
    for s in (0, 3):                      # first token of a chunk: softmax over one key
        for h in range(q.shape[1]):
            np.testing.assert_allclose(a[s, h], v[s, h // 2], rtol=1e-13)


def test_finite_key_bias_is_added_unscaled_to_cached_logits_only():
    """Approximation-style caches carry one additive logit term per cached key (Sec. 3.1).  A literal
    per-key loop fixes where it enters: after the 1/sqrt(hd) scaling, on cache keys only, never on the
    chunk's own keys."""
    q, k, v, Kc, Vc = rand_attn_inputs(seed=3, rows=(9, 5))
    r = np.random.default_rng(7)
    bias = [r.uniform(-2.0, 2.0, len(K)) for K in Kc]
    n, Hq, hd = q.shape
    for chunks in ([0, 7], [0, 3, 7]):
        a = orc.attention(q, k, v, Kc, Vc, chunks, key_bias=bias).reshape(q.shape)
        for c in range(len(chunks) - 1):
            s, e = chunks[c], chunks[c + 1]
            for i in range(s, e):
                for h in range(Hq):
                    kh = h // 2
                    lg = [sum(q[i, h, t] * Kc[kh][j][t] for t in range(hd)) / math.sqrt(hd) + bias[kh][j]
                          for j in range(len(Kc[kh]))]
                    lg += [sum(q[i, h, t] * k[j, kh, t] for t in range(hd)) / math.sqrt(hd) for j in range(s, i + 1)]
                    vals = [Vc[kh][j] for j in range(len(Vc[kh]))] + [v[j, kh] for j in range(s, i + 1)]
                    mx = max(lg)
                    ex = [math.exp(x - mx) for x in lg]
                    want = sum(w_ * val for w_, val in zip(ex, vals)) / sum(ex)
                    np.testing.assert_allclose(a[i, h], want, rtol=1e-12, atol=1e-13)
    assert not np.allclose(a, orc.attention(q, k, v, Kc, Vc, chunks).reshape(q.shape))


def test_finite_key_bias_closed_form_with_equal_keys():
    """All keys equal: a cached key with bias beta weighs e^beta, a chunk key weighs 1, whatever hd is
    (a bias multiplied by 1/sqrt(hd), or applied to the chunk keys too, fails this)."""
    q, k, v, Kc, Vc = rand_attn_inputs(seed=4, hd=16, rows=(6, 6))
    one = np.ones(q.shape[2])
    Kc = [np.tile(one, (6, 1)) for _ in range(2)]
    k = np.tile(one, (q.shape[0], 2, 1))
    beta = [np.array([0.0, 1.0, -1.0, 2.0, 0.5, -0.5]), np.array([3.0, 0.0, 0.0, -2.0, 1.5, 0.25])]
    a = orc.attention(q, k, v, Kc, Vc, [0, q.shape[0]], key_bias=beta).reshape(q.shape)
    for i in range(q.shape[0]):
        for h in range(q.shape[1]):
            kh = h // 2
            wgt = np.exp(beta[kh])
            want = (wgt @ Vc[kh] + v[:i + 1, kh].sum(0)) / (wgt.sum() + i + 1)
            np.testing.assert_allclose(a[i, h], want, rtol=1e-12)


def test_prefill_cache_then_cached_forward_equals_one_causal_pass():
    """prefill_kv pins: the cache it builds from context rows, attended to by reference tokens at
    positions L.., gives what one causal pass over [context; reference] gives on the reference rows."""
    cfg = tiny_cfg(L=19, N=6)
    w, _, _, x, _ = tiny_problem(cfg, seed=9)
    r = np.random.default_rng(10)
    ctx = r.standard_normal((cfg.L, cfg.d))
    K, V, q_ctx = orc.prefill_kv(ctx, w, cfg)
    assert K.shape == (cfg.Hkv, cfg.L, cfg.hd) and V.shape == K.shape and q_ctx.shape == (cfg.L, cfg.Hq, cfg.hd)
    cached = orc.block_forward(x, w, list(K), list(V), [0, cfg.N], cfg.L, cfg)
    empty = [np.zeros((0, cfg.hd))] * cfg.Hkv
    whole = orc.block_forward(np.concatenate([ctx, x]), w, empty, empty, [0, cfg.L + cfg.N], 0, cfg)
    np.testing.assert_allclose(cached["a"], whole["a"][cfg.L:], rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(cached["h"], whole["h"][cfg.L:], rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(q_ctx, whole["q"][:cfg.L], rtol=1e-12, atol=1e-13)
    # a context row moved to another position changes the result: positions matter
    K2, V2, _ = orc.prefill_kv(ctx[::-1].copy(), w, cfg)
    assert not np.allclose(orc.block_forward(x, w, list(K2[:, ::-1]), list(V2[:, ::-1]), [0, cfg.N], cfg.L, cfg)["a"],
                           cached["a"])


def test_quantised_cache_decode_on_hand_written_bytes_and_closed_forms():
    """The storage format of quantised compact caches: nibble order, sign extension, group scales, and the
    element type of the decoded value."""
    # 4 bits: byte 0xA3 holds element 0 = 3 (low nibble) and element 1 = 0xA = -6 (two's complement)
    codes4 = np.array([[0xA3, 0x7F, 0x80, 0x01]], dtype=np.uint8)           # 8 elements, hd = 8
    scales = np.array([[0.5]], dtype=np.float32)
    got = orc.dequantize_cache(codes4, scales, 4, 8, "fp32")
    np.testing.assert_array_equal(got, np.array([[1.5, -3.0, -0.5, 3.5, 0.0, -4.0, 0.5, 0.0]], dtype=np.float32))
    # 8 bits, two groups with their own scales
    codes8 = np.array([[127, -127, 1, 0, -1, 64, -64, 2] * 2], dtype=np.int8)   # hd = 16, group = 8
    sc = np.array([[0.25, 2.0]], dtype=np.float32)
    got = orc.dequantize_cache(codes8, sc, 8, 8, "fp32")
    want = np.concatenate([0.25 * codes8[0, :8].astype(np.float64), 2.0 * codes8[0, 8:].astype(np.float64)])[None]
    np.testing.assert_array_equal(got.astype(np.float64), want)
    # bf16 caches: the decoded value is the bf16 rounding of the fp32 product (checked against torch)
    import torch
    r = np.random.default_rng(12)
    c = r.integers(-127, 128, size=(5, 32)).astype(np.int8)
    s2 = r.uniform(0.01, 0.1, size=(5, 2)).astype(np.float32)
    got = orc.dequantize_cache(c, s2, 8, 16, "bf16")
    ref = (torch.from_numpy(np.repeat(s2, 16, axis=1)) * torch.from_numpy(c.astype(np.float32))).to(torch.bfloat16).float().numpy()
    np.testing.assert_array_equal(got, ref)
    # a round trip through the harness quantiser is within half a step of every element
    x = r.standard_normal((6, 64)).astype(np.float32)
    for bits in (8, 4):
        q, sc3 = gen.quantize_rows(x, bits, 32)
        back = orc.dequantize_cache(q, sc3, bits, 32, "fp32")
        step = np.repeat(sc3, 32, axis=1)
        assert np.all(np.abs(back - x) <= 0.5 * step * (1 + 1e-6))


# ------------------------------------------------------------------ backbone conventions

def test_rope_is_a_rotation_and_relative():
    r = np.random.default_rng(0)
    t = r.standard_normal((5, 3, 8))
    pos = np.array([0, 1, 7, 100, 4096])
    rt = orc.rope(t, pos, 1e4)
    np.testing.assert_allclose(np.linalg.norm(rt, axis=-1), np.linalg.norm(t, axis=-1), rtol=1e-12)
    np.testing.assert_allclose(rt[0], t[0], rtol=0, atol=0)                 # position 0: identity
    # inner products depend on position differences only
    a, b = r.standard_normal((1, 1, 8)), r.standard_normal((1, 1, 8))
    d1 = np.sum(orc.rope(a, np.array([10]), 1e4) * orc.rope(b, np.array([3]), 1e4))
    d2 = np.sum(orc.rope(a, np.array([110]), 1e4) * orc.rope(b, np.array([103]), 1e4))
    assert abs(d1 - d2) < 1e-12
    # first pair (c = 0, partner hd/2) turns by exactly pos radians
    e = np.zeros((1, 1, 8)); e[0, 0, 0] = 1.0
    out = orc.rope(e, np.array([2]), 1e4)[0, 0]
    np.testing.assert_allclose([out[0], out[4]], [math.cos(2.0), math.sin(2.0)], rtol=1e-13)


def test_rmsnorm_and_silu_closed_forms():
    x = np.array([[3.0, 4.0, 0.0, 0.0]])
    u = orc.rmsnorm(x, np.array([1.0, 2.0, 1.0, 1.0]), 0.0)
    np.testing.assert_allclose(u, [[3 / 2.5, 2 * 4 / 2.5, 0, 0]], rtol=1e-14)
    assert abs(orc.silu(np.array([0.0]))[0]) == 0.0
    np.testing.assert_allclose(orc.silu(np.array([2.0])), 2.0 / (1 + math.exp(-2.0)), rtol=1e-15)


# ------------------------------------------------------------------ ridge regression ---

def rand_XR(seed, N, F, d):
    r = np.random.default_rng(seed)
    return r.standard_normal((N, F)), r.standard_normal((N, d))


@pytest.mark.parametrize("N,F,d", [(40, 12, 9), (7, 12, 9)])
def test_ridge_solution_stationarity_and_other_routes(N, F, d):
    X, R = rand_XR(3, N, F, d)
    lam = 0.37
    S_H, S_T = orc.sufficient_statistics(X, R)
    dW = orc.ridge_solve(S_H, S_T, lam)                       # [d][F]
    B = dW.T                                                  # [F][d] = G^{-1} C
    C = X.T @ R
    grad = X.T @ (X @ B - R) + lam * B                        # stationarity of Eq. 6
    assert np.linalg.norm(grad) <= 1e-10 * np.linalg.norm(C)
    # least squares on the augmented system never forms G
    A = np.vstack([X, math.sqrt(lam) * np.eye(F)])
    b = np.vstack([R, np.zeros((F, d))])
    np.testing.assert_allclose(B, np.linalg.lstsq(A, b, rcond=None)[0], rtol=1e-9, atol=1e-11)
    # dual form
    np.testing.assert_allclose(B, X.T @ np.linalg.solve(X @ X.T + lam * np.eye(N), R), rtol=1e-9, atol=1e-11)
    # paper orientation: dW = T^T H' (H'^T H' + lam I)^{-1}
    np.testing.assert_allclose(dW, R.T @ X @ np.linalg.inv(X.T @ X + lam * np.eye(F)), rtol=1e-9, atol=1e-11)
    # objective identities and optimality under perturbation
    J = lambda Bm: np.sum((X @ Bm - R) ** 2) + lam * np.sum(Bm ** 2)
    np.testing.assert_allclose(J(B), np.sum(R * R) - np.sum(C * B), rtol=1e-10)
    np.testing.assert_allclose(np.sum((R - X @ B) ** 2), np.sum(R * R) - np.sum(C * B) - lam * np.sum(B * B), rtol=1e-9)
    r = np.random.default_rng(9)
    for _ in range(5):
        assert J(B + 1e-3 * r.standard_normal(B.shape)) > J(B)


def test_ridge_single_token_rank_one_closed_form():
    X, R = rand_XR(4, 1, 10, 6)
    lam = 0.2
    S_H, S_T = orc.sufficient_statistics(X, R)
    dW = orc.ridge_solve(S_H, S_T, lam)
    want = np.outer(R[0], X[0]) / (X[0] @ X[0] + lam)
    np.testing.assert_allclose(dW, want, rtol=1e-11)


def test_ridge_large_lambda_limit_and_zero_target():
    X, R = rand_XR(5, 9, 10, 6)
    S_H, S_T = orc.sufficient_statistics(X, R)
    lam = 1e9
    gap = np.linalg.norm(lam * orc.ridge_solve(S_H, S_T, lam) - S_T)      # = O(||S_H|| / lam)
    assert gap <= 2.0 * np.linalg.norm(S_H, 2) / lam * np.linalg.norm(S_T)
    assert np.all(orc.ridge_solve(S_H, np.zeros_like(S_T), 0.1) == 0.0)
    with pytest.raises(ValueError):
        orc.ridge_solve(S_H, S_T, 0.0)


def test_statistics_chunk_additivity():
    X, R = rand_XR(6, 23, 8, 5)
    a = orc.sufficient_statistics(X, R)
    b = orc.sufficient_statistics(X, R, [0, 4, 5, 17, 23])
    np.testing.assert_allclose(a[0], b[0], rtol=1e-13)
    np.testing.assert_allclose(a[1], b[1], rtol=1e-13)
    np.testing.assert_allclose(a[1], R.T @ X, rtol=1e-13)          # S_T = T^T H' is [d][F]


def test_adaptive_lambda_is_weighted_eigenvalue_mean():
    X, _ = rand_XR(7, 6, 10, 1)
    S = X.T @ X
    ev = np.linalg.eigvalsh(S)
    lam = orc.ridge_lambda(S, 0.5)
    np.testing.assert_allclose(lam, 0.5 * np.sum(ev ** 2) / np.sum(ev), rtol=1e-10)
    assert np.trace(S) / S.shape[0] <= lam / 0.5 <= ev.max() * (1 + 1e-12)
    assert orc.ridge_lambda(S, 0.5, orc.LAMBDA_ABSOLUTE) == 0.5
    np.testing.assert_allclose(orc.ridge_lambda(S, 0.5, orc.LAMBDA_TRACE_MEAN), 0.5 * np.trace(S) / 10)
    with pytest.raises(ZeroDivisionError):
        orc.ridge_lambda(np.zeros((3, 3)), 0.1)


def test_low_rank_patch_is_the_reduced_rank_regression_optimum():
    """Appendix, low-rank patches.  On the reference set the loss of a patch B against the ridge
    patch is ||H'(dW - B)^T||_F^2 = ||(dW - B) S_H^{1/2}||_F^2, so the best rank-r B is the
    truncated SVD of dW S_H^{1/2} mapped back (Eckart-Young) -- a route that never forms the
    d x d eigenproblem the method uses."""
    r0 = np.random.default_rng(21)
    N, F, d, r = 40, 14, 9, 3
    H = r0.standard_normal((N, F)) * (0.2 + r0.random(F))
    T = r0.standard_normal((N, d)) + H @ r0.standard_normal((F, d))
    S_H, S_T = H.T @ H, T.T @ H
    dW = orc.ridge_solve(S_H, S_T, 0.3)
    U, B, dWr, ev = orc.low_rank_patch(dW, S_H, r)
    assert U.shape == (d, r) and B.shape == (r, F) and dWr.shape == (d, F)
    np.testing.assert_allclose(U.T @ U, np.eye(r), atol=1e-12)
    assert np.linalg.matrix_rank(dWr, tol=1e-9) == r
    # other route: symmetric square root by eigen-decomposition of S_H, SVD, truncate, map back
    w, Q = np.linalg.eigh(S_H)
    root, iroot = (Q * np.sqrt(w)) @ Q.T, (Q / np.sqrt(w)) @ Q.T
    Us, sv, Vt = np.linalg.svd(dW @ root, full_matrices=False)
    want = (Us[:, :r] * sv[:r]) @ Vt[:r] @ iroot
    np.testing.assert_allclose(dWr, want, rtol=1e-8, atol=1e-10)
    np.testing.assert_allclose(ev[:d], sv ** 2, rtol=1e-9, atol=1e-10)
    # what the truncation costs on the reference set is the discarded eigenvalues
    loss = np.linalg.norm(H @ (dW - dWr).T) ** 2
    np.testing.assert_allclose(loss, ev[r:].sum(), rtol=1e-9)
    # no random rank-r competitor, nor a plain (unweighted) truncated SVD of dW, does better
    for _ in range(200):
        C = dWr + 0.05 * r0.standard_normal((d, r)) @ r0.standard_normal((r, F))
        A = r0.standard_normal((d, r)) @ r0.standard_normal((r, F))
        assert np.linalg.norm(H @ (dW - A).T) ** 2 >= loss
        if np.linalg.matrix_rank(C, tol=1e-9) <= r:
            assert np.linalg.norm(H @ (dW - C).T) ** 2 >= loss * (1 - 1e-12)
    Up, sp, Vp = np.linalg.svd(dW, full_matrices=False)
    plain = (Up[:, :r] * sp[:r]) @ Vp[:r]
    assert np.linalg.norm(H @ (dW - plain).T) ** 2 > loss
    # limits: full rank returns the ridge patch, rank 0 the zero patch; the projector is idempotent
    np.testing.assert_allclose(orc.low_rank_patch(dW, S_H, d)[2], dW, rtol=1e-10, atol=1e-12)
    assert np.all(orc.low_rank_patch(dW, S_H, 0)[2] == 0.0)
    np.testing.assert_allclose(orc.low_rank_patch(dWr, S_H, r)[2], dWr, rtol=1e-8, atol=1e-11)
    # a patch that already has rank r is returned unchanged
    low = r0.standard_normal((d, r)) @ r0.standard_normal((r, F))
    np.testing.assert_allclose(orc.low_rank_patch(low, S_H, r)[2], low, rtol=1e-8, atol=1e-10)
    with pytest.raises(ValueError):
        orc.low_rank_patch(dW, S_H, d + 1)


# ------------------------------------------------------------------ block identities ---

def test_identical_caches_give_zero_target_and_zero_patch():
    cfg = tiny_cfg()
    w, K, V, x, _ = tiny_problem(cfg)
    full = [np.arange(cfg.L, dtype=np.int32)] * cfg.Hkv
    out = orc.build_patch(w, K, V, full, x, x, [0, cfg.N], cfg.L, 0.1, cfg, keep_intermediates=True)
    assert np.all(out["T"] == 0.0)
    assert np.all(out["dW"] == 0.0)
    np.testing.assert_array_equal(out["xF_next"], out["xC_next"])


def test_patched_student_block_output_gap_is_ridge_residual():
    """Eq. 4: teacher block output minus the patched student's equals T - H' dW^T, where the
    patched output is obtained by actually running the block with W + dW."""
    cfg = tiny_cfg()
    w, K, V, x, kept = tiny_problem(cfg)
    xC = x + 0.05 * np.random.default_rng(3).standard_normal(x.shape)
    chunks = [0, 5, cfg.N]
    out = orc.build_patch(w, K, V, kept, x, xC, chunks, cfg.L, 0.05, cfg, keep_intermediates=True)
    Kc, Vc = orc.gather_cache(K, V, kept)
    w2 = dict(w); w2["Wdown"] = w["Wdown"] + out["dW"]
    stu = orc.block_forward(xC, w2, Kc, Vc, chunks, cfg.L, cfg)
    tea = orc.block_forward(x, w, list(K), list(V), chunks, cfg.L, cfg)
    yF = tea["z"] + tea["h"] @ w["Wdown"].T
    yC = stu["z"] + stu["h"] @ w2["Wdown"].T
    np.testing.assert_allclose(out["xF_next"], yF, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(out["xC_next"], yC, rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(yF - yC, out["T"] - out["H"] @ out["dW"].T, rtol=1e-8, atol=1e-11)
    # the ridge-optimal residual reduction: ||T - H'dW^T||^2 = ||T||^2 - <S_T, dW> - lam ||dW||^2
    want = out["T_fro2"] - np.sum(out["S_T"] * out["dW"]) - out["lam"] * out["dW_fro"] ** 2
    np.testing.assert_allclose(out["res_fro2"], want, rtol=1e-9)
    assert out["res_fro2"] < out["T_fro2"]


def test_small_lambda_with_fewer_tokens_than_features_reproduces_teacher():
    cfg = tiny_cfg(N=6, F=24)
    w, K, V, x, kept = tiny_problem(cfg)
    out = orc.build_patch(w, K, V, kept, x, x, [0, cfg.N], cfg.L, 1e-9, cfg)
    assert out["res_fro2"] < 1e-12 * out["T_fro2"]
    np.testing.assert_allclose(out["xC_next"], out["xF_next"], rtol=1e-5, atol=1e-6)


def test_chunks_are_independent_and_restart_positions():
    cfg = tiny_cfg()
    w, K, V, x, kept = tiny_problem(cfg)
    Kc, Vc = orc.gather_cache(K, V, kept)
    both = orc.block_forward(x, w, Kc, Vc, [0, 5, cfg.N], cfg.L, cfg)
    second = orc.block_forward(x[5:], w, Kc, Vc, [0, cfg.N - 5], cfg.L, cfg)
    np.testing.assert_allclose(both["h"][5:], second["h"], rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(both["z"][5:], second["z"], rtol=1e-12, atol=1e-13)


def test_greedy_chain_over_blocks_matches_running_the_patched_model():
    """Algorithm 1 over blocks: feeding each block the states the block below produced must equal
    (a) for the teacher, the unpatched model run on the full caches, whatever was kept or patched;
    (b) for the student, the model with every patch merged so far run on the compressed caches."""
    cfg = tiny_cfg()
    nl, chunks = 3, [0, 7, 12]
    blocks = [tiny_problem(cfg, seed=10 + l) for l in range(nl)]
    x0 = blocks[0][3]

    def chain(kept_of, lam0):
        xF, xC, outs = x0, x0, []
        for l, (w, K, V, _, kept) in enumerate(blocks):
            o = orc.build_patch(w, K, V, kept_of(l, kept), xF, xC, chunks, cfg.L, lam0, cfg)
            outs.append(o)
            xF, xC = o["xF_next"], o["xC_next"]
        return xF, xC, outs

    xF, xC, outs = chain(lambda l, k: k, 0.05)
    # (a) teacher: plain forward through the unpatched blocks
    t = x0
    for w, K, V, _, _ in blocks:
        f = orc.block_forward(t, w, list(K), list(V), chunks, cfg.L, cfg)
        t = f["z"] + f["h"] @ w["Wdown"].T
    np.testing.assert_allclose(xF, t, rtol=1e-11, atol=1e-12)
    # ... and it does not depend on the kept sets or on lambda
    xF2, xC2, _ = chain(lambda l, k: [k[0][:3], k[1][2:]], 0.7)
    np.testing.assert_allclose(xF2, xF, rtol=1e-12, atol=1e-13)
    assert np.linalg.norm(xC2 - xC) > 1e-3 * np.linalg.norm(xC)
    # (b) student: forward through the patched blocks on the compressed caches
    s = x0
    for (w, K, V, _, kept), o in zip(blocks, outs):
        Kc, Vc = orc.gather_cache(K, V, kept)
        f = orc.block_forward(s, w, Kc, Vc, chunks, cfg.L, cfg)
        s = f["z"] + f["h"] @ (w["Wdown"] + o["dW"]).T
    np.testing.assert_allclose(xC, s, rtol=1e-9, atol=1e-10)
    # the patched student ends closer to the teacher than the unpatched one
    u = x0
    for w, K, V, _, kept in blocks:
        Kc, Vc = orc.gather_cache(K, V, kept)
        f = orc.block_forward(u, w, Kc, Vc, chunks, cfg.L, cfg)
        u = f["z"] + f["h"] @ w["Wdown"].T
    assert np.linalg.norm(xF - xC) < np.linalg.norm(xF - u)
    # full caches in every block: every patch is exactly zero and the streams never part
    full = [np.arange(cfg.L, dtype=np.int32)] * cfg.Hkv
    xF3, xC3, outs3 = chain(lambda l, k: full, 0.05)
    assert all(np.all(o["dW"] == 0.0) for o in outs3)
    np.testing.assert_array_equal(xF3, xC3)


def test_build_patch_rejects_bad_index_sets():
    cfg = tiny_cfg()
    w, K, V, x, kept = tiny_problem(cfg)
    for bad in ([3, 3, 5], [5, 4], [-1, 2], [0, cfg.L]):
        k2 = [np.array(bad, dtype=np.int32), kept[1]]
        assert orc.check_kept(k2, cfg.L) is not None
        with pytest.raises(IndexError):
            orc.build_patch(w, K, V, k2, x, x, [0, cfg.N], cfg.L, 0.1, cfg)
    assert orc.check_kept(kept, cfg.L) is None
    assert orc.check_kept([np.zeros(0, dtype=np.int32)] * 2, cfg.L) is None


# ------------------------------------------------------------------ merge and formats --

def test_bf16_rounding_and_merge_match_torch():
    import torch
    r = np.random.default_rng(0)
    a = (r.standard_normal(4096) * np.exp(r.uniform(-20, 20, 4096))).astype(np.float32)
    a[:4] = [1.0 + 2 ** -8, 1.0 + 3 * 2 ** -8, -(1.0 + 2 ** -8), 0.0]          # ties
    want = torch.from_numpy(a).to(torch.bfloat16).to(torch.float32).numpy()
    np.testing.assert_array_equal(orc.round_bf16(a), want)
    np.testing.assert_array_equal(gen.round_to_bf16(a), want)
    W = gen.round_to_bf16(r.standard_normal((8, 8)).astype(np.float32) * 0.02)
    dW = (r.standard_normal((8, 8)) * 1e-3).astype(np.float32)
    want = (torch.from_numpy(W) + torch.from_numpy(dW)).to(torch.bfloat16).to(torch.float32).numpy()
    np.testing.assert_array_equal(orc.merge(W, dW, "bf16"), want)
    np.testing.assert_array_equal(orc.merge(W, dW, "fp32"), W + dW)


def test_oracle_reproduces_its_stored_values_on_config1():
    """Drift guard, not a pin: the stored numbers are the oracle's own (the paper prints none), written by
    tests/golden/make_oracle_fixture.py.  An unintended change of the oracle or of the input recipe shows here."""
    import importlib.util
    import os
    here = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")
    spec = importlib.util.spec_from_file_location("make_oracle_fixture", os.path.join(here, "make_oracle_fixture.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    stored = {}
    for line in open(os.path.join(here, "config1_oracle.txt")):
        if line.startswith("#") or not line.strip():
            continue
        name, v = line.rstrip("\n").split("\t")
        stored[name] = float(v)
    now = dict(mod.values())
    assert set(now) == set(stored)
    for name, v in now.items():
        np.testing.assert_allclose(v, stored[name], rtol=1e-9, err_msg=name)

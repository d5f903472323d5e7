"""CUDA path vs the fp64 oracle, element by element on the same seeded inputs, through the C ABI.

Tolerances: attention outputs max relative error <= 2e-2 (relative to max|a| per head), dW relative
Frobenius error <= 5e-3, index handling / compaction / merge bit-exact."""
import numpy as np
import pytest

from oracle import pkv_oracle as orc
from paper_2609_39329_b200 import inputs as gen
from tests import helpers as H

pytestmark = pytest.mark.gpu

ATTN_TOL = 2e-2
DW_TOL = 5e-3


@pytest.fixture(scope="module")
def B():
    import torch
    from paper_2609_39329_b200 import binding
    assert torch.cuda.is_available()
    binding.lib()
    return binding


def small_cfg(dtype="bf16", **kw):
    base = gen.benchmark_config(2)
    d = dict(dtype=dtype, d=256, Hq=8, Hkv=2, hd=64, F=192, L=1000, N=70, window=16, budget=100, n_obs=8,
             name="small")
    d.update(kw)
    return gen.scaled_config(base, **d)


def engines(B, cfg):
    """Engines a config must be checked on: fp32 -> SIMT; bf16 -> tensor-core path and SIMT."""
    if cfg.dtype == "fp32":
        return [B.ENGINE_SIMT]
    return [B.ENGINE_AUTO, B.ENGINE_SIMT]


def gpu_build(B, cfg, lay, xF, xC, chunk_off, lam0, engine, mode=0, kv_split=0, want_next=True, solver=0, refine=0):
    import torch
    ctx = B.PkvContext(B.dims_from_config(cfg, N_max=xF.shape[0], b_max=max(len(k) for k in lay["kept"])),
                       engine=engine, kv_split=kv_split, solver=solver)
    if refine:
        ctx.set_refinement(refine)
    w = B.to_device(lay["weights"], cfg.dtype)
    kv = B.to_device({"K": lay["K"], "V": lay["V"]}, cfg.dtype)
    off, idx = gen.kept_to_csr(lay["kept"])
    idx_t = torch.from_numpy(idx).cuda() if len(idx) else None
    xF_t = torch.from_numpy(np.ascontiguousarray(xF, dtype=np.float32)).cuda()
    xC_t = xF_t if xC is xF else torch.from_numpy(np.ascontiguousarray(xC, dtype=np.float32)).cuda()
    if idx_t is None:   # empty compressed cache: explicit form with zero rows
        dummy = torch.zeros((1, cfg.hd), dtype=kv["K"].dtype, device="cuda")
        out = ctx.build_patch(w, kv["K"], kv["V"], off, None, xF_t, xC_t, chunk_off, cfg.L, lam0, mode, want_next,
                              Kc=dummy, Vc=dummy)
    else:
        out = ctx.build_patch(w, kv["K"], kv["V"], off, idx_t, xF_t, xC_t, chunk_off, cfg.L, lam0, mode, want_next)
    res = {k: (v.cpu().numpy() if hasattr(v, "cpu") else v) for k, v in out.items()}
    res["launches"] = ctx.launch_count()
    ctx.close()
    return res


def check_build(B, cfg, lay, xF, xC, chunk_off, lam0, engine, mode=0, kv_split=0, solver=0):
    ref = H.run_oracle(cfg, lay, xF, xC, chunk_off, lam0, mode)
    got = gpu_build(B, cfg, lay, xF, xC, chunk_off, lam0, engine, mode, kv_split, solver=solver)
    e_dw = H.rel_fro(got["dW"], ref["dW"])
    assert e_dw <= DW_TOL, "dW rel fro %.3e" % e_dw
    np.testing.assert_allclose(got["stats"]["lambda_eff"], ref["lam"], rtol=2e-3)
    np.testing.assert_allclose(got["stats"]["trace"], ref["tr"], rtol=2e-3)
    assert H.rel_fro(got["xF_next"], ref["xF_next"]) <= 1e-3
    assert H.rel_fro(got["xC_next"], ref["xC_next"]) <= 1e-3
    # the gap between the next states is the ridge residual (Eq. 4); compare it on its own scale
    gap_ref = ref["xF_next"] - ref["xC_next"]
    assert H.rel_fro(got["xF_next"].astype(np.float64) - got["xC_next"], gap_ref) <= 2e-2
    np.testing.assert_allclose(got["stats"]["target_fro2"], ref["T_fro2"], rtol=2e-2)
    assert got["launches"] > 0
    return e_dw


# ------------------------------------------------------------------ S0 + merge: bit-exact

@pytest.mark.parametrize("dtype", ["bf16", "fp32"])
def test_gather_kept_bit_exact_and_bad_sets_reported(B, dtype):
    import torch
    cfg = small_cfg(dtype, hd=128, Hq=6, Hkv=3, L=777)
    r = np.random.default_rng(0)
    K = gen._to_dtype(r.standard_normal((cfg.Hkv, cfg.L, cfg.hd)).astype(np.float32), dtype)
    V = gen._to_dtype(r.standard_normal((cfg.Hkv, cfg.L, cfg.hd)).astype(np.float32), dtype)
    kept = [np.sort(r.choice(cfg.L, size=b, replace=False)).astype(np.int32) for b in (100, 0, 37)]
    kept[2][-1] = cfg.L - 1
    kept[0][0] = 0
    off, idx = gen.kept_to_csr(kept)
    ctx = B.PkvContext(B.dims_from_config(cfg, b_max=100), engine=B.ENGINE_SIMT)
    kv = B.to_device({"K": K, "V": V}, dtype)
    Kc, Vc = ctx.gather_kept(kv["K"], kv["V"], off, torch.from_numpy(idx).cuda())
    Ko, Vo = orc.gather_cache(K, V, kept)
    np.testing.assert_array_equal(Kc.float().cpu().numpy(), np.concatenate(Ko))
    np.testing.assert_array_equal(Vc.float().cpu().numpy(), np.concatenate(Vo))
    # invalid sets: duplicate, descending, negative, == L; the first offender is reported
    for pos, val in ((5, int(idx[4])), (50, int(idx[49]) - 1), (0, -1), (136, cfg.L)):
        bad = idx.copy()
        bad[pos] = val
        badk = [bad[off[h]:off[h + 1]] for h in range(cfg.Hkv)]
        want = orc.check_kept(badk, cfg.L)
        with pytest.raises(B.PkvError) as ei:
            ctx.gather_kept(kv["K"], kv["V"], off, torch.from_numpy(bad).cuda())
        assert ei.value.code == -3 and tuple(ei.value.info) == want
    # the context stays usable after an error
    Kc2, _ = ctx.gather_kept(kv["K"], kv["V"], off, torch.from_numpy(idx).cuda())
    assert torch.equal(Kc, Kc2)
    ctx.close()


@pytest.mark.parametrize("dtype", ["bf16", "fp32"])
def test_merge_bit_exact(B, dtype):
    import torch
    r = np.random.default_rng(1)
    n = (130, 77)      # 10010 entries: not a multiple of the vector width
    W = gen._to_dtype((r.standard_normal(n) * 0.02).astype(np.float32), dtype)
    dW = (r.standard_normal(n) * 1e-3).astype(np.float32)
    want = orc.merge(W, dW, dtype)
    cfg = small_cfg(dtype)
    ctx = B.PkvContext(B.dims_from_config(cfg), engine=B.ENGINE_SIMT)
    Wt = torch.from_numpy(W).cuda().to(torch.bfloat16 if dtype == "bf16" else torch.float32)
    ctx.merge(Wt, torch.from_numpy(dW).cuda())
    torch.cuda.synchronize()
    np.testing.assert_array_equal(Wt.float().cpu().numpy(), want)
    ctx.close()


# ------------------------------------------------------------------ S3 alone

def attention_case(B, cfg, engine, chunk_off, budgets, kv_split=0, seed=0):
    import torch
    r = np.random.default_rng(seed)
    N = chunk_off[-1]
    q = r.standard_normal((2, N, cfg.Hq, cfg.hd)).astype(np.float32) * 1.3
    k = r.standard_normal((2, N, cfg.Hkv, cfg.hd)).astype(np.float32)
    v = r.standard_normal((2, N, cfg.Hkv, cfg.hd)).astype(np.float32)
    kvd = gen.gen_cache(cfg, 0) if cfg.dtype == "bf16" else {
        "K": r.standard_normal((cfg.Hkv, cfg.L, cfg.hd)).astype(np.float32),
        "V": r.standard_normal((cfg.Hkv, cfg.L, cfg.hd)).astype(np.float32)}
    kept = gen.select_kept(gen.scaled_config(cfg, kept_rule="random"), 0, per_head_budget=budgets)
    Kg, Vg = orc.gather_cache(kvd["K"], kvd["V"], kept)
    aF = orc.attention(q[0], k[0], v[0], list(kvd["K"]), list(kvd["V"]), chunk_off)
    aC = orc.attention(q[1], k[1], v[1], Kg, Vg, chunk_off)
    ctx = B.PkvContext(B.dims_from_config(cfg, N_max=N, b_max=max(max(budgets), 1)), engine=engine, kv_split=kv_split)
    kv = B.to_device({"K": kvd["K"], "V": kvd["V"]}, cfg.dtype)
    off, idx = gen.kept_to_csr(kept)
    tq, tk, tv = (torch.from_numpy(t.reshape(2, N, -1)).cuda() for t in (q, k, v))
    if len(idx):
        gF, gC, gD = ctx.attention(tq, tk, tv, kv["K"], kv["V"], off, torch.from_numpy(idx).cuda(), chunk_off)
    else:
        dummy = torch.zeros((1, cfg.hd), dtype=kv["K"].dtype, device="cuda")
        gF, gC, gD = ctx.attention(tq, tk, tv, kv["K"], kv["V"], off, None, chunk_off, Kc=dummy, Vc=dummy)
    gF, gC, gD = (t.cpu().numpy() for t in (gF, gC, gD))
    ctx.close()
    assert H.attn_max_rel(gF, aF, cfg.Hq, cfg.hd) <= ATTN_TOL
    assert H.attn_max_rel(gC, aC, cfg.Hq, cfg.hd) <= ATTN_TOL
    assert H.attn_max_rel(gD, aF - aC, cfg.Hq, cfg.hd) <= ATTN_TOL
    np.testing.assert_array_equal(gD, gF - gC)
    return gF, aF


@pytest.mark.parametrize("dtype,hd", [("bf16", 128), ("bf16", 64), ("fp32", 64)])
def test_attention_parity_ragged_chunks_and_splits(B, dtype, hd):
    cfg = small_cfg(dtype, hd=hd, Hq=8, Hkv=2, L=1500)
    for engine in engines(B, cfg):
        attention_case(B, cfg, engine, [0, 70], [100, 100])
        attention_case(B, cfg, engine, [0, 13, 14, 70, 131], [257, 31], kv_split=256)   # ragged heads, 4 chunks
        attention_case(B, cfg, engine, [0, 33], [0, 0])                                  # empty compressed cache


def test_attention_group_of_seven_and_odd_lengths(B):
    cfg = small_cfg("bf16", hd=128, Hq=14, Hkv=2, L=1237)
    for engine in engines(B, cfg):
        attention_case(B, cfg, engine, [0, 45], [19, 123], kv_split=320)


# ------------------------------------------------------------------ explicit compact cache with per-key bias

def explicit_cache(cfg, budgets, seed):
    """A compact cache that is not a subset of the full one (an approximation-style compressor refits keys and
    values and attaches one additive logit term per key): per-head lists plus the packed device layout."""
    r = np.random.default_rng(seed)
    Kc = [gen._to_dtype(r.standard_normal((b, cfg.hd)).astype(np.float32), cfg.dtype) for b in budgets]
    Vc = [gen._to_dtype(r.standard_normal((b, cfg.hd)).astype(np.float32), cfg.dtype) for b in budgets]
    bias = [r.uniform(-2.0, 2.0, b).astype(np.float32) for b in budgets]
    off = np.zeros(len(budgets) + 1, dtype=np.int32)
    off[1:] = np.cumsum(budgets)
    return Kc, Vc, bias, off


def pack_explicit(B, cfg, Kc, Vc, bias):
    import torch
    wd = torch.bfloat16 if cfg.dtype == "bf16" else torch.float32
    tK = torch.from_numpy(np.concatenate(Kc)).cuda().to(wd).contiguous()
    tV = torch.from_numpy(np.concatenate(Vc)).cuda().to(wd).contiguous()
    tb = torch.from_numpy(np.concatenate(bias)).cuda().contiguous()
    return tK, tV, tb


@pytest.mark.parametrize("dtype,hd", [("bf16", 128), ("bf16", 64), ("fp32", 64)])
def test_attention_with_explicit_cache_and_finite_key_bias(B, dtype, hd):
    """Student stream against an explicit K', V' with ragged heads and a finite bias on every cached key
    (Sec. 3.1, approximation compressors), through pkv_attention, against the oracle; the teacher stream
    and the difference dA keep their meaning.  A second call without the bias must differ."""
    import torch
    cfg = small_cfg(dtype, hd=hd, Hq=8, Hkv=2, L=900)
    r = np.random.default_rng(21)
    chunk_off = [0, 13, 70, 131]
    N = chunk_off[-1]
    budgets = [257, 31]
    q = r.standard_normal((2, N, cfg.Hq, cfg.hd)).astype(np.float32) * 1.3
    k = r.standard_normal((2, N, cfg.Hkv, cfg.hd)).astype(np.float32)
    v = r.standard_normal((2, N, cfg.Hkv, cfg.hd)).astype(np.float32)
    kvd = gen.gen_cache(cfg, 0) if dtype == "bf16" else {
        "K": r.standard_normal((cfg.Hkv, cfg.L, cfg.hd)).astype(np.float32),
        "V": r.standard_normal((cfg.Hkv, cfg.L, cfg.hd)).astype(np.float32)}
    Kc, Vc, bias, off = explicit_cache(cfg, budgets, 22)
    aF = orc.attention(q[0], k[0], v[0], list(kvd["K"]), list(kvd["V"]), chunk_off)
    aC = orc.attention(q[1], k[1], v[1], Kc, Vc, chunk_off, key_bias=bias)
    aC_nobias = orc.attention(q[1], k[1], v[1], Kc, Vc, chunk_off)
    assert H.attn_max_rel(aC_nobias, aC, cfg.Hq, cfg.hd) > 10 * ATTN_TOL      # the bias matters on this input
    for engine in engines(B, cfg):
        ctx = B.PkvContext(B.dims_from_config(cfg, N_max=N, b_max=max(budgets)), engine=engine, kv_split=256)
        kv = B.to_device({"K": kvd["K"], "V": kvd["V"]}, cfg.dtype)
        tK, tV, tb = pack_explicit(B, cfg, Kc, Vc, bias)
        tq, tk, tv = (torch.from_numpy(t.reshape(2, N, -1)).cuda() for t in (q, k, v))
        gF, gC, gD = (t.cpu().numpy() for t in
                      ctx.attention(tq, tk, tv, kv["K"], kv["V"], off, None, chunk_off, Kc=tK, Vc=tV, bias=tb))
        eF, eC = H.attn_max_rel(gF, aF, cfg.Hq, cfg.hd), H.attn_max_rel(gC, aC, cfg.Hq, cfg.hd)
        print("explicit cache + bias, %s hd %d engine %d: aF err %.2e, aC err %.2e" % (dtype, hd, engine, eF, eC))
        assert eF <= ATTN_TOL and eC <= ATTN_TOL
        assert H.attn_max_rel(gD, aF - aC, cfg.Hq, cfg.hd) <= ATTN_TOL
        np.testing.assert_array_equal(gD, gF - gC)
        _, gC0, _ = ctx.attention(tq, tk, tv, kv["K"], kv["V"], off, None, chunk_off, Kc=tK, Vc=tV)
        assert H.attn_max_rel(gC0.cpu().numpy(), aC_nobias, cfg.Hq, cfg.hd) <= ATTN_TOL
        ctx.close()


@pytest.mark.parametrize("hd,Hq,Hkv", [(64, 8, 2), (128, 4, 2)])
def test_block_with_explicit_cache_and_key_bias_matches_oracle(B, hd, Hq, Hkv):
    """pkv_build_patch with the compressed cache given explicitly (K', V', bias) instead of a kept-index set."""
    import torch
    cfg = small_cfg("bf16", hd=hd, Hq=Hq, Hkv=Hkv, d=256, F=192, L=1000, N=150)
    lay = H.make_problem(cfg)
    budgets = [100, 37]
    Kc, Vc, bias, off = explicit_cache(cfg, budgets, 23)
    xF = lay["x0"]
    xC = (xF + 0.02 * np.random.default_rng(5).standard_normal(xF.shape)).astype(np.float32)
    chunk_off = [0, 40, 150]
    ref = orc.build_patch(lay["weights"], lay["K"], lay["V"], None, xF, xC, chunk_off, cfg.L, 0.1, cfg,
                          compressed=(Kc, Vc, bias))
    ref0 = orc.build_patch(lay["weights"], lay["K"], lay["V"], None, xF, xC, chunk_off, cfg.L, 0.1, cfg,
                           compressed=(Kc, Vc, None))
    assert H.rel_fro(ref0["dW"], ref["dW"]) > 10 * DW_TOL                     # the bias matters on this input
    for engine in engines(B, cfg):
        ctx = B.PkvContext(B.dims_from_config(cfg, N_max=cfg.N, b_max=max(budgets)), engine=engine)
        w = B.to_device(lay["weights"], cfg.dtype)
        kv = B.to_device({"K": lay["K"], "V": lay["V"]}, cfg.dtype)
        tK, tV, tb = pack_explicit(B, cfg, Kc, Vc, bias)
        xF_t, xC_t = torch.from_numpy(xF).cuda(), torch.from_numpy(xC).cuda()
        out = ctx.build_patch(w, kv["K"], kv["V"], off, None, xF_t, xC_t, chunk_off, cfg.L, 0.1, Kc=tK, Vc=tV, bias=tb)
        err = H.rel_fro(out["dW"].cpu().numpy(), ref["dW"])
        print("block with explicit cache + bias, hd %d engine %d: dW rel fro err %.3e" % (hd, engine, err))
        assert err <= DW_TOL
        assert H.rel_fro(out["xC_next"].cpu().numpy(), ref["xC_next"]) <= 1e-3
        ctx.close()


@pytest.mark.parametrize("dtype,hd,bits", [("bf16", 128, 8), ("bf16", 128, 4), ("bf16", 64, 4), ("fp32", 64, 8)])
def test_quantised_compact_cache_decode_bit_exact_and_attention(B, dtype, hd, bits):
    """INT8 / INT4 compact cache with group scales (appendix, quantised caches): the decode in the student's load
    path is bit-exact against the oracle's, and attention on the quantised cache matches the oracle's attention on
    the decoded cache; a finite key bias rides along."""
    import torch
    cfg = small_cfg(dtype, hd=hd, Hq=8, Hkv=2, L=700)
    r = np.random.default_rng(41)
    budgets, group = [150, 33], 32
    off = np.zeros(3, dtype=np.int32)
    off[1:] = np.cumsum(budgets)
    Kraw = r.standard_normal((sum(budgets), hd)).astype(np.float32) * np.exp(r.uniform(-1, 1, hd)).astype(np.float32)
    Vraw = r.standard_normal((sum(budgets), hd)).astype(np.float32)
    Kq, Ks = gen.quantize_rows(Kraw, bits, group)
    Vq, Vs = gen.quantize_rows(Vraw, bits, group)
    Kd = orc.dequantize_cache(Kq, Ks, bits, group, dtype)
    Vd = orc.dequantize_cache(Vq, Vs, bits, group, dtype)
    bias = r.uniform(-1.0, 1.0, sum(budgets)).astype(np.float32)
    chunk_off = [0, 40, 97]
    N = chunk_off[-1]
    q = r.standard_normal((2, N, cfg.Hq, hd)).astype(np.float32) * 1.3
    k = r.standard_normal((2, N, cfg.Hkv, hd)).astype(np.float32)
    v = r.standard_normal((2, N, cfg.Hkv, hd)).astype(np.float32)
    kvd = gen.gen_cache(cfg, 0) if dtype == "bf16" else {
        "K": r.standard_normal((cfg.Hkv, cfg.L, hd)).astype(np.float32),
        "V": r.standard_normal((cfg.Hkv, cfg.L, hd)).astype(np.float32)}
    split = lambda a: [a[off[h]:off[h + 1]] for h in range(cfg.Hkv)]
    aC = orc.attention(q[1], k[1], v[1], split(Kd), split(Vd), chunk_off, key_bias=split(bias))
    quant = {"k_scale": torch.from_numpy(Ks).cuda(), "v_scale": torch.from_numpy(Vs).cuda(), "bits": bits, "group": group}
    tKq, tVq = torch.from_numpy(Kq).cuda(), torch.from_numpy(Vq).cuda()
    for engine in engines(B, cfg):
        ctx = B.PkvContext(B.dims_from_config(cfg, N_max=N, b_max=max(budgets)), engine=engine)
        gK, gV = ctx.dequant_cache(off, tKq, tVq, quant)
        np.testing.assert_array_equal(gK.float().cpu().numpy(), Kd)
        np.testing.assert_array_equal(gV.float().cpu().numpy(), Vd)
        kv = B.to_device({"K": kvd["K"], "V": kvd["V"]}, cfg.dtype)
        tq, tk, tv = (torch.from_numpy(t.reshape(2, N, -1)).cuda() for t in (q, k, v))
        _, gC, _ = ctx.attention(tq, tk, tv, kv["K"], kv["V"], off, None, chunk_off, Kc=tKq, Vc=tVq,
                                 bias=torch.from_numpy(bias).cuda(), quant=quant)
        e = H.attn_max_rel(gC.cpu().numpy(), aC, cfg.Hq, hd)
        print("quantised cache, %s hd %d int%d engine %d: aC err %.2e" % (dtype, hd, bits, engine, e))
        assert e <= ATTN_TOL
        # malformed descriptions are refused
        bad = dict(quant, group=12)
        with pytest.raises(B.PkvError) as ei:
            ctx.dequant_cache(off, tKq, tVq, bad)
        assert ei.value.code == -2
        ctx.close()


def test_block_with_int4_compact_cache_matches_oracle(B):
    """pkv_build_patch against an INT4 compact cache: the patch is the oracle's patch for the decoded cache."""
    import torch
    cfg = small_cfg("bf16", hd=128, Hq=4, Hkv=2, d=256, F=192, L=1000, N=120)
    lay = H.make_problem(cfg)
    # the compact cache is a quantised copy of the kept rows of the full cache
    Kg, Vg = orc.gather_cache(lay["K"], lay["V"], lay["kept"])
    off, _ = gen.kept_to_csr(lay["kept"])
    Kq, Ks = gen.quantize_rows(np.concatenate(Kg), 4, 32)
    Vq, Vs = gen.quantize_rows(np.concatenate(Vg), 4, 32)
    Kd = orc.dequantize_cache(Kq, Ks, 4, 32, "bf16")
    Vd = orc.dequantize_cache(Vq, Vs, 4, 32, "bf16")
    split = lambda a: [a[off[h]:off[h + 1]] for h in range(cfg.Hkv)]
    x = lay["x0"]
    ref = orc.build_patch(lay["weights"], lay["K"], lay["V"], None, x, x, [0, cfg.N], cfg.L, 0.1, cfg,
                          compressed=(split(Kd), split(Vd), None))
    exact = H.run_oracle(cfg, lay, x, x, [0, cfg.N], 0.1)
    assert H.rel_fro(exact["dW"], ref["dW"]) > 10 * DW_TOL          # quantisation changes the patch: it must be seen
    ctx = B.PkvContext(B.dims_from_config(cfg, b_max=max(len(k) for k in lay["kept"])), engine=B.ENGINE_AUTO)
    w = B.to_device(lay["weights"], cfg.dtype)
    kv = B.to_device({"K": lay["K"], "V": lay["V"]}, cfg.dtype)
    quant = {"k_scale": torch.from_numpy(Ks).cuda(), "v_scale": torch.from_numpy(Vs).cuda(), "bits": 4, "group": 32}
    xt = torch.from_numpy(x).cuda()
    out = ctx.build_patch(w, kv["K"], kv["V"], off, None, xt, xt, [0, cfg.N], cfg.L, 0.1,
                          Kc=torch.from_numpy(Kq).cuda(), Vc=torch.from_numpy(Vq).cuda(), quant=quant)
    err = H.rel_fro(out["dW"].cpu().numpy(), ref["dW"])
    print("block with INT4 compact cache: dW rel fro err %.3e" % err)
    assert err <= DW_TOL
    ctx.close()


# ------------------------------------------------------------------ S7, S8 alone

@pytest.mark.parametrize("n,F,d", [(70, 192, 256), (300, 256, 128)])
def test_gram_parity_and_accumulation(B, n, F, d):
    import torch
    cfg = small_cfg("bf16", F=F, d=d, Hq=d // 64, Hkv=1, N=n)
    r = np.random.default_rng(2)
    X = (r.standard_normal((n, F)) * np.exp(r.uniform(-1, 1, F))).astype(np.float32)
    R = (r.standard_normal((n, d)) * 0.1).astype(np.float32)
    S_H, S_T = orc.sufficient_statistics(X, R)
    for engine in engines(B, cfg):
        ctx = B.PkvContext(B.dims_from_config(cfg, N_max=n), engine=engine)
        Xt, Rt = torch.from_numpy(X).cuda(), torch.from_numpy(R).cuda()
        gH, gT = ctx.gram(Xt, Rt)
        assert H.rel_fro(gH.cpu().numpy(), S_H) <= 2e-4
        assert H.rel_fro(gT.cpu().numpy(), S_T) <= 2e-4
        # Eq. 9: running sums over chunks
        h = n // 3
        aH, aT = ctx.gram(Xt[:h].contiguous(), Rt[:h].contiguous())
        ctx.gram(Xt[h:].contiguous(), Rt[h:].contiguous(), aH, aT, accumulate=True)
        assert H.rel_fro(aH.cpu().numpy(), S_H) <= 2e-4
        assert H.rel_fro(aT.cpu().numpy(), S_T) <= 2e-4
        ctx.close()


@pytest.mark.parametrize("F,d,n", [(192, 256, 70), (200, 64, 500), (64, 64, 10)])
def test_ridge_solve_parity_modes_and_errors(B, F, d, n):
    import torch
    cfg = small_cfg("bf16", F=F, d=d, Hq=max(d // 64, 1), Hkv=1)
    r = np.random.default_rng(3)
    X = r.standard_normal((n, F))
    R = r.standard_normal((n, d))
    S_H, S_T = orc.sufficient_statistics(X, R)
    for engine in engines(B, cfg):
        ctx = B.PkvContext(B.dims_from_config(cfg), engine=engine)
        tH = torch.from_numpy(S_H.astype(np.float32)).cuda()
        tT = torch.from_numpy(S_T.astype(np.float32)).cuda()
        for mode, lam0 in ((B.LAMBDA_PAPER, 0.1), (B.LAMBDA_PAPER, 1e-3), (B.LAMBDA_ABSOLUTE, 5.0),
                           (B.LAMBDA_TRACE_MEAN, 0.1)):
            lam = orc.ridge_lambda(S_H, lam0, mode)
            want = orc.ridge_solve(S_H, S_T, lam)
            dW, st = ctx.ridge_solve(tH, tT, lam0, mode)
            assert H.rel_fro(dW.cpu().numpy(), want) <= 1e-3, (mode, lam0)
            np.testing.assert_allclose(st["lambda_eff"], lam, rtol=1e-4)
            np.testing.assert_allclose(st["dW_fro2"], np.sum(want * want), rtol=2e-3)
            assert st["min_pivot"] > 0
            # the reported bounds bracket the condition number of the ridge matrix
            ev = np.linalg.eigvalsh(S_H + lam * np.eye(F))
            cond = ev[-1] / ev[0]
            assert st["cond_lower_bound"] <= cond * (1 + 1e-3) and cond <= st["cond_upper_bound"] * (1 + 1e-3), (mode, lam0)
            assert st["cond_warning"] == 0
        # a ridge far below the spectrum of a rank-deficient S_H (n < F): flagged, the patch is still returned
        if n < F:
            dW, st = ctx.ridge_solve(tH, tT, 2e-3, B.LAMBDA_ABSOLUTE)
            assert st["cond_warning"] == 1 and st["cond_lower_bound"] > 1e4 and torch.isfinite(dW).all()
        # not positive definite: a negative diagonal entry that the ridge does not lift
        bad = S_H.astype(np.float32).copy()
        bad[5, 5] = -1e6
        with pytest.raises(B.PkvError) as ei:
            ctx.ridge_solve(torch.from_numpy(bad).cuda(), tT, 1e-3, B.LAMBDA_ABSOLUTE)
        assert ei.value.code == -4 and ei.value.info["err_info"][0] == 5
        with pytest.raises(B.PkvError) as ei:
            ctx.ridge_solve(torch.zeros_like(tH), tT, 0.1, B.LAMBDA_PAPER)
        assert ei.value.code == -5
        with pytest.raises(B.PkvError) as ei:
            ctx.ridge_solve(tH, tT, 0.0, B.LAMBDA_PAPER)
        assert ei.value.code == -1
        dW, _ = ctx.ridge_solve(tH, tT, 0.1, B.LAMBDA_PAPER)      # still usable
        assert torch.isfinite(dW).all()
        ctx.close()


def ill_conditioned_statistics(F, d, n, seed=5):
    r = np.random.default_rng(seed)
    S_H, S_T = orc.sufficient_statistics(r.standard_normal((n, F)), r.standard_normal((n, d)))
    # what the device is handed is the fp32 rounding; the oracle solves exactly that system in fp64
    return S_H.astype(np.float32), S_T.astype(np.float32)


def test_iterative_refinement_for_a_small_absolute_ridge(B):
    """Eq. 6 with lambda as written (absolute mode) on a rank-deficient S_H (n < F): cond(G) = 4.6e4, the plain
    fp32-equivalent solve misses the 5e-3 tolerance, one correction brings it inside; the reported residual norm falls
    from step to step; zero steps is the plain solve bit for bit."""
    import torch
    F = d = 2048
    cfg = small_cfg("bf16", F=F, d=d, Hq=16, Hkv=2, hd=128, N=64)
    S_H, S_T = ill_conditioned_statistics(F, d, 512)
    want = orc.ridge_solve(S_H.astype(np.float64), S_T.astype(np.float64), 0.1)
    ctx = B.PkvContext(B.dims_from_config(cfg), engine=B.ENGINE_AUTO)
    tH, tT = torch.from_numpy(S_H).cuda(), torch.from_numpy(S_T).cuda()
    plain, st0 = ctx.ridge_solve(tH, tT, 0.1, B.LAMBDA_ABSOLUTE)
    assert st0["cond_warning"] == 1
    errs, resid = [H.rel_fro(plain.cpu().numpy(), want)], []
    for steps in (1, 2):
        dW, st = ctx.ridge_solve(tH, tT, 0.1, B.LAMBDA_ABSOLUTE, refine_steps=steps)
        errs.append(H.rel_fro(dW.cpu().numpy(), want))
        resid.append(np.sqrt(st["resid_fro2"]) / np.linalg.norm(S_T))
        np.testing.assert_allclose(st["dW_fro2"], np.sum(want * want), rtol=1e-2)
    print("refinement at cond 4.6e4: error %.2e -> %.2e -> %.2e, residual before the last step %.1e, %.1e" %
          (errs[0], errs[1], errs[2], resid[0], resid[1]))
    assert errs[0] > DW_TOL > errs[1] and errs[1] <= errs[0] / 4 and errs[2] <= DW_TOL
    assert resid[1] < resid[0] / 4
    # the context's own setting applies the same correction to a plain solve call; switched off again it is gone
    ctx.set_refinement(1)
    dW1, _ = ctx.ridge_solve(tH, tT, 0.1, B.LAMBDA_ABSOLUTE)
    assert H.rel_fro(dW1.cpu().numpy(), want) <= DW_TOL
    ctx.set_refinement(0)
    again, _ = ctx.ridge_solve(tH, tT, 0.1, B.LAMBDA_ABSOLUTE)
    assert torch.equal(again, plain)
    with pytest.raises(B.PkvError):
        ctx.set_refinement(9)
    ctx.close()
    # well conditioned (Eq. 7, lambda0 = 0.1): refinement changes nothing that matters
    S_H, S_T = ill_conditioned_statistics(448, 256, 900, seed=6)
    cfg = small_cfg("bf16", F=448, d=256, Hq=4, Hkv=1)
    ctx = B.PkvContext(B.dims_from_config(cfg), engine=B.ENGINE_AUTO)
    lam = orc.ridge_lambda(S_H.astype(np.float64), 0.1, B.LAMBDA_PAPER)
    want = orc.ridge_solve(S_H.astype(np.float64), S_T.astype(np.float64), lam)
    for steps in (0, 1):
        dW, _ = ctx.ridge_solve(torch.from_numpy(S_H).cuda(), torch.from_numpy(S_T).cuda(), 0.1, B.LAMBDA_PAPER,
                                refine_steps=steps)
        assert H.rel_fro(dW.cpu().numpy(), want) <= 1e-4, steps
    ctx.close()
    simt = B.PkvContext(B.dims_from_config(cfg), engine=B.ENGINE_SIMT)
    with pytest.raises(B.PkvError) as ei:
        simt.set_refinement(1)
    assert ei.value.code == -2
    simt.close()


def test_solve_with_more_operand_sets_than_cached_graphs(B):
    """The solve is replayed from a graph captured per operand set, a few of which are kept: six different S_T
    buffers in turn (older graphs are dropped), then the first again, each against the oracle; the result address
    changes from call to call as well."""
    import torch
    F, d, n = 320, 256, 90
    cfg = small_cfg("bf16", F=F, d=d, Hq=4, Hkv=1)
    r = np.random.default_rng(11)
    X = r.standard_normal((n, F))
    S_H, _ = orc.sufficient_statistics(X, r.standard_normal((n, d)))
    lam = orc.ridge_lambda(S_H, 0.1, B.LAMBDA_PAPER)
    ctx = B.PkvContext(B.dims_from_config(cfg), engine=B.ENGINE_AUTO)
    tH = torch.from_numpy(S_H.astype(np.float32)).cuda()
    sets = []
    for i in range(6):
        _, S_T = orc.sufficient_statistics(X, r.standard_normal((n, d)))
        sets.append((S_T, torch.from_numpy(S_T.astype(np.float32)).cuda()))
    for i in list(range(6)) + [0, 3]:
        S_T, tT = sets[i]
        dW, _ = ctx.ridge_solve(tH, tT, 0.1, B.LAMBDA_PAPER)
        assert H.rel_fro(dW.cpu().numpy(), orc.ridge_solve(S_H, S_T, lam)) <= 1e-3, i
    ctx.close()


def test_standalone_solve_after_a_build_uses_the_callers_statistics(B):
    """A build leaves its own S_T split into bf16 parts inside the context; a later pkv_ridge_solve must take the
    S_T it is handed."""
    import torch
    cfg = small_cfg("bf16", hd=128, Hq=4, Hkv=2, d=256, F=192, L=600, N=64)
    lay = H.make_problem(cfg)
    ctx = B.PkvContext(B.dims_from_config(cfg, b_max=max(len(k) for k in lay["kept"])), engine=B.ENGINE_AUTO)
    w = B.to_device(lay["weights"], cfg.dtype)
    kv = B.to_device({"K": lay["K"], "V": lay["V"]}, cfg.dtype)
    off, idx = gen.kept_to_csr(lay["kept"])
    xt = torch.from_numpy(lay["x0"]).cuda()
    ctx.build_patch(w, kv["K"], kv["V"], off, torch.from_numpy(idx).cuda(), xt, xt, [0, cfg.N], cfg.L, 0.1)
    r = np.random.default_rng(31)
    X, R = r.standard_normal((90, cfg.F)), r.standard_normal((90, cfg.d))
    S_H, S_T = orc.sufficient_statistics(X, R)
    want = orc.ridge_solve(S_H, S_T, orc.ridge_lambda(S_H, 0.1))
    dW, _ = ctx.ridge_solve(torch.from_numpy(S_H.astype(np.float32)).cuda(), torch.from_numpy(S_T.astype(np.float32)).cuda(), 0.1)
    assert H.rel_fro(dW.cpu().numpy(), want) <= 1e-3
    ctx.close()


@pytest.mark.parametrize("M,N,K", [(200, 136, 128), (128, 128, 1000)])
def test_fp32_equivalent_product_and_its_accumulation_bias(B, M, N, K):
    """The split-bf16 product of the solve against an fp64 product of the same fp32 operands.  With all terms of
    one sign the tensor core's truncating accumulation shows as a one-sided error; kept in separate
    accumulators (the configuration the factorisation uses) it stays within a few fp32 roundings of the sum."""
    import torch
    cfg = small_cfg("bf16", hd=128, Hq=8, Hkv=2, d=1024, F=1024, L=256, N=64)
    ctx = B.PkvContext(B.dims_from_config(cfg), engine=B.ENGINE_AUTO)
    r = np.random.default_rng(32)
    for positive in (True, False):
        A = r.standard_normal((M, K)).astype(np.float32)
        Bm = r.standard_normal((N, K)).astype(np.float32)
        if positive:
            A, Bm = np.abs(A), np.abs(Bm)
        want = A.astype(np.float64) @ Bm.astype(np.float64).T
        scale = np.abs(A).astype(np.float64) @ np.abs(Bm).astype(np.float64).T
        tA, tB = torch.from_numpy(A).cuda(), torch.from_numpy(Bm).cuda()
        rms = {}
        for acc in (1, 4):
            got = ctx.fp32_product(tA, tB, passes=6, accumulators=acc).cpu().numpy().astype(np.float64)
            rms[acc] = float(np.sqrt((((got - want) / scale) ** 2).mean()))
        print("M %d N %d K %d %s terms: rms error / sum|terms|: one accumulator %.2e, separated %.2e"
              % (M, N, K, "positive" if positive else "signed", rms[1], rms[4]))
        assert rms[4] <= 2e-7 * max(1.0, K / 128.0)
        if positive:
            assert rms[4] < 0.5 * rms[1]
        # pairs: about 16 bits
        got3 = ctx.fp32_product(tA, tB, passes=3, accumulators=2).cpu().numpy().astype(np.float64)
        assert float(np.sqrt((((got3 - want) / scale) ** 2).mean())) <= 2e-5
        # C <- C - A B^T (the form of the trailing update)
        C0 = r.standard_normal((M, N)).astype(np.float32)
        tC = torch.from_numpy(C0).cuda()
        ctx.fp32_product(tA, tB, alpha=-1.0, C_out=tC, accumulate=True, passes=6, accumulators=4)
        np.testing.assert_allclose(tC.cpu().numpy(), C0 - want, rtol=0, atol=1e-5 * scale.max())
    ctx.close()


@pytest.mark.parametrize("M,N,K", [(2048, 2048, 512), (4096, 1024, 200), (2048, 2048, 64)])
def test_product_on_cta_pairs_matches_fp64(B, M, N, K):
    """Products whose M and N are multiples of 256 and that fill the machine run on pairs of CTAs (256 x 256 tiles,
    each CTA loading its own half of the operands): against an fp64 product of the same fp32 operands, per 128 x 128
    block so that a misplaced half tile cannot hide in a norm; ragged K; overwrite and accumulate."""
    import torch
    cfg = small_cfg("bf16", hd=128, Hq=16, Hkv=2, d=2048, F=2048, L=256, N=64)
    ctx = B.PkvContext(B.dims_from_config(cfg), engine=B.ENGINE_AUTO)
    r = np.random.default_rng(33)
    A = r.standard_normal((M, K)).astype(np.float32)
    Bm = r.standard_normal((N, K)).astype(np.float32)
    want = A.astype(np.float64) @ Bm.astype(np.float64).T
    tA, tB = torch.from_numpy(A).cuda(), torch.from_numpy(Bm).cuda()
    got = ctx.fp32_product(tA, tB, passes=3, accumulators=1).cpu().numpy().astype(np.float64)
    blk = np.abs(got - want).reshape(M // 128, 128, N // 128, 128).max(axis=(1, 3)) / np.abs(want).max()
    assert blk.max() <= 3e-5, (blk.max(), np.unravel_index(blk.argmax(), blk.shape))
    C0 = r.standard_normal((M, N)).astype(np.float32)
    tC = torch.from_numpy(C0).cuda()
    ctx.fp32_product(tA, tB, alpha=-0.5, C_out=tC, accumulate=True, passes=3, accumulators=1)
    np.testing.assert_allclose(tC.cpu().numpy(), C0 - 0.5 * want, rtol=0, atol=3e-5 * np.abs(want).max())
    ctx.close()


@pytest.mark.parametrize("d,F,n,r", [(256, 192, 500, 32), (128, 128, 60, 8)])
def test_low_rank_patch_matches_oracle(B, d, F, n, r):
    """Appendix, low-rank weight patches: dW_r = U_r U_r^T dW with U_r the leading eigenvectors of dW S_H dW^T,
    against the oracle's eigendecomposition; the weighted loss of the truncation is the sum of the discarded
    eigenvalues; the stored factors have (d + F) r numbers."""
    import torch
    cfg = small_cfg("bf16", F=F, d=d, Hq=max(d // 64, 1), Hkv=1)
    rng = np.random.default_rng(51)
    X = rng.standard_normal((n, F))
    # targets with a decaying spectrum so that the r-th eigenvalue gap is open
    basis = rng.standard_normal((F, d))
    R = (X @ basis) * (0.85 ** np.arange(d))[None, :] + 1e-3 * rng.standard_normal((n, d))
    S_H, S_T = orc.sufficient_statistics(X, R)
    dW = orc.ridge_solve(S_H, S_T, orc.ridge_lambda(S_H, 0.1))
    U_o, B_o, dWr_o, ev_o = orc.low_rank_patch(dW, S_H, r)
    assert ev_o[r - 1] > 1.3 * ev_o[r]                       # an open gap: dW_r is then well determined
    ctx = B.PkvContext(B.dims_from_config(cfg), engine=B.ENGINE_AUTO)
    t_dW = torch.from_numpy(dW.astype(np.float32)).cuda()
    t_SH = torch.from_numpy(S_H.astype(np.float32)).cuda()
    out = ctx.low_rank(t_dW, t_SH, r)
    dWr = out["dW_r"].cpu().numpy().astype(np.float64)
    err = H.rel_fro(dWr, dWr_o)
    # loss identity: tr((dW - dW_r) S_H (dW - dW_r)^T) = sum of the discarded eigenvalues
    E = dW - dWr
    loss = np.trace(E @ S_H @ E.T)
    print("rank-%d patch (d %d, F %d): dW_r rel fro err %.3e; weighted loss %.6g vs discarded eigenvalues %.6g"
          % (r, d, F, err, loss, ev_o[r:].sum()))
    assert err <= DW_TOL
    np.testing.assert_allclose(loss, ev_o[r:].sum(), rtol=2e-3)
    np.testing.assert_allclose(out["ritz"].cpu().numpy()[:r], ev_o[:r], rtol=2e-3)
    U = out["U"].cpu().numpy().astype(np.float64)
    np.testing.assert_allclose(U.T @ U, np.eye(r), atol=1e-5)                      # orthonormal columns
    np.testing.assert_allclose(out["Br"].cpu().numpy(), U.T @ dW, rtol=0, atol=1e-4 * np.abs(dW).max() * np.sqrt(d))
    np.testing.assert_allclose(dWr, U @ out["Br"].cpu().numpy().astype(np.float64), rtol=0, atol=1e-5 * np.abs(dW).max())
    ctx.close()


# ------------------------------------------------------------------ whole block

def test_config1_tiny_fp32_end_to_end(B):
    cfg = gen.benchmark_config(1)
    lay = H.make_problem(cfg)
    x = lay["x0"]
    check_build(B, cfg, lay, x, x, [0, cfg.N], cfg.lam0, B.ENGINE_SIMT)
    check_build(B, cfg, lay, x, x, [0, cfg.N], 1e-2, B.ENGINE_SIMT, mode=B.LAMBDA_ABSOLUTE)


@pytest.mark.parametrize("hd,Hq,Hkv", [(64, 8, 2), (128, 4, 2)])
def test_small_bf16_block_chunks_ragged_distinct_states(B, hd, Hq, Hkv):
    cfg = small_cfg("bf16", hd=hd, Hq=Hq, Hkv=Hkv, d=256, F=192, L=1000, N=150)
    lay = H.make_problem(cfg, per_head_budget=[100, 37][:Hkv])
    xF = lay["x0"]
    xC = (xF + 0.02 * np.random.default_rng(5).standard_normal(xF.shape)).astype(np.float32)
    for engine in engines(B, cfg):
        check_build(B, cfg, lay, xF, xC, [0, 40, 41, 150], 0.1, engine, kv_split=256)
        check_build(B, cfg, lay, xF, xF, [0, 150], 1e-3, engine)


@pytest.mark.parametrize("N,F", [(150, 192), (70, 448), (128, 128)])
def test_dual_solver_gives_the_same_patch(B, N, F):
    """dW through the N x N system (Woodbury) against the oracle's F x F solve, ragged N, several modes."""
    cfg = small_cfg("bf16", hd=128, Hq=4, Hkv=2, d=256, F=F, L=1000, N=N)
    lay = H.make_problem(cfg, per_head_budget=[100, 37])
    xF = lay["x0"]
    xC = (xF + 0.02 * np.random.default_rng(5).standard_normal(xF.shape)).astype(np.float32)
    check_build(B, cfg, lay, xF, xC, [0, N // 3, N], 0.1, B.ENGINE_AUTO, solver=B.SOLVER_DUAL)
    check_build(B, cfg, lay, xF, xF, [0, N], 1e-3, B.ENGINE_AUTO, solver=B.SOLVER_DUAL)
    check_build(B, cfg, lay, xF, xF, [0, N], 0.05, B.ENGINE_AUTO, mode=B.LAMBDA_TRACE_MEAN, solver=B.SOLVER_DUAL)
    # the dual form needs N <= F and the tensor-core engine
    with pytest.raises(B.PkvError) as ei:
        B.PkvContext(B.dims_from_config(gen.scaled_config(cfg, N=F + 8)), solver=B.SOLVER_DUAL)
    assert ei.value.code == -2


def test_block_and_stack_with_refinement_match_the_oracle(B):
    """pkv_set_refinement on the building calls: a block in absolute-lambda mode with fewer reference tokens than
    features (ill conditioned: the condition warning is raised) and a three-block stack, each with one correction,
    against the oracle; the student's next state is formed with the refined patch."""
    import torch
    cfg = small_cfg("bf16", hd=128, Hq=4, Hkv=2, d=256, F=448, L=700, N=70)
    lay = H.make_problem(cfg)
    x = lay["x0"]
    # the absolute coefficient: 5e-5 of the eigenvalue mean of S_H (the oracle under Eq. 7 gives its value)
    ref = H.run_oracle(cfg, lay, x, x, [0, cfg.N], 5e-5)
    lam_abs = float(ref["lam"])
    errs = []
    for refine in (0, 1):
        got = gpu_build(B, cfg, lay, x, x, [0, cfg.N], lam_abs, B.ENGINE_AUTO, mode=B.LAMBDA_ABSOLUTE, refine=refine)
        errs.append(H.rel_fro(got["dW"], ref["dW"]))
        assert got["stats"]["cond_warning"] == 1
        if refine:
            assert H.rel_fro(got["xC_next"], ref["xC_next"]) <= 1e-3
            gap = got["xF_next"].astype(np.float64) - got["xC_next"]
            np.testing.assert_allclose(got["stats"]["resid_fro2"], np.sum(gap * gap), rtol=1e-2)
            np.testing.assert_allclose(got["stats"]["dW_fro2"], np.sum(ref["dW"] ** 2), rtol=2e-2)
    print("block, absolute lambda (5e-5 of the eigenvalue mean), cond lower bound %.1e: dW error %.2e plain, %.2e with one correction" %
          (got["stats"]["cond_lower_bound"], errs[0], errs[1]))
    assert errs[1] <= DW_TOL and errs[1] <= errs[0]
    nl = 3
    cfg = small_cfg("bf16", n_layers=nl, N=64, hd=128, Hq=4, Hkv=2)
    lays = [H.make_problem(cfg, layer=l) for l in range(nl)]
    x0 = lays[0]["x0"]
    xF, xC = x0.astype(np.float64), x0.astype(np.float64)
    refs = []
    for l in range(nl):
        refs.append(H.run_oracle(cfg, lays[l], xF, xC, [0, cfg.N], 1e-3))
        xF, xC = refs[-1]["xF_next"], refs[-1]["xC_next"]
    ctx = B.PkvContext(B.dims_from_config(cfg), engine=B.ENGINE_AUTO)
    ctx.set_refinement(1)
    dl = []
    for l in range(nl):
        off, idx = gen.kept_to_csr(lays[l]["kept"])
        kv = B.to_device({"K": lays[l]["K"], "V": lays[l]["V"]}, cfg.dtype)
        dl.append({"w": B.to_device(lays[l]["weights"], cfg.dtype), "K": kv["K"], "V": kv["V"], "head_off": off,
                   "idx": torch.from_numpy(idx).cuda()})
    xt = torch.from_numpy(x0).cuda()
    out = ctx.build_stack(dl, xt, xt, [0, cfg.N], cfg.L, 1e-3)
    for l in range(nl):
        assert H.rel_fro(out["dW"][l].cpu().numpy(), refs[l]["dW"]) <= DW_TOL, l
    assert H.rel_fro(out["xC_final"].cpu().numpy(), refs[-1]["xC_next"]) <= 2e-3
    ctx.close()


def test_identical_caches_give_zero_patch(B):
    cfg = small_cfg("bf16", L=300, budget=300, N=40)
    lay = H.make_problem(cfg)
    lay["kept"] = [np.arange(cfg.L, dtype=np.int32)] * cfg.Hkv
    for engine in engines(B, cfg):
        got = gpu_build(B, cfg, lay, lay["x0"], lay["x0"], [0, cfg.N], 0.1, engine)
        ref = H.run_oracle(cfg, lay, lay["x0"], lay["x0"], [0, cfg.N], 0.1)
        assert np.all(ref["dW"] == 0.0)
        # dA, dz, dh are formed as differences of identical numbers: exactly zero, hence dW = 0
        assert np.all(got["dW"] == 0.0)
        np.testing.assert_array_equal(got["xF_next"], got["xC_next"])


def test_reduced_config2_shape(B):
    """Llama-3-8B head layout (g = 4, hd = 128) at reduced width and length: several tiles in
    every dimension and ragged tails."""
    cfg = small_cfg("bf16", hd=128, Hq=8, Hkv=2, d=512, F=448, L=5000, N=200, window=32, budget=500, n_obs=32,
                    kept_rule="window_topk")
    lay = H.make_problem(cfg)
    for engine in engines(B, cfg):
        check_build(B, cfg, lay, lay["x0"], lay["x0"], [0, cfg.N], 0.1, engine)


@pytest.mark.parametrize("nl,solver,hd", [(2, 0, 64), (5, 0, 128), (4, 1, 128), (8, 0, 128)])
def test_stack_matches_oracle_chain(B, nl, solver, hd):
    """Free-running stack: GPU and oracle each propagate their own states through all blocks (the tensor-core
    engine runs the teacher ahead on its own stream; five blocks reuse its three-slot ring of teacher outputs, eight
    blocks go round it twice and once round the five-slot ring of the teacher's next states)."""
    import torch
    cfg = small_cfg("bf16", n_layers=nl, N=64, hd=hd, Hq=4 if hd == 128 else 8, Hkv=2)
    lays = [H.make_problem(cfg, layer=l) for l in range(nl)]
    x0 = lays[0]["x0"]
    xF, xC = x0.astype(np.float64), x0.astype(np.float64)
    refs = []
    for l in range(nl):
        o = H.run_oracle(cfg, lays[l], xF, xC, [0, cfg.N], 0.1)
        refs.append(o)
        xF, xC = o["xF_next"], o["xC_next"]
    for engine in (engines(B, cfg) if solver == 0 else [B.ENGINE_AUTO]):
        ctx = B.PkvContext(B.dims_from_config(cfg), engine=engine, solver=solver)
        dl = []
        for l in range(nl):
            off, idx = gen.kept_to_csr(lays[l]["kept"])
            kv = B.to_device({"K": lays[l]["K"], "V": lays[l]["V"]}, cfg.dtype)
            dl.append({"w": B.to_device(lays[l]["weights"], cfg.dtype), "K": kv["K"], "V": kv["V"],
                       "head_off": off, "idx": torch.from_numpy(idx).cuda()})
        xt = torch.from_numpy(x0).cuda()
        out = ctx.build_stack(dl, xt, xt, [0, cfg.N], cfg.L, 0.1)
        for l in range(nl):
            assert H.rel_fro(out["dW"][l].cpu().numpy(), refs[l]["dW"]) <= DW_TOL, l
            np.testing.assert_allclose(out["stats"][l]["lambda_eff"], refs[l]["lam"], rtol=5e-3)
        assert H.rel_fro(out["xC_final"].cpu().numpy(), refs[-1]["xC_next"]) <= 2e-3
        assert H.rel_fro(out["xF_final"].cpu().numpy(), refs[-1]["xF_next"]) <= 2e-3
        # resuming from a later block with the states of the block before gives the same patches
        if nl >= 4 and engine == B.ENGINE_AUTO:
            mid = 2
            xFm = torch.from_numpy(refs[mid - 1]["xF_next"].astype(np.float32)).cuda()
            xCm = torch.from_numpy(refs[mid - 1]["xC_next"].astype(np.float32)).cuda()
            out2 = ctx.build_stack(dl, xFm, xCm, [0, cfg.N], cfg.L, 0.1, first_layer=mid)
            for l in range(mid, nl):
                assert H.rel_fro(out2["dW"][l].cpu().numpy(), refs[l]["dW"]) <= DW_TOL, l
        # an invalid kept set in a later block is reported with its position
        if engine == B.ENGINE_AUTO and solver == 0:
            bad = dict(dl[-1])
            bi = dl[-1]["idx"].clone()
            bi[3] = bi[2]
            bad["idx"] = bi
            with pytest.raises(B.PkvError) as ei:
                ctx.build_stack(dl[:-1] + [bad], xt, xt, [0, cfg.N], cfg.L, 0.1)
            assert ei.value.code == -3
        ctx.close()


def test_lambda_sweep_with_the_teacher_run_once_matches_separate_stacks(B):
    """pkv_build_stack_sweep (teacher outputs cached, student + solve replayed per ridge coefficient) against
    one pkv_build_stack per coefficient and against the oracle chain."""
    import torch
    nl = 4
    cfg = small_cfg("bf16", n_layers=nl, N=64, hd=128, Hq=4, Hkv=2)
    lays = [H.make_problem(cfg, layer=l) for l in range(nl)]
    x0 = lays[0]["x0"]
    ctx = B.PkvContext(B.dims_from_config(cfg), engine=B.ENGINE_AUTO)
    dl = []
    for l in range(nl):
        off, idx = gen.kept_to_csr(lays[l]["kept"])
        kv = B.to_device({"K": lays[l]["K"], "V": lays[l]["V"]}, cfg.dtype)
        dl.append({"w": B.to_device(lays[l]["weights"], cfg.dtype), "K": kv["K"], "V": kv["V"], "head_off": off,
                   "idx": torch.from_numpy(idx).cuda()})
    xt = torch.from_numpy(x0).cuda()
    lams = [1e-3, 0.1, 10.0]
    sweep = ctx.build_stack_sweep(dl, xt, xt, [0, cfg.N], cfg.L, lams)
    for j, lam0 in enumerate(lams):
        single = ctx.build_stack(dl, xt, xt, [0, cfg.N], cfg.L, lam0)
        xF, xC = x0.astype(np.float64), x0.astype(np.float64)
        for l in range(nl):
            o = H.run_oracle(cfg, lays[l], xF, xC, [0, cfg.N], lam0)
            xF, xC = o["xF_next"], o["xC_next"]
            got = sweep["dW"][j][l].cpu().numpy()
            assert H.rel_fro(got, single["dW"][l].cpu().numpy()) <= 1e-5, (lam0, l)
            assert H.rel_fro(got, o["dW"]) <= DW_TOL, (lam0, l)
            np.testing.assert_allclose(sweep["stats"][j][l]["lambda_eff"], o["lam"], rtol=5e-3)
    ctx.close()


@pytest.mark.parametrize("engine_name,lam0", [("tc", 0.1), ("tc", 1e-3), ("simt", 0.1)])
def test_streamed_reference_set_equals_one_call_and_the_oracle(B, engine_name, lam0):
    """Sec. 2.3 / Eq. 9: the reference set fed in three parts (whole chunks each), only S_H and S_T kept between the
    calls, against one pkv_build_patch on all tokens and against the oracle; the teacher's next states come out of
    the parts, the student's from the propagation call with the patched block (Algorithm 1)."""
    import torch
    cfg = small_cfg("bf16", hd=128, Hq=4, Hkv=2, d=256, F=192, L=1000, N=210)
    engine = B.ENGINE_AUTO if engine_name == "tc" else B.ENGINE_SIMT
    lay = H.make_problem(cfg, per_head_budget=[100, 37])
    xF = lay["x0"]
    xC = (xF + 0.02 * np.random.default_rng(5).standard_normal(xF.shape)).astype(np.float32)
    chunk_off = [0, 40, 41, 100, 150, 210]
    parts = [(0, 41, [0, 40, 41]), (41, 150, [0, 59, 109]), (150, 210, [0, 60])]       # token range, local chunk offsets
    ref = H.run_oracle(cfg, lay, xF, xC, chunk_off, lam0)
    ctx = B.PkvContext(B.dims_from_config(cfg, N_max=cfg.N, b_max=100), engine=engine)
    w = B.to_device(lay["weights"], cfg.dtype)
    kv = B.to_device({"K": lay["K"], "V": lay["V"]}, cfg.dtype)
    off, idx = gen.kept_to_csr(lay["kept"])
    idx_t = torch.from_numpy(idx).cuda()
    tF, tC = torch.from_numpy(xF).cuda(), torch.from_numpy(xC).cuda()
    whole = ctx.build_patch(w, kv["K"], kv["V"], off, idx_t, tF, tC, chunk_off, cfg.L, lam0)
    ctx.stream_begin(lam0)
    xFn = []
    for a, e, co in parts:
        xFn.append(ctx.stream_add(w, kv["K"], kv["V"], off, idx_t, tF[a:e].contiguous(), tC[a:e].contiguous(), co, cfg.L,
                                  want_next=True))
    dW, st = ctx.stream_finish()
    e_or = H.rel_fro(dW.cpu().numpy(), ref["dW"])
    e_one = H.rel_fro(dW.cpu().numpy(), whole["dW"].cpu().numpy())
    print("streamed in 3 parts (%s, lambda0 %g): dW vs oracle %.3e, vs one call %.3e" % (engine_name, lam0, e_or, e_one))
    assert e_or <= DW_TOL and e_one <= 2e-3
    np.testing.assert_allclose(st["lambda_eff"], ref["lam"], rtol=2e-3)
    np.testing.assert_allclose(st["target_fro2"], ref["T_fro2"], rtol=2e-2)
    assert H.rel_fro(torch.cat(xFn).cpu().numpy(), ref["xF_next"]) <= 1e-3
    if engine_name == "tc":
        xCn = torch.cat([ctx.stream_propagate(w, kv["K"], kv["V"], off, idx_t, tC[a:e].contiguous(), co, cfg.L, dW)
                         for a, e, co in parts])
        assert H.rel_fro(xCn.cpu().numpy(), ref["xC_next"]) <= 1e-3
    # a second stream on the same context starts from zero sums
    ctx.stream_begin(lam0)
    ctx.stream_add(w, kv["K"], kv["V"], off, idx_t, tF, tC, chunk_off, cfg.L)
    dW2, _ = ctx.stream_finish()
    assert H.rel_fro(dW2.cpu().numpy(), ref["dW"]) <= DW_TOL
    with pytest.raises(B.PkvError):                      # no stream open
        ctx.stream_finish()
    # the streamed solve with one correction of iterative refinement (the sums are kept as a full symmetric matrix)
    if engine_name == "tc":
        ctx.set_refinement(1)
        ctx.stream_begin(lam0)
        for a, e, co in parts:
            ctx.stream_add(w, kv["K"], kv["V"], off, idx_t, tF[a:e].contiguous(), tC[a:e].contiguous(), co, cfg.L)
        dW3, _ = ctx.stream_finish()
        e3 = H.rel_fro(dW3.cpu().numpy(), ref["dW"])
        print("   with one correction: dW vs oracle %.3e" % e3)
        assert e3 <= DW_TOL and e3 <= e_or * 1.05 + 1e-5
    ctx.close()


def test_statistics_survive_massive_activations(B):
    """The build's statistics take one pass over fp16 copies scaled by a power of two from each array's maximum.
    A few features 256 times larger than the rest (rows of Wup scaled by a power of two, so that they stay bf16
    values) must not cost the others their bits: same tolerance against the oracle as everywhere."""
    cfg = small_cfg("bf16", hd=128, Hq=8, Hkv=2, d=512, F=448, L=3000, N=200, window=32, budget=300, n_obs=16)
    lay = H.make_problem(cfg)
    w = dict(lay["weights"])
    wu = np.array(w["Wup"], dtype=np.float32, copy=True)
    wu[::37] *= 256.0
    w["Wup"] = wu
    lay = dict(lay, weights=w)
    rng = np.random.default_rng(11)
    xF = lay["x0"]
    xC = (xF + 0.05 * rng.standard_normal(xF.shape)).astype(np.float32)
    e = check_build(B, cfg, lay, xF, xC, [0, 120, cfg.N], 0.1, B.ENGINE_AUTO)
    print("features x256: dW rel fro err %.3e" % e)


def test_repeated_builds_on_one_context_are_stable(B):
    """The build spreads one block over several internal streams (student half, teacher half on an SM partition,
    targets and S_T beside the solve, the solve's own four).  Forty builds back to back on one context, alternating
    between two problems, must each reproduce the first result of their problem: an ordering hole between the
    streams would show up as a result that depends on what ran before."""
    import torch
    cfg = small_cfg("bf16", hd=128, Hq=8, Hkv=2, d=512, F=448, L=3000, N=200, window=32, budget=300, n_obs=16)
    lay = H.make_problem(cfg)
    rng = np.random.default_rng(17)
    xF = lay["x0"]
    xCs = [(xF + s_ * rng.standard_normal(xF.shape)).astype(np.float32) for s_ in (0.05, 0.2)]
    chunk_off = [0, 120, cfg.N]
    ctx = B.PkvContext(B.dims_from_config(cfg, N_max=cfg.N, b_max=max(len(k) for k in lay["kept"])), engine=B.ENGINE_AUTO)
    w = B.to_device(lay["weights"], cfg.dtype)
    kv = B.to_device({"K": lay["K"], "V": lay["V"]}, cfg.dtype)
    off, idx = gen.kept_to_csr(lay["kept"])
    idx_t = torch.from_numpy(idx).cuda()
    tF = torch.from_numpy(xF).cuda()
    tCs = [torch.from_numpy(x).cuda() for x in xCs]
    first = [None, None]
    worst = 0.0
    for i in range(40):
        k = i & 1
        o = ctx.build_patch(w, kv["K"], kv["V"], off, idx_t, tF, tCs[k], chunk_off, cfg.L, 0.1, 0, True)
        got = {n: o[n].cpu().numpy() for n in ("dW", "xF_next", "xC_next")}
        got["t"] = o["stats"]["target_fro2"]
        if first[k] is None:
            first[k] = got
            ref = H.run_oracle(cfg, lay, xF, xCs[k], chunk_off, 0.1, 0)
            assert H.rel_fro(got["dW"], ref["dW"]) <= DW_TOL
            continue
        for n in ("dW", "xF_next", "xC_next"):
            e = H.rel_fro(got[n], first[k][n])
            worst = max(worst, e)
            assert e <= 1e-5, (i, n, e)
        np.testing.assert_allclose(got["t"], first[k]["t"], rtol=1e-6)
    ctx.close()
    print("40 alternating builds: largest deviation from the first result %.2e" % worst)


def test_timed_build_uses_the_stacked_schedule_and_agrees(B):
    """With stage timing on, a block runs teacher and student stacked on one stream (so that the stage marks mean
    something); without, the student half runs first and the teacher half beside the solve.  Same patch either way,
    and both against the oracle."""
    import torch
    cfg = small_cfg("bf16", hd=128, Hq=8, Hkv=2, d=512, F=448, L=3000, N=200, window=32, budget=300, n_obs=16)
    lay = H.make_problem(cfg)
    rng = np.random.default_rng(5)
    xF = lay["x0"]
    xC = (xF + 0.05 * rng.standard_normal(xF.shape)).astype(np.float32)
    chunk_off = [0, 120, cfg.N]
    ref = H.run_oracle(cfg, lay, xF, xC, chunk_off, 0.1, 0)
    ctx = B.PkvContext(B.dims_from_config(cfg, N_max=cfg.N, b_max=max(len(k) for k in lay["kept"])), engine=B.ENGINE_AUTO)
    w = B.to_device(lay["weights"], cfg.dtype)
    kv = B.to_device({"K": lay["K"], "V": lay["V"]}, cfg.dtype)
    off, idx = gen.kept_to_csr(lay["kept"])
    idx_t = torch.from_numpy(idx).cuda()
    tF, tC = torch.from_numpy(xF).cuda(), torch.from_numpy(xC).cuda()
    outs = []
    for timed in (False, True, False, 2):
        ctx.set_timing(timed)
        o = ctx.build_patch(w, kv["K"], kv["V"], off, idx_t, tF, tC, chunk_off, cfg.L, 0.1, 0, True)
        outs.append({k: (v.cpu().numpy() if hasattr(v, "cpu") else v) for k, v in o.items()})
    ctx.close()
    errs = [H.rel_fro(o["dW"], ref["dW"]) for o in outs]
    cross = H.rel_fro(outs[1]["dW"], outs[0]["dW"])
    print("untimed / timed / untimed / solve-only timing vs oracle: %.3e %.3e %.3e %.3e; timed vs untimed %.3e" % (*errs, cross))
    # mode 2 times the solve alone and leaves the schedule as it is
    sm = outs[3]["stats"]["stage_ms"]
    assert sm[7] > 0 and sum(sm) == sm[7]
    assert H.rel_fro(outs[3]["dW"], outs[0]["dW"]) <= 1e-5
    assert max(errs) <= DW_TOL and cross <= 2e-3
    assert sum(outs[1]["stats"]["stage_ms"]) > 0 and sum(outs[0]["stats"]["stage_ms"]) == 0
    for o in outs:
        assert H.rel_fro(o["xF_next"], ref["xF_next"]) <= 1e-3 and H.rel_fro(o["xC_next"], ref["xC_next"]) <= 1e-3
        np.testing.assert_allclose(o["stats"]["target_fro2"], ref["T_fro2"], rtol=2e-2)


# ------------------------------------------------------------------ boundary

_ALT_CASE = '''
import sys
sys.path.insert(0, %r)
from paper_2609_39329_b200 import binding as B
from tests import test_gpu_parity as T
from tests import helpers as H
cfg = T.small_cfg("bf16", hd=128, Hq=8, Hkv=2, d=512, F=448, L=3000, N=200, window=32, budget=300, n_obs=16)
lay = H.make_problem(cfg)
e = T.check_build(B, cfg, lay, lay["x0"], lay["x0"], [0, 120, cfg.N], 0.1, B.ENGINE_AUTO)
print("ALT_OK %%.3e" %% e)
'''


@pytest.mark.parametrize("env", [{"PKV_ATTN_Q": "pair"}, {"PKV_SOLVE_GRAPH": "0"}, {"PKV_SOLVE_TRACE": "1"},
                                 {"PKV_BUILD_OVERLAP": "0"}, {"PKV_SIDE_STREAM": "0"}, {"PKV_BUILD_RESERVE_SMS": "0"},
                                 {"PKV_BUILD_TRACE": "1"}, {"PKV_STATS_F16": "0"}, {"PKV_SM_PARTITIONS": "0"}])
def test_alternate_paths_selected_by_environment(env):
    """Paths the environment selects at start-up, each in a process of its own on one small hd-128 block against the
    oracle: bf16 query pairs against bf16 keys (the attention path for caches outside fp16's range), the solve
    issued launch by launch instead of replayed as a graph, the solve's phase trace, the block with teacher and
    student stacked on one stream (no teacher half beside the solve), nothing at all beside the solve, the teacher
    half on the stack driver's partition instead of the build's own, the build's timeline, the statistics from
    bf16 pairs in three passes instead of one scaled fp16 pass, and ordinary streams in place of SM partitions."""
    import os
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    r = subprocess.run([sys.executable, "-c", _ALT_CASE % root], env={**os.environ, **env}, capture_output=True, text=True,
                       timeout=900, cwd=root)
    assert r.returncode == 0 and "ALT_OK" in r.stdout, r.stdout[-2000:] + r.stderr[-2000:]
    if "PKV_SOLVE_TRACE" in env:
        assert "solve timeline" in r.stderr
    if "PKV_BUILD_TRACE" in env:
        assert "build timeline" in r.stderr


_PAIR_CASE = '''
import sys
sys.path.insert(0, %r)
import numpy as np, torch
from paper_2609_39329_b200 import binding as B
from tests import test_gpu_parity as T
cfg = T.small_cfg("bf16", hd=128, Hq=16, Hkv=2, d=2048, F=2048, L=256, N=64)
ctx = B.PkvContext(B.dims_from_config(cfg), engine=B.ENGINE_AUTO)
r = np.random.default_rng(34)
A = r.standard_normal((2048, 320)).astype(np.float32)
Bm = r.standard_normal((2048, 320)).astype(np.float32)
got = ctx.fp32_product(torch.from_numpy(A).cuda(), torch.from_numpy(Bm).cuda(), passes=3, accumulators=1).cpu().numpy()
want = A.astype(np.float64) @ Bm.astype(np.float64).T
print("PAIR_CASE %%.9e %%s" %% (np.abs(got - want).max() / np.abs(want).max(), got.tobytes()[:64].hex()))
'''


def test_products_agree_with_and_without_cta_pairs():
    """PKV_GEMM_PAIR=0 sends every product to single CTAs: the same 2048 x 2048 x 320 product in two processes, one per
    setting, both against fp64 and against each other (same passes in the same order on the same accumulator width:
    the two kernels give the same bits)."""
    import os
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    outs = []
    for v in ("1", "0"):
        r = subprocess.run([sys.executable, "-c", _PAIR_CASE % root], env={**os.environ, "PKV_GEMM_PAIR": v}, capture_output=True,
                           text=True, timeout=600, cwd=root)
        assert r.returncode == 0 and "PAIR_CASE" in r.stdout, r.stdout[-2000:] + r.stderr[-2000:]
        line = [x for x in r.stdout.splitlines() if x.startswith("PAIR_CASE")][-1].split()
        assert float(line[1]) <= 3e-5
        outs.append(line[2])
    assert outs[0] == outs[1]


def test_boundary_rejects_bad_arguments(B):
    import torch
    cfg = small_cfg("bf16")
    with pytest.raises(B.PkvError) as ei:
        B.PkvContext(B.dims_from_config(gen.scaled_config(cfg, hd=96)), engine=B.ENGINE_SIMT)
    assert ei.value.code == -2
    with pytest.raises(B.PkvError) as ei:
        B.PkvContext(B.dims_from_config(gen.scaled_config(cfg, F=40000)), engine=B.ENGINE_SIMT)
    assert ei.value.code == -2
    lay = H.make_problem(cfg)
    x = lay["x0"]
    for lam in (0.0, -1.0, float("nan"), float("inf")):
        with pytest.raises(B.PkvError) as ei:
            gpu_build(B, cfg, lay, x, x, [0, cfg.N], lam, B.ENGINE_SIMT)
        assert ei.value.code == -1
    for chunks in ([0, 10, 10, cfg.N], [1, cfg.N], [0, cfg.N - 1]):
        with pytest.raises(B.PkvError) as ei:
            gpu_build(B, cfg, lay, x, x, chunks, 0.1, B.ENGINE_SIMT)
        assert ei.value.code == -1
    bad = dict(lay)
    bad["kept"] = [lay["kept"][0].copy(), lay["kept"][1].copy()]
    bad["kept"][1][7] = bad["kept"][1][6]
    with pytest.raises(B.PkvError) as ei:
        gpu_build(B, cfg, bad, x, x, [0, cfg.N], 0.1, B.ENGINE_SIMT)
    assert ei.value.code == -3 and ei.value.info["err_info"] == (1, 7)


def test_bounded_wait_gives_timeout_status_and_context_survives(B):
    """Failure detection without a fault: a pipeline wait on a barrier nothing completes runs out of its
    (short) limit, the call returns PKV_ERR_TIMEOUT with the wait site, and the context keeps working."""
    import torch
    cfg = small_cfg("bf16", hd=128, Hq=4, Hkv=2)
    ctx = B.PkvContext(B.dims_from_config(cfg), engine=B.ENGINE_AUTO)
    rc, site = ctx.selftest_bounded_wait()
    assert rc == -7 and site == 99
    r = np.random.default_rng(0)
    X = torch.from_numpy(r.standard_normal((cfg.N, cfg.F)).astype(np.float32)).cuda()
    R = torch.from_numpy(r.standard_normal((cfg.N, cfg.d)).astype(np.float32)).cuda()
    gH, _ = ctx.gram(X, R)
    assert H.rel_fro(gH.cpu().numpy(), X.double().cpu().numpy().T @ X.double().cpu().numpy()) <= 2e-4
    ctx.close()


def test_nonfinite_inputs_are_reported_and_caller_workspace_is_accepted(B):
    import torch
    cfg = small_cfg("bf16", hd=128, Hq=4, Hkv=2, N=64)
    lay = H.make_problem(cfg)
    x = lay["x0"].copy()
    x[3, 5] = np.nan
    with pytest.raises(B.PkvError) as ei:
        gpu_build(B, cfg, lay, x, x, [0, cfg.N], 0.1, B.ENGINE_AUTO)
    assert ei.value.code == -6
    # a cached key beyond fp16's range cannot go through the fp16 key copies of the hd-128 attention: reported
    lay2 = dict(lay)
    lay2["K"] = lay["K"].copy()
    lay2["K"][0, 7, 3] = 1.0e5
    with pytest.raises(B.PkvError) as ei:
        gpu_build(B, cfg, lay2, lay["x0"], lay["x0"], [0, cfg.N], 0.1, B.ENGINE_AUTO)
    assert ei.value.code == -6
    # caller-provided workspace: same result as the context-owned one; an undersized one is refused
    dims = B.dims_from_config(cfg, b_max=max(len(k) for k in lay["kept"]))
    probe = B.PkvContext(dims, engine=B.ENGINE_AUTO)
    need = probe.workspace_bytes()
    probe.close()
    ws = torch.empty(need, dtype=torch.uint8, device="cuda")
    ctx = B.PkvContext(dims, engine=B.ENGINE_AUTO, workspace=ws)
    w = B.to_device(lay["weights"], cfg.dtype)
    kv = B.to_device({"K": lay["K"], "V": lay["V"]}, cfg.dtype)
    off, idx = gen.kept_to_csr(lay["kept"])
    xt = torch.from_numpy(lay["x0"]).cuda()
    out = ctx.build_patch(w, kv["K"], kv["V"], off, torch.from_numpy(idx).cuda(), xt, xt, [0, cfg.N], cfg.L, 0.1)
    ref = H.run_oracle(cfg, lay, lay["x0"], lay["x0"], [0, cfg.N], 0.1)
    assert H.rel_fro(out["dW"].cpu().numpy(), ref["dW"]) <= DW_TOL
    ctx.close()
    with pytest.raises(B.PkvError) as ei:
        B.PkvContext(dims, engine=B.ENGINE_AUTO, workspace=ws[:need // 2])
    assert ei.value.code == -9

"""Full-size checks in the launch configuration bench.py times (tensor-core engine, default split plan).

Config 2 (the benchmark workload) is compared with the fp64 oracle element by element.  Configs 3-5 are
compared with the oracle as whole blocks at their full cache length, width, head layout and kept rule, with
the number of reference tokens cut to 256 (the oracle's time grows with it; every other size is the
config's own), and as a three-block stack at config 3's shape, free-running and re-anchored per block.
Beside that every stage is checked at the full reference-set size on what the oracle can compute one by
one (sampled attention rows at full cache length, the full Gram, the full ridge solve) and on properties
that hold at any size (stationarity of the ridge solution, the ridge residual identity between the
returned states)."""
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
    return binding


@pytest.mark.parametrize("solver", [0, 1])
def test_config2_whole_block_matches_oracle(B, solver):
    import torch
    cfg = gen.benchmark_config(2)
    lay = gen.gen_layer(cfg, 0)
    x = gen.gen_reference(cfg)
    ref = orc.build_patch(lay["weights"], lay["K"], lay["V"], lay["kept"], x, x, [0, cfg.N], cfg.L, cfg.lam0, cfg)
    ctx = B.PkvContext(B.dims_from_config(cfg), engine=B.ENGINE_AUTO, solver=solver)
    w = B.to_device(lay["weights"], cfg.dtype)
    kv = B.to_device({"K": lay["K"], "V": lay["V"]}, cfg.dtype)
    off, idx = gen.kept_to_csr(lay["kept"])
    xt = torch.from_numpy(x).cuda()
    out = ctx.build_patch(w, kv["K"], kv["V"], off, torch.from_numpy(idx).cuda(), xt, xt, [0, cfg.N], cfg.L, cfg.lam0)
    dW = out["dW"].cpu().numpy()
    err = H.rel_fro(dW, ref["dW"])
    print("solver %d:" % solver, "config 2 dW rel fro err %.3e  lambda %.5g (oracle %.5g)" % (err, out["stats"]["lambda_eff"], ref["lam"]))
    assert err <= DW_TOL
    np.testing.assert_allclose(out["stats"]["lambda_eff"], ref["lam"], rtol=1e-3)
    assert H.rel_fro(out["xF_next"].cpu().numpy(), ref["xF_next"]) <= 1e-3
    assert H.rel_fro(out["xC_next"].cpu().numpy(), ref["xC_next"]) <= 1e-3
    gap = out["xF_next"].double() - out["xC_next"].double()
    assert H.rel_fro(gap.cpu().numpy(), ref["xF_next"] - ref["xC_next"]) <= 2e-2
    np.testing.assert_allclose(out["stats"]["resid_fro2"], float((gap * gap).sum()), rtol=1e-3)
    np.testing.assert_allclose(out["stats"]["resid_fro2"], ref["res_fro2"], rtol=3e-2)
    # merge: bit-exact against the two stated roundings
    Wm = w["Wdown"].clone()
    ctx.merge(Wm, out["dW"])
    torch.cuda.synchronize()
    np.testing.assert_array_equal(Wm.float().cpu().numpy(), orc.merge(lay["weights"]["Wdown"], dW, "bf16"))
    ctx.close()


def sampled_attention_check(B, cfg, n_samples=48, seed=0):
    import torch
    r = np.random.default_rng(seed)
    N = cfg.N
    kvd = gen.gen_cache(cfg, 0)
    q = (r.standard_normal((2, N, cfg.Hq, cfg.hd)) * 1.3).astype(np.float32)
    k = r.standard_normal((2, N, cfg.Hkv, cfg.hd)).astype(np.float32)
    v = r.standard_normal((2, N, cfg.Hkv, cfg.hd)).astype(np.float32)
    kept = gen.select_kept(cfg, 0, kvd["K"], gen.gen_obs_queries(cfg, 0) if cfg.kept_rule == "window_topk" else None)
    off, idx = gen.kept_to_csr(kept)
    ctx = B.PkvContext(B.dims_from_config(cfg), engine=B.ENGINE_AUTO)
    kv = B.to_device({"K": kvd["K"], "V": kvd["V"]}, cfg.dtype)
    tq, tk, tv = (torch.from_numpy(t.reshape(2, N, -1)).cuda() for t in (q, k, v))
    gF, gC, gD = ctx.attention(tq, tk, tv, kv["K"], kv["V"], off, torch.from_numpy(idx).cuda(), [0, N])
    # compaction is bit-exact on every kept row
    Kc, Vc = ctx.gather_kept(kv["K"], kv["V"], off, torch.from_numpy(idx).cuda())
    Ko, Vo = orc.gather_cache(kvd["K"], kvd["V"], kept)
    np.testing.assert_array_equal(Kc.float().cpu().numpy(), np.concatenate(Ko))
    np.testing.assert_array_equal(Vc.float().cpu().numpy(), np.concatenate(Vo))
    gF, gC, gD = (t.cpu().numpy().reshape(N, cfg.Hq, cfg.hd) for t in (gF, gC, gD))
    ctx.close()
    toks = np.unique(np.concatenate([[0, 1, N - 1], r.integers(0, N, n_samples)]))
    worst = 0.0
    for h in r.choice(cfg.Hq, size=min(cfg.Hq, 6), replace=False):
        kh = h // cfg.g
        for stream, got, Kh, Vh in ((0, gF, kvd["K"][kh], kvd["V"][kh]), (1, gC, Ko[kh], Vo[kh])):
            # one query row at a time: cache rows + causal part of the chunk
            keys = np.concatenate([Kh.astype(np.float64), k[stream, :, kh].astype(np.float64)])
            vals = np.concatenate([Vh.astype(np.float64), v[stream, :, kh].astype(np.float64)])
            rows = len(Kh)
            want = np.zeros((len(toks), cfg.hd))
            for n, t in enumerate(toks):
                lg = keys[:rows + t + 1] @ q[stream, t, h].astype(np.float64) / np.sqrt(cfg.hd)
                p = np.exp(lg - lg.max())
                want[n] = (p / p.sum()) @ vals[:rows + t + 1]
            scale = np.abs(got[:, h]).max()
            worst = max(worst, np.abs(got[toks, h] - want).max() / scale)
    np.testing.assert_array_equal(gD, gF - gC)
    return worst


@pytest.mark.parametrize("cfg_id", [2, 3, 4, 5])
def test_attention_sampled_rows_at_full_cache_length(B, cfg_id):
    cfg = gen.benchmark_config(cfg_id)
    worst = sampled_attention_check(B, cfg)
    print("config %d attention sampled max rel err %.3e" % (cfg_id, worst))
    assert worst <= ATTN_TOL


@pytest.mark.parametrize("cfg_id", [3, 4, 5])
def test_statistics_and_ridge_solve_at_full_width(B, cfg_id):
    import torch
    cfg = gen.benchmark_config(cfg_id)
    r = np.random.default_rng(cfg_id)
    N, F, d = cfg.N, cfg.F, cfg.d
    # features with a decaying spectrum and a dominant direction, targets small differences
    X = (r.standard_normal((N, F)) * np.exp(r.uniform(-2, 0.5, F)) + 0.5 * r.standard_normal((N, 1))).astype(np.float32)
    R = (0.05 * r.standard_normal((N, d))).astype(np.float32)
    S_H, S_T = orc.sufficient_statistics(X, R)
    ctx = B.PkvContext(B.dims_from_config(cfg), engine=B.ENGINE_AUTO)
    gH, gT = ctx.gram(torch.from_numpy(X).cuda(), torch.from_numpy(R).cuda())
    assert H.rel_fro(gH.cpu().numpy(), S_H) <= 2e-4
    assert H.rel_fro(gT.cpu().numpy(), S_T) <= 2e-4
    lams = cfg.lam_sweep if cfg.lam_sweep else (cfg.lam0,)
    for lam0 in lams:
        lam = orc.ridge_lambda(S_H, lam0)
        dW, st = ctx.ridge_solve(gH, gT, lam0, B.LAMBDA_PAPER)
        dWn = dW.cpu().numpy().astype(np.float64)
        # stationarity of Eq. 6 in fp64 with the GPU's own statistics
        Hg, Tg = gH.cpu().numpy().astype(np.float64), gT.cpu().numpy().astype(np.float64)
        lam_g = st["lambda_eff"]
        stat = np.linalg.norm(dWn @ Hg + lam_g * dWn - Tg) / np.linalg.norm(Tg)
        want = orc.ridge_solve(S_H, S_T, lam)
        err = H.rel_fro(dWn, want)
        print("config %d lambda0 %g: dW rel fro err %.3e, stationarity %.3e, min pivot %.3g" %
              (cfg_id, lam0, err, stat, st["min_pivot"]))
        np.testing.assert_allclose(lam_g, lam, rtol=1e-3)
        assert err <= 2e-3
        assert stat <= 2e-3
    ctx.close()


@pytest.mark.parametrize("cfg_id", [3, 4, 5])
def test_whole_block_runs_at_full_size_and_keeps_the_ridge_identities(B, cfg_id):
    import torch
    cfg = gen.benchmark_config(cfg_id)
    lay = gen.gen_layer(cfg, 0)
    x = gen.gen_reference(cfg)
    ctx = B.PkvContext(B.dims_from_config(cfg), engine=B.ENGINE_AUTO)
    w = B.to_device(lay["weights"], cfg.dtype)
    kv = B.to_device({"K": lay["K"], "V": lay["V"]}, cfg.dtype)
    off, idx = gen.kept_to_csr(lay["kept"])
    xt = torch.from_numpy(x).cuda()
    out = ctx.build_patch(w, kv["K"], kv["V"], off, torch.from_numpy(idx).cuda(), xt, xt, [0, cfg.N], cfg.L, cfg.lam0)
    st = out["stats"]
    assert torch.isfinite(out["dW"]).all() and st["min_pivot"] > 0
    np.testing.assert_allclose(st["lambda_eff"], cfg.lam0 * st["fro2"] / st["trace"], rtol=1e-5)    # Eq. 7
    gap = out["xF_next"].double() - out["xC_next"].double()
    np.testing.assert_allclose(float((gap * gap).sum()), st["resid_fro2"], rtol=1e-3)
    assert 0 < st["resid_fro2"] < st["target_fro2"]          # the patch reduces the block-output gap
    np.testing.assert_allclose(float((out["dW"].double() ** 2).sum()), st["dW_fro2"], rtol=1e-4)
    print("config %d: lambda %.4g, ||T||^2 %.4g -> residual %.4g" % (cfg_id, st["lambda_eff"], st["target_fro2"],
                                                                     st["resid_fro2"]))
    ctx.close()


# ------------------------------------------------------------------ whole blocks of configs 3-5 vs the oracle

N_CUT = 256        # reference tokens of the whole-block comparisons below (the configs' own N is 1024-4096)


def device_layer(B, cfg, lay):
    import torch
    off, idx = gen.kept_to_csr(lay["kept"])
    kv = B.to_device({"K": lay["K"], "V": lay["V"]}, cfg.dtype)
    return {"w": B.to_device(lay["weights"], cfg.dtype), "K": kv["K"], "V": kv["V"], "head_off": off,
            "idx": torch.from_numpy(idx).cuda()}


@pytest.mark.parametrize("cfg_id", [3, 4, 5])
def test_whole_block_matches_oracle_at_the_shapes_of_configs_3_to_5(B, cfg_id):
    """Full L, d, F, head layout and kept rule of the config; N cut to N_CUT to bound the oracle's time.
    Config 4 is checked at the three ridge coefficients of its sweep (one oracle forward, three solves)."""
    import torch
    cfg = gen.scaled_config(gen.benchmark_config(cfg_id), N=N_CUT)
    lay = gen.gen_layer(cfg, 0)
    x = gen.gen_reference(cfg)
    lams = cfg.lam_sweep if cfg.lam_sweep else (cfg.lam0,)
    ref = orc.build_patch(lay["weights"], lay["K"], lay["V"], lay["kept"], x, x, [0, cfg.N], cfg.L, lams[0], cfg,
                          keep_intermediates=True)
    ctx = B.PkvContext(B.dims_from_config(cfg), engine=B.ENGINE_AUTO)
    dl = device_layer(B, cfg, lay)
    xt = torch.from_numpy(x).cuda()
    for lam0 in lams:
        lam = orc.ridge_lambda(ref["S_H"], lam0)
        want = orc.ridge_solve(ref["S_H"], ref["S_T"], lam)
        out = ctx.build_patch(dl["w"], dl["K"], dl["V"], dl["head_off"], dl["idx"], xt, xt, [0, cfg.N], cfg.L, lam0)
        err = H.rel_fro(out["dW"].cpu().numpy(), want)
        eF = H.rel_fro(out["xF_next"].cpu().numpy(), ref["xF_next"])
        xC_want = ref["stu"]["z"] + ref["H"] @ (lay["weights"]["Wdown"].astype(np.float64) + want).T
        eC = H.rel_fro(out["xC_next"].cpu().numpy(), xC_want)
        print("config %d shape, N=%d, lambda0 %g: dW rel fro err %.3e, xF_next %.2e, xC_next %.2e, lambda %.5g (oracle %.5g)"
              % (cfg_id, cfg.N, lam0, err, eF, eC, out["stats"]["lambda_eff"], lam))
        assert err <= DW_TOL
        np.testing.assert_allclose(out["stats"]["lambda_eff"], lam, rtol=1e-3)
        np.testing.assert_allclose(out["stats"]["target_fro2"], ref["T_fro2"], rtol=2e-2)
        assert eF <= 1e-3 and eC <= 1e-3
    ctx.close()


def test_three_block_stack_at_config3_shape_free_running_and_reanchored(B):
    """Algorithm 1 over blocks through pkv_build_stack (teacher run ahead on its own stream) at config 3's
    full L, d, F and kept rule; N cut to 128, three blocks.  Free-running: both sides propagate their own
    states.  Re-anchored: the oracle's block l is fed the states the CUDA path produced for it, which is the
    contract of one block; those states come from a stack call over the blocks before l, and the patch from a
    call that resumes at first_layer = l."""
    import torch
    nl = 3
    cfg = gen.scaled_config(gen.benchmark_config(3), N=128, n_layers=nl)
    lays = [gen.gen_layer(cfg, l) for l in range(nl)]
    x0 = gen.gen_reference(cfg)
    ctx = B.PkvContext(B.dims_from_config(cfg), engine=B.ENGINE_AUTO)
    dl = [device_layer(B, cfg, lay) for lay in lays]
    xt = torch.from_numpy(x0).cuda()
    out = ctx.build_stack(dl, xt, xt, [0, cfg.N], cfg.L, cfg.lam0)
    xF, xC = x0.astype(np.float64), x0.astype(np.float64)
    for l in range(nl):
        lay = lays[l]
        o = orc.build_patch(lay["weights"], lay["K"], lay["V"], lay["kept"], xF, xC, [0, cfg.N], cfg.L, cfg.lam0, cfg)
        e_free = H.rel_fro(out["dW"][l].cpu().numpy(), o["dW"])
        msg = "block %d: free-running dW rel fro err %.3e" % (l, e_free)
        assert e_free <= DW_TOL, msg
        if l > 0:
            pre = ctx.build_stack(dl[:l], xt, xt, [0, cfg.N], cfg.L, cfg.lam0)          # states entering block l
            res = ctx.build_stack(dl, pre["xF_final"], pre["xC_final"], [0, cfg.N], cfg.L, cfg.lam0, first_layer=l)
            oa = orc.build_patch(lay["weights"], lay["K"], lay["V"], lay["kept"], pre["xF_final"].cpu().numpy(),
                                 pre["xC_final"].cpu().numpy(), [0, cfg.N], cfg.L, cfg.lam0, cfg)
            e_anch = H.rel_fro(res["dW"][l].cpu().numpy(), oa["dW"])
            msg += ", re-anchored %.3e" % e_anch
            assert e_anch <= DW_TOL, msg
            # resuming reproduces the uninterrupted run up to the rounding of the attention's split merge: the states
            # entering block l come from a stack call whose launches (one block: both streams in one launch; more:
            # teacher and student apart) cut the cache into different numbers of splits
            assert H.rel_fro(res["dW"][l].cpu().numpy(), out["dW"][l].cpu().numpy()) <= 2e-3
        print(msg)
        xF, xC = o["xF_next"], o["xC_next"]
    eF = H.rel_fro(out["xF_final"].cpu().numpy(), xF)
    eC = H.rel_fro(out["xC_final"].cpu().numpy(), xC)
    print("final states: xF %.2e, xC %.2e" % (eF, eC))
    assert eF <= 1e-3 and eC <= 1e-3
    ctx.close()


def test_ridge_solve_at_the_true_mlp_width_of_llama3_8b(B):
    """F = d_ff = 14336 (the width the paper's W in R^{d x d_ff} has in the Llama-3-8B-shaped model): statistics from
    1024 reference tokens (rank-deficient, as in every benchmark config), solve against the oracle's fp64 Cholesky.
    d is cut to 256 rows of dW to bound the oracle's time; the F x F system is the full one."""
    import torch
    cfg = gen.scaled_config(gen.benchmark_config(2), F=14336, d=256, Hq=2, Hkv=1, N=1024, L=256, budget=16)
    r = np.random.default_rng(7)
    X = (r.standard_normal((cfg.N, cfg.F)) * np.exp(r.uniform(-1.5, 0.5, cfg.F))).astype(np.float32)
    R = (0.05 * r.standard_normal((cfg.N, cfg.d))).astype(np.float32)
    ctx = B.PkvContext(B.dims_from_config(cfg), engine=B.ENGINE_AUTO)
    gH, gT = ctx.gram(torch.from_numpy(X).cuda(), torch.from_numpy(R).cuda())
    S_H, S_T = orc.sufficient_statistics(X, R)
    assert H.rel_fro(gT.cpu().numpy(), S_T) <= 2e-4
    lam = orc.ridge_lambda(S_H, 0.1)
    want = orc.ridge_solve(S_H, S_T, lam)
    dW, st = ctx.ridge_solve(gH, gT, 0.1)
    err = H.rel_fro(dW.cpu().numpy(), want)
    print("F = 14336: dW rel fro err %.3e, lambda %.5g (oracle %.5g), min pivot %.3g" % (err, st["lambda_eff"], lam, st["min_pivot"]))
    np.testing.assert_allclose(st["lambda_eff"], lam, rtol=1e-3)
    assert err <= 2e-3
    ctx.close()


def test_low_rank_patch_at_config2_width(B):
    """Rank-32 patch (appendix) at d = F = 4096: the weighted truncation loss tr((dW - dW_r) S_H (dW - dW_r)^T) equals
    the sum of the discarded eigenvalues of dW S_H dW^T (the oracle's), the leading eigenvalues agree, and the
    factors have orthonormal columns.  The loss is insensitive to the order inside eigenvalue clusters, so this
    holds whether or not the 32nd gap is open."""
    import torch
    cfg = gen.benchmark_config(2)
    r, n = 32, 512
    rng = np.random.default_rng(61)
    X = rng.standard_normal((n, cfg.F)).astype(np.float32)
    basis = rng.standard_normal((cfg.F, 64)).astype(np.float32)
    mix = rng.standard_normal((64, cfg.d)).astype(np.float32)
    R = ((X @ basis) * (0.9 ** np.arange(64, dtype=np.float32))[None, :]) @ mix * np.float32(1e-2)
    S_H, S_T = orc.sufficient_statistics(X, R)
    dW = orc.ridge_solve(S_H, S_T, orc.ridge_lambda(S_H, 0.1))
    _, _, _, ev_o = orc.low_rank_patch(dW, S_H, r)
    ctx = B.PkvContext(B.dims_from_config(cfg), engine=B.ENGINE_AUTO)
    out = ctx.low_rank(torch.from_numpy(dW.astype(np.float32)).cuda(), torch.from_numpy(S_H.astype(np.float32)).cuda(), r)
    dWr = out["dW_r"].cpu().numpy().astype(np.float64)
    E = dW - dWr
    loss = float(np.sum((E @ S_H) * E))
    U = out["U"].cpu().numpy().astype(np.float64)
    print("rank-32 patch at d = F = 4096: weighted loss %.6g vs discarded eigenvalues %.6g (kept %.6g)"
          % (loss, ev_o[r:].sum(), ev_o[:r].sum()))
    np.testing.assert_allclose(loss, ev_o[r:].sum(), rtol=5e-3)
    np.testing.assert_allclose(out["ritz"].cpu().numpy()[:8], ev_o[:8], rtol=2e-3)
    np.testing.assert_allclose(U.T @ U, np.eye(r), atol=1e-5)
    ctx.close()

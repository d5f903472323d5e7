#!/usr/bin/env python
"""Benchmark of PatchKV patch construction.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--config 2] [--impl ours|reference]

A step is one pass of the whole path over one synthetic context: for the single-block workload (config 2, the
default and the headline) index check + compaction, teacher and student forward, targets, statistics, ridge
solve, next states and merge of one block; for the stack workloads (configs 3-5) the same for every block in
sequence (Algorithm 1's outer loop).  Prints ONE JSON line.  The default run also carries a `configs` block
(stack workloads, few steps each) and a `kernels` block (attention / statistics / solve alone, per config).
With --impl reference the fp64 CPU oracle is timed on a bounded sample of the same workload instead (host
cores; a deliberately slow baseline).
"""
from __future__ import annotations

import argparse
import gc
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2609_39329_b200 import dist_util as du  # noqa: E402
from paper_2609_39329_b200 import inputs as gen  # noqa: E402

# DRAM traffic of the ridge-solve stage at config 2, bytes per solve: dram__bytes_read.sum + dram__bytes_write.sum
# summed over every kernel of one pkv_ridge_solve call (profiles/ridge_solve_config2.md gives the command).
SOLVE_STAGE_TRAFFIC_CONFIG2 = 1.243e9


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            d = json.load(open(p))
            return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d["bf16_tflops"]),
                    "bf16_tflops_sustained": float(d.get("bf16_tflops_sustained", d["bf16_tflops"])),
                    "sm_max_mhz": float(d.get("sm_max_mhz", 1965.0)), "source": "measured"}
        except Exception:
            pass
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "sm_max_mhz": 1965.0,
            "source": "fallback"}


def stage_work(cfg, b_sum):
    """Algorithmic work per stage of one block: (name, flops, bytes, bound)."""
    N, d, F, L, Dq, Dkv, hd = cfg.N, cfg.d, cfg.F, cfg.L, cfg.Dq, cfg.Dkv, cfg.hd
    eb = 2 if cfg.dtype == "bf16" else 4
    b_mean = b_sum / cfg.Hkv
    return [
        ("S0 index check + compaction", 0.0, 2.0 * (2.0 * b_sum * hd * eb), "hbm"),
        ("S1-S2 norm + QKV + RoPE", 4.0 * N * d * (Dq + 2 * Dkv), 0.0, "tensor"),
        ("S3 dual-cache attention", 4.0 * N * L * Dq + 4.0 * N * b_mean * Dq + 4.0 * N * N * Dq,
         2.0 * (L + b_mean) * Dkv * eb, "tensor"),
        ("S4 o-proj + residual", 4.0 * N * Dq * d, 0.0, "tensor"),
        ("S5 norm + gate/up + SiLU", 8.0 * N * d * F, 0.0, "tensor"),
        ("S6 targets", 2.0 * N * F * d, 0.0, "tensor"),
        ("S7 Gram + cross statistics", float(N) * F * (F + 1) + 2.0 * N * F * d, 4.0 * (F * F + F * d), "tensor"),
        ("S8 ridge solve", F ** 3 / 3.0 + 2.0 * F * F * d, 0.0, "alu"),
        ("S9 next states", 4.0 * N * F * d, 0.0, "tensor"),
    ]


def layer_bounds(cfg, b_sum, peaks, fma_tflops):
    """Roofline time of one block, ms: tensor-eligible flops at the sustained bf16 peak, the solve's fp32 flops at the
    fp32 FMA peak, cache + weight + statistics bytes at the HBM peak.  Returns (sum, max) = without / with perfect
    overlap of the three."""
    work = stage_work(cfg, b_sum)
    tensor = sum(w[1] for w in work if w[3] == "tensor")
    alu = sum(w[1] for w in work if w[3] == "alu")
    eb = 2
    weights = eb * (cfg.d * (cfg.Dq + 2 * cfg.Dkv) + cfg.Dq * cfg.d + 3 * cfg.d * cfg.F)
    byts = sum(w[2] for w in work) + weights + 8.0 * cfg.F * cfg.d
    t_t = tensor / (peaks["bf16_tflops_sustained"] * 1e12) * 1e3
    t_a = alu / (fma_tflops * 1e12) * 1e3
    t_h = byts / (peaks["hbm_gbs"] * 1e9) * 1e3
    return t_t + t_a + t_h, max(t_t, t_a, t_h)


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.th = threading.Thread(target=self._read, daemon=True)
            self.th.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            pass
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
                for n, v in zip(names, r[2:6]):
                    if v.lower().startswith("active"):
                        reasons.add(n)
            except Exception:
                continue
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def build_inputs(cfg, layer=0):
    lay = gen.gen_layer(cfg, layer)
    lay["x0"] = gen.gen_reference(cfg)
    return lay


def oracle_sample(cfg, lay, n_sample):
    """Times the fp64 oracle on the first n_sample reference tokens (full cache, full d x F solve) and
    scales the token-proportional part to the workload's N.  Returns (ms per context, seconds spent)."""
    from oracle import pkv_oracle as orc
    sub = gen.scaled_config(cfg, N=n_sample)
    x = lay["x0"][:n_sample]
    t0 = time.perf_counter()
    out = orc.build_patch(lay["weights"], lay["K"], lay["V"], lay["kept"], x, x, [0, n_sample], cfg.L, cfg.lam0, sub,
                          keep_intermediates=True)
    t1 = time.perf_counter()
    lam = out["lam"]
    orc.ridge_solve(out["S_H"], out["S_T"], lam)
    t2 = time.perf_counter()
    t_solve = t2 - t1
    t_fwd = (t1 - t0) - t_solve
    est = t_fwd * (cfg.N / n_sample) + t_solve
    return est * 1e3, t2 - t0


def oracle_full(cfg, lay):
    """The fp64 oracle on the whole reference set of one block; returns (ms, seconds spent)."""
    from oracle import pkv_oracle as orc
    t0 = time.perf_counter()
    orc.build_patch(lay["weights"], lay["K"], lay["V"], lay["kept"], lay["x0"], lay["x0"], [0, cfg.N], cfg.L, cfg.lam0, cfg)
    dt = time.perf_counter() - t0
    return dt * 1e3, dt


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cfg = gen.benchmark_config(args.config)
    lay = build_inputs(cfg)
    cores = os.cpu_count() or 1
    if cfg.n_layers == 1 and args.ref_sample <= 0:
        # single-block workload: the oracle runs the whole workload every step (about 10 s per step on 16 cores)
        for _ in range(min(args.warmup, 1)):
            oracle_sample(cfg, lay, 8)
        vals = [oracle_full(cfg, lay)[0] for _ in range(args.steps)]
        val = float(np.mean(vals))
        sample = "fp64 numpy oracle on the whole workload (all %d reference tokens, L=%d cache, %dx%d solve), every step" % (
            cfg.N, cfg.L, cfg.d, cfg.F)
    else:
        n_sample = min(cfg.N, args.ref_sample if args.ref_sample > 0 else 32)
        for _ in range(min(args.warmup, 1)):
            oracle_sample(cfg, lay, max(n_sample // 4, 4))
        vals = [oracle_sample(cfg, lay, n_sample)[0] for _ in range(args.steps)]
        val = float(np.mean(vals)) * cfg.n_layers
        sample = ("fp64 numpy oracle on the first %d of %d reference tokens of one block (full L=%d cache, full %dx%d solve), "
                  "token-proportional part scaled by %d/%d (an over-estimate: the oracle's per-head set-up does not grow "
                  "with the tokens)%s" % (n_sample, cfg.N, cfg.L, cfg.d, cfg.F, cfg.N, n_sample,
                                          "" if cfg.n_layers == 1 else ", multiplied by %d blocks" % cfg.n_layers))
    line = {"impl": "reference", "metric": "patch_build_ms_per_context", "value": val, "unit": "ms",
            "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": val,
            "higher_is_better": False, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": workload_config(cfg, lay),
            "cpu_baseline": {"value": val, "unit": "ms", "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": val, "unit": "ms", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def workload_config(cfg, lay):
    b = [int(len(k)) for k in lay["kept"]]
    return {"workload": "config %d: %s" % (cfg.cfg_id, cfg.name), "layers_per_step": cfg.n_layers, "d": cfg.d,
            "F": cfg.F, "Hq": cfg.Hq, "Hkv": cfg.Hkv, "hd": cfg.hd, "L": cfg.L, "n_ref": cfg.N, "kept_per_head": b[0],
            "lambda0": cfg.lam0, "lambda_mode": "paper (Eq. 7)", "seed": cfg.seed,
            "l2": "inputs (weights + caches, >300 MB) exceed L2 and a 512 MB buffer is written between steps"}


def timed(torch, fn, steps, flush):
    """Mean device time of fn over `steps` calls, CUDA events on the current stream, L2 flushed before each."""
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    for i in range(steps):
        flush.fill_(i & 0xFF)
        ev[i][0].record()
        fn()
        ev[i][1].record()
    torch.cuda.synchronize()
    return float(sum(a.elapsed_time(b) for a, b in ev) / steps)


def measure_kernel(kind, cfg, B, torch, peaks, fma_tflops, steps, warmup, flush):
    """One stage alone, through its single-stage entry point, on the shapes of a benchmark config."""
    r = np.random.default_rng(cfg.seed)
    N, F, d = cfg.N, cfg.F, cfg.d
    if kind == "attention":
        kvd = gen.gen_cache(cfg, 0)
        kept = gen.select_kept(cfg, 0, kvd["K"], gen.gen_obs_queries(cfg, 0) if cfg.kept_rule == "window_topk" else None)
        off, idx = gen.kept_to_csr(kept)
        ctx = B.PkvContext(B.dims_from_config(cfg, b_max=max(len(k) for k in kept)))
        kv = B.to_device({"K": kvd["K"], "V": kvd["V"]}, cfg.dtype)
        q = torch.from_numpy((r.standard_normal((2, N, cfg.Dq)) * 1.3).astype(np.float32)).cuda()
        k = torch.from_numpy(r.standard_normal((2, N, cfg.Dkv)).astype(np.float32)).cuda()
        v = torch.from_numpy(r.standard_normal((2, N, cfg.Dkv)).astype(np.float32)).cuda()
        idx_t = torch.from_numpy(idx).cuda()
        fn = lambda: ctx.attention(q, k, v, kv["K"], kv["V"], off, idx_t, [0, N])
        b_mean = sum(len(k_) for k_ in kept) / cfg.Hkv
        flops = 4.0 * N * cfg.L * cfg.Dq + 4.0 * N * b_mean * cfg.Dq + 4.0 * N * N * cfg.Dq
        bound, note = "tensor", "key conversion to fp16 + operand preparation + attention kernel + combine; executed MMA work = algorithmic work (fp16 Q against fp16 K, bf16 P against bf16 V)"
    elif kind == "gram":
        ctx = B.PkvContext(B.dims_from_config(cfg, b_max=16))
        X = torch.from_numpy(r.standard_normal((N, F)).astype(np.float32)).cuda()
        R = torch.from_numpy((0.1 * r.standard_normal((N, d))).astype(np.float32)).cuda()
        S_H = torch.zeros((F, F), dtype=torch.float32, device="cuda")
        S_T = torch.zeros((d, F), dtype=torch.float32, device="cuda")
        fn = lambda: ctx.gram(X, R, S_H, S_T)
        flops = float(N) * F * (F + 1) + 2.0 * N * F * d
        bound, note = "tensor", "two transposing splits + two three-pass products; symmetric half counted once"
    else:
        ctx = B.PkvContext(B.dims_from_config(cfg, b_max=16))
        X = r.standard_normal((N, F)).astype(np.float32)
        S_H = torch.from_numpy(X.T @ X).cuda()
        S_T = torch.from_numpy((0.1 * r.standard_normal((d, F))).astype(np.float32)).cuda()
        fn = lambda: ctx.ridge_solve(S_H, S_T, cfg.lam0, B.LAMBDA_PAPER)
        flops = F ** 3 / 3.0 + 2.0 * F * F * d
        bound = "alu"
        note = ("fp32-equivalent solve executed as multi-pass tensor-core products plus one single-CTA factor kernel per "
                "128 columns (latency-bound chain of F/128 steps); measured fp32 FMA rate as the reference")
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    ms = timed(torch, fn, steps, flush)
    peak = peaks["bf16_tflops_sustained"] if bound == "tensor" else fma_tflops
    ach = flops / (ms * 1e-3) / 1e12
    ctx.close()
    del ctx
    gc.collect()
    torch.cuda.empty_cache()
    return {"kernel": kind, "config": cfg.cfg_id, "ms": ms, "algorithmic_flops": flops, "bound": bound,
            "achieved_tflops": ach, "peak_tflops": peak, "frac": ach / peak, "note": note}


def measure_stack(cfg, B, torch, peaks, fma_tflops, steps, warmup, flush, distinct, reserve_sms, engine, world=1,
                  rank=0, dist=None, want_stages=True):
    """Patches for all blocks of a stack workload built in sequence (pkv_build_stack).  `distinct` layers are
    generated with their own seeded weights and caches and the stack cycles through them (every layer has the same
    shapes and the per-layer working set is far larger than L2 either way)."""
    D = max(1, min(distinct, cfg.n_layers))
    lays = [build_inputs(cfg, l) for l in range(D)]
    b_max = max(len(k) for lay in lays for k in lay["kept"])
    ctx = B.PkvContext(B.dims_from_config(cfg, b_max=b_max), engine=engine, reserve_sms=reserve_sms)
    dev = []
    for lay in lays:
        off, idx = gen.kept_to_csr(lay["kept"])
        kv = B.to_device({"K": lay["K"], "V": lay["V"]}, cfg.dtype)
        dev.append({"w": B.to_device(lay["weights"], cfg.dtype), "K": kv["K"], "V": kv["V"], "head_off": off,
                    "idx": torch.from_numpy(idx).cuda()})
    layers = [dev[l % D] for l in range(cfg.n_layers)]
    x_t = torch.from_numpy(lays[0]["x0"]).cuda()
    W_merged = [d_["w"]["Wdown"].clone() for d_ in dev]
    chunk_off = [0, cfg.N]
    lams = list(cfg.lam_sweep) if cfg.lam_sweep else [cfg.lam0]

    def step(lam):
        out = ctx.build_stack(layers, x_t, x_t, chunk_off, cfg.L, lam, B.LAMBDA_PAPER, want_final=True)
        for l, dWl in enumerate(out["dW"]):
            ctx.merge(W_merged[l % D], dWl)
        return out

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(warmup):
        step(lams[0])
    barrier()
    l0 = ctx.launch_count()
    per_lam, n_steps = [], 0
    for lam in lams:
        per_lam.append(timed(torch, lambda: step(lam), steps, flush))
        n_steps += steps
        barrier()
    launches = ctx.launch_count() - l0 + n_steps * cfg.n_layers
    ms = float(sum(per_lam) / len(per_lam))
    res = {"ms_overlapped": ms, "ms_per_lambda": per_lam, "launches": int(launches), "steps": steps,
           "teacher_sms": ctx.teacher_sm_count()}
    # the same stack block by block (one host synchronisation per block, no teacher running ahead): every block takes the
    # single block's schedule, student half first and teacher half beside its own solve
    if engine != B.ENGINE_SIMT:
        ctx.set_stack_schedule(True)
        step(lams[0])
        res["ms_sequential"] = timed(torch, lambda: step(lams[0]), max(1, min(steps, 2)), flush)
        ctx.set_stack_schedule(False)
    # ridge-coefficient sweep with the teacher run once (pkv_build_stack_sweep)
    if len(lams) > 1 and engine != B.ENGINE_SIMT:
        cache = None

        def sweep():
            nonlocal cache
            out = ctx.build_stack_sweep(layers, x_t, x_t, chunk_off, cfg.L, lams, B.LAMBDA_PAPER, cache=cache)
            cache = out["cache"]
            return out
        sweep()
        res["ms_sweep_teacher_once"] = timed(torch, sweep, max(1, min(steps, 2)), flush)
        res["ms_sweep_separate_stacks"] = float(sum(per_lam))
        del cache
    if want_stages:
        ctx.set_timing(True)
        step(lams[-1])
        st = step(lams[-1])["stats"]
        ctx.set_timing(False)
        res["stage_ms_sequential_driver"] = [round(sum(s_["stage_ms"][i] for s_ in st), 3) for i in range(9)]
    b_list = [len(k) for k in lays[0]["kept"]]
    work = stage_work(cfg, sum(b_list))
    res["flops"] = sum(wk[1] for wk in work) * cfg.n_layers
    b_no, b_ov = layer_bounds(cfg, sum(b_list), peaks, fma_tflops)
    res["bound_ms_no_overlap"] = b_no * cfg.n_layers
    res["bound_ms_perfect_overlap"] = b_ov * cfg.n_layers
    res["lays0"] = lays[0]
    res["lams"] = lams
    res["distinct"] = D
    ctx.close()
    del ctx, dev, layers, W_merged
    gc.collect()
    torch.cuda.empty_cache()
    return res


def stack_summary(cfg, r, peaks):
    ms = r["ms_overlapped"]
    out = {"workload": "config %d: %s" % (cfg.cfg_id, cfg.name), "layers": cfg.n_layers, "n_ref": cfg.N, "L": cfg.L,
           "steps": r["steps"], "ms_per_context": ms, "ms_per_layer": ms / cfg.n_layers,
           "driver": "teacher run ahead on its own stream (%d of the SMs), student + solve beside it" % r["teacher_sms"],
           "ms_per_context_block_by_block": r.get("ms_sequential"),
           "algorithmic_tflops": r["flops"] / (ms * 1e-3) / 1e12,
           "frac_bf16_peak_all_flops": r["flops"] / (ms * 1e-3) / 1e12 / peaks["bf16_tflops_sustained"],
           "bound_ms": {"no_overlap": r["bound_ms_no_overlap"], "perfect_overlap": r["bound_ms_perfect_overlap"]},
           "time_over_bound_no_overlap": ms / r["bound_ms_no_overlap"],
           "distinct_layers_generated": r["distinct"], "lambda0": r["lams"] if len(r["lams"]) > 1 else r["lams"][0]}
    if len(r["lams"]) > 1:
        out["ms_per_lambda"] = r["ms_per_lambda"]
        out["sweep_ms"] = {"teacher_once": r.get("ms_sweep_teacher_once"), "separate_stacks": r.get("ms_sweep_separate_stacks")}
    if "stage_ms_sequential_driver" in r:
        out["stage_ms_sequential_driver"] = r["stage_ms_sequential_driver"]
    return out


def run_stack(args, cfg, B, torch, dist, world, rank, local, peaks):
    """Configs 3-5 as the headline: a step is one context = n_layers blocks."""
    if world > 1:
        cfg = gen.scaled_config(cfg, seed=du.rank_seed(cfg.seed, rank))
    engine = B.ENGINE_SIMT if args.engine == "simt" else B.ENGINE_AUTO
    flush = torch.empty(512 << 20, dtype=torch.uint8, device="cuda")
    probe = B.PkvContext(B.dims_from_config(gen.benchmark_config(2), b_max=16))
    fma = probe.measure_fma_peak()
    probe.close()
    sampler = ClockSampler(local)
    sampler.start()
    r = measure_stack(cfg, B, torch, peaks, fma, args.steps, args.warmup if args.quick else max(args.warmup, 3), flush,
                      args.distinct_layers, args.reserve_sms, engine, world, rank, dist)
    clocks = sampler.stop()
    ms = du.max_over_ranks(r["ms_overlapped"], "cuda")
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return
    summ = stack_summary(cfg, r, peaks)
    stage_ms = r.get("stage_ms_sequential_driver", [0] * 9)
    b_list = [len(k) for k in r["lays0"]["kept"]]
    work = stage_work(cfg, sum(b_list))
    dom = int(np.argmax(stage_ms))
    name, fl, by, bound = work[dom]
    dur_ms = stage_ms[dom]      # stage times of a stack come from the block-by-block driver's own pass
    dur = dur_ms * 1e-3
    fl *= cfg.n_layers
    if bound == "tensor":
        peak, unit, ach, note = peaks["bf16_tflops_sustained"], "TFLOP/s", fl / dur / 1e12, "bf16 dense, sustained, %s" % peaks["source"]
    elif bound == "alu":
        peak, unit, ach = fma, "TFLOP/s", fl / dur / 1e12
        note = ("fp32 FMA rate measured in this run; the stage runs as tensor-core products plus a latency-bound chain of "
                "single-CTA factor kernels")
    else:
        peak, unit, ach, note = peaks["hbm_gbs"], "GB/s", by * cfg.n_layers / dur / 1e9, "HBM copy, %s" % peaks["source"]
    cpu = None
    if not args.no_cpu_baseline and world == 1 and not args.quick:
        n_sample = min(cfg.N, 16)
        v, spent = oracle_sample(cfg, r["lays0"], n_sample)
        cpu = {"value": v * cfg.n_layers, "unit": "ms", "cores": os.cpu_count() or 1, "kind": "oracle",
               "sample": "fp64 numpy oracle on layer 0, first %d of %d reference tokens, full cache and full solve, token "
                         "part scaled by %d/%d, extrapolated from 1 layer to %d; %.1f s of CPU wall time" %
                         (n_sample, cfg.N, cfg.N, n_sample, cfg.n_layers, spent)}
    conf = workload_config(cfg, r["lays0"])
    conf.update({"distinct_layers_generated": r["distinct"], "lambda0": r["lams"] if len(r["lams"]) > 1 else r["lams"][0]})
    line = {"metric": "patch_build_ms_per_context", "value": ms / world, "unit": "ms", "n_gpus": world,
            "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms, "ms_per_layer": ms / cfg.n_layers,
            "higher_is_better": False, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
            "data": "synthetic", "config": conf, "engine": "simt-fp32" if engine == B.ENGINE_SIMT else "tcgen05",
            "timed_driver": "overlapped (teacher run ahead); stage times below come from the sequential driver",
            "stack": summ,
            "algorithmic_tflops": r["flops"] / (ms * 1e-3) / 1e12,
            "frac_bf16_peak_all_flops": r["flops"] / (ms * 1e-3) / 1e12 / peaks["bf16_tflops_sustained"],
            "roofline": {"kernel": name + " (stage, sequential driver)", "bound": bound, "achieved": ach, "peak": peak,
                         "unit": unit, "frac": ach / peak, "traffic": None, "peak_note": note, "stage_ms": stage_ms[dom]},
            "stages": [{"stage": wk[0], "ms": round(t_, 3)} for wk, t_ in zip(work, stage_ms)],
            "cpu_baseline": cpu, "clocks": clocks,
            "e2e": {"value": None, "unit": "ms", "h2d_bytes_per_step": None, "d2h_bytes_per_step": None,
                    "note": "end-to-end with host buffers is measured on the single-block workload (default config 2)"},
            "gpu_launches": r["launches"], "peaks": dict(peaks, fp32_fma_tflops_measured=fma)}
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", type=int, default=2)
    ap.add_argument("--impl", default="ours")
    ap.add_argument("--engine", default="auto", choices=["auto", "simt"])
    ap.add_argument("--ref-sample", type=int, default=0,
                    help="reference tokens the oracle is timed on (token-proportional part scaled to the workload); "
                         "0 = the whole workload for the single-block config, 32 for the stack configs")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extras", action="store_true",
                    help="default workload only: skip the `configs` (stack workloads) and `kernels` blocks")
    ap.add_argument("--distinct-layers", type=int, default=2,
                    help="stack configs: layers generated with their own weights/caches; the stack cycles through them")
    ap.add_argument("--kernel", default=None, choices=["attention", "gram", "solve"],
                    help="time one stage alone through its own entry point (pkv_attention / pkv_gram / pkv_ridge_solve) "
                         "on the shapes of --config, with seeded random operands")
    ap.add_argument("--reserve-sms", type=int, default=0,
                    help="stack configs: SMs the teacher stream leaves free (0 = library default, negative = none)")
    ap.add_argument("--quick", action="store_true",
                    help="timed steps only (no stage pass, no end-to-end pass, no CPU baseline): for profiler runs")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
        return

    import torch
    import torch.distributed as dist
    from paper_2609_39329_b200 import binding as B

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    peaks = measured_peaks()
    cfg = gen.benchmark_config(args.config)
    if args.kernel:
        flush = torch.empty(512 << 20, dtype=torch.uint8, device="cuda")
        probe = B.PkvContext(B.dims_from_config(gen.benchmark_config(2), b_max=16))
        fma = probe.measure_fma_peak()
        probe.close()
        k = measure_kernel(args.kernel, cfg, B, torch, peaks, fma, args.steps,
                           args.warmup if args.quick else max(args.warmup, 3), flush)
        print(json.dumps({"kernel": k["kernel"], "config": "config %d: %s" % (cfg.cfg_id, cfg.name), "ms": k["ms"],
                          "algorithmic_flops": k["algorithmic_flops"],
                          "roofline": {"bound": k["bound"], "achieved": k["achieved_tflops"], "peak": k["peak_tflops"],
                                       "unit": "TFLOP/s", "frac": k["frac"], "note": k["note"]}, "steps": args.steps}))
        return
    if cfg.n_layers > 1:
        run_stack(args, cfg, B, torch, dist, world, rank, local, peaks)
        return
    if world > 1:      # replicas only: every rank builds the patch of its own context
        cfg = gen.scaled_config(cfg, seed=du.rank_seed(cfg.seed, rank))
    lay = build_inputs(cfg)
    b_list = [len(k) for k in lay["kept"]]
    off, idx = gen.kept_to_csr(lay["kept"])

    engine = B.ENGINE_SIMT if args.engine == "simt" else B.ENGINE_AUTO
    ctx = B.PkvContext(B.dims_from_config(cfg, b_max=max(b_list)), engine=engine)
    w = B.to_device(lay["weights"], cfg.dtype)
    kv = B.to_device({"K": lay["K"], "V": lay["V"]}, cfg.dtype)
    idx_t = torch.from_numpy(idx).cuda()
    x_t = torch.from_numpy(lay["x0"]).cuda()
    W_merged = w["Wdown"].clone()
    dW = torch.empty((cfg.d, cfg.F), dtype=torch.float32, device="cuda")
    flush = torch.empty(512 << 20, dtype=torch.uint8, device="cuda")
    chunk_off = [0, cfg.N]

    def step():
        out = ctx.build_patch(w, kv["K"], kv["V"], off, idx_t, x_t, x_t, chunk_off, cfg.L, cfg.lam0, B.LAMBDA_PAPER,
                              True, dW=dW)
        ctx.merge(W_merged, dW)
        return out

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup if args.quick else max(args.warmup, 3)):
        step()
    barrier()
    sampler = ClockSampler(local)
    sampler.start()
    l0 = ctx.launch_count()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    for i in range(args.steps):
        flush.fill_(i & 0xFF)           # L2 flush, outside the timed events
        ev[i][0].record()
        step()
        ev[i][1].record()
    barrier()
    launches = ctx.launch_count() - l0 + args.steps      # + one merge kernel per step
    times = [a.elapsed_time(b) for a, b in ev]
    ms = float(sum(times) / len(times))
    ms = du.max_over_ranks(ms, "cuda")

    if args.quick:
        sampler.stop()
        if rank == 0:
            print(json.dumps({"metric": "patch_build_ms_per_context", "value": ms / world, "unit": "ms",
                              "n_gpus": world, "steps": args.steps, "quick": True, "gpu_launches": int(launches)}))
        if world > 1:
            dist.destroy_process_group()
        return

    # per-stage device times (separate pass with the library's stage events)
    ctx.set_timing(True)
    step()                  # the stacked schedule's first call captures its own solve graph: not a timed one
    stage_acc = None
    for i in range(5):
        flush.fill_(i)
        st = step()["stats"]["stage_ms"][:9]
        stage_acc = st if stage_acc is None else [a + b for a, b in zip(stage_acc, st)]
    stage_ms = [a / 5 for a in stage_acc]
    # the ridge solve's interval inside the schedule that `value` is timed on (the teacher half runs beside it)
    ctx.set_timing(2)
    step()
    s8_acc = 0.0
    for i in range(5):
        flush.fill_(i)
        s8_acc += step()["stats"]["stage_ms"][7]
    s8_timed_schedule = s8_acc / 5
    ctx.set_timing(False)
    work = stage_work(cfg, sum(b_list))
    total_flops = sum(wk[1] for wk in work)
    fma = ctx.measure_fma_peak()

    # end to end through the public call with host buffers: H2D of every input, D2H of the patch
    host = {k: v.cpu().pin_memory() for k, v in {**w, "K": kv["K"], "V": kv["V"], "idx": idx_t, "x": x_t}.items()}
    dev = {k: torch.empty_like(v, device="cuda") for k, v in host.items()}
    dW_host = torch.empty((cfg.d, cfg.F), dtype=torch.float32).pin_memory()
    h2d = sum(v.numel() * v.element_size() for v in host.values())
    d2h = dW_host.numel() * 4

    def e2e_step():
        for k in host:
            dev[k].copy_(host[k], non_blocking=True)
        wd = {k: dev[k] for k in w}
        ctx.build_patch(wd, dev["K"], dev["V"], off, dev["idx"], dev["x"], dev["x"], chunk_off, cfg.L, cfg.lam0,
                        B.LAMBDA_PAPER, True, dW=dW)
        dW_host.copy_(dW, non_blocking=True)
        torch.cuda.synchronize()

    e2e_step()
    barrier()
    e2e_n = max(3, min(args.steps, 5))
    t0 = time.perf_counter()
    for _ in range(e2e_n):
        e2e_step()
    barrier()
    e2e_ms = (time.perf_counter() - t0) * 1e3 / e2e_n
    clocks = sampler.stop()      # sampled over the timed steps, the stage pass and the end-to-end pass
    e2e_ms = du.max_over_ranks(e2e_ms, "cuda")
    del host, dev

    # the same block through the dual (N x N) solver option: same dW, reported beside the headline
    dual_ms = None
    if cfg.N <= cfg.F and engine != B.ENGINE_SIMT:
        ctx_d = B.PkvContext(B.dims_from_config(cfg, b_max=max(b_list)), engine=engine, solver=B.SOLVER_DUAL)

        def step_d():
            ctx_d.build_patch(w, kv["K"], kv["V"], off, idx_t, x_t, x_t, chunk_off, cfg.L, cfg.lam0, B.LAMBDA_PAPER,
                              True, dW=dW)
            ctx_d.merge(W_merged, dW)
        for _ in range(3):
            step_d()
        dual_ms = timed(torch, step_d, 5, flush)
        ctx_d.close()
        del ctx_d

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # roofline of the dominant stage
    dom = int(np.argmax(stage_ms))
    name, fl, by, bound = work[dom]
    dur_ms = s8_timed_schedule if (dom == 7 and s8_timed_schedule > 0) else stage_ms[dom]
    dur = dur_ms * 1e-3
    traffic = None
    if bound == "tensor":
        peak, unit, ach = peaks["bf16_tflops_sustained"], "TFLOP/s", fl / dur / 1e12
        peak_note = "bf16 dense, sustained, %s" % peaks["source"]
    elif bound == "alu":
        peak, unit, ach = fma, "TFLOP/s", fl / dur / 1e12
        nsteps = (cfg.F + 127) // 128
        peak_note = ("fp32 FMA rate measured in this run (register-resident FMA kernel, CUDA events); the stage stands "
                     "for fp32 arithmetic but runs as multi-pass tensor-core products plus a chain of %d single-CTA factor "
                     "kernels, one per 128 columns: it is bound by that chain's latency (%.1f us per step if the whole stage "
                     "were chain), not by FMA throughput; the stage is timed inside the schedule of `value`, with the "
                     "teacher half running beside it (%.3f ms; %.3f ms with nothing beside it, stacked schedule)"
                     % (nsteps, dur_ms * 1e3 / nsteps, dur_ms, stage_ms[dom]))
        if cfg.cfg_id == 2:
            traffic = SOLVE_STAGE_TRAFFIC_CONFIG2
    else:
        peak, unit, ach = peaks["hbm_gbs"], "GB/s", by / dur / 1e9
        peak_note = "HBM copy, %s" % peaks["source"]
    roofline = {"kernel": name + " (stage: k_chain128 chain + k_gemm_tc products)" if bound == "alu" else name,
                "bound": bound, "achieved": ach, "peak": peak, "unit": unit, "frac": ach / peak,
                "traffic": traffic, "peak_note": peak_note, "stage_ms": dur_ms,
                "stage_ms_stacked_schedule": stage_ms[dom]}
    stages = [{"stage": wk[0], "ms": round(t, 4), "algorithmic_tflops": (wk[1] / (t * 1e-3) / 1e12) if t > 0 else None}
              for wk, t in zip(work, stage_ms)]
    tensor_flops = sum(wk[1] for wk in work if wk[3] == "tensor")
    tensor_ms = sum(t for wk, t in zip(work, stage_ms) if wk[3] == "tensor")
    b_no, b_ov = layer_bounds(cfg, sum(b_list), peaks, fma)

    cpu = None
    if not args.no_cpu_baseline and world == 1:
        v, spent = oracle_full(cfg, lay)
        cpu = {"value": v, "unit": "ms", "cores": os.cpu_count() or 1, "kind": "oracle",
               "sample": "fp64 numpy oracle on the whole workload once (all %d reference tokens, full cache, full solve); "
                         "%.1f s of CPU wall time" % (cfg.N, spent)}
        n_sample = min(cfg.N, args.ref_sample if args.ref_sample > 0 else 32)
        v2, _ = oracle_sample(cfg, lay, n_sample)
        cpu["extrapolated_from_%d_tokens_ms" % n_sample] = v2      # what a token-proportional scaling of a sample predicts

    ctx.close()
    del ctx, kv, w
    gc.collect()
    torch.cuda.empty_cache()

    # side blocks of the default run: the stack workloads (few steps each) and the three hot kernels alone
    configs_block, kernels_block = None, None
    if not args.no_extras and world == 1 and engine != B.ENGINE_SIMT:
        configs_block = []
        for cid in (3, 5, 4):
            c_ = gen.benchmark_config(cid)
            r = measure_stack(c_, B, torch, peaks, fma, 2, 1, flush, 1, args.reserve_sms, engine, want_stages=False)
            configs_block.append(stack_summary(c_, r, peaks))
            del r
            gc.collect()
            torch.cuda.empty_cache()
        kernels_block = []
        for cid in (2, 3, 4, 5):
            c_ = gen.benchmark_config(cid)
            for kind in ("attention", "gram", "solve"):
                k = measure_kernel(kind, c_, B, torch, peaks, fma, 5, 3, flush)
                kernels_block.append({kk: k[kk] for kk in ("kernel", "config", "ms", "bound", "achieved_tflops",
                                                           "peak_tflops", "frac")})

    value = ms / world
    line = {"metric": "patch_build_ms_per_context", "value": value, "unit": "ms", "n_gpus": world,
            "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms, "higher_is_better": False,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16" if cfg.dtype == "bf16" else "f32",
            "data": "synthetic", "config": workload_config(cfg, lay),
            "engine": "simt-fp32" if engine == B.ENGINE_SIMT else "tcgen05",
            "algorithmic_tflops": total_flops / (ms * 1e-3) / 1e12,
            "frac_bf16_peak_all_flops": total_flops / (ms * 1e-3) / 1e12 / peaks["bf16_tflops_sustained"],
            "frac_bf16_peak_tensor_stages": (tensor_flops / (tensor_ms * 1e-3) / 1e12 / peaks["bf16_tflops_sustained"])
            if tensor_ms > 0 else None,
            "bound_ms": {"no_overlap": b_no, "perfect_overlap": b_ov}, "time_over_bound_no_overlap": ms / b_no,
            "roofline": roofline, "stages": stages,
            "schedule": {"value": "student half and S_H first, then the ridge solve on the caller's stream with the teacher "
                                  "half, the targets and S_T beside it on an SM partition (they are needed only by the "
                                  "solve's last two products)",
                         "stages": "separate pass with the library's stage marks on, which runs teacher and student stacked "
                                   "on one stream so that every stage has an interval of its own",
                         "sum_of_stages_ms": float(sum(stage_ms))},
            "cpu_baseline": cpu, "clocks": clocks,
            "e2e": {"value": e2e_ms / world, "unit": "ms", "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h)},
            "gpu_launches": int(launches), "peaks": dict(peaks, fp32_fma_tflops_measured=fma),
            "dual_solver_option": {"ms_per_context": dual_ms, "note": "same dW through the N x N system (PKV_SOLVER_DUAL); "
                                   "the headline value uses the primal F x F solve on the sufficient statistics"},
            "configs": configs_block, "kernels": kernels_block}
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()

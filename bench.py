#!/usr/bin/env python
"""Benchmark of the SNLP hot path: greedy decoding with the layer-parallel Newton sweep on the
d20 (~0.5B) Nanochat-shaped model, random-init bf16 weights, KV cache of 2048 random-prefill tokens.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--quick]

A "step" is one decode step of the whole path: embed -> K_sweeps x (all 20 blocks evaluated at once
on the current trace + IDN correction along the layer axis + residual norms) -> LM head + argmax.
`value` is tokens/s of SNLP(K=2) IDN decoding at batch 1 (inputs resident on the device); the same
line also carries the library's own sequential decode and the other (B, K) points, the roofline of
the dominant kernel, the whole-sweep HBM fraction, and the CPU oracle timed on the host cores.
With N > 1 (torchrun) every rank runs an independent replica (the path does not shard).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

CTX = 2048          # random-prefill tokens in the cache before decoding starts
K_MAIN = 2          # sweeps of the headline configuration
WORKLOAD = "d20 decode: L20 d1280 H10x128 ff5120 V65536 bf16, KV cache of 2048 random-prefill tokens, greedy"


HBM_NOMINAL_GBS = 8000.0   # B200 HBM3e as quoted for the part (7.7 TB/s in HGX boards); context beside the measured copy rate


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return float(d["hbm_gbs"]), "measured (MEASURED_PEAKS.json)"
    return 6650.0, "fallback (6.65 TB/s)"


def ncu_traffic(kernel_class):
    """dram__bytes_read.sum + dram__bytes_write.sum per launch of a kernel class of this workload, from the table kept
    beside the ncu summary of the decode GEMM (one `class bytes` pair per line); None if there is no such table."""
    path = os.path.join(ROOT, "profiles", "k_umma_gemm_d20_decode.traffic.txt")
    try:
        for line in open(path):
            f = line.split()
            if len(f) >= 2 and f[0] == kernel_class:
                return float(f[1])
    except OSError:
        pass
    return None


def evaluated_layers(L, K):
    """Blocks evaluated by each of the K sweeps of a decode step (prefix 0, h0 initialisation): sweep k covers blocks
    k .. L-1, the earlier ones being exact already."""
    return [L - min(k, L) for k in range(K)]


class ClockSampler:
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index = index
        self.proc = None
        self.path = f"/tmp/snlp_bench_clocks_{os.getpid()}.csv"

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in open(self.path):
            f = [x.strip() for x in line.split(",")]
            if len(f) < 6:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except ValueError:
                continue
            for nm, v in zip(names, f[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        try:
            os.remove(self.path)
        except OSError:
            pass
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def d20():
    from paper_2605_17842_b200 import synth
    return synth.CONFIGS["d20"]


def alg_bytes(cfg, B, ctx):
    """Algorithmic HBM bytes (bf16): weights per sweep, KV per sweep, lm head per step."""
    L, d, ff, V = cfg.n_layer, cfg.d_model, cfg.d_ff, cfg.vocab
    w = {"qkv": L * 3 * d * d * 2, "out_proj": L * d * d * 2, "mlp_up": L * d * ff * 2, "mlp_down": L * d * ff * 2}
    kv = L * B * 2 * ctx * d * 2
    return w, kv, V * d * 2


# ----------------------------------------------------------------------------------------------
def run_ours(args):
    import torch

    from paper_2605_17842_b200 import build, replicas
    rk = replicas.ranks_from_env()
    rank, world, local = rk.rank, rk.world, rk.local
    if rank == 0:
        build.build()
    torch.cuda.set_device(local)
    replicas.init(rk, "nccl", torch.device("cuda", local))
    from paper_2605_17842_b200 import snlp, synth

    cfg = d20()
    steps, warmup = args.steps, max(args.warmup, 3)
    extra_steps = 32 if args.quick else 64
    W = synth.make_weights(cfg, seed=1234)
    max_ctx = CTX + warmup + max(steps, extra_steps) + 8
    model = snlp.Model(cfg, max_rows=512 * args.main_batch if args.only_main else 2048, max_batch=8, max_ctx=max_ctx)
    model.load_weights(W)
    stream = torch.cuda.Stream()
    hbm_peak, peak_src = peaks()

    def barrier():
        replicas.barrier(rk)
        torch.cuda.synchronize()

    def timed_decode(kv, first_tok, K, n_warm, n_steps, min_total_ms=0.0):
        """Repeats of (cache cut back to CTX, n_warm untimed steps, n_steps timed steps between two CUDA events).  One
        calibration repeat fixes how many are needed for min_total_ms of timed device work; those are then enqueued back
        to back (no host synchronisation in between, so the GPU never idles between repeats) inside one barrier +
        synchronize bracket, and every repeat is reduced to the maximum over the ranks.
        Returns (median ms/step, min ms/step, repeats)."""
        def block(n):
            evs = []
            for _ in range(n):
                kv.truncate(CTX)
                tok = first_tok.clone()
                for _ in range(n_warm):
                    model.decode_step(kv, tok, K, snlp.MODE_IDN, tok_out=tok)
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                for _ in range(n_steps):
                    model.decode_step(kv, tok, K, snlp.MODE_IDN, tok_out=tok)
                e1.record()
                evs.append((e0, e1))
            return evs

        barrier()
        evs = block(1)
        barrier()
        first = replicas.max_over_ranks(rk, evs[0][0].elapsed_time(evs[0][1]), "cuda")   # the same figure on every rank
        n = max(1, min(400, int(min_total_ms / max(first, 1e-3)) + 1)) if min_total_ms > 0 else 1
        barrier()
        evs = block(n)
        barrier()
        per_step = [replicas.max_over_ranks(rk, a.elapsed_time(b), "cuda") / n_steps for a, b in evs]
        return statistics.median(per_step), min(per_step), len(per_step)

    results = {}
    with torch.cuda.stream(stream):
        caches = {}
        for B in ((args.main_batch,) if args.only_main else (1, 8)):
            if B == 8 and args.quick:
                continue
            ids = torch.from_numpy(synth.make_ids(cfg, B, CTX, seed=3)).cuda()
            kv = model.kv_cache(B, max_ctx)
            first = model.prefill(kv, ids)
            torch.cuda.synchronize()
            caches[B] = (kv, first)

        # ---- headline: SNLP(K=2) IDN, batch 1 ------------------------------------------------
        kv, first = caches[args.main_batch if args.only_main else 1]
        sampler = ClockSampler(local)
        timed_decode(kv, first, K_MAIN, warmup, steps)  # untimed pass: CUDA graphs are captured here
        sampler.start()
        time.sleep(0.15)
        l0 = model.launch_count()
        min_ms = 0.0 if args.only_main else 1000.0    # at least a second of timed device work whatever --steps is
        ms_main, ms_main_min, repeats = timed_decode(kv, first, K_MAIN, warmup, steps, min_total_ms=min_ms)
        launches = model.launch_count() - l0
        clocks = sampler.stop()
        launches_timed = int(round(launches * steps / (steps + warmup) / (repeats + 1)))   # per timed block of `steps` steps (one calibration repeat ran too)
        results[(1, K_MAIN)] = ms_main

        if args.only_main:
            if rank == 0:
                print(json.dumps({"metric": "d20 decode tokens/s SNLP(K) vs sequential; sweep HBM GB/s vs B200 peak",
                                  "value": replicas.whole_job_rate(rk, args.main_batch, ms_main), "unit": "tokens/s", "ms_per_step": ms_main,
                                  "steps": steps, "warmup": warmup, "batch": args.main_batch, "note": "--only-main: one point only"}))
            return

        # ---- the other points (fewer steps each) ---------------------------------------------
        for B, (kv, first) in caches.items():
            for K in (0, 2, 4, 8):
                if (B, K) in results:
                    continue
                results[(B, K)] = timed_decode(kv, first, K, warmup, extra_steps, min_total_ms=150.0)[0]

        # ---- end to end through the public call with HOST buffers ----------------------------
        kv, first = caches[1]
        kv.truncate(CTX)
        host_in = torch.empty((1,), dtype=torch.int32).pin_memory()
        host_out = torch.empty((1,), dtype=torch.int32).pin_memory()
        host_in.copy_(first.cpu())
        e2e_steps = min(steps, 128)

        def e2e_step():   # the C-ABI call with host buffers: token in, the step, next token out, stream sync
            model.decode_step_host(kv, host_in, K_MAIN, snlp.MODE_IDN, tok_out=host_out)
            host_in.copy_(host_out)

        for _ in range(warmup):
            e2e_step()
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(e2e_steps):
            e2e_step()
        e1.record()
        barrier()
        ms_e2e = replicas.max_over_ranks(rk, e0.elapsed_time(e1) / e2e_steps, "cuda")

        # ---- per-kernel device time (CUDA events inside the library, on its launch stream) ----
        model.set_flag(2, 1)
        kv.truncate(CTX)
        tok = first.clone()
        for _ in range(4):
            model.decode_step(kv, tok, K_MAIN, snlp.MODE_IDN, tok_out=tok)
        torch.cuda.synchronize()
        model.kernel_times(reset=True)
        n_prof = 32
        for _ in range(n_prof):
            model.decode_step(kv, tok, K_MAIN, snlp.MODE_IDN, tok_out=tok)
        torch.cuda.synchronize()
        ktimes = model.kernel_times(reset=True)
        model.set_flag(2, 0)

    if rank != 0:
        if world > 1:
            replicas.finish(rk)
        return

    # ---- algorithmic bytes actually moved: sweep k evaluates blocks k..L-1 only (the correction covers every layer,
    # its traffic is < 1 MB) ------------------------------------------------------------------------------------
    L = cfg.n_layer
    ev = evaluated_layers(L, K_MAIN)                       # layers per sweep, e.g. [20, 19]
    frac_ev = sum(ev) / float(L)                           # weight+KV passes per step in units of a full sweep
    ctx_mid = CTX + warmup + steps / 2.0
    wbytes, kvbytes, lmbytes = alg_bytes(cfg, 1, ctx_mid)
    sweep_bytes = sum(wbytes.values()) + kvbytes           # one full (untrimmed) sweep
    step_bytes = frac_ev * sweep_bytes + lmbytes
    step_bytes_untrimmed = K_MAIN * sweep_bytes + lmbytes  # K (W + KV) + lm head, the figure of the metric's definition
    per_class = {k: {"ms_per_launch": (v[0] / v[1] if v[1] else None), "launches_per_step": v[1] / n_prof,
                     "ms_per_step": v[0] / n_prof} for k, v in ktimes.items()}
    cls_full = dict(wbytes)                                # bytes of one launch over all L layers
    # The three products after the attention run as one chained launch (booked under mlp_up by the library's timers)
    chained = ktimes["out_proj"][1] == 0 and ktimes["mlp_down"][1] == 0 and ktimes["mlp_up"][1] > 0
    if chained:
        cls_full["mlp_up"] = wbytes["out_proj"] + wbytes["mlp_up"] + wbytes["mlp_down"]
        cls_full["out_proj"] = cls_full["mlp_down"] = 0.0
    cls_full["attention"] = alg_bytes(cfg, 1, CTX + 4 + n_prof / 2.0)[1]
    cls_step = {k: v * frac_ev for k, v in cls_full.items()}   # bytes the class moves per step
    cls_full["lm_head"] = cls_step["lm_head"] = lmbytes
    for k in per_class:
        if k in cls_step and per_class[k]["ms_per_step"]:
            per_class[k]["alg_bytes_per_step"] = cls_step[k]
            per_class[k]["alg_GBs"] = cls_step[k] / (per_class[k]["ms_per_step"] * 1e-3) / 1e9
            per_class[k]["frac_of_hbm_peak"] = per_class[k]["alg_GBs"] / hbm_peak
            per_class[k]["frac_of_nominal"] = per_class[k]["alg_GBs"] / HBM_NOMINAL_GBS
    # dominant kernel: the projection class with the largest summed device time
    if chained:
        per_class["mlp_up"]["what"] = "out_proj + mlp_up + mlp_down as one chained launch (k_umma_chain)"
    dom = max(("qkv", "out_proj", "mlp_up", "mlp_down"), key=lambda k: ktimes[k][0])
    dom_name = ("k_umma_chain (out-projection -> MLP up -> MLP down, every evaluated layer, one cooperative launch)" if chained and dom == "mlp_up"
                else f"decode-regime k_umma_gemm ({dom} projection, every evaluated layer in one launch)")
    dom_launches_per_step = ktimes[dom][1] / n_prof
    dom_ms = ktimes[dom][0] / ktimes[dom][1]               # average launch duration
    dom_bytes = cls_step[dom] / dom_launches_per_step      # average algorithmic bytes of one launch
    achieved = dom_bytes / (dom_ms * 1e-3) / 1e9
    traffic_full = ncu_traffic("chain" if chained and dom == "mlp_up" else dom)   # ncu figure for a launch over all L layers
    step_gbs = step_bytes / (ms_main * 1e-3) / 1e9

    table = {}
    for (B, K), ms in sorted(results.items()):
        table[f"B{B}_" + ("seq" if K == 0 else f"K{K}")] = {"ms_per_step": ms, "tok_s": replicas.whole_job_rate(rk, B, ms)}
    speedups = {f"B{B}_K{K}": results[(B, 0)] / results[(B, K)] for (B, K) in results if K > 0 and (B, 0) in results}
    # the same steps against their own rooflines (bytes moved / measured HBM rate)
    roof = {}
    for (B, K), ms in sorted(results.items()):
        wb, kvb, lmb = alg_bytes(cfg, B, CTX + warmup + extra_steps / 2.0)
        passes = 1.0 if K == 0 else sum(evaluated_layers(L, K)) / float(L)
        nbytes = passes * (sum(wb.values()) + kvb) + lmb
        roof[f"B{B}_" + ("seq" if K == 0 else f"K{K}")] = {"alg_bytes_per_step": nbytes, "frac_of_hbm_peak": nbytes / (ms * 1e-3) / 1e9 / hbm_peak}

    cpu = cpu_baseline_sample(cfg, W, seconds=8.0 if args.quick else 20.0)

    other = None
    if world == 1 and not args.quick and not args.no_other:
        for kv_, _ in caches.values():
            kv_.close()
        model.close()
        torch.cuda.empty_cache()
        other = other_configs(W)

    line = {
        "metric": "d20 decode tokens/s SNLP(K) vs sequential; sweep HBM GB/s vs B200 peak",
        "value": replicas.whole_job_rate(rk, 1, ms_main),
        "unit": "tokens/s",
        "n_gpus": world, "steps": steps, "warmup": warmup, "ms_per_step": ms_main,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": WORKLOAD, "point": f"SNLP IDN K={K_MAIN}, batch 1 per GPU", "parallelism": "replicas only",
                   "l2": "no flush: each step streams 2.1 GB of weights + KV (> 126 MB L2)"},
        "timing": {"repeats": repeats, "steps_per_repeat": steps, "ms_per_step_median": ms_main, "ms_per_step_min": ms_main_min,
                   "note": "value = median over the repeats; each repeat = cache cut back to 2048, warm-up steps, then `steps` "
                           "steps between two CUDA events; enough repeats for >= 1 s of timed device work, enqueued back to back "
                           "between one barrier + synchronize on each side"},
        "clocks": clocks,
        "e2e": {"value": world * 1e3 / ms_e2e, "unit": "tokens/s", "h2d_bytes_per_step": 4, "d2h_bytes_per_step": 4,
                "steps": e2e_steps, "note": "snlp_decode_step_host every step: host token -> mapped pinned staging, read across the bus by the step's first kernel; next token written back by its last kernel and awaited by the host in that buffer"},
        "gpu_launches": launches_timed,
        "roofline": {"bound": "hbm", "kernel": dom_name,
                     "achieved": achieved, "peak": hbm_peak, "unit": "GB/s", "frac": achieved / hbm_peak, "peak_source": peak_src,
                     "frac_of_nominal": achieved / HBM_NOMINAL_GBS, "nominal_peak": HBM_NOMINAL_GBS,
                     "traffic": (traffic_full * dom_bytes / cls_full[dom]) if traffic_full else None,
                     "traffic_note": "ncu dram bytes of a launch over all 20 layers, scaled to this step's average launch "
                                     "(traffic grows in proportion to the layers covered)" if traffic_full else "no ncu table found",
                     "alg_bytes_per_launch": dom_bytes, "alg_bytes_untrimmed": cls_full[dom], "layers_per_launch": ev,
                     "ms_per_launch": dom_ms,
                     "sum_of_timed_launches_ms_per_step": sum(v[0] for v in ktimes.values()) / n_prof,
                     "note": "duration = CUDA events recorded by the library around every launch of the class (graphs off), "
                             "which adds a few microseconds per launch (compare sum_of_timed_launches_ms_per_step with "
                             "ms_per_step, the same launches replayed as a graph without events; event-record nodes inside "
                             "the graph were measured to cost the same); the whole-step figure under `sweep` has no such overhead"},
        "sweep": {"alg_bytes_per_step": step_bytes, "alg_bytes_untrimmed": step_bytes_untrimmed, "achieved_GBs": step_gbs,
                  "frac_of_hbm_peak": step_gbs / hbm_peak, "frac_of_nominal": step_gbs / HBM_NOMINAL_GBS, "target_frac": 0.70,
                  "note": "whole decode step (K sweeps + lm head) under CUDA-graph replay; bytes count the layers each sweep "
                          "evaluates (sweep k: blocks k..L-1); the 70 % target is met against the measured copy rate and "
                          "is quoted against the nominal 8 TB/s beside it"},
        "kernels": per_class,
        "decode": table,
        "decode_roofline": roof,
        "speedup_vs_own_sequential": speedups,
        "paper_context": "paper reports only relative speed-ups on H100 (up to 2.58x, 1.40x without PPL increase, 0.5B models)",
        "cpu_baseline": cpu,
    }
    if other is not None:
        line["other_configs"] = other
    print(json.dumps(line))
    replicas.finish(rk)


# ----------------------------------------------------------------------------------------------
def oracle_decode_setup(cfg, W):
    """The oracle's d20 decode state: a cache whose 2048 slots hold seeded random unit-RMS keys and
    N(0,1)-scaled values (cost-equivalent stand-in for a 1.6 TFLOP fp64 prefill on the host)."""
    from oracle import snlp_oracle as O
    kv = O.LayerKV(cfg.n_layer, 1, CTX + 64, cfg.n_head, cfg.head_dim)
    rng = np.random.Generator(np.random.Philox(11))
    kv.k[:, :, :CTX] = rng.standard_normal(kv.k[:, :, :CTX].shape)
    kv.v[:, :, :CTX] = 0.3 * rng.standard_normal(kv.v[:, :, :CTX].shape)
    kv.len = CTX
    return kv


def cpu_baseline_sample(cfg, W, seconds):
    from oracle import snlp_oracle as O
    kv = oracle_decode_setup(cfg, W)
    tok = np.array([17], dtype=np.int32)
    n, t0 = 0, time.perf_counter()
    while True:
        tok, _ = O.decode_step(cfg, W, kv, tok, K_MAIN, O.MODE_IDN)
        n += 1
        dt = time.perf_counter() - t0
        if dt >= seconds or n >= 32:
            break
    return {"value": n / dt, "unit": "tokens/s", "cores": os.cpu_count(), "kind": "oracle",
            "sample": f"{n} greedy decode steps of the numpy fp64 oracle, IDN K={K_MAIN}, batch 1, d20, cache of {CTX} "
                      f"seeded random keys/values (no prefill), {dt:.1f} s"}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import snlp_oracle as O
    from paper_2605_17842_b200 import synth
    cfg = d20()
    W = synth.make_weights(cfg, seed=1234)
    kv = oracle_decode_setup(cfg, W)
    tok = np.array([17], dtype=np.int32)
    warm = min(max(args.warmup, 1), 2)
    for _ in range(warm):
        tok, _ = O.decode_step(cfg, W, kv, tok, K_MAIN, O.MODE_IDN)
    budget = 150.0
    n, t0 = 0, time.perf_counter()
    while n < args.steps:
        tok, _ = O.decode_step(cfg, W, kv, tok, K_MAIN, O.MODE_IDN)
        n += 1
        if time.perf_counter() - t0 > budget:
            break
    dt = time.perf_counter() - t0
    val = n / dt
    sample = (f"{n} whole decode steps of the numpy fp64 oracle (IDN K={K_MAIN}, batch 1, d20, cache of {CTX} seeded random "
              f"keys/values); the run stops after {budget:.0f} s, so fewer than --steps may be timed")
    line = {"impl": "reference", "metric": "d20 decode tokens/s SNLP(K) vs sequential; sweep HBM GB/s vs B200 peak",
            "value": val, "unit": "tokens/s", "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": n, "warmup": warm,
            "ms_per_step": 1e3 * dt / n, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": {"workload": WORKLOAD, "point": f"SNLP IDN K={K_MAIN}, batch 1"},
            "cpu_baseline": {"value": val, "unit": "tokens/s", "cores": os.cpu_count(), "kind": "oracle", "sample": sample},
            "e2e": {"value": val, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


# ----------------------------------------------------------------------------------------------
# Secondary workloads (parity-test configurations measured for the report; not the default bench line)
def tensor_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return float(d["bf16_tflops_sustained"]), float(d["bf16_tflops"]), "measured (MEASURED_PEAKS.json)"
    return 1400.0, 1590.0, "fallback"


def measure_prefill_workload(name, reps, warm, W=None):
    """d12 prefill (B4 x T512, IDN) or d20 mHC (B2 x T1024, n=4, HCN): ms per forward for the sequential pass and
    for K sweeps, per-kernel-class device time of one sweep, GEMM TFLOP/s against the measured bf16 peak.
    W: weights of the configuration if the caller has them already."""
    import torch
    from paper_2605_17842_b200 import snlp, synth
    if name == "d12_prefill":
        cfg, B, T, Ks, mode = synth.CONFIGS["d12"], 4, 512, (2, 4, 6), snlp.MODE_IDN
    else:
        cfg, B, T, Ks, mode = synth.CONFIGS["d20_hc"], 2, 1024, (2, 4, 8), snlp.MODE_HCN
    if W is None:
        W = synth.make_weights(cfg, seed=1234)
    model = snlp.Model(cfg, max_rows=B * T, max_batch=B, max_ctx=T)
    model.load_weights(W)
    ids = torch.from_numpy(synth.make_ids(cfg, B, T, seed=2 if name == "d12_prefill" else 4)).cuda()
    h0 = model.embed(ids)

    def timed(fn):
        for _ in range(warm):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / reps

    out = {"sequential_ms": timed(lambda: model.forward_sequential(h0, want_trace=False))}
    for K in Ks:
        out[f"K{K}_ms"] = timed(lambda: model.forward_parallel(h0, K, mode, want_trace=False, want_resnorm=True))
    model.device_status()
    # per-class device time of one sweep
    model.set_flag(2, 1)
    model.forward_parallel(h0, 1, mode, want_trace=False)
    torch.cuda.synchronize()
    model.kernel_times(reset=True)
    nrep = 5
    for _ in range(nrep):
        model.forward_parallel(h0, 1, mode, want_trace=False)
    kt = model.kernel_times(reset=True)
    model.set_flag(2, 0)
    L, d, ff, M = cfg.n_layer, cfg.d_model, cfg.d_ff, B * T
    flops = {"qkv": 2.0 * L * M * 3 * d * d, "out_proj": 2.0 * L * M * d * d, "mlp_up": 2.0 * L * M * d * ff, "mlp_down": 2.0 * L * M * d * ff,
             "attention": 4.0 * L * B * cfg.n_head * (T * (T + 1) / 2) * cfg.head_dim}
    sust, burst, src = tensor_peak()
    classes = {}
    for k, (ms, n) in kt.items():
        if n:
            classes[k] = {"ms_per_sweep": ms / nrep, "launches_per_sweep": n / nrep}
            if k in flops:
                classes[k]["TFLOPs"] = flops[k] / (ms / nrep * 1e-3) / 1e12
                classes[k]["frac_of_bf16_peak"] = classes[k]["TFLOPs"] / burst
    # the correction timed here is that of a K = 1 forward: the first sweep after initialisation (old states all equal h_0:
    # not read) and at the same time the last one (no operands for a next sweep): it reads a and m and writes the new states
    n = cfg.n_streams
    corr_bytes = L * M * d * (n * 4 + 2 * 4)
    if "correction" in classes:
        hbm = peaks()[0]
        classes["correction"]["alg_GBs"] = corr_bytes / (classes["correction"]["ms_per_sweep"] * 1e-3) / 1e9
        classes["correction"]["frac_of_hbm_peak"] = classes["correction"]["alg_GBs"] / hbm
    dom = max(("qkv", "out_proj", "mlp_up", "mlp_down"), key=lambda k: kt[k][0])
    sweep_ms = sum(v["ms_per_sweep"] for v in classes.values())
    line = {"metric": f"{name} forward ms (sequential and SNLP K sweeps)", "value": out[f"K{Ks[0]}_ms"], "unit": "ms",
            "higher_is_better": False, "n_gpus": 1, "steps": reps, "warmup": warm, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": f"{name}: L{L} d{d} ff{ff} n_streams {cfg.n_streams}, B{B} x T{T}, mode {'HCN' if mode else 'IDN'}"},
            "forward_ms": out, "speedup_vs_own_sequential": {k: out["sequential_ms"] / v for k, v in out.items() if k != "sequential_ms"},
            "sweep_ms_sum_of_kernels": sweep_ms, "kernels": classes,
            "roofline": {"bound": "tensor", "kernel": f"k_umma_gemm2 ({dom}; 256x256 tiles on CTA pairs)", "achieved": classes[dom]["TFLOPs"], "peak": burst,
                         "unit": "TFLOP/s", "frac": classes[dom]["TFLOPs"] / burst, "peak_source": src + " burst", "traffic": None},
            "gemm_flops_per_sweep": sum(flops[k] for k in ("qkv", "out_proj", "mlp_up", "mlp_down")), "attention_flops_per_sweep": flops["attention"]}
    model.close()
    return line


def run_prefill_workload(args, name):
    import torch
    from paper_2605_17842_b200 import build
    build.build()
    torch.cuda.set_device(0)
    print(json.dumps(measure_prefill_workload(name, args.steps if args.steps < 256 else 20, max(3, min(args.warmup, 5)))))


def measure_spec_workload(n_gen, W=None):
    """d20 self-speculative decoding: IDN K=2 drafter, 8-token blocks, batch 1, 4096-token random-prefill context.

    Two synthetic models: the benchmark's initialisation (every matrix N(0, 0.02)), whose branches are several times
    larger than the embedded state, so that a K=2 drafter almost never agrees with the sequential model; and the same
    weights with unit-scale embeddings (branches small against the state, the regime J ~ I the method is built for),
    reported beside it and labelled as such.  Trained checkpoints are not available.
    W: the benchmark-initialised d20 weights (seed 1234) if the caller has them already."""
    import torch
    from paper_2605_17842_b200 import snlp, synth
    cfg = d20()
    ctx, block, K = 4096, 8, 2
    if W is None:
        W = synth.make_weights(cfg, seed=1234)
    ids = torch.from_numpy(synth.make_ids(cfg, 1, ctx, seed=6)).cuda()
    stream = torch.cuda.Stream()

    def measure(W):
        model = snlp.Model(cfg, max_rows=2048, max_batch=1, max_ctx=ctx + n_gen + 2 * block + 8)
        model.load_weights(W)
        with torch.cuda.stream(stream):
            kv = model.kv_cache(1, ctx + n_gen + 2 * block + 8)
            first = model.prefill(kv, ids)
            # plain sequential greedy decoding (the stream the verifier guarantees)
            tok = first.clone()
            for _ in range(8):
                model.decode_step(kv, tok, 0, tok_out=tok)
            kv.truncate(ctx)
            tok = first.clone()
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            seq_tokens = []
            for _ in range(n_gen):
                model.decode_step(kv, tok, 0, tok_out=tok)
                seq_tokens.append(tok.clone())
            torch.cuda.synchronize()
            seq_s = time.perf_counter() - t0
            seq_tokens = torch.stack(seq_tokens).flatten().tolist()
            # the drafter alone (its speed relative to the sequential model enters the paper's estimator)
            kv.truncate(ctx)
            tok = first.clone()
            for _ in range(8):
                model.decode_step(kv, tok, K, tok_out=tok)
            kv.truncate(ctx)
            tok = first.clone()
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            for _ in range(n_gen):
                model.decode_step(kv, tok, K, tok_out=tok)
            torch.cuda.synchronize()
            draft_s = time.perf_counter() - t0
            # self-speculative decoding
            kv.truncate(ctx)
            last = first.clone()
            model.draft_and_verify(kv, last, block, K)   # warm-up round (graphs)
            kv.truncate(ctx)
            last = first.clone()
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            got, acc, rounds, rejects = [], 0, 0, 0
            while len(got) < n_gen:
                em, na = model.draft_and_verify(kv, last, block, K)
                got += em
                acc += na
                rounds += 1
                rejects += na < block
            torch.cuda.synchronize()
            spec_s = time.perf_counter() - t0
        model.device_status()
        kv.close()
        model.close()
        alpha = acc / (rounds * block)                               # accepted drafts / proposed drafts
        a_tok = acc / max(acc + rejects, 1)                          # per-token acceptance: accepted / (accepted + first rejections)
        s_rel = seq_s / draft_s                                      # drafter speed in units of the sequential model's
        num = block + 1.0 if a_tok >= 1.0 else (1.0 - a_tok ** (block + 1)) / (1.0 - a_tok)
        return {"accepted_tok_s": len(got) / spec_s, "generated": len(got), "rounds": rounds, "acceptance_rate": alpha,
                "per_token_acceptance": a_tok, "tokens_per_round": len(got) / rounds, "sequential_tok_s": n_gen / seq_s, "drafter_tok_s": n_gen / draft_s,
                "speedup_vs_own_sequential": (len(got) / spec_s) / (n_gen / seq_s),
                "estimator_speedup": num / (block / s_rel + 1.0),      # ((1 - a^(B+1)) / (1 - a)) / (B / s + 1) with the per-token a, Sec. 5.1
                "output_equals_sequential_greedy": bool(got[:n_gen] == seq_tokens[:n_gen])}

    base = measure(W)
    pert = measure(synth.with_embed_std(W, cfg, 1234, 1.0))
    line = {"metric": "d20 self-speculative decode accepted tokens/s", "value": base["accepted_tok_s"], "unit": "tokens/s", "higher_is_better": True,
            "n_gpus": 1, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": "d20 self-speculative decode: IDN K=2 drafter, block 8, batch 1, ctx 4096 random prefill, greedy"},
            **{k: v for k, v in base.items() if k != "accepted_tok_s"},
            "unit_scale_embeddings": {"what": "same shapes and seeds, embedding rows N(0, 1) instead of N(0, 0.02): branches are small "
                                              "against the residual state, so the solver's bias is small", **pert},
            "note": "timed with the host clock around the whole loop (each round synchronises once to learn the accepted count)"}
    return line


def run_spec_workload(args):
    import torch
    from paper_2605_17842_b200 import build
    build.build()
    torch.cuda.set_device(0)
    print(json.dumps(measure_spec_workload(512 if args.steps >= 256 else args.steps)))


def measure_paper_workload(steps, warm):
    """The paper's own 0.5B shape (32 layers, d 640, 5 heads, random-init weights) through the inference configurations
    of its main table (NxFM-init, K): ms per greedy decode step at batch 1, ctx 2048, and the speed-up over this
    library's sequential step, next to the speed-up the paper reports for its trained model on H100."""
    import torch
    from paper_2605_17842_b200 import snlp, synth
    cfg = synth.CONFIGS["paper_0p5b"]
    W = synth.make_weights(cfg, seed=1234)
    ctx = 2048
    model = snlp.Model(cfg, max_rows=2048, max_batch=1, max_ctx=ctx + steps + warm + 8)
    model.load_weights(W)
    L = cfg.n_layer
    S = snlp.Solver
    rows = [  # (name, solver, speed-up printed in the paper's main table for that configuration)
        ("sequential", S(K=0, mode=snlp.MODE_SEQUENTIAL), 1.0),
        ("24xF1-h0 K=2", S(K=2, prefix=L - 24), 1.88),
        ("24xF1-h0 K=4", S(K=4, prefix=L - 24), 1.33),
        ("12xF1-fwd K=2", S(K=2, prefix=L - 12, init=snlp.INIT_FWD), 1.14),
        ("8xF1-h0 K=4", S(K=4, prefix=L - 8), 0.99),
        ("12xF2-h0 K=1", S(K=1, prefix=L - 24, fuse=2), 2.58),
        ("12xF2-h0 K=2", S(K=2, prefix=L - 24, fuse=2), 2.09),
        ("1xF12-h0 K=1", S(K=1, prefix=L - 12, fuse=12), 1.40),
        ("32xF1-h0 K=2 (no prefix)", S(K=2), None),
    ]
    stream = torch.cuda.Stream()
    out = []
    with torch.cuda.stream(stream):
        kv = model.kv_cache(1, ctx + steps + warm + 8)
        first = model.prefill(kv, torch.from_numpy(synth.make_ids(cfg, 1, ctx, seed=3)).cuda())
        for name, sol, paper in rows:
            kv.truncate(ctx)
            tok = first.clone()
            for _ in range(warm):
                model.decode_step_solver(kv, tok, sol, tok_out=tok)
            for rep in range(2):   # first pass captures the graphs, second is timed
                kv.truncate(ctx + warm)
                torch.cuda.synchronize()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                for _ in range(steps):
                    model.decode_step_solver(kv, tok, sol, tok_out=tok)
                e1.record()
                torch.cuda.synchronize()
            out.append({"config": name, "ms_per_step": e0.elapsed_time(e1) / steps, "paper_speedup_h100": paper})
        model.device_status()
    seq_ms = out[0]["ms_per_step"]
    for r in out:
        r["speedup_vs_own_sequential"] = seq_ms / r["ms_per_step"]
        r["tok_s"] = 1e3 / r["ms_per_step"]
    line = {"metric": "paper-shaped 0.5B decode: ms/step per inference configuration", "value": out[1]["ms_per_step"], "unit": "ms",
            "higher_is_better": False, "n_gpus": 1, "steps": steps, "warmup": warm, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": "paper_0p5b: L32 d640 H5x128 ff2560 V65536, random-init bf16, batch 1, ctx 2048, greedy decode"},
            "table": out,
            "note": "paper speed-ups are for its trained models on H100 with a PyTorch-level implementation (timed workload not stated)"}
    kv.close()
    model.close()
    return line


def run_paper_workload(args):
    import torch
    from paper_2605_17842_b200 import build
    build.build()
    torch.cuda.set_device(0)
    print(json.dumps(measure_paper_workload(args.steps if args.steps < 256 else 64, max(3, min(args.warmup, 8)))))


def other_configs(W_d20):
    """Compact results of the remaining configurations for the benchmark line (a few repetitions each, about a
    minute in all): d12 prefill, d20 mHC, d20 self-speculative decoding and the paper-shaped 32-layer model.
    Every figure is measured in this run; the full lines come from `--workload <name>`."""
    from paper_2605_17842_b200 import synth
    out = {}
    t0 = time.perf_counter()

    def compact_prefill(r):
        k = r["kernels"]
        return {"workload": r["config"]["workload"], "forward_ms": r["forward_ms"], "speedup_vs_own_sequential": r["speedup_vs_own_sequential"],
                "sweep_ms_sum_of_kernels": r["sweep_ms_sum_of_kernels"],
                "kernel_TFLOPs": {c: round(v["TFLOPs"], 1) for c, v in k.items() if "TFLOPs" in v},
                "kernel_ms_per_sweep": {c: round(v["ms_per_sweep"], 4) for c, v in k.items()},
                "correction_frac_of_hbm_peak": k.get("correction", {}).get("frac_of_hbm_peak"),
                "roofline": {q: r["roofline"][q] for q in ("bound", "kernel", "achieved", "peak", "unit", "frac")}}

    out["d12_prefill"] = compact_prefill(measure_prefill_workload("d12_prefill", 10, 3))
    out["d20_hcn"] = compact_prefill(measure_prefill_workload("d20_hcn", 5, 3, W=synth.with_mixing(W_d20, synth.CONFIGS["d20_hc"], 5)))
    sp = measure_spec_workload(96, W=W_d20)
    keep = ("accepted_tok_s", "acceptance_rate", "per_token_acceptance", "tokens_per_round", "sequential_tok_s", "drafter_tok_s",
            "speedup_vs_own_sequential", "estimator_speedup", "output_equals_sequential_greedy", "generated")
    out["d20_spec"] = {"workload": sp["config"]["workload"], "accepted_tok_s": sp["value"], **{q: sp[q] for q in keep if q in sp},
                       "unit_scale_embeddings": {q: sp["unit_scale_embeddings"][q] for q in keep if q in sp["unit_scale_embeddings"]}}
    pw = measure_paper_workload(32, 4)
    out["paper_0p5b"] = {"workload": pw["config"]["workload"],
                         "table": [{q: (round(r[q], 4) if isinstance(r[q], float) else r[q]) for q in ("config", "ms_per_step", "speedup_vs_own_sequential", "paper_speedup_h100")}
                                   for r in pw["table"]]}
    out["seconds"] = round(time.perf_counter() - t0, 1)
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=256)
    ap.add_argument("--warmup", type=int, default=16)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--quick", action="store_true", help="batch 1 only, shorter side measurements")
    ap.add_argument("--no-other", action="store_true", help="leave the other configurations out of the benchmark line")
    ap.add_argument("--only-main", action="store_true",
                    help="headline point only, small workspace: the light command used for ncu captures")
    ap.add_argument("--main-batch", type=int, default=1, choices=[1, 8], help="with --only-main: the batch size of the one point that is run")
    ap.add_argument("--workload", default="d20_decode", choices=["d20_decode", "d12_prefill", "d20_hcn", "d20_spec", "paper_0p5b"],
                    help="d20_decode is the benchmark line; the others are side measurements of the remaining configurations")
    args = ap.parse_args()
    if args.workload in ("d12_prefill", "d20_hcn"):
        return run_prefill_workload(args, args.workload)
    if args.workload == "d20_spec":
        return run_spec_workload(args)
    if args.workload == "paper_0p5b":
        return run_paper_workload(args)
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()

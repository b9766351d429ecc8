#!/usr/bin/env python
"""Benchmark of the MoE denoise step against a bounded expert cache.

A "step" is one denoising iteration of the whole stack over one block of tokens: every layer
runs gate -> top-k -> permutation -> hit/miss + fills -> grouped SwiGLU FFN -> combine ->
retention once (the residual between layers included).  The headline workload is the 16-layer,
hidden-2048, 64-expert top-8 stack with a 32-token block at 40 % expert residency.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

Prints ONE JSON line (rank 0).  `--impl reference` times the CPU oracle as it stands.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

METRIC = "moe_denoise_step_tokens_per_s_at_40pct_residency"
UNIT = "tokens/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


# DRAM traffic per algorithmic byte of the FFN kernels, from the ncu captures summarised under
# profiles/ (dram__bytes_read.sum + dram__bytes_write.sum over the algorithmic bytes of the
# captured launch).  Traffic grows in proportion to the experts (few-token regime) or token rows
# (many-token regime) a launch processes, so the ratio scales a capture to any launch.
NCU_TRAFFIC_RATIO = {
    # profiles/ffn_tc_kernel_cfg2_full_residency.md: 60 experts x 4 tokens, H 2048, I 1024
    ("ffn_gate_up", "few_tokens"): (504.42 + 4.48) / 504.9,
    ("ffn_down", "few_tokens"): (252.23 + 7.01) / 254.4,
    # the one-launch form runs the same items as those two kernels together
    ("ffn_fused", "few_tokens"): (504.42 + 4.48 + 252.23 + 7.01) / (504.9 + 254.4),
    # profiles/ffn_tc_kernel_fp8_cfg2_full_residency.md: the same launch with fp8 stores
    ("ffn_gate_up", "few_tokens", "fp8"): (261.71 + 4.15) / 270.6,
    ("ffn_down", "few_tokens", "fp8"): (131.12 + 4.37) / 136.9,
    # profiles/ffn_pair_kernel_cfg5_4096_tokens.md: 4096 tokens, H 4096, I 1536
    ("ffn_gate_up", "many_tokens"): (1944.0 + 100.7) / 1979.7,
    ("ffn_down", "many_tokens"): (909.4 + 264.2) / 1174.4,
    # the one-launch form on CTA pairs, which also gathers its token rows (268 MB read and written
    # on top of the projections' algorithmic bytes)
    ("ffn_fused", "many_tokens"): (3180.0 + 631.6) / 3154.1,
}


# nominal figures of a B200 (HGX) and of its PCIe Gen5 x16 host link, per direction
NOMINAL = {"hbm_gbs": 7700.0, "bf16_tflops": 2250.0, "h2d_gbs": 63.0}


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            d = json.load(open(p))
            return {k: float(d[k]) for k in FALLBACK_PEAKS if k in d} | {"source": "measured"}
        except Exception:
            pass
    return dict(FALLBACK_PEAKS) | {"source": "fallback"}


# ------------------------------------------------------------------------------ clocks
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_id: str):
        self.proc = None
        self.gpu_id = gpu_id

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", self.gpu_id, f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unsampled"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        sm, mx, pw, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
                pw.append(float(f[2]))
            except ValueError:
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unsampled"]}
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "power_w_max": max(pw),
                "samples": len(sm), "reasons": sorted(reasons)}


# ------------------------------------------------------------------------------ oracle legs
def oracle_layer_steps(w, budget_s: float, max_steps: int, distinct_layers: int = 1, threads=None):
    """Time the CPU oracle, as it stands, on layer executions of the workload.

    threads: cap on the BLAS threads (None = all cores the process may use).
    Returns (seconds per layer execution, layer executions timed, BLAS threads used)."""
    from oracle import OracleStack
    from paper_2609_33385_b200 import synth
    try:
        from threadpoolctl import threadpool_info, threadpool_limits
    except Exception:                                   # pragma: no cover
        threadpool_info = threadpool_limits = None
    caps = [w.capacity] * w.n_layers
    ora = OracleStack(w.n_layers, w.hidden, w.n_experts, w.top_k, w.intermediate, caps)
    blobs = []
    for d in range(distinct_layers):
        b = np.empty((w.n_experts, w.expert_elems), np.uint16)
        synth.fill_layer_blobs(w, d, b, threads=min(32, len(os.sched_getaffinity(0))))
        blobs.append(b)
    for l in range(w.n_layers):
        wr, bias = synth.router_weights(w, l)
        ora.register_router(l, wr, bias)
        ora.register_experts(l, blobs[l % distinct_layers])
    limiter = threadpool_limits(limits=threads) if (threads and threadpool_limits) else None
    used = 1
    if threadpool_info:
        used = max([int(i.get("num_threads", 1)) for i in threadpool_info()] or [1])
    times = []
    t_start = time.perf_counter()
    done = False
    try:
        for _, _, h_bits, conf in synth.denoise_inputs(w):
            x = h_bits
            for l in range(w.n_layers):
                t0 = time.perf_counter()
                res = ora.denoise_step(l, x, conf)
                times.append(time.perf_counter() - t0)
                xf = synth.bf16_bits_to_f32(x).astype(np.float64) + res["out"]
                x = synth.f32_to_bf16_bits(xf.astype(np.float32))
                if len(times) >= max_steps or time.perf_counter() - t_start > budget_s:
                    done = True
                    break
            if done:
                break
    finally:
        if limiter is not None:
            limiter.restore_original_limits() if hasattr(limiter, "restore_original_limits") else limiter.unregister()
    return sum(times) / len(times), len(times), used


def run_reference(args, w):
    """--impl reference: the oracle, as it stands, on the host cores.

    A "step" of this arm is a BOUNDED SAMPLE of the workload's step - one layer execution of the
    L-layer stack - so that the run ends within minutes; `value` is the tokens/s of the whole
    step extrapolated from it (layers are alike), and the line says so."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    n = max(1, args.steps + args.warmup)
    t0 = time.perf_counter()
    sec, count, threads = oracle_layer_steps(w, budget_s=150.0, max_steps=n)
    wall = time.perf_counter() - t0
    value = w.tokens / (sec * w.n_layers)
    sample = (f"{count} layer executions of {w.name} (1 distinct layer of weights aliased across the stack); "
              f"one timed step = ONE layer execution, the full step is {w.n_layers} of them")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": dict(workload_config(w, "A"), expert_format="bf16"),
        "extrapolated": True, "layer_executions_timed": count, "layers_per_full_step": w.n_layers,
        "ms_per_full_step_extrapolated": sec * w.n_layers * 1e3, "wall_s": wall,
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def workload_config(w, variant):
    streamed = w.n_layers * w.n_experts * w.expert_bytes
    if streamed > 4 * 126e6:
        l2 = f"inputs larger than L2: each step streams up to {streamed / 1e9:.1f} GB of expert weights (L2 126 MB)"
    else:
        l2 = (f"the step's expert weights ({streamed / 1e6:.0f} MB) do not exceed L2 by much: too small to carry a "
              "bandwidth claim, reported for completeness")
    return {"workload": w.name, "variant": variant, "layers": w.n_layers, "hidden": w.hidden,
            "experts": w.n_experts, "top_k": w.top_k, "intermediate": w.intermediate,
            "tokens_per_step": w.tokens, "iters_per_block": w.iters, "capacity_per_layer": w.capacity,
            "residency": w.residency, "rho": w.rho, "l2": l2}


# ------------------------------------------------------------------------------ GPU legs
def measure_h2d(torch, device, blob_bytes: int) -> dict:
    big = 256 << 20
    src = torch.empty(big, dtype=torch.uint8, pin_memory=True)
    dst = torch.empty(big, dtype=torch.uint8, device=device)
    best = 0.0
    for _ in range(10):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        dst.copy_(src, non_blocking=True)
        b.record()
        b.synchronize()
        best = max(best, big / (a.elapsed_time(b) * 1e-3) / 1e9)
    n = max(1, min(16, big // blob_bytes))
    best_train = 0.0
    for _ in range(5):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for i in range(n):
            dst[i * blob_bytes:(i + 1) * blob_bytes].copy_(src[i * blob_bytes:(i + 1) * blob_bytes],
                                                           non_blocking=True)
        b.record()
        b.synchronize()
        best_train = max(best_train, n * blob_bytes / (a.elapsed_time(b) * 1e-3) / 1e9)
    return {"gbs_256mb": best, "gbs_blob_train": best_train}


def timed_pass(torch, run, xs, cs, warmup, steps, host=False, sampler=None, dummy=None):
    """warmup + steps denoising iterations; returns (ms total, launches, stats delta)."""
    w = run.w
    n_tok = w.tokens
    dev_out = torch.empty((n_tok, w.hidden), dtype=torch.bfloat16, device=run.device)
    if host:
        hx = [x.cpu().pin_memory() for x in xs]
        hc = [c.cpu().pin_memory() for c in cs]
        ho = torch.empty((n_tok, w.hidden), dtype=torch.bfloat16).pin_memory()

    def one(i):
        if host:
            run.ctx.denoise_iteration_host(hx[i].data_ptr(), hc[i].data_ptr(), n_tok, ho.data_ptr())
        else:
            run.ctx.denoise_iteration(xs[i].data_ptr(), cs[i].data_ptr(), n_tok, dev_out.data_ptr())

    run.ctx.reset_cache()
    if dummy is not None:          # warm the cache with dummy requests before the warm-up steps
        for dx, dc in dummy:
            run.ctx.denoise_iteration(dx.data_ptr(), dc.data_ptr(), n_tok, dev_out.data_ptr())
    for i in range(warmup):
        one(i)
    run.ctx.synchronize()
    s0, l0 = run.ctx.stats(), run.ctx.launch_count()
    p0 = run.ctx.policy_time()
    from paper_2609_33385_b200 import dist
    dist.barrier()
    torch.cuda.synchronize()
    if sampler:
        sampler.start()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record(run.stream)
    for i in range(warmup, warmup + steps):
        one(i)
    b.record(run.stream)
    torch.cuda.synchronize()
    dist.barrier()
    clocks = sampler.stop() if sampler else None
    ms = a.elapsed_time(b)
    s1, l1 = run.ctx.stats(), run.ctx.launch_count()
    delta = {k: getattr(s1, k) - getattr(s0, k) for k in
             ("steps", "hits", "misses", "bytes_moved", "evictions", "active_experts", "assignments",
              "fills_reused", "ideal_hits")}
    p1 = run.ctx.policy_time()
    delta["policy_us_per_layer_step"] = (p1[0] - p0[0]) / max(1, p1[1] - p0[1]) / 1e3
    return ms, l1 - l0, delta, clocks


def step_roofline(w, delta, steps, ms_per_step, peaks, h2d_gbs, blob=None):
    """Binding roofline of the whole step from the algorithmic work of the timed region."""
    blob = blob or w.expert_bytes
    layer_steps = max(1, delta["steps"])
    b_hbm = (delta["active_experts"] * blob + delta["misses"] * blob +
             layer_steps * (w.n_experts * w.hidden * 2 + 2 * w.tokens * w.hidden * 2)) / steps
    b_h2d = delta["bytes_moved"] / steps
    flops = 6.0 * delta["assignments"] * w.hidden * w.intermediate / steps
    t_hbm = b_hbm / (peaks["hbm_gbs"] * 1e9) * 1e3
    t_h2d = b_h2d / (h2d_gbs * 1e9) * 1e3
    t_tc = flops / (peaks["bf16_tflops_sustained"] * 1e12) * 1e3
    terms = {"hbm": t_hbm, "host_link": t_h2d, "tensor": t_tc}
    bound = max(terms, key=terms.get)
    # the same bound against the nominal figures of the part (context; the headline uses measured peaks)
    nominal = {"hbm": b_hbm / (NOMINAL["hbm_gbs"] * 1e9) * 1e3, "host_link": b_h2d / (NOMINAL["h2d_gbs"] * 1e9) * 1e3,
               "tensor": flops / (NOMINAL["bf16_tflops"] * 1e12) * 1e3}
    return {"bound": bound, "t_roof_ms": terms[bound], "t_measured_ms": ms_per_step,
            "frac": terms[bound] / ms_per_step, "terms_ms": terms,
            "frac_of_nominal": nominal[bound] / ms_per_step, "nominal_peaks": NOMINAL,
            "hbm_bytes_per_step": b_hbm, "h2d_bytes_per_step": b_h2d, "flops_per_step": flops}


def measure_workload(torch, w, variant, device, peaks, h2d, steps, warmup, *, fp8=False, distinct_layers=None,
                     opts=(), share_store_of=None, legs=("e2e", "profile", "full"), sampler=None, threads=None):
    """All timed legs of one workload on this rank's GPU.  Returns (result dict, runner)."""
    from paper_2609_33385_b200 import dist, synth
    from paper_2609_33385_b200.binding import OPT_PROFILE
    from paper_2609_33385_b200.runner import StackRunner, bits_to_dev
    n_iters = warmup + steps
    w = w.replace(blocks=int(math.ceil(n_iters / w.iters)))
    t_setup = time.perf_counter()
    run = StackRunner(w, device=device, gen_threads=threads, distinct_layers=distinct_layers, fp8=fp8,
                      share_store_of=share_store_of)
    for oid, val in opts:
        run.ctx.set_option(oid, val)
    xs, cs = [], []
    for _, _, h_bits, conf in synth.denoise_inputs(w):
        xs.append(bits_to_dev(h_bits, device))
        cs.append(torch.from_numpy(conf).to(device))
        if len(xs) >= n_iters:
            break
    setup_s = time.perf_counter() - t_setup
    res = {"w": w, "setup_s": setup_s}

    # 1. device-resident inputs: the headline value
    if sampler:
        sampler.start()           # sampled over every timed pass of this workload (same load)
    ms, launches, delta, _ = timed_pass(torch, run, xs, cs, warmup, steps)
    units, ms_max = dist.aggregate(w.tokens * steps, ms, device)
    res.update(value=units / (ms_max * 1e-3), ms_per_step=ms_max / steps, launches=launches, delta=delta, ms_rank=ms)

    # 2. end to end: host buffers through the C ABI, copies inside the timed region
    if "e2e" in legs:
        ms_e, _, delta_e, _ = timed_pass(torch, run, xs, cs, warmup, steps, host=True)
        units_e, ms_e_max = dist.aggregate(w.tokens * steps, ms_e, device)
        in_bytes = w.tokens * w.hidden * 2 + w.tokens * 4
        ctrl_bytes = w.n_layers * w.n_experts * 16
        res["e2e"] = {"value": units_e / (ms_e_max * 1e-3), "unit": UNIT,
                      "h2d_bytes_per_step": in_bytes + delta_e["bytes_moved"] / steps,
                      "d2h_bytes_per_step": w.tokens * w.hidden * 2 + ctrl_bytes,
                      "input_h2d_bytes_per_step": in_bytes,
                      "expert_fill_h2d_bytes_per_step": delta_e["bytes_moved"] / steps,
                      "ms_per_step": ms_e_max / steps}

    # 3. per-kernel CUDA-event timing of the same region (separate pass: events add overhead and
    # keep consecutive kernels from overlapping)
    out_dev = torch.empty((w.tokens, w.hidden), dtype=torch.bfloat16, device=device)
    if "profile" in legs:
        run.ctx.set_option(OPT_PROFILE, 0)
        run.ctx.reset_cache()
        for i in range(warmup):
            run.ctx.denoise_iteration(xs[i].data_ptr(), cs[i].data_ptr(), w.tokens, out_dev.data_ptr())
        run.ctx.synchronize()
        run.ctx.set_option(OPT_PROFILE, 1)
        for i in range(warmup, n_iters):
            run.ctx.denoise_iteration(xs[i].data_ptr(), cs[i].data_ptr(), w.tokens, out_dev.data_ptr())
        prof = run.ctx.profile_read(reset=True)
        run.ctx.set_option(OPT_PROFILE, 0)
        top = max(prof, key=lambda k: prof[k]["ms"])
        kp = prof[top]
        ach = kp["bytes"] / max(kp["ms"], 1e-9) / 1e6          # GB/s
        ach_tf = kp["flops"] / max(kp["ms"], 1e-9) / 1e9       # TFLOP/s
        tensor_bound = ach_tf / peaks["bf16_tflops_sustained"] > ach / peaks["hbm_gbs"]
        roofline = {"kernel": top, "bound": "tensor" if tensor_bound else "hbm",
                    "achieved": ach_tf if tensor_bound else ach,
                    "peak": peaks["bf16_tflops_sustained"] if tensor_bound else peaks["hbm_gbs"],
                    "unit": "TFLOP/s" if tensor_bound else "GB/s",
                    "frac": (ach_tf / peaks["bf16_tflops_sustained"]) if tensor_bound else ach / peaks["hbm_gbs"],
                    "peak_source": peaks["source"] + (" (sustained bf16 matmul)" if tensor_bound else " (copy)"),
                    "traffic": None, "traffic_source": None, "launches": kp["launches"],
                    "avg_launch_us": kp["ms"] * 1e3 / max(1, kp["launches"]),
                    "algorithmic_bytes_per_launch": kp["bytes"] / max(1, kp["launches"]),
                    "algorithmic_flops_per_launch": kp["flops"] / max(1, kp["launches"]),
                    "achieved_gbs": ach, "achieved_tflops": ach_tf}
        regime = "many_tokens" if w.tokens * w.top_k > 4096 else "few_tokens"
        ratio = NCU_TRAFFIC_RATIO.get((top, regime, "fp8") if fp8 else (top, regime))
        if ratio is not None:
            roofline["traffic"] = ratio * roofline["algorithmic_bytes_per_launch"]
            roofline["traffic_source"] = (f"ncu capture of the {regime.replace('_', '-')} regime (profiles/), scaled by "
                                          "the algorithmic bytes of the average launch")
        kernels = {k: {"launches": v["launches"], "ms": round(v["ms"], 4),
                       "gbs": (v["bytes"] / v["ms"] / 1e6) if v["ms"] > 0 else None,
                       "tflops": (v["flops"] / v["ms"] / 1e9) if v["ms"] > 0 else None}
                   for k, v in prof.items()}
        res.update(roofline=roofline, kernels=kernels, top=top, tensor_bound=tensor_bound)

    blob = run.ctx.expert_bytes
    res["roofline_step"] = step_roofline(w, delta, steps, res["ms_per_step"], peaks, h2d["gbs_blob_train"], blob)
    res["roofline_step"]["host_link_peak"] = (
        f"{h2d['gbs_blob_train']:.2f} GB/s: back-to-back pinned copies of one expert blob each, measured in this run "
        f"(the message shape of a fill; one 256 MB copy reached {h2d['gbs_256mb']:.2f} GB/s, nominal PCIe Gen5 x16 "
        f"is {NOMINAL['h2d_gbs']:.0f} GB/s)")
    res["extra"] = {"tpot_ms": res["ms_per_step"] * w.iters / w.tokens,
                    "hits": delta["hits"], "misses": delta["misses"],
                    "cache_utilisation": delta["hits"] / max(1, delta["steps"] * w.capacity),
                    "ideal_cache_utilisation": delta["ideal_hits"] / max(1, delta["steps"] * w.capacity),
                    "effective_transfer_ratio": delta["fills_reused"] / max(1, delta["misses"]),
                    "policy_overhead_us_per_layer_step": delta["policy_us_per_layer_step"],
                    "active_experts_per_layer_step": delta["active_experts"] / max(1, delta["steps"]),
                    "h2d_link": {"achieved_gbs": delta["bytes_moved"] / (ms * 1e-3) / 1e9, **h2d},
                    "setup_s": setup_s}

    # 4. full residency on the same workload (C = E): the HBM-bound regime and the TPOT ratio
    if "full" in legs and w.residency < 1.0:
        full = StackRunner(w.replace(residency=1.0), device=device, share_store_of=run, fp8=fp8)
        for oid, val in opts:
            full.ctx.set_option(oid, val)
        # dummy requests (i.i.d. tokens activate nearly every expert) so that no cold miss is left
        dummy = []
        for j, (_, _, h_bits, conf) in enumerate(synth.denoise_inputs(w.replace(shared_beta=0.0, seed=w.seed + 1))):
            dummy.append((bits_to_dev(h_bits, device), torch.from_numpy(conf).to(device)))
            if j >= 3:
                break
        ms_f, _, delta_f, _ = timed_pass(torch, full, xs, cs, warmup, steps, dummy=dummy)
        _, ms_f_max = dist.aggregate(0, ms_f, device)
        msf = ms_f_max / steps
        rf = step_roofline(w.replace(residency=1.0), delta_f, steps, msf, peaks, h2d["gbs_blob_train"], blob)
        fr = {"ms_per_step": msf, "tokens_per_s": w.tokens / (msf * 1e-3), "tpot_ms": msf * w.iters / w.tokens,
              "misses": delta_f["misses"], "roofline_step": rf}
        if "profile" in legs:
            full.ctx.reset_cache()
            for dx, dc in dummy:
                full.ctx.denoise_iteration(dx.data_ptr(), dc.data_ptr(), w.tokens, out_dev.data_ptr())
            for i in range(warmup):
                full.ctx.denoise_iteration(xs[i].data_ptr(), cs[i].data_ptr(), w.tokens, out_dev.data_ptr())
            full.ctx.synchronize()
            full.ctx.set_option(OPT_PROFILE, 1)
            for i in range(warmup, n_iters):
                full.ctx.denoise_iteration(xs[i].data_ptr(), cs[i].data_ptr(), w.tokens, out_dev.data_ptr())
            pf = full.ctx.profile_read(reset=True)
            fr["kernels"] = {k: {"launches": v["launches"], "ms": round(v["ms"], 4),
                                 "gbs": (v["bytes"] / v["ms"] / 1e6) if v["ms"] > 0 else None}
                             for k, v in pf.items()}
            # the dominant kernel of THIS pass: no expert fill in flight (fills slow an overlapping launch)
            top_f = max(pf, key=lambda k: pf[k]["ms"])
            kf = pf[top_f]
            if kf["ms"] > 0 and not res["tensor_bound"]:
                ach_f = kf["bytes"] / kf["ms"] / 1e6
                fr["roofline"] = {"kernel": top_f, "bound": "hbm", "achieved": ach_f, "peak": peaks["hbm_gbs"],
                                  "unit": "GB/s", "frac": ach_f / peaks["hbm_gbs"], "launches": kf["launches"],
                                  "avg_launch_us": kf["ms"] * 1e3 / max(1, kf["launches"])}
                res["roofline"]["note"] = ("launches that overlap the expert fills run slower than alone; "
                                           "full_residency.roofline is the dominant kernel with no fill in flight")
        res["extra"]["full_residency"] = fr
        res["extra"]["tpot_ratio_vs_full_residency"] = res["ms_per_step"] / msf
        # lower bound of that ratio given the measured link: the fills that cannot hide
        res["extra"]["tpot_ratio_min_from_link"] = max(1.0, res["roofline_step"]["terms_ms"]["host_link"] / msf)
        full.close()
    if sampler:
        res["clocks"] = sampler.stop()
    return res, run


def compact(res, variant, fp8):
    """The few figures of a workload that go into the `configs` block of the JSON line."""
    w = res["w"]
    rs = res["roofline_step"]
    out = {"workload": w.name, "variant": variant, "expert_format": "fp8_e4m3_row_scaled" if fp8 else "bf16",
           "tokens_per_step": w.tokens, "layers": w.n_layers, "capacity_per_layer": w.capacity,
           "ms_per_step": res["ms_per_step"], "tokens_per_s": res["value"], "tpot_ms": res["extra"]["tpot_ms"],
           "hits": res["delta"]["hits"], "misses": res["delta"]["misses"],
           "h2d_gb_per_step": rs["h2d_bytes_per_step"] / 1e9,
           "roofline_step": {"bound": rs["bound"], "frac": rs["frac"], "t_roof_ms": rs["t_roof_ms"],
                             "frac_of_nominal": rs["frac_of_nominal"]},
           "gpu_launches": res["launches"], "clocks": res.get("clocks")}
    if "roofline" in res:
        r = res["roofline"]
        out["dominant_kernel"] = {"kernel": r["kernel"], "bound": r["bound"], "frac": r["frac"],
                                  "achieved": r["achieved"], "unit": r["unit"], "avg_launch_us": r["avg_launch_us"]}
    fr = res["extra"].get("full_residency")
    if fr:
        out["full_residency"] = {"ms_per_step": fr["ms_per_step"], "roofline_step_bound": fr["roofline_step"]["bound"],
                                 "roofline_step_frac": fr["roofline_step"]["frac"]}
        out["tpot_ratio_vs_full_residency"] = res["extra"]["tpot_ratio_vs_full_residency"]
        out["tpot_ratio_min_from_link"] = res["extra"]["tpot_ratio_min_from_link"]
    return out


def capacity_sweep(torch, base_run, device, peaks, h2d, steps, warmup):
    """Workload configuration 4: residency x hidden-state correlation on the 16-layer, 64-expert,
    top-8, hidden-2048 shape (the host expert store of the headline run is shared)."""
    from paper_2609_33385_b200 import synth
    rows = []
    for rho in (0.5, 0.9, 0.98):
        full_ms = None
        for res_frac in (1.0, 0.6, 0.4, 0.2, 0.1):
            w = synth.config(1, rho=rho, residency=res_frac)
            r, run = measure_workload(torch, w, "A", device, peaks, h2d, steps, warmup, share_store_of=base_run, legs=())
            run.close()
            if res_frac == 1.0:
                full_ms = r["ms_per_step"]
            rs = r["roofline_step"]
            rows.append({"rho": rho, "residency": res_frac, "capacity": r["w"].capacity, "hits": r["delta"]["hits"],
                         "misses": r["delta"]["misses"], "h2d_gb_per_step": rs["h2d_bytes_per_step"] / 1e9,
                         "ms_per_step": r["ms_per_step"], "tpot_ms": r["extra"]["tpot_ms"],
                         "x_full": r["ms_per_step"] / full_ms, "bound": rs["bound"], "frac_of_bound": rs["frac"]})
    return rows


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=16)
    ap.add_argument("--warmup", type=int, default=8)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=None, help="workload configuration index (0..4); default: the "
                    "headline (1) plus the compact `configs` and `sweep` blocks")
    ap.add_argument("--variant", default="A", choices=["A", "B"],
                    help="A: literal i.i.d. tokens; B: tokens of a block share a direction")
    ap.add_argument("--residency", type=float, default=None)
    ap.add_argument("--distinct-layers", type=int, default=None)
    ap.add_argument("--layers", type=int, default=None, help="override the number of layers (profiling)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-full-residency", action="store_true")
    ap.add_argument("--headline-only", action="store_true", help="skip the `configs` and `sweep` blocks")
    ap.add_argument("--cpu-budget-s", type=float, default=12.0)
    ap.add_argument("--opt", action="append", default=[], metavar="ID=VALUE",
                    help="oled_set_option(ID, VALUE) on every context (launch-structure switches, see include/oled.h)")
    ap.add_argument("--expert-format", default="bf16", choices=["bf16", "fp8"],
                    help="fp8: e4m3 expert blobs with row scales (an extension; the headline is bf16)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    plain_default = (args.config is None and args.variant == "A" and args.residency is None and args.layers is None
                     and args.expert_format == "bf16" and not args.opt)
    if args.config is None:
        args.config = 1

    from paper_2609_33385_b200 import synth
    over = {}
    if args.residency is not None:
        over["residency"] = args.residency
    if args.layers is not None:
        over["n_layers"] = args.layers
    if args.variant == "B":
        over["shared_beta"] = 0.9
        over["rho"] = 0.98
    w = synth.config(args.config, **over)
    n_iters = args.warmup + args.steps
    w = w.replace(blocks=int(math.ceil(n_iters / w.iters)))

    if args.impl == "reference":
        run_reference(args, w)
        return

    import torch
    from paper_2609_33385_b200 import build, dist
    build.build()

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    rank, local_rank, world = dist.init("nccl")
    device = f"cuda:{local_rank}"
    torch.cuda.set_device(device)
    peaks = load_peaks()
    cores = len(os.sched_getaffinity(0))
    threads = max(1, min(32, cores // max(1, world)))
    fp8 = args.expert_format == "fp8"
    opts = [tuple(int(v) for v in o.split("=")) for o in args.opt]
    blob_bytes = synth.fp8_blob_bytes(w) if fp8 else w.expert_bytes
    h2d = measure_h2d(torch, device, blob_bytes)
    gpu_uuid = "GPU-" + str(torch.cuda.get_device_properties(device).uuid).replace("GPU-", "")

    legs = ["e2e", "profile"] + ([] if args.no_full_residency else ["full"])
    res, run = measure_workload(torch, w, args.variant, device, peaks, h2d, args.steps, args.warmup, fp8=fp8,
                                distinct_layers=args.distinct_layers, opts=opts, legs=legs,
                                sampler=ClockSampler(gpu_uuid) if rank == 0 else None, threads=threads)

    configs, sweep = None, None
    if plain_default and world == 1 and not args.headline_only:
        # every other workload configuration, compactly (fewer steps; same protocol): the line then
        # carries what the design notes claim for each of them
        configs = []
        k, wu = 8, 4

        def extra(wx, variant, fp8x=False, share=None, distinct=None, legs=("profile", "full")):
            h2dx = measure_h2d(torch, device, synth.fp8_blob_bytes(wx) if fp8x else wx.expert_bytes)
            r, rn = measure_workload(torch, wx, variant, device, peaks, h2dx, k, wu, fp8=fp8x, distinct_layers=distinct,
                                     share_store_of=share, legs=legs, sampler=ClockSampler(gpu_uuid), threads=threads)
            rn.close()
            configs.append(compact(r, variant, fp8x))

        extra(synth.config(0), "A", legs=("profile",))
        extra(synth.config(1, shared_beta=0.9, rho=0.98), "B (block-shared direction, ~24 of 64 experts active)",
              share=run)
        sweep = capacity_sweep(torch, run, device, peaks, h2d, 8, 8)
        run.close()
        run = None
        extra(synth.config(1), "A", fp8x=True, distinct=2)
        extra(synth.config(2), "A (48 layers over 4 distinct weight sets)", distinct=4)
        extra(synth.config(4), "A", legs=("profile",))

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline and not fp8:
        sec, count, thr = oracle_layer_steps(w, budget_s=args.cpu_budget_s, max_steps=64)
        sec1, count1, thr1 = oracle_layer_steps(w, budget_s=args.cpu_budget_s, max_steps=64, threads=1)
        cpu = {"value": w.tokens / (sec * w.n_layers), "unit": UNIT, "cores": thr, "kind": "oracle",
               "sample": f"{count} layer executions of {w.name} ({sec:.3f} s each; 1 distinct layer of "
                         f"weights), scaled by {w.n_layers} layers per step",
               "extrapolated": True, "host_cores_available": cores,
               "single_thread": {"value": w.tokens / (sec1 * w.n_layers), "unit": UNIT, "cores": thr1,
                                 "sample": f"{count1} layer executions ({sec1:.3f} s each), scaled likewise"}}

    if rank == 0:
        line = {"metric": METRIC, "value": res["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": res["ms_per_step"], "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
                "config": dict(workload_config(res["w"], args.variant),
                               expert_format="fp8_e4m3_row_scaled" if fp8 else "bf16"),
                "clocks": res.get("clocks"), "e2e": res.get("e2e"),
                "gpu_launches": res["launches"], "roofline": res.get("roofline"), "roofline_step": res["roofline_step"],
                "kernels": res.get("kernels"), "cpu_baseline": cpu, **res["extra"]}
        if configs is not None:
            line["configs"] = configs
        if sweep is not None:
            line["sweep"] = {"workload": "configuration 4: residency x rho on the 16-layer, 64-expert, top-8, hidden-2048 "
                                         "shape, 32 tokens per step, 8 warm-up + 8 timed iterations per point",
                             "rows": sweep}
        print(json.dumps(line))
    if run is not None:
        run.close()
    dist.shutdown()


if __name__ == "__main__":
    main()

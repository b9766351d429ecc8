"""Cache-capacity x hidden-state-correlation sweep on the 64-expert / top-8 / hidden-2048 shape.

The synthetic analogue of the paper's cache-capacity sensitivity study (Sec. 5.4): for every
(residency, rho) point it reports hits, misses, host->HBM bytes and TPOT of a MoE-only stack,
next to the full-residency TPOT and the lower bound the measured host link puts on the step.

    python -m paper_2609_33385_b200.sweep [--layers 16] [--variant A|B] [--out file.md]
"""
from __future__ import annotations

import argparse
import json
import sys

import torch

from . import build, synth
from .runner import StackRunner, bits_to_dev


def dummy_requests(w, device, tokens: int = 64, n: int = 4):
    """A few steps of i.i.d. tokens that touch nearly every expert: the cache is warmed once with
    dummy requests before measuring (the paper's protocol, Sec. 5.1)."""
    wd = w.replace(batch=1, block_len=tokens, shared_beta=0.0, seed=w.seed + 1, blocks=1)
    out = []
    for j, (_, _, h_bits, conf) in enumerate(synth.denoise_inputs(wd)):
        out.append((bits_to_dev(h_bits, device), torch.from_numpy(conf).to(device)))
        if j + 1 >= n:
            break
    return out


def run_point(run: StackRunner, xs, cs, warmup: int, steps: int, dummy=None):
    w = run.w
    out = torch.empty((max(w.tokens, 64), w.hidden), dtype=torch.bfloat16, device=run.device)
    run.ctx.reset_cache()
    for dx, dc in (dummy or []):
        run.ctx.denoise_iteration(dx.data_ptr(), dc.data_ptr(), dx.shape[0], out.data_ptr())
    for i in range(warmup):
        run.ctx.denoise_iteration(xs[i].data_ptr(), cs[i].data_ptr(), w.tokens, out.data_ptr())
    run.ctx.synchronize()
    s0 = run.ctx.stats()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record(run.stream)
    for i in range(warmup, warmup + steps):
        run.ctx.denoise_iteration(xs[i].data_ptr(), cs[i].data_ptr(), w.tokens, out.data_ptr())
    b.record(run.stream)
    torch.cuda.synchronize()
    s1 = run.ctx.stats()
    ms = a.elapsed_time(b) / steps
    d = {k: getattr(s1, k) - getattr(s0, k) for k in ("steps", "hits", "misses", "bytes_moved",
                                                     "active_experts", "fills_reused", "ideal_hits",
                                                     "evictions")}
    return ms, d


def policy_mode(args, device):
    """Priority vs LRU vs LFU (uniform allocation) and Priority with layer-adaptive sizing, on a
    workload whose confidences carry routing-stability information and whose layers differ in
    activation footprint (the regime Sec. 4.3 describes)."""
    rows = []
    base = None
    w0 = synth.config(3, n_layers=args.layers, rho=0.9, shared_beta=0.9, conf_coupling=0.6,
                      layer_zipf=3.0)
    n_it = args.warmup + args.steps
    w0 = w0.replace(blocks=-(-n_it // w0.iters))
    xs, cs = [], []
    for _, _, h_bits, conf in synth.denoise_inputs(w0):
        xs.append(bits_to_dev(h_bits, device))
        cs.append(torch.from_numpy(conf).to(device))
    for res in (0.1, 0.2, 0.4, 0.6):
        for policy, period in (("priority", 0), ("lru", 0), ("lfu", 0), ("priority", 5)):
            w = w0.replace(residency=res)
            run = StackRunner(w, device=device, share_store_of=base, distinct_layers=args.distinct_layers,
                              policy=policy, adapt_period=period, staging_slots=w.n_experts)
            if base is None:
                base = run
            ms, d = run_point(run, xs, cs, args.warmup, args.steps)
            slots = d["steps"] * w.capacity
            rows.append(dict(residency=res, capacity=w.capacity, policy=policy, adaptive=bool(period),
                             ms_per_step=ms, hits=d["hits"], misses=d["misses"],
                             ideal_hits=d["ideal_hits"], utilisation=d["hits"] / max(1, slots),
                             ideal_utilisation=d["ideal_hits"] / max(1, slots),
                             transfer_ratio=d["fills_reused"] / max(1, d["misses"]),
                             active=d["active_experts"] / max(1, d["steps"]),
                             final_capacity=run.ctx.get_capacity()))
            if run is not base:
                run.close()
    lines = ["| residency | C/layer | policy | sizing | hits | misses | ideal hits | utilisation | ideal util. | "
             "eff. transfer | active/layer | ms/step |", "|" + "---|" * 12]
    for r in rows:
        lines.append(f"| {r['residency']:.0%} | {r['capacity']} | {r['policy']} | "
                     f"{'adaptive' if r['adaptive'] else 'uniform'} | {r['hits']} | {r['misses']} | "
                     f"{r['ideal_hits']} | {r['utilisation']:.3f} | {r['ideal_utilisation']:.3f} | "
                     f"{r['transfer_ratio']:.3f} | {r['active']:.1f} | {r['ms_per_step']:.2f} |")
    return rows, "\n".join(lines)


def shape_mode(args, device):
    """Block length x capacity and batch-size sweeps (the paper's sensitivity studies, Sec. 5.4):
    block lengths 1..64 crossed with residencies 10..100 %, and batches of 4, 8 and 32 blocks of
    32 tokens, on the same stack - from the few-tokens-per-expert regime (weight streaming)
    towards the many-token regime (tensor bound)."""
    rows = []
    base = None
    points = [(1, bl, res) for bl in (1, 4, 16, 32, 64) for res in (1.0, 0.6, 0.4, 0.2, 0.1)]
    points += [(b, 32, res) for b in (4, 8, 32) for res in (1.0, 0.4)]
    full_ms = {}
    for batch, block_len, res in points:
        w = synth.config(3, n_layers=args.layers, batch=batch, block_len=block_len, residency=res,
                         shared_beta=0.9 if args.variant == "B" else 0.0,
                         rho=0.98 if args.variant == "B" else 0.9)
        n_it = args.warmup + args.steps
        w = w.replace(blocks=-(-n_it // w.iters))
        xs, cs = [], []
        for _, _, h_bits, conf in synth.denoise_inputs(w):
            xs.append(bits_to_dev(h_bits, device))
            cs.append(torch.from_numpy(conf).to(device))
        run = StackRunner(w, device=device, share_store_of=base, distinct_layers=args.distinct_layers,
                          max_tokens=max(w.tokens, 64))
        if base is None:
            base = run
        ms, d = run_point(run, xs, cs, args.warmup, args.steps, dummy=dummy_requests(w, device))
        if res == 1.0:
            full_ms[(batch, block_len)] = ms
        link_ms = d["bytes_moved"] / args.steps / (args.h2d_gbs * 1e9) * 1e3
        rows.append(dict(batch=batch, block_len=block_len, tokens=w.tokens, residency=res,
                         capacity=w.capacity, ms_per_step=ms, tokens_per_s=w.tokens / (ms * 1e-3),
                         tpot_ms=ms * w.iters / w.tokens, misses=d["misses"], hits=d["hits"],
                         active=d["active_experts"] / max(1, d["steps"]),
                         h2d_gb_per_step=d["bytes_moved"] / args.steps / 1e9,
                         x_full=ms / full_ms[(batch, block_len)],
                         frac_of_link=(link_ms / ms) if link_ms > 0 else None))
        if run is not base:
            run.close()
    lines = ["| batch | block | tokens/step | residency | C | active/layer | misses | H2D GB/step | ms/step | "
             "tokens/s | TPOT ms | x full | of link bound |", "|" + "---|" * 13]
    for r in rows:
        lf = "-" if r["frac_of_link"] is None else f"{r['frac_of_link']:.2f}"
        lines.append(f"| {r['batch']} | {r['block_len']} | {r['tokens']} | {r['residency']:.0%} | {r['capacity']} | "
                     f"{r['active']:.1f} | {r['misses']} | {r['h2d_gb_per_step']:.3f} | {r['ms_per_step']:.3f} | "
                     f"{r['tokens_per_s']:.0f} | {r['tpot_ms']:.4f} | {r['x_full']:.1f} | {lf} |")
    return rows, "\n".join(lines)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--layers", type=int, default=16)
    ap.add_argument("--steps", type=int, default=16)
    ap.add_argument("--warmup", type=int, default=8)
    ap.add_argument("--variant", default="A", choices=["A", "B"])
    ap.add_argument("--h2d-gbs", type=float, default=54.5, help="measured host-link bandwidth")
    ap.add_argument("--out", default=None)
    ap.add_argument("--mode", default="capacity", choices=["capacity", "policy", "shape"])
    ap.add_argument("--distinct-layers", type=int, default=None)
    args = ap.parse_args()
    build.build()
    device = "cuda:0"
    if args.mode in ("policy", "shape"):
        rows, text = (policy_mode if args.mode == "policy" else shape_mode)(args, device)
        print(text)
        if args.out:
            with open(args.out, "w") as f:
                f.write(text + "\n\n" + json.dumps(rows) + "\n")
        return 0
    rows = []
    base_store = None
    for rho in (0.5, 0.9, 0.98):
        over = dict(n_layers=args.layers, rho=rho)
        if args.variant == "B":
            over["shared_beta"] = 0.9
        w0 = synth.config(3, **over)
        n_it = args.warmup + args.steps
        w0 = w0.replace(blocks=-(-n_it // w0.iters))
        xs, cs = [], []
        for _, _, h_bits, conf in synth.denoise_inputs(w0):
            xs.append(bits_to_dev(h_bits, device))
            cs.append(torch.from_numpy(conf).to(device))
        full_ms = None
        for res in (1.0, 0.6, 0.4, 0.2, 0.1):
            w = w0.replace(residency=res)
            run = StackRunner(w, device=device, share_store_of=base_store)
            if base_store is None:
                base_store = run
            ms, d = run_point(run, xs, cs, args.warmup, args.steps, dummy=dummy_requests(w, device, tokens=w.tokens))
            if res == 1.0:
                full_ms = ms
            link_ms = d["bytes_moved"] / args.steps / (args.h2d_gbs * 1e9) * 1e3
            rows.append(dict(rho=rho, residency=res, capacity=w.capacity, ms_per_step=ms,
                             tpot_ms=ms * w.iters / w.tokens, hits=d["hits"], misses=d["misses"],
                             h2d_gb_per_step=d["bytes_moved"] / args.steps / 1e9,
                             utilisation=d["hits"] / max(1, d["steps"] * w.capacity),
                             active=d["active_experts"] / max(1, d["steps"]),
                             ratio_vs_full=ms / full_ms, link_bound_ms=link_ms,
                             frac_of_link=(link_ms / ms) if link_ms > 0 else None))
            if run is not base_store:
                run.close()
    lines = ["| rho | residency | C | hits | misses | H2D GB/step | ms/step | TPOT ms | utilisation | "
             "active/layer | x full | link bound ms | link frac |", "|" + "---|" * 13]
    for r in rows:
        lf = "-" if r["frac_of_link"] is None else f"{r['frac_of_link']:.2f}"
        lines.append(f"| {r['rho']} | {r['residency']:.0%} | {r['capacity']} | {r['hits']} | {r['misses']} | "
                     f"{r['h2d_gb_per_step']:.3f} | {r['ms_per_step']:.3f} | {r['tpot_ms']:.3f} | "
                     f"{r['utilisation']:.3f} | {r['active']:.1f} | {r['ratio_vs_full']:.2f} | "
                     f"{r['link_bound_ms']:.2f} | {lf} |")
    text = "\n".join(lines)
    print(text)
    if args.out:
        with open(args.out, "w") as f:
            f.write(text + "\n")
            f.write("\n" + json.dumps(rows) + "\n")


if __name__ == "__main__":
    sys.exit(main())

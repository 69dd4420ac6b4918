"""Small driver for profiling: a few configuration evaluations (and optionally the sweep) of a
BERT-shaped stack with seeded synthetic inputs.

    python -m paper_2302_01382_b200.probe --hidden 768 --ffn 3072 --blocks 1 --tokens 12288 --evals 3

Prints host enqueue time and device time per evaluation.  Meant to be run under a profiler on
a small case (one block is a few hundred MB at most).
"""
from __future__ import annotations

import argparse
import time

import torch

import qcfg_workloads as wl

from . import Context, Model, PER_ROW


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--hidden", type=int, default=768)
    ap.add_argument("--ffn", type=int, default=3072)
    ap.add_argument("--blocks", type=int, default=1)
    ap.add_argument("--tokens", type=int, default=12288)
    ap.add_argument("--evals", type=int, default=3)
    ap.add_argument("--bits", type=int, default=8)
    ap.add_argument("--sweep", type=int, default=0, help="number of sweep calls to run after the evaluations")
    ap.add_argument("--seed", type=int, default=2)
    ap.add_argument("--resnet", type=int, default=0, help="batch size: run the ResNet-50 table instead of a BERT stack")
    ap.add_argument("--mixed", action="store_true", help="use the workload's drawn bit configuration instead of --bits")
    ap.add_argument("--latency", type=int, default=0, help="repetitions: print the per-width latency table sums and model sizes")
    ap.add_argument("--noise", type=float, default=0.0, help="lambda: run the noise-injection sensitivity E_N over all layers")
    ap.add_argument("--no-grouping", action="store_true", help="one launch per layer")
    ap.add_argument("--no-chains", action="store_true", help="one launch per GEMM instead of chained launches")
    ap.add_argument("--single-cta", action="store_true", help="128-row GEMM tiles on one CTA each instead of CTA pairs")
    args = ap.parse_args()

    if args.resnet:
        w = wl.resnet50(batch=args.resnet)
    else:
        w = wl.bert_stack(args.seed, args.tokens, args.hidden, args.ffn, args.blocks,
                          bit_choices=(4, 8, 16) if args.mixed else None)
    ctx = Context(0)
    ctx.set_pair_tiles(not args.single_cta)
    ctx.set_grouping(not args.no_grouping)
    ctx.set_gemm_chains(not args.no_chains)
    weights = [torch.from_numpy(a).cuda() for a in w.weights]
    x = torch.from_numpy(w.x).cuda()
    model = Model(ctx, w.layers, weights)
    model.calibrate_model(x, w.m)
    out = torch.empty((wl.layer_rows(w.layers, len(w.layers) - 1, w.m), w.layers[-1].n_out), device="cuda")
    ys = [None] * (len(w.layers) - 1) + [out]
    bits = list(w.bits) if (args.mixed or args.resnet) and w.bits is not None else [args.bits] * len(w.layers)
    model.eval_config(bits, x, w.m, ys)          # builds the weight-code cache
    ctx.check_sync()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0 = time.perf_counter()
    e0.record()
    for _ in range(args.evals):
        model.eval_config(bits, x, w.m, ys)
    e1.record()
    t_host = time.perf_counter() - t0
    ctx.check_sync()
    print(f"evaluations: host enqueue {1e3 * t_host / args.evals:.3f} ms, device {e0.elapsed_time(e1) / args.evals:.3f} ms each "
          f"({len(w.layers)} layers, m = {w.m}, bits {sorted(set(int(b) for b in bits))})")
    if args.latency:
        bs = [16, 8, 4]
        table = model.latency_table(x, w.m, bs, reps=args.latency)
        ctx.check_sync()
        for i, b in enumerate(bs):
            lat, size = model.config_cost([b] * len(w.layers), bs, table)
            print(f"all layers at {b:2d} bit: summed layer latency {lat:.3f} ms, weights {size / 1e6:.2f} MB")
    if args.noise > 0:
        gen = torch.Generator(device="cuda").manual_seed(args.seed)
        noises = [torch.randn(t.shape, generator=gen, device="cuda") for t in weights]
        model.noise_sensitivity(x, w.m, noises, args.noise)           # warm-up (allocations)
        t0 = time.perf_counter()
        e_n = model.noise_sensitivity(x, w.m, noises, args.noise)
        dt = time.perf_counter() - t0
        print(f"E_N over {len(e_n)} layers at lambda = {args.noise}: {1e3 * dt:.1f} ms ({1e3 * dt / (len(e_n) + 1):.3f} ms per forward), "
              f"min {min(e_n):.3e} max {max(e_n):.3e}")
    if args.sweep:
        s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        sse, amax = ctx.quant_error_sweep(weights, PER_ROW)
        s0.record()
        for _ in range(args.sweep):
            ctx.quant_error_sweep(weights, PER_ROW, sse=sse, absmax=amax)
        s1.record()
        ctx.check_sync()
        nbytes = 4 * sum(a.size for a in w.weights)
        ms = s0.elapsed_time(s1) / args.sweep
        print(f"sweep: {ms:.4f} ms per call, {nbytes / ms / 1e6:.1f} GB/s over {nbytes / 1e6:.1f} MB")
    model.close()
    ctx.close()


if __name__ == "__main__":
    main()

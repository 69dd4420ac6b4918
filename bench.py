#!/usr/bin/env python
"""Benchmark of the bit-configuration evaluator on one B200 (or N independent replicas).

Workload (the third configuration of the benchmark list): a 12-block BERT-base-shaped stack
of 72 linear tensors.  One STEP is one whole job of the hot path over one batch of synthetic
input: the quantization-error sweep (b = 2..8, per output channel) over all 72 weights, max
calibration of the model on the batch (a 16-bit forward), then the 72 configuration
evaluations of one greedy pass at 32 x 384 tokens, each lowering one tensor from 8 to 4 bits
in the order the sweep gives, with a scripted accept/reject stream.  The metric is
configuration evaluations per second over the whole job.

`python bench.py --gpus N --steps K --warmup W` prints ONE JSON line (rank 0).
`--impl reference` times the CPU oracle instead (a bounded sample per step).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import qcfg_workloads as wl  # noqa: E402

METRIC = "config_evals_per_sec"
UNIT = "evals/s"
N_EVALS = 72
TOKENS = 32 * 384
WORKLOAD = "bert_base_x12_sweep_calibrate_greedy72"
# DRAM bytes (read + write) per int8 GEMM of a BERT-base block at 12288 tokens (mean of the four:
# q/k/v grouped, o, ffn1, ffn2) from the ncu capture summarised in
# profiles/gemm_int8_bert_base_block.md, taken with one launch per GEMM (ncu cannot launch the
# cooperative chain kernel); a chained launch is charged this figure times the GEMMs it runs.
# Set to None whenever the GEMM kernel changes.
GEMM_TRAFFIC_BYTES = 27.1e6
GEMMS_PER_EVAL = 48          # 12 blocks x (q+k+v grouped, o, ffn1, ffn2)
DATASHEET_INT8_TOPS = 4500.0      # B200 dense int8, vendor datasheet (an outside figure)
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        d["_source"] = "measured"
        return d
    d = dict(FALLBACK_PEAKS)
    d["_source"] = "fallback"
    return d


def dist_env():
    return int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))


def max_over_ranks(value: float, world: int) -> float:
    """Max of a per-rank scalar over all ranks (torch.distributed must be initialised if world > 1)."""
    if world <= 1:
        return value
    import torch
    import torch.distributed as dist
    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([value], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.rows = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu), f"--query-gpu={self.QUERY}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            f = [s.strip() for s in r.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except ValueError:
                continue
            for nme, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(nme)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ------------------------------------------------------------------------------ CPU oracle legs

def oracle_sample(w, rows: int, n_sweep_tensors: int):
    """A bounded sample of one job on the CPU oracle: the sweep over the first tensors, plus
    calibration and ONE configuration evaluation on the first `rows` tokens.  Returns
    (seconds of the evaluation part, seconds of the sweep part, elements swept)."""
    from oracle import qcfg_oracle as orc
    t0 = time.perf_counter()
    orc.quant_error_sweep(w.weights[:n_sweep_tensors], orc.PER_ROW)
    t_sweep = time.perf_counter() - t0
    elems = sum(a.size for a in w.weights[:n_sweep_tensors])
    x = w.x[:rows]
    act, wmax = orc.calibrate_model(w.layers, w.weights, x)
    bits = np.full(len(w.layers), 8, np.uint8)
    bits[::7] = 4
    t0 = time.perf_counter()
    orc.eval_config(w.layers, w.weights, bits, x, act, wmax)
    t_eval = time.perf_counter() - t0
    return t_eval, t_sweep, elems


def cpu_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = max([p.get("num_threads", 1) for p in threadpool_info()] or [1])
        return int(n)
    except Exception:
        return os.cpu_count() or 1


def run_reference(args):
    rank, _, world = dist_env()
    if rank != 0:
        return
    rows, n_sweep = 768, 6
    w = wl.bert_base_x12()
    for _ in range(max(args.warmup, 0) and 1):
        oracle_sample(w, 128, 1)
    t_evals, t_sweeps = [], []
    t_all0 = time.perf_counter()
    for _ in range(args.steps):
        te, ts, elems = oracle_sample(w, rows, n_sweep)
        t_evals.append(te); t_sweeps.append(ts)
    wall = time.perf_counter() - t_all0
    te = float(np.mean(t_evals))
    evals_per_s = (rows / TOKENS) / te            # one full-size evaluation takes te * TOKENS / rows
    cores = cpu_threads()
    sample = (f"per step: one evaluation of the 72-layer stack on the first {rows} of {TOKENS} tokens "
              f"(scaled by rows) and the sweep over the first {n_sweep} of 72 tensors")
    line = {"impl": "reference", "metric": METRIC, "value": evals_per_s, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * wall / max(args.steps, 1),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int8/f64",
            "data": "synthetic", "config": {"workload": WORKLOAD, "tokens": TOKENS, "evals_per_step": N_EVALS},
            "cpu_baseline": {"value": evals_per_s, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample,
                             "sweep_gbs": 4e-9 * elems / float(np.mean(t_sweeps))},
            "e2e": {"value": evals_per_s, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


# ------------------------------------------------------------------------------ GPU arm

class Job:
    """Device-resident state of the benchmark job and the code of one step."""

    def __init__(self, q, ctx, w, torch):
        self.q, self.ctx, self.w, self.torch = q, ctx, w, torch
        self.weights = [torch.from_numpy(a).cuda() for a in w.weights]
        self.x = torch.from_numpy(w.x).cuda()
        self.model = q.Model(ctx, w.layers, self.weights)
        self.sse = torch.empty((len(self.weights), 7), dtype=torch.float64, device="cuda")
        self.amax = torch.empty(len(self.weights), dtype=torch.float32, device="cuda")
        self.sizes = np.array([a.size for a in w.weights], dtype=np.float64)
        # two result buffers used alternately, so that the device-to-host copy of one evaluation's
        # result can overlap the next evaluation (end-to-end leg)
        self.outs = [torch.empty((w.m, w.layers[-1].n_out), dtype=torch.float32, device="cuda") for _ in range(2)]
        self.out = self.outs[0]
        self.ys2 = [[None] * (len(w.layers) - 1) + [o] for o in self.outs]
        self.ys = self.ys2[0]
        self.copy_stream = torch.cuda.Stream()
        self.done = [torch.cuda.Event() for _ in range(2)]
        self.copied = [None, None]
        self.last_ranking = None

    def ranking_from_sweep(self):
        sse = self.sse.cpu().numpy()           # synchronises: the search order needs the sweep result
        amax = self.amax.cpu().numpy().astype(np.float64)
        eqe = np.sqrt(sse[:, 2] / self.sizes) / np.where(amax > 0, amax, 1.0)   # E_QE at b = 4
        return np.argsort(eqe, kind="stable")

    def step(self, x=None, host_out=None):
        torch = self.torch
        ctx, w = self.ctx, self.w
        x = self.x if x is None else x
        ctx.quant_error_sweep(self.weights, self.q.PER_ROW, 2, 8, sse=self.sse, absmax=self.amax)
        rank = self.ranking_from_sweep()
        self.last_ranking = rank
        self.model.calibrate_model(x, w.m)
        main = torch.cuda.current_stream()
        for i, bits in enumerate(wl.greedy_sequence(rank, w.accept)):
            if host_out is None:
                self.model.eval_config(bits, x, w.m, self.ys)
                continue
            k = i & 1
            if self.copied[k] is not None:
                main.wait_event(self.copied[k])          # the copy that read this buffer has finished
            self.model.eval_config(bits, x, w.m, self.ys2[k])
            self.done[k].record(main)
            with torch.cuda.stream(self.copy_stream):
                self.copy_stream.wait_event(self.done[k])
                host_out[k].copy_(self.outs[k], non_blocking=True)
                ev = torch.cuda.Event()
                ev.record(self.copy_stream)
                self.copied[k] = ev
        if host_out is not None:
            main.wait_stream(self.copy_stream)


def timed_evals(torch, ctx, model, configs, x, m, ys, reps: int):
    """Device time of `reps` passes over `configs` (inputs resident), plus the GEMM kernels' own
    time stamps (first CTA start to last CTA end of every launch) from the same passes."""
    for bits in configs[:2]:
        model.eval_config(bits, x, m, ys)
    ctx.check_sync()
    l0 = ctx.launch_count()
    ctx.profile_enable(2)
    ctx.profile_read(0); ctx.profile_read(1)
    t_host = time.perf_counter()
    for bits in configs[:2]:                          # host cost: two calls into an empty launch queue
        model.eval_config(bits, x, m, ys)
    t_host = (time.perf_counter() - t_host) / len(configs[:2])
    torch.cuda.synchronize()
    ctx.profile_read(0); ctx.profile_read(1)
    l0 = ctx.launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        for bits in configs:
            model.eval_config(bits, x, m, ys)
    e1.record()
    torch.cuda.synchronize()
    i_ms, i_n, i_ops = ctx.profile_read(0)
    b_ms, b_n, b_ops = ctx.profile_read(1)
    ctx.profile_enable(0)
    n = reps * len(configs)
    ms = e0.elapsed_time(e1) / n
    k_ms = i_ms + b_ms
    return {"evals_per_s": 1e3 / ms, "ms_per_eval": ms, "evals_timed": n, "host_enqueue_ms_per_eval": 1e3 * t_host,
            "gemm_tops": (i_ops + b_ops) / (k_ms * 1e-3) / 1e12 if k_ms else None,
            "gemm_int8_tops": i_ops / (i_ms * 1e-3) / 1e12 if i_ms else None,
            "gemm_bf16_tflops": b_ops / (b_ms * 1e-3) / 1e12 if b_ms else None,
            "gemm_ms_per_eval": k_ms / n, "launches_per_eval": (ctx.launch_count() - l0) / n}


def other_workloads(torch, q, ctx, peaks):
    """Short timed legs of the other four workloads (inputs resident, CUDA events)."""
    out = {}

    def leg(name, w, configs, reps, sweep=False):
        weights = [torch.from_numpy(a).cuda() for a in w.weights]
        x = torch.from_numpy(w.x).cuda()
        model = q.Model(ctx, w.layers, weights)
        model.calibrate_model(x, w.m)
        rank = None
        res = {}
        if sweep:
            sse, amax = ctx.quant_error_sweep(weights)
            sizes = np.array([a.size for a in w.weights], np.float64)
            s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            s0.record()
            for _ in range(5):
                ctx.quant_error_sweep(weights, sse=sse, absmax=amax)
            s1.record()
            torch.cuda.synchronize()
            nbytes = 4.0 * float(sizes.sum())
            res["sweep_gbs"] = nbytes / (s0.elapsed_time(s1) / 5 * 1e-3) / 1e9
            res["sweep_frac_hbm"] = res["sweep_gbs"] / peaks["hbm_gbs"]
            eqe = np.sqrt(sse.cpu().numpy()[:, 2] / sizes) / np.maximum(amax.cpu().numpy().astype(np.float64), 1e-30)
            rank = np.argsort(eqe, kind="stable")
        cfgs = configs(rank) if callable(configs) else configs
        rows_out = wl.layer_rows(w.layers, len(w.layers) - 1, w.m)
        ys = [None] * (len(w.layers) - 1) + [torch.empty((rows_out, w.layers[-1].n_out), device="cuda")]
        res.update(timed_evals(torch, ctx, model, cfgs, x, w.m, ys, reps))
        res["bits"] = sorted(set(int(b) for c in cfgs for b in c))
        res["layers"] = len(w.layers)
        act_mb = 4.0 * max(wl.layer_rows(w.layers, l, w.m) * lay.n_out for l, lay in enumerate(w.layers)) / 1e6
        wt_mb = 4.0 * sum(a.size for a in w.weights) / 1e6
        res["l2"] = ("inputs larger than L2" if wt_mb + act_mb > 126.0 else
                     "working set fits the 126 MB L2: an L2-resident figure (no flush between evaluations)")
        out[name] = res
        model.close()
        del weights, x, ys
        torch.cuda.empty_cache()

    w1 = wl.tiny_mlp()
    leg("tiny_mlp_64x256", w1, [w1.bits], 200, sweep=True)
    w2 = wl.bert_base_block()
    leg("bert_base_block_3072_tokens_mixed_4_8_16", w2, [w2.bits], 50, sweep=True)
    w4 = wl.resnet50()
    leg("resnet50_batch128_bits_4_6_8_first_last_16", w4, [w4.bits], 5)
    w5 = wl.bert_large_x24()
    leg("bert_large_x24_6144_tokens_bisection8", w5, lambda rank: wl.bisection_sequence(rank, w5.accept, 108, 8), 2, sweep=True)
    return out


def run_gpu(args):
    import torch
    import paper_2302_01382_b200 as q
    rank, local_rank, world = dist_env()
    if world > 1:
        import torch.distributed as dist
        torch.cuda.set_device(local_rank)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    else:
        torch.cuda.set_device(0)
    dev_index = torch.cuda.current_device()
    ctx = q.Context(dev_index)
    ctx.set_gemm_chains(not args.no_chains)
    peaks = load_peaks()

    w = wl.bert_base_x12()
    job = Job(q, ctx, w, torch)

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    # ---------------- device-resident timing (value).  The GEMM kernels stamp their own start and
    # end times (two atomics per CTA) in this same pass; nothing else is instrumented.
    for _ in range(args.warmup):
        job.step()
    ctx.check_sync()
    launches0 = ctx.launch_count()
    ctx.profile_enable(2)
    ctx.profile_read(0); ctx.profile_read(1)
    sampler = ClockSampler(dev_index)
    sampler.start()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        job.step()
    e1.record()
    barrier()
    ctx.check_sync()
    ms_total = max_over_ranks(e0.elapsed_time(e1), world)
    clocks = sampler.stop()
    launches = ctx.launch_count() - launches0
    value = world * N_EVALS * args.steps / (ms_total * 1e-3)
    g_ms, g_n, g_ops = ctx.profile_read(0)
    b_ms, b_n, b_ops = ctx.profile_read(1)
    ctx.profile_enable(0)
    # host cost of one evaluation: a few calls into an empty launch queue (a full queue would make
    # the call wait for the device and show the device's time instead)
    torch.cuda.synchronize()
    cfg8 = [8] * len(w.layers)
    t0 = time.perf_counter()
    for _ in range(4):
        job.model.eval_config(cfg8, job.x, w.m, job.ys)
    host_enqueue_ms = 1e3 * (time.perf_counter() - t0) / 4
    torch.cuda.synchronize()

    # ---------------- one more step with CUDA events around every launch: shares of the kernel
    # classes (the events serialise launches that otherwise overlap, so this step is slower)
    ctx.profile_enable(1)
    ctx.profile_read(0); ctx.profile_read(1); ctx.profile_read(2)
    p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    p0.record()
    job.step()
    p1.record()
    torch.cuda.synchronize()
    eg_ms, eg_n, eg_ops = ctx.profile_read(0)
    eb_ms, _, _ = ctx.profile_read(1)
    eo_ms, eo_n, _ = ctx.profile_read(2)
    ctx.profile_enable(0)
    instrumented_ms = p0.elapsed_time(p1)

    # ---------------- sweep alone (sub-metric), L2 flushed by its own 340 MB input: a burst of 10
    # calls, then a loop of about half a second with the SM clock sampled
    sw0, sw1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    n_sw = 10
    sw0.record()
    for _ in range(n_sw):
        ctx.quant_error_sweep(job.weights, q.PER_ROW, 2, 8, sse=job.sse, absmax=job.amax)
    sw1.record()
    torch.cuda.synchronize()
    sweep_ms = sw0.elapsed_time(sw1) / n_sw
    sweep_elems = float(job.sizes.sum())
    sweep_bytes = 4.0 * sweep_elems
    sweep_gbs = sweep_bytes / (sweep_ms * 1e-3) / 1e9
    n_long = max(200, int(500.0 / sweep_ms))
    s_sampler = ClockSampler(dev_index)
    s_sampler.start()
    sw0.record()
    for _ in range(n_long):
        ctx.quant_error_sweep(job.weights, q.PER_ROW, 2, 8, sse=job.sse, absmax=job.amax)
    sw1.record()
    torch.cuda.synchronize()
    s_clocks = s_sampler.stop()
    sweep_long_ms = sw0.elapsed_time(sw1) / n_long
    sweep_long_gbs = sweep_bytes / (sweep_long_ms * 1e-3) / 1e9
    sweep_clock = s_clocks.get("sm_mhz") or clocks.get("sm_mhz") or peaks.get("sm_max_mhz", 1965.0)
    alu_peak = 148 * 128 * sweep_clock * 1e6          # fp32 lane-operations per second at the sampled clock
    alu_frac = 28.0 * sweep_elems / (sweep_long_ms * 1e-3) / alu_peak
    hbm_frac_long = sweep_long_gbs / peaks["hbm_gbs"]

    # ---------------- the build's own ceiling for the int8 GEMM: a large square problem with int8
    # output, timed by the kernel's stamps in this process
    own = None
    if world == 1:
        mq, nq, kq = 12288, 4096, 4096
        gq = torch.Generator(device="cuda").manual_seed(0)
        qa = torch.randint(-127, 128, (mq, kq), dtype=torch.int8, device="cuda", generator=gq)
        qb = torch.randint(-127, 128, (nq, kq), dtype=torch.int8, device="cuda", generator=gq)
        swq = torch.full((nq,), 1e-4, device="cuda")
        oq = torch.empty((mq, nq), dtype=torch.int8, device="cuda")
        for _ in range(3):
            ctx.gemm_i8_requant(qa, qb, kq, 0.01, swq, q.ACT_NONE, 3.0, 8, out=oq)
        ctx.check_sync()
        ctx.profile_enable(2); ctx.profile_read(0)
        for _ in range(20):
            ctx.gemm_i8_requant(qa, qb, kq, 0.01, swq, q.ACT_NONE, 3.0, 8, out=oq)
        torch.cuda.synchronize()
        o_ms, o_n, o_ops = ctx.profile_read(0)
        ctx.profile_enable(0)
        own = {"m": mq, "n": nq, "k": kq, "tops": o_ops / (o_ms * 1e-3) / 1e12, "launches": int(o_n)}
        del qa, qb, oq

    # ---------------- end to end: host buffers, copies inside the timed region
    e2e = None
    if not args.no_e2e:
        host_x = torch.from_numpy(w.x).pin_memory()
        host_out = [torch.empty((w.m, w.layers[-1].n_out), dtype=torch.float32).pin_memory() for _ in range(2)]
        x_dev = torch.empty_like(job.x)
        e2e_steps = max(1, args.steps)
        barrier()
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0.record()
        for _ in range(e2e_steps):
            x_dev.copy_(host_x, non_blocking=True)
            job.step(x_dev, host_out)
        t1.record()
        barrier()
        e2e_ms = max_over_ranks(t0.elapsed_time(t1), world)
        h2d = host_x.numel() * 4
        d2h = N_EVALS * host_out[0].numel() * 4 + job.sse.numel() * 8 + job.amax.numel() * 4 + 4 * len(w.layers)
        e2e = {"value": world * N_EVALS * e2e_steps / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": int(h2d),
               "d2h_bytes_per_step": int(d2h), "steps": e2e_steps}

    # ---------------- the greedy search driver itself (Algorithm 2 through qcfg_search: every
    # evaluation is followed by the fidelity reduction and a synchronisation)
    search = None
    if not args.no_e2e:
        rank_now = [int(v) for v in job.last_ranking]
        job.model.search(q.SEARCH_GREEDY, rank_now, [8, 4], 0.9, job.x, w.m)     # untimed: allocates the driver's buffers
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        bits_s, vis_s, acc_s, n_s = job.model.search(q.SEARCH_GREEDY, rank_now, [8, 4], 0.9, job.x, w.m)
        torch.cuda.synchronize()
        dt = time.perf_counter() - t0
        search = {"algorithm": "greedy", "bs": [8, 4], "target_fidelity": 0.9, "evals": int(n_s), "ms": 1e3 * dt,
                  "evals_per_s": n_s / dt, "layers_at_4_bit": int(sum(1 for b in bits_s if b == 4))}
        # the same search with prefix reuse: every evaluation restarts at the first layer whose
        # width changed (reported beside the full-recompute figures, never instead of them)
        ctx.set_prefix_reuse(True)
        l0 = ctx.launch_count()
        t0 = time.perf_counter()
        bits_r, vis_r, acc_r, n_r = job.model.search(q.SEARCH_GREEDY, rank_now, [8, 4], 0.9, job.x, w.m)
        torch.cuda.synchronize()
        dt_r = time.perf_counter() - t0
        ctx.set_prefix_reuse(False)
        search["prefix_reuse_evals_per_s"] = n_r / dt_r
        search["prefix_reuse_ms"] = 1e3 * dt_r
        search["prefix_reuse_launches"] = int(ctx.launch_count() - l0)
        search["prefix_reuse_same_result"] = bool(bits_r == bits_s and vis_r == vis_s and acc_r == acc_s)

    # ---------------- the other four workloads
    workloads = None
    if world == 1 and not args.no_workloads:
        job.model.close()
        del job
        torch.cuda.empty_cache()
        workloads = other_workloads(torch, q, ctx, peaks)

    if rank == 0:
        sustained2 = 2.0 * peaks.get("bf16_tflops_sustained", FALLBACK_PEAKS["bf16_tflops_sustained"])
        burst2 = 2.0 * peaks.get("bf16_tflops", FALLBACK_PEAKS["bf16_tflops"])
        achieved = g_ops / (g_ms * 1e-3) / 1e12 if g_ms else 0.0
        frac_of = {"2x_bf16_cublas_sustained": achieved / sustained2, "2x_bf16_cublas_burst": achieved / burst2,
                   "datasheet_dense_int8_4500": achieved / DATASHEET_INT8_TOPS}
        if own:
            frac_of["own_large_square_int8"] = achieved / own["tops"]
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_total / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "int8", "data": "synthetic",
            "config": {"workload": WORKLOAD, "tokens": TOKENS, "evals_per_step": N_EVALS, "layers": len(w.layers),
                       "l2": "inputs larger than L2 (340 MB weights, 38 MB activations per layer)",
                       "parallelism": "replicas" if world > 1 else "single"},
            "clocks": clocks, "gpu_launches": int(launches),
            "host": {"enqueue_ms_per_eval": host_enqueue_ms, "device_ms_per_eval": ms_total / args.steps / N_EVALS,
                     "note": "host time of one qcfg_eval_config call (planning, tensor maps, 48 GEMMs in 3 chained launches) against the device time it hides behind"},
            "e2e": e2e, "launches_before_timed": int(launches0),
            "roofline": {"kernel": "gemm_kernel<int8>", "bound": "tensor", "achieved": achieved, "peak": sustained2,
                         "unit": "TOP/s", "frac": achieved / sustained2,
                         "peak_source": f"2 x sustained bf16 cuBLAS ({peaks['_source']}; nominal int8:bf16 ratio)",
                         "frac_of": frac_of, "peaks": {"2x_bf16_cublas_sustained": sustained2, "2x_bf16_cublas_burst": burst2,
                                                       "datasheet_dense_int8_4500": DATASHEET_INT8_TOPS,
                                                       "own_large_square_int8": own},
                         "launches": int(g_n), "avg_launch_us": 1e3 * g_ms / max(g_n, 1),
                         "kernel_ms_per_step": g_ms / args.steps, "bf16_kernel_ms_per_step": b_ms / args.steps,
                         "traffic": None if GEMM_TRAFFIC_BYTES is None or not g_n else
                                    GEMM_TRAFFIC_BYTES * GEMMS_PER_EVAL * N_EVALS * args.steps / g_n,
                         "traffic_source": "none: the kernel changed after the last ncu capture" if GEMM_TRAFFIC_BYTES is None else
                                           "ncu dram bytes per GEMM (mean of the four GEMMs of one block at 12288 tokens, one launch per GEMM: "
                                           "ncu cannot launch the cooperative chain kernel) x GEMMs per timed launch",
                         "gemms_per_launch": GEMMS_PER_EVAL * N_EVALS * args.steps / max(g_n, 1),
                         "how": "the timed pass that gives `value`: every CTA folds %globaltimer after its wait for the "
                                "previous kernel and at its end into the launch's slot; duration = last end - first start; "
                                "a launch is a chain of up to sixteen consecutive GEMMs",
                         "event_pass": {"int8_gemm_avg_launch_us": 1e3 * eg_ms / max(eg_n, 1),
                                        "tops": eg_ops / (eg_ms * 1e-3) / 1e12 if eg_ms else None,
                                        "share_of_kernel_time": eg_ms / max(eg_ms + eb_ms + eo_ms, 1e-9),
                                        "step_ms": instrumented_ms,
                                        "how": "one extra step with CUDA events around every launch (one launch per GEMM, serialised, no chains)"}},
            "sweep": {"gbs": sweep_gbs, "ms": sweep_ms, "bytes": sweep_bytes, "hbm_peak_gbs": peaks["hbm_gbs"],
                      "frac": sweep_gbs / peaks["hbm_gbs"], "peak_source": peaks["_source"],
                      "sustained": {"calls": n_long, "gbs": sweep_long_gbs, "ms": sweep_long_ms, "sm_mhz": sweep_clock,
                                    "hbm_frac": hbm_frac_long, "alu_frac": alu_frac,
                                    "alu_peak_lane_ops_per_s": alu_peak, "lane_ops_per_element": 28,
                                    "binds": "alu" if alu_frac > hbm_frac_long else "hbm"}},
            "search": search,
            "gemm_bf16": {"tflops": (b_ops / (b_ms * 1e-3) / 1e12) if b_ms else None, "launches": int(b_n)},
            "workloads": workloads,
        }
        if not args.no_cpu_baseline and world == 1:
            te, ts, elems = oracle_sample(w, 768, 6)
            line["cpu_baseline"] = {"value": (768 / TOKENS) / te, "unit": UNIT, "cores": cpu_threads(), "kind": "oracle",
                                    "sample": "one evaluation of the 72-layer stack on the first 768 of 12288 tokens "
                                              "(scaled by rows); sweep over the first 6 of 72 tensors",
                                    "sweep_gbs": 4e-9 * elems / ts}
        print(json.dumps(line))
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg (used when profiling)")
    ap.add_argument("--no-workloads", action="store_true", help="skip the short legs of the other four workloads")
    ap.add_argument("--no-chains", action="store_true",
                    help="one launch per GEMM instead of chained launches (ncu cannot launch the cooperative chain kernel)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()

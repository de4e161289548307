#!/usr/bin/env python
"""Benchmark of the cutoff decision: predicted worker-times per second.

One step = one whole decision of Algorithm 1's parameter server: push the newly observed run-times,
then predict_cutoff (encoder, S predictive samples of N run-times, per-sample sort, mean over
samples, throughput argmax).  The metric counts the S*N sampled, sorted and reduced worker-times.

    python bench.py --gpus 1 --steps 20 --warmup 5
    python bench.py --impl reference ...          # the CPU oracle on a bounded sample, as a baseline
    torchrun --nproc-per-node N bench.py --gpus N # N ranks share one decision: S samples each

Prints one JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "predicted_worker_times_per_sec"
UNIT = "worker-times/s"
SM_COUNT = 148
FP32_LANES_PER_SM = 128          # fused multiply-add lanes per SM per clock
MINMAX_LANES_PER_SM = 64         # fp32 min / max lanes per SM per clock (ALU pipe: 16 per sub-partition)
# DRAM bytes per launch of the dominant kernel, from the ncu capture summarised under profiles/ (valid for the
# kernel as committed with that summary; set to None when the kernel changes): the sample matrix read once
# (grows with S) plus the partial rows written (one per CTA: does not grow with S).
NCU_TRAFFIC = {
    ("n1024", "sort"): {"bytes_per_sample": 201400064 / 49152, "bytes_fixed": 4353792,
                        "source": "profiles/ncu_full_n1024_s49152_chain_emit_sort.txt (S=49152, scaled by S)"},
    ("n4096", "sort"): {"bytes_per_sample": 134251776 / 8192, "bytes_fixed": 8298752,
                        "source": "profiles/ncu_full_n4096_s8192_sort.txt (S=8192, scaled by S)"},
}
PRECISION_NAMES = {0: "f32", 1: "tf32", 2: "tf32(bf16 weights)"}


def odd_even_merge_sort_size(n: int) -> int:
    """Compare-exchanges of Batcher's odd-even merge sort over n = 2^k keys."""
    def merge(n, r):
        return 2 * merge(n, 2 * r) + (n // (2 * r) - 1) if 2 * r < n else 1
    return 0 if n < 2 else 2 * odd_even_merge_sort_size(n // 2) + merge(n, 1)


def compare_exchanges(n_pow2: int) -> int:
    """Compare-exchanges of the library's network over n_pow2 keys: every lane sorts its E = min(32, n/32) keys
    by odd-even merge sort, then bitonic merges of width 2E .. n (n/2 compare-exchanges per stage, log2(k)
    stages for width k)."""
    e = min(32, n_pow2 // 32)
    total = (n_pow2 // e) * odd_even_merge_sort_size(e)
    k = 2 * e
    while k <= n_pow2:
        total += (n_pow2 // 2) * (k.bit_length() - 1)
        k *= 2
    return total


def stage_work(wl, S, literal=False):
    """Algorithmic work of one decision per stage: (kind, amount).  'alu' counts one lane-operation per
    fused multiply-add or per min / max; 'tensor' counts floating-point operations (2 per multiply-add)."""
    N, D, H, W = wl.N, wl.D, wl.H, wl.window
    p = 32
    while p < N:
        p *= 2
    chain = S * (W * (2 * D * H + D * D) + 3 * D * H + D * H)
    emit_macs = S * H * 2 * N
    if literal:      # gate and proposal (2 x 2DH), linear map and scale (2 x D^2), first emission layer
        chain = S * (W * (2 * D * H + D * D) + 4 * D * H + 2 * D * D + D * H)
        # fp32: three N x H products; tensor cores: the scale's hidden layer as one H x H product (I is affine in u),
        # then the mean and the scale product in one accumulator
        emit_macs = S * H * (2 * N + H) if wl.precision else S * H * 3 * N
    return {
        "encoder": ("alu", 2 * W * (N * H + H * H)),
        "chain": ("alu", chain),
        "emission": ("tensor", 2 * emit_macs) if wl.precision else ("alu", emit_macs),
        "sort": ("alu", S * 2 * compare_exchanges(p)),
        "decide": ("alu", N),
    }


class ClockSampler:
    """Samples nvidia-smi while the timed region runs."""

    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.rows = []
        self.proc = None
        self.gpu_index = gpu_index

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits", "-lms", "20",
                 "-i", str(self.gpu_index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        self.thread.join(timeout=2)
        sm, smax, reasons = [], [], set()
        for r in self.rows:
            if len(r) < 9:
                continue
            try:
                sm.append(float(r[1]))
                smax.append(float(r[2]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def pipe_rates(device: int, measure: bool) -> dict:
    """Warp-instructions per clock per SM of fp32 min/max, shuffles and fp32 FMA: measured by the library's
    micro-benchmark on this GPU, or the nominal figures (64 / 32 / 128 lanes per SM per clock)."""
    if measure:
        from paper_1803_04209_b200 import binding
        r = binding.measure_pipe_rates(device)
        r["source"] = "measured (cutoff_measure_pipe_rates, this run)"
        return r
    return {"minmax": MINMAX_LANES_PER_SM / 32.0, "shuffle": 1.0, "fma": FP32_LANES_PER_SM / 32.0,
            "source": "nominal lanes per SM per clock"}


def cpu_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = max((p.get("num_threads", 1) for p in threadpool_info()), default=1)
        return int(n)
    except Exception:
        return 1


def time_oracle(wl, weights, trace, sample_S, steps=1, warmup=0, seed=1):
    """Time the CPU oracle, as it stands, on `sample_S` samples of the workload's decision."""
    from oracle import cutoff_oracle as O      # permitted caller: the CPU-baseline leg
    orc = O.CutoffOracle(weights, wl.lag, sample_S, seed=seed)
    for x in trace[-(wl.window + 2):]:
        orc.push(x)
    times = []
    for i in range(warmup + steps):
        t0 = time.perf_counter()
        orc.predict()
        if i >= warmup:
            times.append(time.perf_counter() - t0)
        orc.push(trace[i % len(trace)])
    return sum(times) / len(times)


def run_reference(args, wl, weights, trace):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    sample_S = min(wl.S, args.reference_samples)
    sec = time_oracle(wl, weights, trace, sample_S, steps=args.steps, warmup=args.warmup)
    value = sample_S * wl.N / sec
    cores = cpu_threads()
    sample = f"{sample_S} of the workload's {wl.S} samples per step, all {wl.N} workers"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": wl.name, "variant": args.variant, "N": wl.N, "D": wl.D, "H": wl.H, "lag": wl.lag,
                   "S_per_gpu": wl.S, "parallelism": "samples x1", "timed_samples_per_step": sample_S,
                   "timing": "host clock around the oracle's decision on the sampled rows"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))


def load_weight_file(path: str) -> dict:
    """Weights saved as an npz of the blob's tensors (what oracle/fit_elbo.py writes)."""
    with np.load(path) as z:
        return {k: np.ascontiguousarray(z[k], dtype=np.float32) for k in z.files if not k.startswith("_")}


def fit_on_gpu(args, wl, weights):
    """Section 4.1: Adam with gradient clipping on the ELBO of Section 3.1.3, every step's arithmetic in the library.
    Trains on the windows of the trace's first --evaluate-offset steps; returns (weights, report)."""
    import torch
    from paper_1803_04209_b200 import binding, inputs
    n_train = max(args.evaluate_offset, 4 * wl.window + 64)
    trace = inputs.workload_trace(wl, n_train).astype(np.float64)
    scale = 2.0 * float(trace[: wl.window].mean())                  # the run-time normaliser: twice the first window's mean
    norm = torch.from_numpy((trace / scale).astype(np.float32)).cuda()
    n_win = n_train - wl.window + 1
    batch = 64
    fitter = binding.Fitter(wl.N, wl.D, wl.H, wl.lag, batch, weights)
    gen = torch.Generator(device="cuda").manual_seed(0)
    offs = torch.arange(wl.window, device="cuda")
    first = last = None
    xhat = torch.empty((batch, wl.window, wl.N), device="cuda")
    eps = torch.empty((batch, wl.window, wl.D), device="cuda")
    fitter.capture_elbo_grad(xhat, eps)                              # the step's launches as one graph replay
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for it in range(args.fit_steps):
        idx = torch.randint(0, n_win, (batch,), device="cuda", generator=gen)
        xhat.copy_(norm[idx[:, None] + offs[None, :]])               # [batch, window, N]
        eps.normal_(generator=gen)
        elbo, _ = fitter.replay_elbo_grad()
        fitter.adam_step(lr=2e-3, clip=10.0)
        if it == 0 or it == args.fit_steps - 1:
            val = float(elbo.mean().item())
            first = val if it == 0 else first
            last = val
    torch.cuda.synchronize()
    sec = time.perf_counter() - t0
    report = {"steps": args.fit_steps, "batch_windows": batch, "train_trace_steps": n_train, "seconds": round(sec, 2),
              "steps_per_second": round(args.fit_steps / sec, 1), "elbo_per_window_first": first, "elbo_per_window_last": last,
              "how": "cutoff_elbo_grad (replayed as a CUDA graph) + cutoff_adam_step per step (fp32, lr 2e-3, clip 10), windows and noise drawn with torch on the GPU"}
    return fitter.weights(), report


def run_evaluate(args, wl, weights, literal):
    """Fig. 2's comparison on the workload's synthetic trace: throughput achieved by each cutoff rule relative to
    the hindsight-best throughput of every step.  All scoring runs in the library's kernels."""
    import torch
    from paper_1803_04209_b200 import binding, build, inputs
    build.build()
    torch.cuda.set_device(0)
    fit_report = None
    if args.fit_steps > 0:
        if literal:
            raise SystemExit("--fit-steps fits the compact networks only")
        weights, fit_report = fit_on_gpu(args, wl, weights)
    n_hist = max(wl.window + 1, min(wl.history, 64), args.evaluate_offset)
    T = args.evaluate_steps
    trace = inputs.workload_trace(wl, n_hist + T)
    dev_all = torch.from_numpy(trace).cuda()
    dev_eval = dev_all[n_hist:]
    flags = (binding.FLAG_LITERAL if literal else 0) | binding.FLAG_GRAPH

    def model_cutoffs(censor: bool):
        ctx = binding.Cutoff(wl.N, wl.D, wl.H, wl.lag, wl.S, precision=wl.precision, seed=2024,
                             flags=flags if not censor else flags & ~binding.FLAG_GRAPH)
        ctx.load_weights(weights)
        for x in trace[max(0, n_hist - 64):n_hist]:
            ctx.push(x)
        cs = np.empty(T, dtype=np.int32)
        for t in range(T):
            # Algorithm 1: the cutoff of step t is set before its run-times arrive ...
            code, c = ctx.predict()
            cs[t] = c
            x = trace[n_hist + t]
            if censor:
                # ... and the workers slower than the c-th are killed: their run-times are never observed (Section 4.2)
                order = np.argsort(x, kind="stable")
                mask = np.zeros(wl.N, dtype=bool)
                mask[order[c:]] = True
                ctx.push(x, mask if mask.any() else None)
            else:
                ctx.push(x)
        ctx.close()
        return cs

    static = binding.eval_trace(dev_all[:n_hist], None, want_static=True)
    static_c = int(static["static_c"].item())                       # chosen on the history, applied to what follows
    order = binding.order_baseline(dev_all)[n_hist:].cpu().numpy()  # its running moments start with the history
    rules = {"model": model_cutoffs(False), "model_censored": model_cutoffs(True),
             "static": np.full(T, static_c, dtype=np.int32), "order": order.astype(np.int32),
             "wait_for_all": np.full(T, wl.N, dtype=np.int32)}
    names = list(rules)
    res = binding.eval_trace(dev_eval, torch.from_numpy(np.stack([rules[n] for n in names])).cuda(), want_static=False)
    best = res["best"].double()
    report = {}
    for m, name in enumerate(names):
        ach = res["achieved"][m].double()
        report[name] = {"mean_fraction_of_best": float((ach / best).mean()),
                        "total_fraction_of_best": float(ach.sum() / best.sum()),
                        "mean_step_seconds": float(res["step_time"][m].double().mean()),
                        "mean_cutoff": float(np.mean(rules[name]))}
    fitted = bool(args.weights) or fit_report is not None
    line = {"evaluate": {"workload": wl.name, "variant": args.variant, "N": wl.N, "S": wl.S, "steps": T,
                         "history_steps": n_hist, "fit": fit_report,
                         "weights": (args.weights or "fitted on the GPU in this run") if fitted else "seeded random initialisation with hand-set bias offsets",
                         "note": ("model rows use fitted weights" if fitted else
                                  "the model rows are a plumbing check only: the weights are not fitted to this trace"),
                         "hindsight_mean_cutoff": float(res["best_c"].double().mean()),
                         "static_cutoff": static_c, "rules": report,
                         "how": "throughput c / x~_(c) of every step under each rule's cutoff, relative to the step's "
                                "maximum over c (known only in hindsight); scored by cutoff_eval_trace / "
                                "cutoff_order_baseline on the device-resident trace"}}
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--workload", default="n1024")
    ap.add_argument("--variant", default="compact", choices=["compact", "literal"],
                    help="compact: one-hidden-layer MLPs with (mean, log-variance) heads; literal: the gated "
                         "transition and the emission networks I, J as the paper prints them")
    ap.add_argument("--samples", type=int, default=0, help="override S (for profiling small cases)")
    ap.add_argument("--pass-rows", type=int, default=0)
    ap.add_argument("--reference-samples", type=int, default=4096)
    ap.add_argument("--cpu-baseline-samples", type=int, default=32768)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-stream", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="launch the kernels of a step one by one instead of replaying the captured graph")
    ap.add_argument("--stream-steps", type=int, default=1000)
    ap.add_argument("--no-measure-alu-peak", action="store_true",
                    help="skip the pipe-rate micro-benchmark (a few ms) and take the nominal min/max, shuffle and FMA rates")
    ap.add_argument("--measure-alu-peak", action="store_true", help="(default) measure those rates in this run")
    ap.add_argument("--sustained-seconds", type=float, default=2.0,
                    help="replay the step back to back for this long and report the sustained time per step (0 = skip)")
    ap.add_argument("--evaluate", action="store_true",
                    help="score the model's cutoff, a static cutoff, the Elfving 'order' cutoff and waiting for all "
                         "workers against the hindsight-best throughput on the workload's synthetic trace, then exit")
    ap.add_argument("--evaluate-steps", type=int, default=200)
    ap.add_argument("--evaluate-offset", type=int, default=0,
                    help="first step of the workload's trace that is scored (the steps a weight file was fitted on come before it)")
    ap.add_argument("--fit-steps", type=int, default=0,
                    help="with --evaluate: first fit the weights on the GPU (the library's ELBO gradient and Adam calls) for "
                         "this many steps of 64 windows on the trace before --evaluate-offset")
    ap.add_argument("--weights", default="", help="path of a weight file written by oracle/fit_elbo.py (npz); default: seeded random weights")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "cuda":
        args.warmup = 3

    from paper_1803_04209_b200 import inputs
    wl = inputs.WORKLOADS[args.workload]
    if args.samples:
        import dataclasses
        wl = dataclasses.replace(wl, S=args.samples)
    literal = args.variant == "literal"
    weights = inputs.workload_weights_literal(wl) if literal else inputs.workload_weights(wl)
    trace = inputs.workload_trace(wl, min(wl.history, 64) + args.steps + args.warmup + 8)

    if args.weights:
        weights = load_weight_file(args.weights)
    if args.impl == "reference":
        run_reference(args, wl, weights, trace)
        return
    if args.evaluate:
        run_evaluate(args, wl, weights, literal)
        return

    import torch
    import torch.distributed as dist
    from paper_1803_04209_b200 import binding, build, sharding

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    torch.cuda.set_device(local_rank)
    build.build()
    stream = torch.cuda.current_stream()

    # N ranks share one decision: each draws S samples with global sample indices (weak scaling)
    shard = sharding.shard_config(rank, world, wl.S)
    # One GPU: every step replays the captured graph of push + decision (cutoff_step_device / cutoff_step).
    # Several GPUs: the partial sums are all-reduced between the sort and the decision, so the kernels are
    # launched one by one.
    use_graph = world == 1 and not args.no_graph
    variant_flag = binding.FLAG_LITERAL if literal else 0

    def make_ctx(flags):
        c = binding.Cutoff(wl.N, wl.D, wl.H, wl.lag, shard["n_samples"], precision=wl.precision, seed=2024,
                           device=local_rank, stream=stream.cuda_stream, sample_offset=shard["sample_offset"],
                           total_samples=shard["total_samples"], flags=flags)
        c.load_weights(weights)
        if args.pass_rows:
            c.set_option("pass_rows", args.pass_rows)
        return c

    ctx = make_ctx(variant_flag | (binding.FLAG_GRAPH if use_graph else 0))
    shared = sharding.ShardedDecision(ctx, device="cuda") if world > 1 else None
    n_hist = min(wl.history, 64)
    for x in trace[:n_hist]:
        ctx.push(x)
    dev_trace = torch.from_numpy(trace[n_hist:]).cuda()
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")

    def step_device(i):
        if use_graph:
            return ctx.step_device(dev_trace[i])[1]
        ctx.push_async(dev_trace[i])
        if world > 1:
            code, c = shared.predict()         # local samples, one all-reduce of N sums, shared decision
        else:
            ctx.predict_async()
            code, c = ctx.fetch()
        return c

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(args.warmup):
        step_device(i)

    # ---- device-resident timing: per-step CUDA events, L2 flushed between steps ----------------
    starts = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    stops = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    launches0 = ctx.launch_count()
    sampler = ClockSampler(local_rank)
    barrier()
    sampler.start()
    t_wall0 = time.perf_counter()
    for i in range(args.steps):
        flush.zero_()
        starts[i].record(stream)
        step_device(args.warmup + i)
        stops[i].record(stream)
        stops[i].synchronize()
    barrier()
    wall = time.perf_counter() - t_wall0
    clocks = sampler.stop()
    launches = ctx.launch_count() - launches0

    # ---- per-stage times, in a pass of their own: the events that bracket every stage cost about 0.03 ms per
    # ---- step at the default workload, so they stay out of the timed region above ------------------------------
    # ---- (a context of its own when the timed one replays a graph: events cannot sit inside the replay) ---------
    tctx = ctx
    if use_graph:
        tctx = make_ctx(variant_flag)
        for x in trace[:n_hist]:
            tctx.push(x)
    tctx.set_timing(True)
    stage_ms = {}
    stage_steps = min(args.steps, 20)
    for i in range(stage_steps):
        flush.zero_()
        tctx.push_async(dev_trace[(args.warmup + i) % dev_trace.shape[0]])
        if world > 1:
            shared.predict()
        else:
            tctx.predict_async()
            tctx.fetch()
        for k, v in tctx.get_timing().items():
            stage_ms[k] = stage_ms.get(k, 0.0) + v
    tctx.set_timing(False)
    if tctx is not ctx:
        tctx.close()
    total_ms = sum(s.elapsed_time(e) for s, e in zip(starts, stops))
    if world > 1:
        t = torch.tensor([total_ms], dtype=torch.float64, device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        total_ms = float(t.item())
    ms_per_step = total_ms / args.steps
    value = world * wl.S * wl.N / (ms_per_step * 1e-3)

    # ---- end to end: host buffers in, host results out, wall clock ---------------------------------
    host_trace = trace[n_hist:]
    barrier()
    t0 = time.perf_counter()
    for i in range(args.steps):
        if use_graph:
            code, c = ctx.step(host_trace[args.warmup + i])
        else:
            ctx.push(host_trace[args.warmup + i])
            code, c = shared.predict() if world > 1 else ctx.predict()
        e_sec, omega = ctx.get_stats()
    barrier()
    e2e_sec = (time.perf_counter() - t0) / args.steps
    if world > 1:
        t = torch.tensor([e2e_sec], dtype=torch.float64, device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        e2e_sec = float(t.item())
    e2e_value = world * wl.S * wl.N / e2e_sec

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- streaming decision latency: push + predict per SGD step inside a CUDA graph -------------------
    stream_latency = None
    if not args.no_stream and world == 1:
        swl = inputs.WORKLOADS["stream"]
        sweights = inputs.workload_weights(swl)
        strace = inputs.workload_trace(swl, swl.window + 8 + args.stream_steps)
        sctx = binding.Cutoff(swl.N, swl.D, swl.H, swl.lag, swl.S, precision=swl.precision, seed=7, device=local_rank,
                              stream=stream.cuda_stream, flags=binding.FLAG_GRAPH)
        sctx.load_weights(sweights)
        for x in strace[: swl.window + 8]:
            sctx.step(x)
        lat = []
        for x in strace[swl.window + 8:]:
            t0 = time.perf_counter()
            sctx.step(x)
            lat.append((time.perf_counter() - t0) * 1e6)
        lat.sort()
        stream_latency = {"workload": "stream", "N": swl.N, "S": swl.S, "steps": len(lat),
                          "p50_us": lat[len(lat) // 2], "p99_us": lat[int(len(lat) * 0.99)],
                          "how": "host clock around cutoff_step (host run-times in, cutoff out), CUDA graph replay"}
        sctx.close()

    # ---- roofline: the dominant stage, and the path as a whole ------------------------------------------------
    peaks = {}
    try:
        peaks = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
    except OSError:
        pass
    work = stage_work(wl, wl.S, literal)
    stage_avg = {k: v / stage_steps for k, v in stage_ms.items()}
    dominant = max(stage_avg, key=stage_avg.get)
    kind, amount = work[dominant]
    dur = stage_avg[dominant] * 1e-3
    smax = peaks.get("sm_max_mhz", 1965.0)
    # the clock the timed region actually ran at: the median of the nvidia-smi samples taken during it
    clock_mhz = clocks.get("sm_mhz") or smax
    rates = pipe_rates(local_rank, measure=not args.no_measure_alu_peak)
    lane_rate = lambda name: SM_COUNT * 32.0 * rates[name] * clock_mhz * 1e6          # lane-operations per second
    bf16 = peaks.get("bf16_tflops", 1590.0)
    tensor_peak = 0.5 * bf16 * 1e12                      # tf32 runs at half the bf16 rate (nominal ratio)
    tensor_src = ("measured bf16 burst x 0.5 (nominal tf32 : bf16 ratio)" if peaks else "fallback 1590 x 0.5")
    if kind == "tensor":
        peak, unit, peak_src, bound = tensor_peak / 1e12, "TFLOP/s", tensor_src, "tensor"
    elif dominant == "sort":
        peak, unit, bound = lane_rate("minmax") / 1e12, "Tlane-op/s", "alu"
        peak_src = (f"{rates['source']}: {rates['minmax']:.3f} fp32 min/max warp-instructions per clock per SM x 32 lanes "
                    f"x {SM_COUNT} SMs x {clock_mhz:.0f} MHz (median SM clock sampled during the timed region)")
    else:
        peak, unit, bound = lane_rate("fma") / 1e12, "Tlane-op/s", "alu"
        peak_src = (f"{rates['source']}: {rates['fma']:.3f} fp32 FMA warp-instructions per clock per SM x 32 lanes "
                    f"x {SM_COUNT} SMs x {clock_mhz:.0f} MHz")
    achieved = amount / dur / 1e12
    traffic = None if literal else NCU_TRAFFIC.get((wl.name, dominant))
    roofline = {"bound": bound, "kernel": dominant, "achieved": achieved, "peak": peak, "unit": unit,
                "frac": achieved / peak, "traffic": traffic["bytes_per_sample"] * wl.S + traffic["bytes_fixed"] if traffic else None,
                "traffic_source": traffic["source"] if traffic else None,
                "algorithmic_per_launch": amount, "peak_source": peak_src,
                "stage_ms": {k: round(v, 4) for k, v in stage_avg.items()}}
    # The path's model time: the slowest of the three resources the whole decision needs -- tensor cores (every
    # product that runs on them), the plain ALUs (the sort's min/max at the measured min/max rate, plus the
    # multiply-adds of whatever does not run on the tensor cores at the measured FMA rate), and the exchange of keys
    # between threads (the network's cross-lane stages at the measured shuffle rate).  path_frac sets it against the
    # measured time of a whole step; frac_vs_nlog2n sets the sort stage against the comparison-sort floor of
    # N log2 N compare-exchanges per row instead of the network's own count.
    p2 = 32
    while p2 < wl.N:
        p2 *= 2
    tensor_flops = sum(a for k, (kd, a) in work.items() if kd == "tensor")
    chain_on_tensor = bool(wl.precision) and wl.D in (16, 32) and not (literal and wl.D == 32)
    if chain_on_tensor:
        tensor_flops += 2 * work["chain"][1]
    fma_ops = sum(a for k, (kd, a) in work.items() if kd == "alu" and k not in ("sort", "chain")) + \
        (0 if chain_on_tensor else work["chain"][1])
    minmax_ops = work["sort"][1]
    e_keys = min(32, p2 // 32)
    lane_bits = (p2 // e_keys).bit_length() - 1                    # cross-lane (and cross-warp) bits of a key's index
    xchg_stages = lane_bits * (lane_bits + 1) // 2                 # stages whose partners sit in another thread
    xchg_ops = wl.S * p2 * xchg_stages                             # one key moved per lane per such stage
    t_tc = tensor_flops / tensor_peak
    t_alu = minmax_ops / lane_rate("minmax") + fma_ops / lane_rate("fma")
    t_xchg = xchg_ops / lane_rate("shuffle")
    t_model = max(t_tc, t_alu, t_xchg)
    # Stage by stage: each of the three large stages against the one unit its arithmetic runs on (tensor cores for the
    # products that use them, the FMA rate for those that do not, the min/max rate for the sort), and their sum against
    # the time the three take one after the other.  Looser than path_frac (it lets no stage overlap another), stricter
    # than the dominant kernel's own fraction.
    ideal = {
        "chain": 2 * work["chain"][1] / tensor_peak if chain_on_tensor else work["chain"][1] / lane_rate("fma"),
        "emission": work["emission"][1] / (tensor_peak if work["emission"][0] == "tensor" else lane_rate("fma")),
        "sort": minmax_ops / lane_rate("minmax"),
    }
    big = ("chain", "emission", "sort")
    roofline.update({
        "stage_frac": {k: round(ideal[k] / (stage_avg[k] * 1e-3), 4) for k in big},
        "path_frac_sum": sum(ideal[k] for k in big) / (sum(stage_avg[k] for k in big) * 1e-3),
        "path_frac": t_model / (ms_per_step * 1e-3),
        "path_model_ms": {"tensor": round(t_tc * 1e3, 4), "alu": round(t_alu * 1e3, 4), "exchange": round(t_xchg * 1e3, 4)},
        "path_model_sources": {
            "tensor": f"{tensor_flops:.4g} FLOP / ({tensor_src})",
            "alu": f"{minmax_ops:.4g} min/max + {fma_ops:.4g} multiply-adds (counted from the kernels' source) at the "
                   f"{rates['source']} min/max and FMA rates, {clock_mhz:.0f} MHz",
            "exchange": f"{xchg_ops:.4g} keys exchanged between threads ({xchg_stages} cross-thread stages of the network) at the "
                        f"{rates['source']} shuffle rate"},
        "frac_vs_nlog2n": (wl.S * p2 * (p2.bit_length() - 1) * 2 / (stage_avg["sort"] * 1e-3)) / lane_rate("minmax"),
        "pipe_rates": {k: round(rates[k], 4) for k in ("minmax", "shuffle", "fma")},
        "pipe_rates_source": rates["source"],
    })

    # The emission output layer on the tensor cores is bound by its operand stream from L2 into shared memory
    # (per 128 x 128 output tile the 128 hidden vectors and the 256 weight rows, 4 * H bytes each).
    # Set it against the rate the library measures for exactly those copies on this GPU: weights from a matrix of a
    # few MB that every SM re-reads, hidden vectors from one of tens of MB.
    if wl.precision and not literal and not args.no_measure_alu_peak:
        from paper_1803_04209_b200 import binding as _b
        op_rates = _b.measure_operand_stream(local_rank)
        n_tiles = -(-wl.S // 128) * -(-wl.N // 128)
        k_bytes = -(-wl.H // 32) * 128                               # bytes of one operand row (K blocks of 32 floats)
        bytes_w, bytes_v = n_tiles * 256 * k_bytes, n_tiles * 128 * k_bytes
        t_stream = bytes_w / (op_rates["weights_2mb"] * 1e9) + bytes_v / (op_rates["hidden_64mb"] * 1e9)
        roofline["emission_stream"] = {
            "bound": "l2 -> shared memory operand stream",
            "bytes_per_launch": bytes_w + bytes_v,
            "achieved_gbs": round((bytes_w + bytes_v) / (stage_avg["emission"] * 1e-3) / 1e9, 1),
            "peak_gbs": {k: round(v, 1) for k, v in op_rates.items()},
            "model_ms": round(t_stream * 1e3, 4),
            "frac": round(t_stream / (stage_avg["emission"] * 1e-3), 4),
            "peak_source": "measured (cutoff_measure_operand_stream, this run): the kernel's own copies, nothing consuming them",
        }

    # ---- sustained: the same step replayed back to back for a few seconds, with the clocks seen -------------
    sustained = None
    if args.sustained_seconds > 0 and world == 1:
        n_rep = max(50, int(args.sustained_seconds / max(ms_per_step * 1e-3, 1e-5)))
        sampler2 = ClockSampler(local_rank)
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        sampler2.start()
        ev0.record(stream)
        for i in range(n_rep):
            step_device((args.warmup + i) % dev_trace.shape[0])
        ev1.record(stream)
        ev1.synchronize()
        clk2 = sampler2.stop()
        ms_sus = ev0.elapsed_time(ev1) / n_rep
        sustained = {"steps": n_rep, "ms_per_step": ms_sus, "value": wl.S * wl.N / (ms_sus * 1e-3), "unit": UNIT,
                     "clocks": clk2, "ms_x_mhz": ms_sus * (clk2.get("sm_mhz") or 0.0),
                     "how": "the same graph replays back to back, no L2 flush in between (the 268 MB sample matrix "
                            "alone exceeds the L2), one pair of CUDA events around all of them"}

    cpu_baseline = None
    if not args.no_cpu_baseline:
        sample_S = min(wl.S, args.cpu_baseline_samples)
        sec = time_oracle(wl, weights, trace, sample_S)
        cpu_baseline = {"value": sample_S * wl.N / sec, "unit": UNIT, "cores": cpu_threads(), "kind": "oracle",
                        "sample": f"one decision on {sample_S} of {wl.S} samples, all {wl.N} workers, {sec:.2f} s"}

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": PRECISION_NAMES[wl.precision], "data": "synthetic",
        "config": {"workload": wl.name, "variant": args.variant, "N": wl.N, "D": wl.D, "H": wl.H, "lag": wl.lag,
                   "S_per_gpu": wl.S, "parallelism": f"samples x{world}", "l2": "flushed between timed steps (256 MiB write)",
                   "timing": "CUDA events per step on the library's stream; stage times from a separate pass",
                   "launch": "CUDA graph replay of push + decision" if use_graph else "kernel by kernel"},
        "e2e": {"value": e2e_value, "unit": UNIT, "ms_per_step": e2e_sec * 1e3,
                "h2d_bytes_per_step": 4 * wl.N, "d2h_bytes_per_step": 40 + 8 * wl.N},
        "gpu_launches": int(launches), "clocks": clocks, "roofline": roofline, "cpu_baseline": cpu_baseline,
        "stream_latency": stream_latency, "sustained": sustained,
        "timed_region_wall_s": round(wall, 3),
    }
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()

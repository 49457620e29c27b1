#!/usr/bin/env python
"""Benchmark of the double-sampled low-precision SGD path.

A "step" is one pass of the whole path over one synthetic workload: quantize the dense fp32
samples into two packed planes (after placing variance-optimal levels, if the workload asks for
them), run the workload's SGD epochs over the planes, evaluate the dense training loss.  The
default workload is the largest configuration (c5).

  value         samples/s per SGD epoch = m / mean duration of a zipml_sgd_epoch launch (CUDA events),
                planes resident in device memory; `whole_path_samples_per_s` beside it counts the
                whole pass (quantize + epochs + loss)
  e2e           the whole pass through zipml_train_host with pinned HOST buffers (copies in the timed region)
  roofline      packed-code bytes per SGD-epoch launch / its CUDA-event duration, against the
                measured HBM copy rate; `latency_model` next to it: what the minibatch chain allows
  cpu_baseline  the CPU oracle as it stands, timed on this host (rank 0, N = 1 only)

`--impl reference` times the oracle alone (the reference arm of this tier).
With N > 1 ranks every rank runs its own replica of the workload (the path is single-GPU; there is
no data-path collective), and value is the sum over ranks divided by the slowest rank's time.
"""
import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

FALLBACK_HBM_GBS = 6650.0
NOMINAL_HBM_GBS = 8000.0
# dram__bytes_read.sum + dram__bytes_write.sum of one epoch launch, quoted from the ncu captures summarised under
# profiles/ (a run cannot measure them itself): (workload, engine) -> (bytes, where they come from)
NCU_TRAFFIC = {
    ("c2", 5): (203.04e6 + 3.76e6, "profiles/sgd_cluster_kernel_c2_full.md"),
    ("c5", 6): (4 * (591.80e6 + 6.29e6), "profiles/sgd_stream_kernel_c5_full.md, 16,384-row capture scaled x4 by the rows"),
    ("c5", 7): (4 * (538.45e6 + 4.86e6), "profiles/sgd_column_kernel_c5_full.md, 16,384-row capture scaled x4 by the rows"),
}
ENGINE_KERNELS = {1: "sgd_kernel (stepwise launches)", 2: "sgd_kernel (persistent)", 3: "sgd_ring_kernel", 4: "sgd_lean_kernel",
                  5: "sgd_cluster_kernel", 6: "sgd_stream_kernel", 7: "sgd_column_kernel"}


def measured_peaks():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "50"], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([t.strip() for t in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.thread.join(timeout=2)
        mhz = sorted(int(r[0]) for r in self.rows if r and r[0].isdigit())
        mx = [int(r[1]) for r in self.rows if len(r) > 1 and r[1].isdigit()]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = [n for i, n in enumerate(names) if any(len(r) > 2 + i and r[2 + i].lower().startswith("active")
                                                         for r in self.rows)]
        return {"sm_mhz": mhz[len(mhz) // 2] if mhz else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": reasons, "samples": len(mhz)}


def latency_model(ctx, engine_ran, n, step_bytes, peak_gbs):
    """What the minibatch chain allows: a step moves step_bytes and cannot start before the previous step's model
    exists, so it costs at least step_bytes / BW plus its exchanges between SMs (measured here with the library's
    communication skeleton: publish through L2, bounded-spin barrier, read the others' data).  ceiling_frac =
    S / (S / BW + k t_exchange) / BW with t_compute taken as zero: an upper bound on roofline.frac."""
    k = 1 if engine_ran in (6, 7) else 2           # stream, column: the dots; the others: gradient parts out, model back
    ctas = {5: 16}.get(engine_ran, 128)            # the cluster engine is one cluster of at most 16 CTAs
    floats = max(4, (n // ctas + 3) // 4 * 4)
    try:
        t_ns = ctx.zipml_barrier_latency(ctas, floats, 2000)
    except Exception:
        return None
    t_stream_us = step_bytes / (peak_gbs * 1e3)
    floor_us = k * t_ns * 1e-3
    return {"exchanges_per_step": k, "ctas": ctas, "t_exchange_us": t_ns * 1e-3, "chain_floor_us": floor_us,
            "us_per_step_at_copy_rate": t_stream_us, "ceiling_frac": t_stream_us / (t_stream_us + floor_us),
            "note": "t_compute = 0; exchange measured with zipml_barrier_latency in this run"}


def run_oracle_pass(w, A, b, max_seconds=None):
    """One pass of the whole path on the CPU oracle; returns (seconds, samples processed, x, loss, seconds in SGD epochs)."""
    import numpy as np
    import oracle
    t0 = time.perf_counter()
    levels = None
    if w.levels == "optimal":
        levels, _ = oracle.optimal_levels(A, w.bits, w.hist_bins)
    ds = oracle.quantize(A, w.bits, seed=w.seed, mode=oracle.TABLE if levels is not None else oracle.UNIFORM,
                         levels=levels)
    x = np.zeros(w.n, np.float32)
    te = time.perf_counter()
    for ep in range(w.epochs):
        x, _ = oracle.sgd_epoch(ds, b, x, w.batch, w.lr, model_bits=w.model_bits, grad_bits=w.grad_bits, seed=w.seed,
                                epoch=ep)
    te = time.perf_counter() - te
    loss = oracle.loss_dense(A, b, x)
    return time.perf_counter() - t0, w.m * w.epochs, x, loss, te


def oracle_sample_rows(w):
    """Rows of the workload the oracle is timed on: about 10-30 s of single-core work."""
    # measured cost on one core: ~75 ns per element to quantize, ~9 ns per element and epoch of SGD
    per_row = w.n * (75e-9 + 9e-9 * w.epochs + 2e-9) + (w.n * 60e-9 if w.levels == "optimal" else 0)
    rows = int(15.0 / per_row)
    rows = max(w.batch * 4, min(w.m, rows))
    return min(w.m, rows // w.batch * w.batch if rows >= w.batch else rows)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c5", help="c1..c5, c4u (see paper_1611_05402_b200/synth.py)")
    ap.add_argument("--m", type=int, default=None, help="override the number of samples (smaller profiling cases)")
    ap.add_argument("--engine", default="auto", choices=["auto", "stepwise", "persistent", "ring", "lean", "cluster", "stream", "column"])
    ap.add_argument("--chunk-rows", type=int, default=0, help="column engine: rows per chunk (0 = automatic)")
    ap.add_argument("--feature-parts", type=int, default=0)
    ap.add_argument("--row-parts", type=int, default=0)
    ap.add_argument("--sharded", action="store_true",
                    help="N > 1: one epoch over all ranks' rows (every minibatch split by rows, one all-reduce of n floats "
                         "per step) instead of N independent replicas")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-others", dest="others", action="store_false",
                    help="skip the brief epoch timings of the other workloads (N = 1 only)")
    args = ap.parse_args()

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))

    from paper_1611_05402_b200 import synth
    base = synth.WORKLOADS[args.workload]
    metric, unit = "samples/sec and packed-code HBM GB/s per SGD epoch (fraction of B200 peak)", "samples/s"

    # ------------------------------------------------------------------ reference arm: the oracle
    if args.impl == "reference":
        if rank != 0:
            return
        import numpy as np
        from oracle.build import build as build_oracle
        build_oracle()
        w0 = synth.Workload(**{**base.__dict__})
        if args.m:
            w0.m = args.m
        rows = oracle_sample_rows(w0)
        # spread the few-minute budget over warmup + steps
        rows = max(w0.batch, int(rows / max(1, (args.steps + args.warmup) / 4)) // w0.batch * w0.batch)
        rows = min(rows, w0.m)
        w, A, b, _ = synth.make(args.workload, m=rows)
        A, b = A.numpy(), b.numpy()
        for _ in range(args.warmup):
            run_oracle_pass(w, A, b)
        t, t_ep = 0.0, 0.0
        for _ in range(args.steps):
            dt, samples, _, _, te = run_oracle_pass(w, A, b)
            t += dt
            t_ep += te
        value = samples * args.steps / t_ep            # samples/s per SGD epoch, like the other arm's value
        sample = (f"first {rows} of {w0.m} rows of {args.workload}, all {w.epochs} epochs, single thread; "
                  f"whole path (quantize + epochs + loss): {samples * args.steps / t:.0f} samples/s")
        print(json.dumps({
            "impl": "reference", "metric": metric, "value": value, "unit": unit, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": 1e3 * t / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": w0.name, "m": w0.m, "n": w0.n, "bits": w0.bits, "batch": w0.batch, "epochs": w0.epochs},
            "cpu_baseline": {"value": value, "unit": unit, "cores": 1, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": unit, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0,
        }))
        return

    # ------------------------------------------------------------------ our arm
    import torch
    import torch.distributed as dist
    from paper_1611_05402_b200 import binding, replicas
    from paper_1611_05402_b200.build import build as build_cuda
    if rank == 0:
        build_cuda()
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
        dist.barrier()
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    engine = {"auto": binding.ENGINE_AUTO, "stepwise": binding.ENGINE_STEPWISE, "persistent": binding.ENGINE_PERSISTENT,
              "ring": binding.ENGINE_RING, "lean": binding.ENGINE_LEAN, "cluster": binding.ENGINE_CLUSTER,
              "stream": binding.ENGINE_STREAM, "column": binding.ENGINE_COLUMN}[args.engine]

    sharded = args.sharded and world > 1
    w, A, b, _ = synth.make(args.workload, m=args.m, device=dev, seed=base.seed + (0 if sharded else rank))
    plan = None
    if sharded:
        # every rank draws the same samples and keeps its rows of every minibatch (quantized with its own draws)
        from paper_1611_05402_b200 import sharded as sh
        plan = sh.ShardPlan(w.m, w.batch, rank, world)
        A, b = sh.take_rows(plan, A), sh.take_rows(plan, b)
    ctx = binding.Context(dev)
    loss_dev = torch.zeros(1, dtype=torch.float64, device=dev)
    kw = dict(model_bits=w.model_bits, grad_bits=w.grad_bits, seed=w.seed, engine=engine,
              grid_feature_parts=args.feature_parts, grid_row_parts=args.row_parts, column_chunk_rows=args.chunk_rows)
    epoch_events, quant_events, loss_events = [], [], []

    def timed(events, record, fn):
        if not record:
            return fn()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        out = fn()
        e1.record()
        events.append((e0, e1))
        return out

    def one_pass(record):
        def quant():
            levels = ctx.zipml_optimal_levels(A, w.bits, w.hist_bins) if w.levels == "optimal" else None
            return ctx.zipml_quantize(A, w.bits, seed=w.seed, level_mode=binding.LEVELS_TABLE if levels is not None else
                                      binding.LEVELS_UNIFORM, levels=levels)
        ds = timed(quant_events, record, quant)
        x = torch.zeros(w.n, dtype=torch.float32, device=dev)
        for ep in range(w.epochs):
            if sharded:
                run = sh.ShardedEpoch(ctx, plan, ds, b, x, w.lr, model_bits=w.model_bits, grad_bits=w.grad_bits, seed=w.seed,
                                      epoch=ep, engine=engine)
                timed(epoch_events, record, run.run)
            else:
                timed(epoch_events, record, lambda: ctx.zipml_sgd_epoch(ds, b, x, w.batch, w.lr, epoch=ep, **kw))
        timed(loss_events, record, lambda: ctx.zipml_loss(binding.LOSS_DENSE, b, x, A=A, out=loss_dev))
        return ds, x

    def fence():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    # (the sampler starts before the warm-up passes -- the same work as the timed ones -- so that its first samples
    # do not wait for nvidia-smi to come up inside a timed region of a fraction of a second)
    sampler = ClockSampler(local_rank)
    sampler.start()
    for _ in range(max(args.warmup, 0)):
        ds, x = one_pass(False)
    ctx.zipml_sync()
    fence()
    launches0 = ctx.zipml_kernel_launches()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    for _ in range(args.steps):
        ds, x = one_pass(True)
    t1.record()
    fence()
    clocks = sampler.stop()
    ctx.zipml_sync()
    launches = ctx.zipml_kernel_launches() - launches0
    units = w.m / world if sharded else w.m           # (whole_job_value multiplies by the ranks)
    whole_value, ms_total = replicas.whole_job_value(units * w.epochs * args.steps, t0.elapsed_time(t1), dev)
    final_loss = float(loss_dev.item())

    # dominant kernel: the SGD epoch launch
    epoch_ms = sorted(a.elapsed_time(b_) for a, b_ in epoch_events)
    epoch_avg_ms = sum(epoch_ms) / len(epoch_ms)
    packed_bytes = ds.packed_bytes
    peak, peak_kind = measured_peaks()
    achieved = packed_bytes / (epoch_avg_ms * 1e-3) / 1e9
    value, _ = replicas.whole_job_value(units, epoch_avg_ms, dev)        # samples/s per SGD epoch, all ranks
    steps_per_epoch = (w.m + w.batch - 1) // w.batch
    step_us = 1e3 * epoch_avg_ms / steps_per_epoch
    step_bytes = packed_bytes / steps_per_epoch
    roofline = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                "traffic": NCU_TRAFFIC.get((args.workload, ctx.zipml_last_engine()), (None, None))[0] if args.m is None else None,
                "traffic_source": NCU_TRAFFIC.get((args.workload, ctx.zipml_last_engine()), (None, None))[1] if args.m is None else None,
                "peak_kind": f"of {peak_kind} copy rate", "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS,
                "kernel": ENGINE_KERNELS.get(ctx.zipml_last_engine(), "?") + " (one launch per epoch)",
                "algorithmic_bytes_per_launch": packed_bytes,
                "launch_ms_avg": epoch_avg_ms, "launch_ms_min": epoch_ms[0],
                "epoch_samples_per_s": w.m / (epoch_avg_ms * 1e-3),
                # the minibatch chain is sequential: a step moves step_bytes and cannot start before the previous
                # step's model exists, so the epoch is bound by steps * (exchange latency), not by bytes / bandwidth
                "steps_per_launch": steps_per_epoch, "us_per_step": step_us, "bytes_per_step": step_bytes,
                "us_per_step_at_hbm_peak": step_bytes / (peak * 1e3),
                "latency_model": latency_model(ctx, ctx.zipml_last_engine(), w.n, step_bytes, peak)}

    def stage(events, nbytes):
        ms_ = sorted(a_.elapsed_time(b_) for a_, b_ in events)
        avg = sum(ms_) / len(ms_)
        return {"ms": avg, "GB/s": nbytes / (avg * 1e-3) / 1e9, "frac_of_copy_rate": nbytes / (avg * 1e-3) / 1e9 / peak,
                "algorithmic_bytes": nbytes}
    a_bytes = 4 * w.m * w.n
    stages = {"quantize" + ("+levels" if w.levels == "optimal" else ""):
              stage(quant_events, a_bytes * (2 if w.levels != "optimal" else 4) + 2 * ds.m * ds.row_bytes),
              "loss_dense": stage(loss_events, a_bytes + 4 * w.m)}
    # the loss estimate straight from the two code planes (outside the timed region: the pass above ends in the dense loss)
    lc_events, lc_dev = [], torch.zeros(1, dtype=torch.float64, device=dev)
    for i in range(4):
        timed(lc_events, i > 0, lambda: ctx.zipml_loss(binding.LOSS_CODES, b, x, data=ds, out=lc_dev))
    ctx.zipml_sync()
    stages["loss_codes"] = stage(lc_events, packed_bytes + 4 * w.m)

    # ------------------------------------------------------------------ end to end from host buffers
    e2e = None
    if not args.no_e2e and not sharded:           # (the host entry point runs one device's rows: a replica's figure)
        Ah = torch.empty(A.shape, dtype=torch.float32, pin_memory=True)
        Ah.copy_(A)
        bh = torch.empty(b.shape, dtype=torch.float32, pin_memory=True)
        bh.copy_(b)
        xh = torch.zeros(w.n, dtype=torch.float32, pin_memory=True)

        def host_pass():
            xh.zero_()
            return ctx.zipml_train_host(Ah, bh, xh, w.bits, w.batch, w.lr, w.epochs, optimal_levels=w.levels == "optimal",
                                        hist_bins=w.hist_bins, quantize_seed=w.seed, **kw)
        host_pass()
        fence()
        k_e2e = max(1, min(args.steps, 3))
        h0, h1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        h0.record()
        for _ in range(k_e2e):
            e2e_loss = host_pass()                # returns the loss read back from the device: the call is synchronous
        h1.record()
        torch.cuda.synchronize()
        e2e_value, _ = replicas.whole_job_value(w.m * w.epochs * k_e2e, h0.elapsed_time(h1), dev)
        e2e = {"value": e2e_value, "unit": unit, "what": "whole pass from pinned host buffers: copies, quantize, epochs, dense loss",
               "h2d_bytes_per_step": int(Ah.numel() * 4 + bh.numel() * 4 + xh.numel() * 4),
               "d2h_bytes_per_step": int(xh.numel() * 4 + 8), "steps": k_e2e, "loss": e2e_loss}
        del Ah

    # ------------------------------------------------------------------ the other workloads, briefly
    others = None
    if world == 1 and args.others:
        others = {}
        del A
        torch.cuda.empty_cache()
        for key in [k for k in ("c1", "c2", "c3", "c4", "c5") if k != args.workload]:
            wo, Ao, bo, _ = synth.make(key, device=dev)
            lev = ctx.zipml_optimal_levels(Ao, wo.bits, wo.hist_bins) if wo.levels == "optimal" else None
            q0, q1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            q0.record()
            dso = ctx.zipml_quantize(Ao, wo.bits, seed=wo.seed, levels=lev,
                                     level_mode=binding.LEVELS_TABLE if lev is not None else binding.LEVELS_UNIFORM)
            q1.record()
            xo = torch.zeros(wo.n, dtype=torch.float32, device=dev)
            kwo = dict(model_bits=wo.model_bits, grad_bits=wo.grad_bits, seed=wo.seed, engine=engine)
            ctx.zipml_sgd_epoch(dso, bo, xo, wo.batch, wo.lr, epoch=0, **kwo)
            evs = []
            for ep in range(1, 4):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                ctx.zipml_sgd_epoch(dso, bo, xo, wo.batch, wo.lr, epoch=ep, **kwo)
                e1.record()
                evs.append((e0, e1))
            l0, l1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            lc = torch.zeros(1, dtype=torch.float64, device=dev)
            l0.record()
            ctx.zipml_loss(binding.LOSS_CODES, bo, xo, data=dso, out=lc)
            l1.record()
            ctx.zipml_sync()
            t_ep = sum(a_.elapsed_time(b_) for a_, b_ in evs) / len(evs)         # a mean, like the headline
            To = (wo.m + wo.batch - 1) // wo.batch
            lm = latency_model(ctx, ctx.zipml_last_engine(), wo.n, dso.packed_bytes / To, peak)
            others[key] = {"workload": wo.name, "kernel": ENGINE_KERNELS.get(ctx.zipml_last_engine(), "?"), "epoch_ms": t_ep, "us_per_step": 1e3 * t_ep / To,
                           "samples_per_s": wo.m / (t_ep * 1e-3), "packed_GB/s": dso.packed_bytes / (t_ep * 1e-3) / 1e9,
                           "frac_of_copy_rate": dso.packed_bytes / (t_ep * 1e-3) / 1e9 / peak,
                           "ceiling_frac": lm["ceiling_frac"] if lm else None, "chain_floor_us": lm["chain_floor_us"] if lm else None,
                           "quantize_GB/s": (8 * wo.m * wo.n + 2 * dso.m * dso.row_bytes) / (q0.elapsed_time(q1) * 1e-3) / 1e9,
                           "loss_codes_GB/s": dso.packed_bytes / (l0.elapsed_time(l1) * 1e-3) / 1e9}
            del Ao, dso, bo, xo
            torch.cuda.empty_cache()

    # ------------------------------------------------------------------ the oracle beside it
    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        rows = oracle_sample_rows(w)
        ws, As, bs, _ = synth.make(args.workload, m=rows)
        dt, samples, _, _, te = run_oracle_pass(ws, As.numpy(), bs.numpy())
        cpu_baseline = {"value": samples / te, "unit": unit, "cores": 1, "kind": "oracle",
                        "whole_path_samples_per_s": samples / dt,
                        "sample": f"first {rows} of {w.m} rows of {args.workload}, all {w.epochs} epochs ({te:.1f} s in the SGD "
                                  f"epochs, {dt:.1f} s for the whole path) on one thread of {os.cpu_count()} host cores"}

    if rank == 0:
        print(json.dumps({
            "metric": metric, "value": value, "unit": unit, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_total / args.steps, "higher_is_better": True, "scaling": "strong" if sharded else "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic",
            "config": {"workload": w.name, "m": w.m, "n": w.n, "bits": w.bits, "batch": w.batch, "epochs": w.epochs,
                       "levels": w.levels, "model_bits": w.model_bits, "grad_bits": w.grad_bits, "engine": args.engine,
                       "l2": "inputs larger than L2 (dense A and both planes are streamed every step)",
                       "multi_gpu": "row-sharded epoch, one all-reduce of n floats per step" if sharded else "replicas only"},
            "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches), "roofline": roofline,
            "cpu_baseline": cpu_baseline, "final_loss": final_loss,
            "packed_gb_per_s_per_epoch": achieved, "whole_path_samples_per_s": whole_value,
            "stages": stages, "other_workloads": others,
        }))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()

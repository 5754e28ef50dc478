#!/usr/bin/env python
"""Benchmark of the dithered-backprop hot path on B200.

    python bench.py --gpus N --steps K --warmup W [--config 5|3|1] [--impl reference]

One *step* is one pass of the whole path (statistics -> NSD quantize/compact -> dX -> dW)
over every layer of the workload, on seeded synthetic inputs already resident in HBM.
The metric is dense-equivalent backward throughput: the FLOPs a dense backward of the same
layers would do (2 per MAC, both products) divided by the measured time.

Default workload (config 5): the ResNet-50 ImageNet-shaped bottleneck layer set, batch 64,
bf16 storage with fp32 accumulation, Delta = 5 std(delta) (about 90 % zeros after NSD).
With N > 1 every rank runs the same layer set on its own batch shard (weak scaling; the
path has no data-path exchange between ranks).

`--impl reference` times the CPU oracle (the plain fp64 definition used for parity checks)
on a bounded sample of the same workload, on the host cores.
"""
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

import workloads as wl  # noqa: E402

METRIC = "dithered backward dense-equiv GFLOP/s and % HBM roofline vs cuBLAS dense"
UNIT = "GFLOP/s (dense-equivalent, dW+dX)"
FMA_PEAK_TFLOPS = 148 * 128 * 2 * 1.965e9 / 1e12      # fp32 FMA lanes x 2 flop x max SM clock


def measured_peaks():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            p = json.load(f)
        return float(p["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


# ------------------------------------------------------------------ workloads

def layer_specs(config, batch):
    """[(Layer factory, multiplicity)] in network order."""
    if config == 1:
        return [(lambda: wl.config1(batch or 128), 1)], "config1: linear 784->300, B128, fp32, s=2"
    if config == 3:
        return [(lambda: wl.config3(batch or 128), 1)], "config3: conv3x3 64->64 @32x32, B128, fp32, s=2"
    if config == 5:
        b = batch or 64
        specs = [((lambda i=i: wl.config5_layer(i, batch=b)), wl.RESNET50_SET[i][5])
                 for i in range(len(wl.RESNET50_SET))]
        return specs, f"config5: ResNet-50 bottleneck layer set (48 convs, 16 shapes), B{b}, bf16, s=5"
    raise SystemExit("--config must be 1, 3 or 5")


def algorithmic_bytes(L):
    """Bytes one layer's backward must move at least: delta read twice (statistics, then
    quantize), sparse structure written once and read by both products, X and W read, dX and
    dW written."""
    e = 2 if L.dtype == "bf16" else 4
    nd, nx, nw = L.delta.size, L.X.size, L.W.size
    return 2 * nd * e + nx * e + nw * e + nx * e + nw * 4


# ------------------------------------------------------------------ clocks

class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.perf_counter(), [c.strip() for c in line.split(",")]))

    def stop(self, t_begin=None, t_end=None, t_fallback=None):
        """Samples taken inside [t_begin, t_end] (the timed region); when the region was shorter
        than the sampling period, the samples since t_fallback (warm-up included) instead."""
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        window = "timed region"
        rows = [r for t, r in self.rows if t_begin is None or (t_begin <= t <= t_end)]
        if not rows and t_fallback is not None:
            rows, window = [r for t, r in self.rows if t_fallback <= t <= t_end + 0.2], "warm-up and timed region"
        if not rows:
            rows, window = [r for _, r in self.rows], "whole run"
        sm = [float(r[0]) for r in rows if r and r[0].replace(".", "").isdigit()]
        mx = [float(r[1]) for r in rows if len(r) > 1 and r[1].replace(".", "").isdigit()]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = [n for j, n in enumerate(names)
                   if any(len(r) > 3 + j and r[3 + j].lower().startswith("active") for r in rows)]
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(mx) if mx else None, "reasons": reasons,
                "samples": len(sm), "window": window}


# ------------------------------------------------------------------ CPU oracle arm

def oracle_layers(config):
    """The bounded sample of the workload that the CPU oracle is timed on."""
    if config == 1:
        return [wl.config1()], "the whole layer (B128)", 200
    if config == 3:
        return [wl.config3(batch=32)], "batch 32 of 128", 4
    layers = [wl.config5_layer(i, batch=16) for i in range(len(wl.RESNET50_SET))]
    return layers, "batch 16 of 64 of all 16 shapes (one instance each)", 3


def oracle_time(layers, passes, budget_s=30.0):
    """Runs the oracle (NSD + fp64 products, as it stands) `passes` times over the sample;
    returns (dense-equivalent GFLOP/s, seconds, passes done)."""
    import oracle
    t0 = time.perf_counter()
    flops, done = 0.0, 0
    for _ in range(passes):
        for L in layers:
            D = oracle.step_size(L.delta, L.scale)
            codes, _, _ = oracle.nsd_codes(L.delta, L.seed, D)
            fn = oracle.linear_backward if L.kind == "linear" else oracle.conv_backward
            fn(codes, D, L.X, L.W)
            flops += L.dense_flops
        done += 1
        if time.perf_counter() - t0 > budget_s:
            break
    dt = time.perf_counter() - t0
    return flops / dt / 1e9, dt, done


def host_cores():
    try:
        return len(os.sched_getaffinity(0))
    except Exception:
        return os.cpu_count()


def oracle_sample(config):
    layers, what, passes = oracle_layers(config)
    v, dt, done = oracle_time(layers, passes)
    return v, dt, f"{what}, {done} passes", host_cores()


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    _, name = layer_specs(args.config, args.batch)
    layers, what, passes = oracle_layers(args.config)
    per_step = max(1, passes // 3)
    for _ in range(min(args.warmup, 1)):
        oracle_time(layers, 1)
    t0 = time.perf_counter()
    vals = [oracle_time(layers, per_step)[0] for _ in range(args.steps)]
    total = time.perf_counter() - t0
    v = float(np.mean(vals))
    what = f"{what}, {per_step} pass(es) per step"
    cores = host_cores()
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": total / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": {"workload": name, "sample": what},
        "cpu_baseline": {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": what},
        "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


# ------------------------------------------------------------------ CUDA arm

def max_over_ranks(value, device, world):
    """The slowest rank's time: every rank runs the same step on its own shard, so the job's
    step time is the maximum (the process group is NCCL on GPUs, gloo in the CPU tests)."""
    if world <= 1:
        return float(value)
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.item()


def job_throughput(flops_per_rank_step, world, ms_per_step):
    """Whole-job dense-equivalent GFLOP/s: the work of all ranks over the slowest rank's time."""
    return flops_per_rank_step * world / (ms_per_step * 1e-3) / 1e9


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", type=int, default=5)
    ap.add_argument("--batch", type=int, default=0, help="override the config's batch size")
    ap.add_argument("--only", default="", help="config 5: comma-separated shape indices to run (profiling aid)")
    ap.add_argument("--single", action="store_true", help="one instance of every shape (profiling aid)")
    ap.add_argument("--impl", default="ours")
    ap.add_argument("--no-dense", action="store_true", help="skip the cuDNN/cuBLAS dense comparison")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl != "reference":
        args.warmup = 3
    if args.impl == "reference":
        return run_reference(args)

    import torch
    import torch.distributed as dist
    import paper_2004_04729_b200 as dbp

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    dev = torch.device("cuda", local)
    ctx = dbp.Context(local)
    sampler = ClockSampler(local)       # nvidia-smi takes a while to deliver its first sample: start it now
    if rank == 0:
        sampler.start()

    specs, name = layer_specs(args.config, args.batch)
    if args.only:
        keep = [int(t) for t in args.only.split(",")]
        specs = [specs[i] for i in keep]
        name += f" [only shapes {keep}]"
    if args.single:
        specs = [(make, 1) for make, _ in specs]
        name += " [one instance per shape]"
    tdt = lambda L: torch.bfloat16 if L.dtype == "bf16" else torch.float32
    layers = []          # one entry per layer instance: (Layer, delta, X, W, dW, dX)
    hosts = []           # one entry per distinct shape: pinned host tensors
    dense_flops = alg_bytes = 0.0
    for make, mult in specs:
        L = make()
        hd, hX, hW = (torch.from_numpy(a).to(tdt(L)).pin_memory() for a in (L.delta, L.X, L.W))
        hosts.append((L, mult, hd, hX, hW,
                      torch.empty(L.W.shape, dtype=torch.float32).pin_memory(),
                      torch.empty(L.X.shape, dtype=tdt(L)).pin_memory()))
        for _ in range(mult):
            d, X, W = hd.to(dev), hX.to(dev), hW.to(dev)
            layers.append((L, d, X, W,
                           torch.empty(L.W.shape, dtype=torch.float32, device=dev),
                           torch.empty(L.X.shape, dtype=tdt(L), device=dev)))
            dense_flops += L.dense_flops
            alg_bytes += algorithmic_bytes(L)
    lib = dbp.load_library()
    import ctypes

    ASYNC = dbp.DBP_DW_ASYNC        # dW of a layer may still run while the next layer is quantized; joined at the step's end

    def run_layer(L, d, X, W, dW, dX):
        code = 1 if L.dtype == "bf16" else 0
        if L.kind == "linear":
            B, N = d.shape
            rc = lib.dithered_linear_backward(ctx._h, d.data_ptr(), X.data_ptr(), W.data_ptr(), code,
                                              B, N, X.shape[1], L.seed, L.scale, None, None,
                                              dW.data_ptr(), dX.data_ptr(), None, ASYNC)
        else:
            B, Co, H, Wd = d.shape
            rc = lib.dithered_conv_backward(ctx._h, d.data_ptr(), X.data_ptr(), W.data_ptr(), code,
                                            B, X.shape[1], Co, H, Wd, L.k, 1, (L.k - 1) // 2, L.seed,
                                            L.scale, None, None, dW.data_ptr(), dX.data_ptr(), None, ASYNC)
        if rc != 0:
            raise RuntimeError(f"library call failed on {L.name}: {rc}")

    def step():
        for item in layers:
            run_layer(*item)
        ctx.join()                  # every dW of the step is ordered into the stream before the step ends

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # Warm-up steps run with every kernel kind bracketed by events: that gives the per-kind table
    # and names the dominant kind. The events cost stream time, so the timed region brackets
    # only the dominant kind (its duration is what the roofline line uses).
    # The first warm-up step grows the context's workspaces (allocations) and is not profiled.
    t_warm = time.perf_counter()
    step()
    barrier()
    ctx.profile_enable(True)
    ctx.profile_select(None)
    ctx.profile_read()
    nprof = max(args.warmup - 1, 1)
    for _ in range(nprof):
        step()
    barrier()
    prof_all = ctx.profile_read()
    top_kind = max(prof_all, key=lambda k: prof_all[k][0])
    ctx.profile_select([top_kind])
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    t_begin = time.perf_counter()
    e0.record()
    for _ in range(args.steps):
        step()
    e1.record()
    barrier()
    t_end = time.perf_counter()
    clocks = sampler.stop(t_begin, t_end, t_warm) if rank == 0 else None
    ms = e0.elapsed_time(e1) / args.steps
    prof_top = ctx.profile_read()
    ctx.profile_enable(False)
    ctx.profile_select(None)
    ms = max_over_ranks(ms, dev, world)
    value = job_throughput(dense_flops, world, ms)

    # host time to enqueue one step (the launch queue is empty and deep enough for one step)
    barrier()
    t0 = time.perf_counter()
    step()
    host_ms = (time.perf_counter() - t0) * 1e3
    barrier()

    # non-zero work actually done (for the arithmetic roofline of the sparse products)
    nnz_flops = 0.0
    for (L, d, X, W, dW, dX) in layers:
        q = dbp.nsd_quantize(ctx, d, L.seed, L.scale)
        nnz_flops += (q.nnz.item() / d.numel()) * L.dense_flops
    torch.cuda.synchronize()
    density = nnz_flops / dense_flops

    # ---- end to end through the host entry points (H2D + kernels + D2H every step)
    e2e = None
    if not args.no_e2e:
        h2d = d2h = 0
        def host_step():
            for (L, mult, hd, hX, hW, odW, odX) in hosts:
                fn = dbp.dithered_linear_backward_host if L.kind == "linear" else dbp.dithered_conv_backward_host
                for _ in range(mult):
                    fn(ctx, hd, hX, hW, L.seed, L.scale, odW, odX)
        for (L, mult, hd, hX, hW, odW, odX) in hosts:
            h2d += mult * (hd.numel() * hd.element_size() + hX.numel() * hX.element_size() + hW.numel() * hW.element_size())
            d2h += mult * (odW.numel() * 4 + odX.numel() * odX.element_size())
        host_step()
        ksteps = max(1, min(args.steps, 3))
        barrier()
        t0 = time.perf_counter()
        for _ in range(ksteps):
            host_step()
        barrier()
        dt = (time.perf_counter() - t0) / ksteps
        dt = max_over_ranks(dt, dev, world)
        e2e = {"value": job_throughput(dense_flops, world, dt * 1e3), "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "ms_per_step": dt * 1e3, "steps": ksteps}

    # ---- dense library backward on the same shapes (context, not the product path)
    dense = None
    if not args.no_dense and rank == 0:
        import torch.nn.functional as F
        def dense_step(allow_tf32):
            torch.backends.cudnn.allow_tf32 = allow_tf32
            torch.backends.cuda.matmul.allow_tf32 = allow_tf32
            for (L, d, X, W, dW, dX) in layers:
                if L.kind == "linear":
                    torch.matmul(d.t(), X)
                    torch.matmul(d, W)
                else:
                    p = (L.k - 1) // 2
                    torch.ops.aten.convolution_backward(d, X, W, None, [1, 1], [p, p], [1, 1], False,
                                                        [0, 0], 1, [True, True, False])
        dense = {}
        for label, tf32 in (("tf32_off", False), ("tf32_on", True)):
            for _ in range(3):
                dense_step(tf32)
            torch.cuda.synchronize()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for _ in range(max(3, args.steps // 2)):
                dense_step(tf32)
            b.record()
            torch.cuda.synchronize()
            dms = a.elapsed_time(b) / max(3, args.steps // 2)
            dense[label] = {"ms_per_step": dms, "gflops": dense_flops / (dms * 1e-3) / 1e9}
        dense["what"] = "torch cuDNN/cuBLAS backward-data + backward-filter on the unquantized delta, same buffers"

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    hbm_peak, peak_src = measured_peaks()
    prof = {k: (v[0] / nprof, v[1] / nprof) for k, v in prof_all.items()}   # per step
    kern = {k: {"ms_per_step": v[0], "launches_per_step": v[1], "measured": "warm-up steps, every kind bracketed by events"}
            for k, v in prof.items() if v[1]}
    # algorithmic work of every kernel kind over one step; a layer counts as dense when the
    # library would run it so at this density (bf16, 1x1/linear or 3x3, channels % 8 == 0)
    e = 2 if layers[0][0].dtype == "bf16" else 4
    dense_on = prof["dx_dense"][1] > 0
    is_dense = lambda L: (dense_on and L.dtype == "bf16" and L.X.shape[1] % 8 == 0 and L.delta.shape[1] % 8 == 0)
    # kernels launched in the timed region: statistics and quantize, then for a dense layer the
    # dX product (after the weight re-layout for 3x3) and the dW product with its split-K sum,
    # for a sparse layer the weight re-layout, dX and dW
    # kernels launched in the timed region, per layer: statistics and quantize; then, dense 1x1:
    # dX, (copy of X to padded planes when H*W % 8 != 0), dW, split-K sum; dense 3x3: weight
    # re-layout, dX, dW, split-K sum; sparse: weight re-layout, dX, dW
    tma = lambda L: is_dense(L) and L.kind == "conv" and L.k == 1 and L.X.shape[2] * L.X.shape[3] >= 16
    per_step = 0
    for (L, d, X, W, dW, dX) in layers:
        if tma(L):
            per_step += 2 + 1 + (1 if (L.X.shape[2] * L.X.shape[3]) % 8 else 0) + 2
        elif is_dense(L):
            per_step += 2 + (2 if (L.kind == "conv" and L.k == 3) else 1) + 2
        else:
            per_step += 2 + 2 + 1
    launches = per_step * args.steps
    work = {k: 0.0 for k in ("statistics", "quantize", "dx", "dw", "dx_dense", "dw_dense")}
    for (L, d, X, W, dW, dX) in layers:
        nd, nx, nw = d.numel(), X.numel(), W.numel()
        cb = 2 if tma(L) else 1                                        # bytes per code the product kernels read
        work["statistics"] += nd * e                                   # bytes
        work["quantize"] += nd * (e + cb)                              # bytes: delta read, codes written
        if is_dense(L):
            work["dx_dense"] += nd * cb + nx * e + nw * e              # bytes: codes, dX, W
            work["dw_dense"] += nd * cb + nx * e + nw * 4              # bytes: codes, X, dW
        else:
            work["dx"] += density * L.dense_flops / 2                  # flops of non-zero codes
            work["dw"] += density * L.dense_flops / 2
    top = top_kind if top_kind in work else max(work, key=lambda k: prof[k][0])
    # duration of the dominant kind inside the timed region (only that kind was bracketed there)
    t_s = (prof_top[top][0] / args.steps if prof_top[top][1] else prof[top][0]) * 1e-3
    if top in kern:
        kern[top]["ms_per_step_timed_region"] = t_s * 1e3
    if top in ("dx", "dw"):
        ach = work[top] / t_s / 1e12
        roof = {"kernel": f"sparse {top} (conv_{top}2_kernel)", "bound": "alu", "achieved": ach,
                "peak": FMA_PEAK_TFLOPS, "unit": "TFLOP/s", "frac": ach / FMA_PEAK_TFLOPS, "traffic": None,
                "peak_source": "derived: 148 SMs x 128 fp32 lanes x 2 flop x 1.965 GHz",
                "note": "non-zero-code FMAs only (2*nnz*K_eff flops per product), summed over the layers that use it"}
    else:
        ach = work[top] / t_s / 1e9
        roof = {"kernel": {"dx_dense": "tensor-core dX (tma_dx_kernel for 1x1, tc3_dx_shift_kernel for 3x3)",
                           "dw_dense": "tensor-core dW (tma_dw_kernel for 1x1, tc3_dw_shift_kernel for 3x3, + split-K sums)"}.get(top, top + "_kernel"),
                "bound": "hbm", "achieved": ach, "peak": hbm_peak, "unit": "GB/s", "frac": ach / hbm_peak,
                "traffic": None, "peak_source": peak_src + " (MEASURED_PEAKS.json hbm_gbs)",
                "note": "algorithmic bytes summed over the layers that use it / summed launch time"}
    for k in work:
        if k in kern:
            kern[k]["work_per_step"] = work[k]
            kern[k]["unit"] = "flop" if k in ("dx", "dw") else "byte"
    path_gbs = alg_bytes / (ms * 1e-3) / 1e9
    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16 storage, f32 accumulate" if layers[0][0].dtype == "bf16" else "f32",
        "data": "synthetic",
        "config": {"workload": name, "layers_per_step": len(layers), "l2": "inputs larger than L2 (distinct buffers per layer instance)"
                   if alg_bytes > 2.5e8 else "working set smaller than L2 (warm)", "nsd_density": density},
        "clocks": clocks, "gpu_launches": launches, "host_enqueue_ms_per_step": host_ms, "e2e": e2e,
        "roofline": roof,
        "hbm_path": {"algorithmic_gb_per_step": alg_bytes / 1e9, "achieved_gbs": path_gbs,
                     "frac_of_measured_hbm": path_gbs / hbm_peak, "peak": hbm_peak, "peak_source": peak_src},
        "kernels": kern, "dense_baseline": dense,
    }
    if not args.no_cpu and world == 1:
        v, dt, what, cores = oracle_sample(args.config)
        out["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": what,
                               "seconds": dt}
    print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()

#!/usr/bin/env python
"""Benchmark of the dithered-backprop hot path on B200.

    python bench.py --gpus N --steps K --warmup W [--config 5|4|3|2|1] [--impl reference]

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


def measured_peaks():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            p = json.load(f)
        return float(p["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


# ------------------------------------------------------------------ workloads

CHAIN_NAMES = {2: "config2: LeNet-300-100 full backward, B256, fp32, s=2",
               4: "config4: VGG-16/CIFAR full backward (13 conv3x3 + FC), B128, fp32, s=2"}


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
    if config in CHAIN_NAMES:
        return [], CHAIN_NAMES[config]
    raise SystemExit("--config must be 1 ... 5")


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
    if config == 2:
        c = wl.mlp_chain(batch=256)
        return [c], "the whole network (B256)", 100
    if config == 4:
        c = wl.vgg_chain(batch=8)
        return [c], "batch 8 of 128", 2
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
            if isinstance(L, wl.Chain):
                oracle.chain_backward(L.kinds, L.X, L.W, L.relu_mask, L.pool_argmax, L.delta_out, L.scale, 0)
                flops += chain_flops(L)
                continue
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


def chain_flops(c):
    """Dense backward FLOPs of a chain (2 per MAC, dW and dX of every layer; the first layer's dX is
    not computed, as in a training step)."""
    f = 0.0
    for l, kind in enumerate(c.kinds):
        X, W = c.X[l], c.W[l]
        macs = X.shape[0] * W.shape[0] * W.shape[1] * (X.shape[2] * X.shape[3] * 9 if kind == "conv" else 1)
        f += 2.0 * macs * (2 if l > 0 else 1)
    return f


def chain_bytes(c):
    """Bytes a chain's backward must move at least: per layer delta twice (statistics, quantize), X and W
    read, dW and (but for the first layer) dX written; fp32."""
    b = 0
    for l in range(len(c.kinds)):
        nx, nw = c.X[l].size, c.W[l].size
        nd = c.X[l].shape[0] * c.W[l].shape[0] * (c.X[l].shape[2] * c.X[l].shape[3] if c.kinds[l] == "conv" else 1)
        b += 4 * (2 * nd + nx + nw + nw + (nx if l > 0 else 0))
    return b


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


def time_events(torch, fn, reps):
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(reps):
        fn()
    b.record()
    torch.cuda.synchronize()
    return a.elapsed_time(b) / reps


def graph_times(torch, ctx, fns, reps):
    """Each closure captured into a CUDA graph on a side stream and replayed: device time without the host's
    per-call cost (which is what bounds eager calls on layers of a few microseconds)."""
    side = torch.cuda.Stream()
    prev = ctx._stream
    torch.cuda.synchronize()
    out = []
    ctx.set_stream(side)
    try:
        with torch.cuda.stream(side):
            for fn in fns:
                fn()                                     # allocations happen outside the capture
                side.synchronize()
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=side):
                    fn()
                for _ in range(5):
                    g.replay()
                side.synchronize()
                out.append(time_events(torch, g.replay, reps))
    finally:
        torch.cuda.synchronize()
        ctx.set_stream(prev)
    return out


def dense_layer_fn(torch, L, d, X, W):
    if L.kind == "linear":
        return lambda: (torch.matmul(d.t(), X), torch.matmul(d, W))
    p = (L.k - 1) // 2
    return lambda: torch.ops.aten.convolution_backward(d, X, W, None, [1, 1], [p, p], [1, 1], False, [0, 0], 1,
                                                       [True, True, False])


def dense_times(torch, fns, reps):
    """cuDNN / cuBLAS backward (autotuned algorithms) on the given closures, TF32 off and on."""
    torch.backends.cudnn.benchmark = True
    out = {}
    for label, tf32 in (("tf32_off", False), ("tf32_on", True)):
        torch.backends.cudnn.allow_tf32 = tf32
        torch.backends.cuda.matmul.allow_tf32 = tf32
        step = lambda: [f() for f in fns]
        for _ in range(3):
            step()
        torch.cuda.synchronize()
        out[label] = time_events(torch, step, reps)
    return out


def per_shape_table(torch, layers, run_layer, ctx, dq, hbm_peak, no_dense):
    """One row per distinct layer shape: time per layer of the whole backward (statistics, quantization, dX, dW)
    with the instances of the shape run back to back on their own buffers, as in the step (dW of one instance may
    run beside the next instance; joined after the last), the dense library's time for the same layers, and the
    layer's algorithmic bytes against the measured bandwidth."""
    groups = {}
    for idx, item in enumerate(layers):
        groups.setdefault(item[0].name, []).append(idx)
    torch.backends.cudnn.benchmark = True
    torch.backends.cudnn.allow_tf32 = False
    torch.backends.cuda.matmul.allow_tf32 = False
    rows = []
    for name, idxs in groups.items():
        L = layers[idxs[0]][0]
        def ours():
            for i in idxs:
                run_layer(*layers[i])
            ctx.join()
        for _ in range(3):
            ours()
        torch.cuda.synchronize()
        ms = time_events(torch, ours, 20) / len(idxs)
        row = {"shape": name, "instances": len(idxs), "ms": ms, "algorithmic_mb": algorithmic_bytes(L) / 1e6,
               "frac_of_measured_hbm": algorithmic_bytes(L) / (ms * 1e-3) / 1e9 / hbm_peak,
               "tflops_dense_equiv": L.dense_flops / (ms * 1e-3) / 1e12}
        if not no_dense and dq is not None:
            fns = [dense_layer_fn(torch, layers[i][0], dq[i], layers[i][2], layers[i][3]) for i in idxs]
            def dense():
                for f in fns:
                    f()
            for _ in range(3):
                dense()
            torch.cuda.synchronize()
            row["dense_ms"] = time_events(torch, dense, 20) / len(idxs)
        rows.append(row)
    return rows


def strided_table(torch, dbp, ctx, hbm_peak, no_dense, batch):
    """The stride-2 layers of the same network (a side measurement, not part of the step): time per layer of the
    whole backward through the library's stride-2 form, the dense library's strided backward on the dequantized
    gradient, and the layer's algorithmic bytes against the measured bandwidth. Two instances of each shape on
    their own buffers, run in turn."""
    dev = torch.device("cuda", ctx.device)
    torch.backends.cudnn.benchmark = True
    torch.backends.cudnn.allow_tf32 = False
    torch.backends.cuda.matmul.allow_tf32 = False
    rows = []
    for idx in range(len(wl.RESNET50_STRIDED)):
        L = wl.resnet50_strided_layer(idx, batch=batch)
        sets = []
        for _ in range(2):
            d, X, W = (torch.from_numpy(a).to(dev).to(torch.bfloat16) for a in (L.delta, L.X, L.W))
            sets.append((d, X, W))
        def ours():
            for d, X, W in sets:
                dbp.dithered_conv_backward(ctx, d, X, W, L.seed, L.scale, stride=2)
        for _ in range(3):
            ours()
        torch.cuda.synchronize()
        ms = time_events(torch, ours, 10) / len(sets)
        q = dbp.nsd_quantize(ctx, sets[0][0], L.seed, L.scale)
        row = {"shape": L.name, "k": L.k, "ms": ms, "algorithmic_mb": algorithmic_bytes(L) / 1e6,
               "frac_of_measured_hbm": algorithmic_bytes(L) / (ms * 1e-3) / 1e9 / hbm_peak,
               "tflops_dense_equiv": L.dense_flops / (ms * 1e-3) / 1e12, "nsd_density": q.nnz.item() / sets[0][0].numel()}
        if not no_dense:
            p = (L.k - 1) // 2
            fns = []
            for d, X, W in sets:
                g = (dbp.nsd_decode_dense(ctx, dbp.nsd_quantize(ctx, d, L.seed, L.scale), d.shape).float() * q.delta).to(d.dtype).contiguous()
                fns.append(lambda g=g, X=X, W=W: torch.ops.aten.convolution_backward(
                    g, X, W, None, [2, 2], [p, p], [1, 1], False, [0, 0], 1, [True, True, False]))
            def dense():
                for f in fns:
                    f()
            for _ in range(3):
                dense()
            torch.cuda.synchronize()
            row["dense_ms"] = time_events(torch, dense, 10) / len(sets)
            del fns
        rows.append(row)
        del sets
        torch.cuda.empty_cache()
    return rows


def tensor_peak():
    """Measured dense bf16 rate (TFLOP/s, burst) and where it comes from."""
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["bf16_tflops"]), "measured (MEASURED_PEAKS.json bf16_tflops, burst)"
    except (OSError, KeyError, ValueError):
        return 1590.0, "fallback (an earlier measurement on this pool)"


def small_config(torch, dbp, ctx, config, hbm_peak, fma_peak):
    """One of configs 1-4 as a short side measurement: layer (or whole-network backward) time, dense-equivalent
    throughput, fraction of the HBM roofline for the algorithmic bytes, fraction of the fp32 FMA peak for the
    non-zero FMAs (meaningful for the linear layers, which run on the gather kernels; the fp32 3x3 convolutions run
    on the tensor cores with operands split into two bf16 pieces), the dense library time."""
    dev = torch.device("cuda", ctx.device)
    if config in (1, 3):
        L = wl.config1() if config == 1 else wl.config3()
        d, X, W = (torch.from_numpy(a).to(dev) for a in (L.delta, L.X, L.W))
        fn = dbp.dithered_linear_backward if L.kind == "linear" else dbp.dithered_conv_backward
        run = lambda: fn(ctx, d, X, W, L.seed, L.scale)
        flops, nbytes = L.dense_flops, algorithmic_bytes(L)
        q = dbp.nsd_quantize(ctx, d, L.seed, L.scale)
        density = q.nnz.item() / d.numel()
        dq = (dbp.nsd_decode_dense(ctx, q, d.shape).float() * q.delta).contiguous()
        dense_fns = [dense_layer_fn(torch, L, dq, X, W)]
        name = layer_specs(config, 0)[1]
    else:
        c = wl.mlp_chain(batch=256) if config == 2 else wl.vgg_chain(batch=128, device=str(dev))
        cu = lambda a: None if a is None else torch.from_numpy(np.ascontiguousarray(a)).to(dev)
        Xs, Ws = [cu(a) for a in c.X], [cu(a) for a in c.W]
        masks = [None if m is None else cu(m.astype(np.uint8)) for m in c.relu_mask]
        pools = [cu(a) for a in c.pool_argmax]
        dout = cu(c.delta_out)
        def run():
            # training order: a layer's dW may still run while the layer below is quantized; joined at the end
            dbp.network_backward(ctx, c.kinds, Xs, Ws, masks, pools, dout, c.scale, 0, with_sparse=False,
                                 flags=dbp.DBP_DW_ASYNC)
            ctx.join()
        res = dbp.network_backward(ctx, c.kinds, Xs, Ws, masks, pools, dout, c.scale, 0, keep_delta_z=True)
        torch.cuda.synchronize()
        flops, nbytes = chain_flops(c), chain_bytes(c)
        nz = sum(r["nnz"].item() for r in res)
        density = nz / sum(r["delta_z"].numel() for r in res)
        dense_fns = []
        for l, kind in enumerate(c.kinds):
            dz = res[l]["delta_z"]
            if kind == "linear":
                dense_fns.append(lambda dz=dz, X=Xs[l], W=Ws[l], l=l: (torch.matmul(dz.t(), X), torch.matmul(dz, W) if l else None))
            else:
                dense_fns.append(lambda dz=dz, X=Xs[l], W=Ws[l], l=l: torch.ops.aten.convolution_backward(
                    dz, X, W, None, [1, 1], [1, 1], [1, 1], False, [0, 0], 1, [l > 0, True, False]))
        name = CHAIN_NAMES[config]
    for _ in range(3):
        run()
    torch.cuda.synchronize()
    n0 = dbp.kernel_launches()
    run()
    launches = dbp.kernel_launches() - n0
    reps = {1: 200, 2: 200, 3: 50, 4: 5}[config]
    ms = time_events(torch, run, reps)
    dt = dense_times(torch, dense_fns, reps)
    graphs = None
    if config in (1, 2):
        # a few launches of a few microseconds each: eager calls are bound by the host on both sides
        torch.backends.cudnn.allow_tf32 = False
        torch.backends.cuda.matmul.allow_tf32 = False
        g_ours, g_dense = graph_times(torch, ctx, [run, lambda: [f() for f in dense_fns]], reps)
        graphs = {"ms": g_ours, "dense_ms_tf32_off": g_dense,
                  "what": "the same work captured into a CUDA graph and replayed (device time without the per-call host cost)"}
    return {"workload": name, "ms": ms, "graph_replay": graphs, "gflops_dense_equiv": flops / (ms * 1e-3) / 1e9,
            "hbm_frac": nbytes / (ms * 1e-3) / 1e9 / hbm_peak, "algorithmic_mb": nbytes / 1e6,
            "nsd_density": density, "fma_frac": density * flops / (ms * 1e-3) / 1e12 / fma_peak,
            "dense_ms": dt, "launches": launches,
            "note": "fp32 linear layers: step size + codes, then both products on warp-level MMAs: two chained launches per layer (small_linear_*_kernel)"
                    if config in (1, 2) else "fp32 3x3 convolutions: tensor-core kernels, weights and activations split into two bf16 pieces "
                                             "(codes are exact in bf16); fma_frac does not apply" + ("; the FC layer runs on the gather kernels" if config == 4 else "")}


def crossover_sweep(torch, dbp, ctx):
    """Sparse gather kernels against the tensor-core path as the gradient gets sparser (larger s): one 1x1,
    one 3x3 and one linear shape, bf16. Prints one JSON line per (shape, s)."""
    shapes = [("conv1x1 128->512 @28x28 B64", lambda s: wl.conv_layer(64, 128, 512, 28, 28, 1, data_seed=71, scale=s, dtype="bf16")),
              ("conv3x3 128->128 @28x28 B64", lambda s: wl.conv_layer(64, 128, 128, 28, 28, 3, data_seed=72, scale=s, dtype="bf16")),
              ("linear 2048->512 B256", lambda s: wl.linear_layer(256, 512, 2048, data_seed=73, scale=s, dtype="bf16"))]
    for name, make in shapes:
        for s in (2.0, 5.0, 10.0, 20.0, 40.0, 80.0):
            L = make(s)
            d, X, W = (torch.from_numpy(a).to(torch.bfloat16).cuda() for a in (L.delta, L.X, L.W))
            fn = dbp.dithered_linear_backward if L.kind == "linear" else dbp.dithered_conv_backward
            q = dbp.nsd_quantize(ctx, d, L.seed, L.scale)
            dens = q.nnz.item() / d.numel()
            row = {"shape": name, "s": s, "density": dens}
            for label, flag in (("sparse_ms", dbp.DBP_FORCE_SPARSE), ("dense_ms", dbp.DBP_FORCE_DENSE)):
                run = lambda: fn(ctx, d, X, W, L.seed, L.scale, flags=flag)
                for _ in range(3):
                    run()
                torch.cuda.synchronize()
                row[label] = time_events(torch, run, 10)
            print(json.dumps(row))


# DRAM bytes (read + written) of one config-5 bench step's launches of each kernel kind, from the ncu capture summarised
# in profiles/bench_step_config5_launch_list.md; None = the kernels of that kind changed after the capture
NCU_DRAM_BYTES_PER_STEP = {"statistics": 1156103424, "quantize": 1331695616, "dx_dense": 1309135360, "dw_dense": 2629219840}


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
    ap.add_argument("--no-others", action="store_true", help="skip the side measurements of configs 1-4")
    ap.add_argument("--crossover-sweep", action="store_true", help="time the sparse and the dense path against density and exit")
    ap.add_argument("--force-sparse", action="store_true", help="gather kernels on every layer (profiling aid)")
    ap.add_argument("--bf16", action="store_true", help="configs 1 and 3 with bf16 storage (profiling aid: the bf16 linear kernels)")
    ap.add_argument("--strided-only", action="store_true", help="time the stride-2 layers of the network and exit (profiling aid)")
    ap.add_argument("--sync-dw", action="store_true", help="every call joins its dW before it returns (no DBP_DW_ASYNC)")
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
    hbm_peak, peak_src = measured_peaks()
    fma_peak = ctx.measure_fma_peak()
    if args.crossover_sweep:
        if rank == 0:
            crossover_sweep(torch, dbp, ctx)
        return
    if args.strided_only:
        if rank == 0:
            print(json.dumps({"strided_layers": strided_table(torch, dbp, ctx, hbm_peak, args.no_dense, args.batch or 64)}))
        return

    if args.config in CHAIN_NAMES:
        # whole-network configurations: the side measurement is the measurement
        r = small_config(torch, dbp, ctx, args.config, hbm_peak, fma_peak)
        clocks = sampler.stop() if rank == 0 else None
        ms = max_over_ranks(r["ms"], dev, world)
        if rank == 0:
            print(json.dumps({
                "metric": METRIC, "value": job_throughput(r["gflops_dense_equiv"] * r["ms"] * 1e6, world, ms), "unit": UNIT,
                "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
                "config": {"workload": r["workload"], "nsd_density": r["nsd_density"], "l2": "working set smaller than L2 (warm)"},
                "clocks": clocks, "gpu_launches": r["launches"] * 20, "e2e": None,
                "roofline": ({"kernel": "sparse gather dX/dW (conv_dx2_kernel, conv_dw2_kernel)", "bound": "alu",
                              "achieved": r["fma_frac"] * fma_peak, "peak": fma_peak, "unit": "TFLOP/s", "frac": r["fma_frac"],
                              "traffic": None, "peak_source": "measured: dependent fp32 FMA chains on every lane"}
                             if args.config == 2 else
                             {"kernel": "tensor-core 3x3 dX/dW (tc3_tma_dx_kernel, tc3_tma_dw_kernel), fp32 operands as two bf16 pieces",
                              "bound": "tensor", "achieved": r["gflops_dense_equiv"] / 1e3, "peak": tensor_peak()[0], "unit": "TFLOP/s",
                              "frac": r["gflops_dense_equiv"] / 1e3 / tensor_peak()[0], "traffic": None,
                              "peak_source": tensor_peak()[1],
                              "note": "dense-equivalent flops of the whole backward pass (every kernel of it, not only the products) / its "
                                      "time; the split operands cost two MMAs per dense-equivalent one"}),
                "hbm_path": {"algorithmic_gb_per_step": r["algorithmic_mb"] / 1e3, "frac_of_measured_hbm": r["hbm_frac"], "peak": hbm_peak},
                "dense_baseline": r["dense_ms"]}))
        if world > 1:
            dist.destroy_process_group()
        return

    specs, name = layer_specs(args.config, args.batch)
    if args.bf16 and args.config in (1, 3):
        def as_bf16(make):
            def f():
                L = make()
                L.delta, L.X, L.W, L.dtype = wl.round_to_bf16(L.delta), wl.round_to_bf16(L.X), wl.round_to_bf16(L.W), "bf16"
                return L
            return f
        specs = [(as_bf16(make), mult) for make, mult in specs]
        name += " [bf16 storage]"
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

    # dW of a layer may still run while the next layer is quantized (the layer below needs dX only); every dW
    # is ordered into the stream before the step ends
    FLAGS = (0 if args.sync_dw else dbp.DBP_DW_ASYNC) | (dbp.DBP_FORCE_SPARSE if args.force_sparse else 0)
    if args.force_sparse:
        name += " [gather kernels forced]"

    def run_layer(L, d, X, W, dW, dX, want_dw=True, want_dx=True):
        code = 1 if L.dtype == "bf16" else 0
        pw, px = (dW.data_ptr() if want_dw else None), (dX.data_ptr() if want_dx else None)
        if L.kind == "linear":
            B, N = d.shape
            rc = lib.dithered_linear_backward(ctx._h, d.data_ptr(), X.data_ptr(), W.data_ptr(), code,
                                              B, N, X.shape[1], L.seed, L.scale, None, None, pw, px, None, FLAGS)
        else:
            B, Co, H, Wd = d.shape
            rc = lib.dithered_conv_backward(ctx._h, d.data_ptr(), X.data_ptr(), W.data_ptr(), code,
                                            B, X.shape[1], Co, H, Wd, L.k, 1, (L.k - 1) // 2, L.seed,
                                            L.scale, None, None, pw, px, None, FLAGS)
        if rc != 0:
            raise RuntimeError(f"library call failed on {L.name}: {rc} {lib.dbp_last_error().decode()}")

    def step(want_dw=True, want_dx=True):
        for item in layers:
            run_layer(*item, want_dw=want_dw, want_dx=want_dx)
        ctx.join()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # Warm-up steps run with every kernel kind bracketed by events: that gives the per-kind table
    # and names the dominant kind. The events cost stream time, so the timed region brackets
    # only the dominant kind (its duration is what the roofline line uses). The dW kinds run on the
    # context's second stream beside the others, so the kinds' times overlap and add up to more than the step.
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
    launches0 = dbp.kernel_launches()
    t_begin = time.perf_counter()
    e0.record()
    for _ in range(args.steps):
        step()
    e1.record()
    barrier()
    t_end = time.perf_counter()
    launches = dbp.kernel_launches() - launches0
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

    # every kind by itself: one product per call, so nothing runs beside anything else (the quantization kinds
    # are taken from the dX-only pass)
    alone = {}
    for want_dw, want_dx in ((False, True), (True, False)):
        step(want_dw, want_dx)
        barrier()
        ctx.profile_enable(True)
        ctx.profile_select(None)
        ctx.profile_read()
        for _ in range(3):
            step(want_dw, want_dx)
        barrier()
        for k, v in ctx.profile_read().items():
            if v[1] and k not in alone:
                alone[k] = v[0] / 3
        ctx.profile_enable(False)

    # non-zero work actually done, and the dequantized gradients the dense comparison is fed
    nnz_flops = 0.0
    dq = []
    for (L, d, X, W, dW, dX) in layers:
        q = dbp.nsd_quantize(ctx, d, L.seed, L.scale)
        nnz_flops += (q.nnz.item() / d.numel()) * L.dense_flops
        if not args.no_dense and rank == 0:
            dq.append((dbp.nsd_decode_dense(ctx, q, d.shape).float() * q.delta).to(d.dtype).contiguous())
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
    dq_by_layer = dq if (not args.no_dense and rank == 0) else None
    if not args.no_dense and rank == 0:
        fns = [dense_layer_fn(torch, L, g, X, W) for (L, d, X, W, dW, dX), g in zip(layers, dq)]
        dt = dense_times(torch, fns, max(20, args.steps // 4))
        dense = {k: {"ms_per_step": v, "gflops": dense_flops / (v * 1e-3) / 1e9} for k, v in dt.items()}
        dense["what"] = ("torch cuDNN/cuBLAS backward-data + backward-filter (cudnn.benchmark autotuning) on the "
                         "dequantized gradient Delta*q in the layers' dtype, same X and W buffers")
        del fns

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    prof = {k: (v[0] / nprof, v[1] / nprof) for k, v in prof_all.items()}   # per step
    kern = {k: {"ms_per_step": v[0], "launches_per_step": v[1],
                "measured": "warm-up steps, every kind bracketed by events (dW kinds run beside the others: times overlap)"}
            for k, v in prof.items() if v[1]}
    # algorithmic work of every kernel kind over one step; a layer counts as dense when the
    # library would run it so at this density (bf16, 1x1/linear or 3x3, channels % 8 == 0)
    e = 2 if layers[0][0].dtype == "bf16" else 4
    dense_on = prof["dx_dense"][1] > 0
    is_dense = lambda L: (dense_on and L.dtype == "bf16" and L.X.shape[1] % 8 == 0 and L.delta.shape[1] % 8 == 0)
    work = {k: 0.0 for k in ("statistics", "quantize", "dx", "dw", "dx_dense", "dw_dense", "fused")}
    for (L, d, X, W, dW, dX) in layers:
        nd, nx, nw = d.numel(), X.numel(), W.numel()
        if prof["fused"][1] > 0:                                       # two chained launches per layer: dense MMAs on the codes
            work["fused"] += L.dense_flops
            continue
        cb = 2 if is_dense(L) else 1                                   # bytes per code the product kernels read
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
    if top == "fused":
        ach = work[top] / t_s / 1e12
        roof = {"kernel": "small linear backward (small_linear_quantize_kernel + small_linear_products_kernel)", "bound": "tensor",
                "achieved": ach, "peak": tensor_peak()[0], "unit": "TFLOP/s", "frac": ach / tensor_peak()[0], "traffic": None,
                "peak_source": tensor_peak()[1],
                "note": "dense-equivalent flops of both products (2 * 2 * B * N * K) / time of the two launches; at these sizes they "
                        "are bound by launch and load latency, not by the tensor pipe (warp-level MMAs, two bf16 pieces per fp32 operand)"}
    elif top in ("dx", "dw"):
        ach = work[top] / t_s / 1e12
        roof = {"kernel": f"sparse {top} (conv_{top}2_kernel)", "bound": "alu", "achieved": ach,
                "peak": fma_peak, "unit": "TFLOP/s", "frac": ach / fma_peak, "traffic": None,
                "peak_source": "measured: dependent fp32 FMA chains on every lane (dbp_measure_fma_peak)",
                "note": "non-zero-code FMAs only (2*nnz*K_eff flops per product), summed over the layers that use it"}
    else:
        ach = work[top] / t_s / 1e9
        # per launch, like the algorithmic bytes: a launch of a kind is one layer's use of it (48 per step)
        per_step = NCU_DRAM_BYTES_PER_STEP.get(top) if (args.config == 5 and not (args.only or args.single or args.batch)) else None
        n_launch = max(prof[top][1], 1)
        traffic = None if per_step is None else per_step / n_launch
        roof = {"kernel": {"dx_dense": "tensor-core dX (tma_dx_kernel for 1x1, tc3_tma_dx_kernel for 3x3)",
                           "dw_dense": "tensor-core dW (tma_dw_kernel for 1x1, tc3_tma_dw_kernel + tc3_dw_finish_kernel for 3x3)",
                           "quantize": "NSD quantizer (quantize_dense_kernel / quantize_planes_odd_kernel for 1x1, quantize_nhwc_kernel for 3x3)"}.get(top, top + "_kernel"),
                "bound": "hbm", "achieved": ach, "peak": hbm_peak, "unit": "GB/s", "frac": ach / hbm_peak,
                "traffic": traffic, "algorithmic_bytes_per_launch": work[top] / n_launch, "launches_per_step": n_launch,
                "peak_source": peak_src + " (MEASURED_PEAKS.json hbm_gbs)",
                "note": "achieved = algorithmic bytes of the kind's launches / their summed duration inside the timed region "
                        "(CUDA events on the stream they run on; the dW kinds run beside the other kernels, which share the "
                        "SMs and the bandwidth with them: kernels[kind].frac_of_measured_hbm_alone is the same ratio with nothing "
                        "else running); traffic: DRAM read+write bytes per launch from the committed ncu launch list "
                        "(profiles/bench_step_config5_launch_list.md; write-back L2: a kernel's own write counters see little of its output)"}
    for k in work:
        if k in kern:
            kern[k]["work_per_step"] = work[k]
            kern[k]["unit"] = "flop" if k in ("dx", "dw", "fused") else "byte"
    for k in kern:
        if k in alone:
            kern[k]["ms_per_step_alone"] = alone[k]
            if k in work and kern[k].get("unit") == "byte":
                kern[k]["frac_of_measured_hbm_alone"] = work[k] / (alone[k] * 1e-3) / 1e9 / hbm_peak
    path_gbs = alg_bytes / (ms * 1e-3) / 1e9
    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16 storage, f32 accumulate" if layers[0][0].dtype == "bf16" else "f32",
        "data": "synthetic",
        "config": {"workload": name, "layers_per_step": len(layers), "l2": "inputs larger than L2 (distinct buffers per layer instance)"
                   if alg_bytes > 2.5e8 else "working set smaller than L2 (warm)", "nsd_density": density,
                   "dw": "joined per call" if args.sync_dw else "DBP_DW_ASYNC, joined at the end of the step"},
        "clocks": clocks, "gpu_launches": launches, "host_enqueue_ms_per_step": host_ms, "e2e": e2e,
        "roofline": roof,
        "hbm_path": {"algorithmic_gb_per_step": alg_bytes / 1e9, "achieved_gbs": path_gbs,
                     "frac_of_measured_hbm": path_gbs / hbm_peak, "peak": hbm_peak, "peak_source": peak_src},
        "fma_peak_tflops": fma_peak,
        "kernels": kern, "dense_baseline": dense,
    }
    if not args.no_others and world == 1 and args.config == 5 and not (args.only or args.single):
        out["other_configs"] = {str(c): small_config(torch, dbp, ctx, c, hbm_peak, fma_peak) for c in (1, 2, 3, 4)}
        out["per_shape"] = per_shape_table(torch, layers, run_layer, ctx, dq_by_layer, hbm_peak, args.no_dense)
        out["strided_layers"] = strided_table(torch, dbp, ctx, hbm_peak, args.no_dense, layers[0][0].delta.shape[0])
    if not args.no_cpu and world == 1:
        v, dt, what, cores = oracle_sample(args.config)
        out["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": what,
                               "seconds": dt}
    print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()

#!/usr/bin/env python
"""Benchmark of the pruned-CNN task path on B200.

A step is one pass of a whole pruned network over one batch of synthetic images: the input
cast, every conv task (fused bias / activation / residual / pool), the pools, the global average
pool and the FC tail -- everything `cprune_model_run` enqueues.  The one-time part of the path
(L1 selection, slicing, weight packing) is timed separately and reported as `prepare_ms`.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload resnet18|mobilenet_v2|vgg16_cifar]
    python bench.py --impl reference ...        # the CPU oracle on the host cores, same metric

Prints ONE JSON line (rank 0).  With N > 1 (torchrun) every rank runs an independent replica on
its own GPU with its own batch: weak scaling, no collective on the data path.
"""
from __future__ import annotations

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

import numpy as np  # noqa: E402

# DRAM bytes (read + write) of all launches of a kernel in one model pass, from the ncu captures summarised under profiles/
# (conv_patch_resnet18_b64_dram_traffic.md); absent where no capture of the current kernel exists.
DRAM_BYTES_PER_STEP = {("resnet18", "conv_patch_kernel"): 258.9e6}

WORKLOADS = {"resnet18": ("resnet18", 64), "mobilenet_v2": ("mobilenet_v2", 64), "vgg16_cifar": ("vgg16_cifar", 128)}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"],
                "bf16_tflops_sustained": p.get("bf16_tflops_sustained", p["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.lines, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._pump, daemon=True).start()
        except OSError:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [t.strip() for t in ln.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
            except ValueError:
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        bins = {}
        for v in sm:
            bins[str(int(round(v / 15.0) * 15))] = bins.get(str(int(round(v / 15.0) * 15)), 0) + 1
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm), "sm_mhz_bins": bins}


def max_over_ranks(values, device=None):
    """Every rank passes its own timings; all get the element-wise maximum (the slowest replica
    decides).  Without an initialised process group the values come back unchanged."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [float(v) for v in values]
    t = torch.tensor(values, dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def replica_seed(base_seed: int, rank: int) -> int:
    """Seed of the input batch of replica `rank`: replicas process different images."""
    return base_seed + 17 * rank


def cpu_reference(args, table_name, batch):
    """The oracle, as it stands, on the host cores: each step runs the pruned network on a bounded
    sample of the batch."""
    import oracle
    import workloads as wl
    table = wl.MODELS[table_name]()
    weights = wl.model_weights(table)
    pw, _ = oracle.prune_model(table, weights)
    sample = {"resnet18": 2, "mobilenet_v2": 4, "vgg16_cifar": 8}[table_name]
    sample = min(sample, batch)
    x = wl.model_input(table, sample)
    for _ in range(min(args.warmup, 1)):
        oracle.model_ref(table, pw, x, matched=True)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle.model_ref(table, pw, x, matched=True)
    dt = time.perf_counter() - t0
    return sample * args.steps / dt, dt * 1e3 / args.steps, sample, oracle.num_threads()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=30)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="resnet18", choices=sorted(WORKLOADS))
    ap.add_argument("--batch", type=int, default=0, help="images per step and GPU (0: the workload's own batch; 1 gives the latency point)")
    ap.add_argument("--no-graph", action="store_true", help="enqueue every launch from the host instead of replaying a CUDA graph")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-sustained", action="store_true", help="skip the 1.2 s sustained run (for profiler launch lists)")
    ap.add_argument("--no-task-times", action="store_true",
                    help="skip the per-task timing passes (and with them the roofline object); for profiler launch lists")
    ap.add_argument("--task", default=None,
                    help="time ONE conv task instead of a model: N,C,H,W,K,R,stride,pad[,groups[,act[,residual[,pool]]]]")
    ap.add_argument("--sweep", action="store_true",
                    help="time every distinct conv shape of the four models while the kept filter count K goes "
                         "from full width down to a quarter (the staircase of latency against K)")
    ap.add_argument("--sweep-stride", type=int, default=0, help="step in K (0: about 24 points per shape; 1: every K)")
    ap.add_argument("--sweep-batch", type=int, default=64)
    ap.add_argument("--sweep-out", default="sweep.jsonl", help="JSON lines, appended to; points already there are skipped")
    ap.add_argument("--sweep-axis", default="K", choices=["K", "C"], help="prune the task's filters (K) or its input channels (C)")
    ap.add_argument("--sweep-shapes", default="", help="comma-separated substrings of model/layer: only those shapes")
    args = ap.parse_args()
    if args.task:
        return task_bench(args)
    if args.sweep:
        return sweep_bench(args)
    table_name, batch = WORKLOADS[args.workload]
    if args.batch > 0:
        batch = args.batch
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    cfg = {"workload": "pruned_%s_batch%d" % (table_name, batch), "batch_per_gpu": batch, "layout": "NHWC bf16",
           "parallelism": "replicas x%d" % world if world > 1 else "single GPU",
           "l2": "activations of one step exceed the 126 MB L2 (inputs larger than L2)" if batch >= 32 else
                 "small batch: the step fits in L2 (latency point, no roofline claim)"}

    if args.impl == "reference":
        if rank != 0:
            return
        steps = max(1, min(args.steps, 5))
        args.steps = steps
        v, ms, sample, cores = cpu_reference(args, table_name, batch)
        line = {"impl": "reference", "metric": "pruned_model_images_per_s", "value": v, "unit": "images/s",
                "n_gpus": 0, "steps": steps, "warmup": min(args.warmup, 1), "ms_per_step": ms, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": cfg,
                "cpu_baseline": {"value": v, "unit": "images/s", "cores": cores, "kind": "oracle",
                                 "sample": "%d images of the %s batch per step" % (sample, cfg["workload"])},
                "e2e": {"value": v, "unit": "images/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
        print(json.dumps(line))
        return

    import torch
    import torch.distributed as dist

    import paper_2207_01260_b200 as cp
    import workloads as wl
    from paper_2207_01260_b200.pipeline import PrunedNetwork

    cp.lib()  # fails loudly if the CUDA library is missing: there is no other path
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize(dev)

    table = wl.MODELS[table_name]()
    weights = wl.model_weights(table)
    x_host = torch.from_numpy(wl.model_input(table, batch, seed=replica_seed(table["seed"], rank))).pin_memory()

    t0 = time.perf_counter()
    net = PrunedNetwork(table, weights, batch, device=dev)
    torch.cuda.synchronize(dev)
    prepare_first_ms = (time.perf_counter() - t0) * 1e3
    t0 = time.perf_counter()
    net2 = PrunedNetwork(table, weights, batch, device=dev)   # second pass: allocator and plan cache warm
    torch.cuda.synchronize(dev)
    prepare_ms = (time.perf_counter() - t0) * 1e3
    del net2
    cp.cprune_poll_device_status()

    x = x_host.to(dev)
    logits = torch.empty((batch, net.model.classes), dtype=torch.float32, device=dev)
    logits_host = torch.empty((batch, net.model.classes), dtype=torch.float32).pin_memory()
    use_graph = not args.no_graph
    stream = torch.cuda.current_stream()

    # ---------------- device-resident throughput
    for _ in range(max(args.warmup, 3)):
        net.run(x, logits, use_graph)
    barrier()
    sampler = ClockSampler(local_rank)
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(args.steps):
        net.run(x, logits, use_graph)
    e1.record(stream)
    barrier()
    ms = e0.elapsed_time(e1)
    clocks = sampler.stop()
    cp.cprune_poll_device_status()

    # ---------------- end to end: pinned host input -> device -> model -> logits back on the host, all inside
    # the C-ABI call cprune_model_run_host (copy of step i+1 overlaps the kernels of step i)
    for _ in range(3):
        net.run_host(x_host, logits_host)
    barrier()
    e2, e3 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e2.record(stream)
    for _ in range(args.steps):
        net.run_host(x_host, logits_host)
    e3.record(stream)
    barrier()
    ms_e2e = e2.elapsed_time(e3)
    if rank == 0 and not torch.equal(logits_host, logits.cpu()):
        raise RuntimeError("host-buffer path and device path disagree")

    # ---------------- sustained: at least 1.2 s of back-to-back replays, so that the clock record covers the timed
    # kernels (the 20 to 50 steps above last a few milliseconds, far less than the 100 ms sampling period)
    n_sus = args.steps if args.no_sustained else max(args.steps, int(1.2 / max(ms / args.steps * 1e-3, 1e-6)) + 1)
    barrier()
    sus_sampler = ClockSampler(local_rank)
    sus_sampler.start()
    time.sleep(0.12)
    e4, e5 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e4.record(stream)
    for _ in range(n_sus):
        net.run(x, logits, use_graph)
    e5.record(stream)
    barrier()
    ms_sus = e4.elapsed_time(e5)
    sus_clocks = sus_sampler.stop()
    cp.cprune_poll_device_status()

    ms, ms_e2e, ms_sus = max_over_ranks([ms, ms_e2e, ms_sus], dev if world > 1 else None)

    # ---------------- per-task timing of the tensor-core kernel (roofline of the dominant kernel)
    roof, per_task = None, []
    if rank == 0 and not args.no_task_times:
        peaks = measured_peaks()
        per_task = net_task_times(cp, net, table)
        # the tensor family has two kernels; the roofline object describes the one that takes more of the step
        tens_all = [t for t in per_task if t["kernel"] == "tensor"]
        by_variant = {v: [t for t in tens_all if min(t["variant"], 1) == v] for v in (0, 1)}   # variants 1 and 2: the patch kernel
        top = max((0, 1), key=lambda v: sum(t["ms"] for t in by_variant[v]))
        tens = by_variant[top]
        tens_name = "conv_patch_kernel" if top == 1 else "conv_tc_kernel"
        dw = [t for t in per_task if t["kernel"] == "depthwise"]
        t_tens, t_dw = sum(t["ms"] for t in tens), sum(t["ms"] for t in dw)
        if t_dw > t_tens and dw:
            gb = sum(t["bytes"] for t in dw) / 1e9
            ach = gb / (t_dw * 1e-3)
            roof = {"kernel": "depthwise3x3_kernel", "bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"],
                    "unit": "GB/s", "frac": ach / peaks["hbm_gbs"], "traffic": None, "peak_source": peaks["source"],
                    "launches_per_step": len(dw), "ms_per_step": t_dw}
        elif tens:
            tf = sum(t["flops"] for t in tens) / 1e12
            ach = tf / (t_tens * 1e-3)
            # each task is timed alone (eight launches, rotating buffers), 20 to 30 us at full clocks and far from the
            # power cap: the burst GEMM figure is the matching denominator; the fraction of the sustained one is alongside
            roof = {"kernel": tens_name, "bound": "tensor", "achieved": ach, "peak": peaks["bf16_tflops"],
                    "unit": "TFLOP/s", "frac": ach / peaks["bf16_tflops"],
                    "frac_of_sustained_peak": ach / peaks["bf16_tflops_sustained"],
                    "traffic": DRAM_BYTES_PER_STEP.get((args.workload, tens_name)),
                    "traffic_note": "DRAM bytes of all launches of this kernel in one step (ncu); algorithmic bytes alongside",
                    "algorithmic_bytes": sum(t["bytes"] for t in tens),
                    "peak_source": peaks["source"] + " (burst bf16 GEMM: the kernels are timed alone)", "launches_per_step": len(tens),
                    "ms_per_step": t_tens}

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    cpu, parity = None, None
    if world == 1 and not args.no_cpu_baseline:
        a = argparse.Namespace(steps=1, warmup=0)
        import oracle  # the CPU-baseline leg is the one place the benchmark may run the oracle
        sample = {"resnet18": 16, "mobilenet_v2": 32, "vgg16_cifar": 96}[table_name]
        pw, _ = oracle.prune_model(table, weights)
        xs = wl.model_input(table, sample)
        t0 = time.perf_counter()
        ref = oracle.model_ref(table, pw, xs, matched=True)
        dt = time.perf_counter() - t0
        cpu = {"value": sample / dt, "unit": "images/s", "cores": oracle.num_threads(), "kind": "oracle",
               "sample": "%d images of %s, one pass, %.1f s" % (sample, cfg["workload"], dt)}
        # parity of the very plans that were timed: the oracle's pass above ran the first images of the timed batch
        # (the generator is counter-based: the first `sample` images of any batch are the same)
        got = logits.cpu().numpy()[:sample].astype(np.float64)
        srt = np.sort(ref, axis=1)
        decided = (srt[:, -1] - srt[:, -2]) > 2.0 * 1e-2 * np.max(np.abs(ref), axis=1)
        agree = np.argmax(got, 1) == np.argmax(ref, 1)
        parity = {"images": int(sample), "rel_l2": float(np.linalg.norm(got - ref) / np.linalg.norm(ref)),
                  "top1_agree_raw": int(agree.sum()), "top1_decided": int(decided.sum()),
                  "top1_agree_decided": int((agree & decided).sum()),
                  "against": "oracle in matched mode (bf16 rounding where the device stores bf16), first images of the timed batch",
                  "ok": bool(np.linalg.norm(got - ref) <= 1e-2 * np.linalg.norm(ref) and np.all(agree[decided]))}

    images = batch * world * args.steps
    in_bytes = x_host.numel() * 4
    out_bytes = logits_host.numel() * 4
    line = {"metric": "pruned_model_images_per_s", "value": images / (ms * 1e-3), "unit": "images/s", "n_gpus": world,
            "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic", "config": cfg,
            "tflops": net.flops() * world * args.steps / (ms * 1e-3) / 1e12,
            "e2e": {"value": images / (ms_e2e * 1e-3), "unit": "images/s", "h2d_bytes_per_step": in_bytes,
                    "d2h_bytes_per_step": out_bytes, "ms_per_step": ms_e2e / args.steps},
            "gpu_launches": net.model.launches * args.steps, "launches_per_step": net.model.launches,
            "cuda_graph": use_graph, "clocks": clocks, "roofline": roof, "cpu_baseline": cpu, "parity": parity,
            "sustained": {"value": batch * world * n_sus / (ms_sus * 1e-3), "unit": "images/s", "steps": n_sus,
                          "seconds": ms_sus * 1e-3, "ms_per_step": ms_sus / n_sus, "clocks": sus_clocks},
            "prepare_ms": prepare_ms, "prepare_first_ms": prepare_first_ms,
            "tasks": per_task}
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def task_bench(args):
    """One conv task, timed with CUDA events over `steps` launches that rotate through enough
    distinct (x, y) buffer sets to exceed twice the L2 size (cold), and again on one set (warm)."""
    import torch

    import paper_2207_01260_b200 as cp
    import workloads as wl
    f = args.task.split(",")
    N, C, H, W, K, R, stride, pad = [int(v) for v in f[:8]]
    groups = int(f[8]) if len(f) > 8 else 1
    act = f[9] if len(f) > 9 else "relu"
    residual = len(f) > 10 and f[10] == "1"
    pool = f[11] if len(f) > 11 and f[11] not in ("", "none") else None
    torch.cuda.set_device(0)
    plan = cp.cprune_task_plan(N, C, H, W, K, R, R, stride, pad, groups, act, residual, pool)
    i = plan.info
    x, w, b, res = wl.conv_task_tensors(7, N, C, H, W, K, R, R, groups, residual, i["P"], i["Q"])
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
    wp, bp = cp.cprune_pack_weights(plan, dev(w), dev(b))
    xb = cp.cprune_cast_input(dev(x))
    rb = cp.cprune_cast_input(dev(res)) if residual else None
    set_bytes = xb.numel() * 2 + N * i["out_h"] * i["out_w"] * i["k_pad"] * 2
    nsets = int(max(1, min(64, -(-2 * 126e6 // set_bytes))))
    xs = [xb] + [xb.clone() for _ in range(nsets - 1)]
    ys = [torch.empty((N, i["out_h"], i["out_w"], i["k_pad"]), dtype=torch.bfloat16, device="cuda") for _ in range(nsets)]
    ws = torch.empty(max(i["workspace_bytes"], 16), dtype=torch.uint8, device="cuda")
    stream = torch.cuda.current_stream()

    def timed(rotate):
        """`steps` launches captured into one CUDA graph (no host launch gaps), replayed and timed."""
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            for j in range(nsets if rotate else 1):       # encodes tensor maps for every buffer set
                cp.cprune_task_run(plan, xs[j], wp, bp, rb, ys[j], ws)
            torch.cuda.synchronize()
            with torch.cuda.graph(graph, stream=side):
                for j in range(args.steps):
                    k = j % nsets if rotate else 0
                    cp.cprune_task_run(plan, xs[k], wp, bp, rb, ys[k], ws)
        for _ in range(max(args.warmup, 3)):
            graph.replay()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        graph.replay()
        e1.record(stream)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / args.steps

    ms_cold, ms_warm = timed(True), timed(False)
    cp.cprune_poll_device_status()
    peaks = measured_peaks()
    line = {"metric": "conv_task_tflops", "task": args.task, "kernel": cp.KERNEL_NAMES[i["kernel"]],
            "ms_cold": ms_cold, "ms_warm": ms_warm, "tflops_cold": i["flops"] / ms_cold / 1e9,
            "tflops_warm": i["flops"] / ms_warm / 1e9, "gbs_cold": i["algorithmic_bytes"] / ms_cold / 1e6,
            "frac_tensor_peak": i["flops"] / ms_cold / 1e9 / peaks["bf16_tflops"],
            "frac_hbm_peak": i["algorithmic_bytes"] / ms_cold / 1e6 / peaks["hbm_gbs"],
            "buffer_sets": nsets, "tile_n": i["tile_n"], "tiles": i["tiles_m"] * i["tiles_n"], "stages": i["stages"],
            "steps": args.steps, "padded_flops_ratio": i["padded_flops"] / i["flops"]}
    print(json.dumps(line))


def sweep_bench(args):
    """Latency and TFLOP/s (or GB/s) of every distinct conv shape against the pruned channel count: the kept filters K
    (--sweep-axis K; depthwise shapes lose the channel with the filter) or the input channels C of dense shapes
    (--sweep-axis C: what pruning the PREVIOUS layer does to this task).  Every point is timed cold (rotating buffer
    sets larger than twice the L2) and warm (one buffer set).  Points already in --sweep-out are skipped, so an
    interrupted sweep resumes where it stopped."""
    import torch

    import paper_2207_01260_b200 as cp
    import workloads as wl
    torch.cuda.set_device(0)
    peaks = measured_peaks()
    N = args.sweep_batch
    done = set()
    if os.path.exists(args.sweep_out):
        for line in open(args.sweep_out):
            try:
                r = json.loads(line)
                done.add((r["model"], r["layer"], r["N"], r["C"], r["K"], r.get("axis", "K")))
            except (ValueError, KeyError):
                continue
    out = open(args.sweep_out, "a")
    npoints, skipped, t0 = 0, 0, time.perf_counter()
    worst = {}
    for si, shp in enumerate(wl.sweep_shapes()):
        if args.sweep_shapes and not any(f in "%s/%s" % (shp["model"], shp["layer"]) for f in args.sweep_shapes.split(",")):
            continue
        dw = shp["groups"] > 1
        if args.sweep_axis == "C" and (dw or shp["C"] < 16):
            continue
        full = shp["C"] if args.sweep_axis == "C" else shp["K"]
        lo = (full + 3) // 4
        stride = args.sweep_stride or max(1, (full - lo) // 24)
        # the layer's own weights (Kaiming-normal from the shape's seed); pruning keeps the leading filters / channels here:
        # which ones survive does not change the time
        _, w, b, _ = wl.conv_task_tensors(9000 + si, 1, shp["C"], 1, 1, shp["K"], shp["R"], shp["S"], shp["groups"])
        w, b = torch.from_numpy(w).cuda(), torch.from_numpy(b).cuda()
        for v in range(full, lo - 1, -stride):
            K = shp["K"] if args.sweep_axis == "C" else v
            C = v if args.sweep_axis == "C" else (K if dw else shp["C"])
            if (shp["model"], shp["layer"], N, C, K, args.sweep_axis) in done:
                skipped += 1
                continue
            plan = cp.cprune_task_plan(N, C, shp["H"], shp["W"], K, shp["R"], shp["S"], shp["stride"], shp["pad"],
                                       K if dw else 1, shp["act"])
            i = plan.info
            wk = w[:K].contiguous() if dw else w[:K, :C].contiguous()
            wp, bp = cp.cprune_pack_weights(plan, wk, b[:K].contiguous())
            ms_cold, nsets = time_task_cold(cp, plan, wp, bp, False, launches=8, reps=2, warmup=1)
            ms_warm, _ = time_task_cold(cp, plan, wp, bp, False, launches=8, reps=2, warmup=1) if nsets == 1 else \
                time_task_warm(cp, plan, wp, bp)
            ai = i["flops"] / i["algorithmic_bytes"]
            bound = "tensor" if ai > peaks["bf16_tflops"] * 1e3 / peaks["hbm_gbs"] else "hbm"
            tf, gbs = i["flops"] / ms_cold / 1e9, i["algorithmic_bytes"] / ms_cold / 1e6
            frac = tf / peaks["bf16_tflops"] if bound == "tensor" else gbs / peaks["hbm_gbs"]
            rec = {"model": shp["model"], "layer": shp["layer"], "axis": args.sweep_axis, "N": N, "C": C, "K": K, "H": shp["H"],
                   "W": shp["W"], "R": shp["R"], "stride": shp["stride"], "depthwise": dw, "kernel": cp.KERNEL_NAMES[i["kernel"]],
                   "ms": ms_cold, "ms_warm": ms_warm, "tflops": tf, "gbs": gbs, "bound": bound, "frac": frac,
                   "tile": [i["tile_m"], i["tile_n"]], "tiles": i["tiles_m"] * i["tiles_n"], "k_alloc": i["k_alloc"],
                   "splits": i["splits"], "est_us": i["est_us"], "prune_step": cp.cprune_prune_step(plan), "buffer_sets": nsets}
            out.write(json.dumps(rec) + "\n")
            out.flush()
            npoints += 1
            key = (shp["model"], shp["layer"])
            worst[key] = min(worst.get(key, 1e9), frac)
        cp.cprune_poll_device_status()
        cp.cprune_cache_clear()
    out.close()
    print(json.dumps({"metric": "conv_task_sweep", "axis": args.sweep_axis, "points": npoints, "skipped_done": skipped, "batch": N,
                      "seconds": time.perf_counter() - t0, "out": args.sweep_out,
                      "min_frac_over_shapes": min(worst.values()) if worst else None,
                      "median_of_min_frac": float(np.median(list(worst.values()))) if worst else None}))


def time_task_warm(cp, plan, wp, bp, launches=8, reps=2):
    """As time_task_cold with ONE buffer set: the operands stay in L2 between launches."""
    import torch
    i = plan.info
    gen = torch.Generator(device="cuda").manual_seed(1234)
    x = torch.randn((i["N"], i["H"], i["W"], i["c_pad"]), device="cuda", generator=gen).to(torch.bfloat16)
    if i["c_pad"] > i["C"]:
        x[..., i["C"]:] = 0
    y = torch.empty((i["N"], i["out_h"], i["out_w"], i["k_pad"]), dtype=torch.bfloat16, device="cuda")
    ws = torch.empty(max(i["workspace_bytes"], 16), dtype=torch.uint8, device="cuda")
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        cp.cprune_task_run(plan, x, wp, bp, None, y, ws)
        torch.cuda.synchronize()
        with torch.cuda.graph(graph, stream=side):
            for _ in range(launches):
                cp.cprune_task_run(plan, x, wp, bp, None, y, ws)
    graph.replay()
    torch.cuda.synchronize()
    best = 1e9
    stream = torch.cuda.current_stream()
    for _ in range(reps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        graph.replay()
        e1.record(stream)
        torch.cuda.synchronize()
        best = min(best, e0.elapsed_time(e1) / launches)
    return best, 1


def time_task_cold(cp, plan, wp, bp, with_res, launches=8, reps=3, warmup=2):
    """Milliseconds of one launch of a task: `launches` back-to-back launches between one pair of CUDA events (a CUDA
    graph, so no host gaps; long enough to be off the event timer's ~2 us grid), rotating through enough distinct
    (x, residual, y) buffer sets to exceed twice the L2 size, so that every launch reads its operands from HBM."""
    import torch
    i = plan.info
    gen = torch.Generator(device="cuda").manual_seed(1234)
    x_elems = i["N"] * i["H"] * i["W"] * i["c_pad"]
    y_elems = i["N"] * i["out_h"] * i["out_w"] * i["k_pad"]
    r_elems = i["N"] * i["P"] * i["Q"] * i["k_pad"] if with_res else 0
    set_bytes = 2 * (x_elems + y_elems + r_elems)
    nsets = int(max(2, min(launches, -(-2 * 126e6 // set_bytes))))
    xs, ys, rs = [], [], []
    for _ in range(nsets):
        x = torch.randn((i["N"], i["H"], i["W"], i["c_pad"]), device="cuda", generator=gen).to(torch.bfloat16)
        if i["c_pad"] > i["C"]:
            x[..., i["C"]:] = 0
        xs.append(x)
        ys.append(torch.empty((i["N"], i["out_h"], i["out_w"], i["k_pad"]), dtype=torch.bfloat16, device="cuda"))
        rs.append(torch.randn((i["N"], i["P"], i["Q"], i["k_pad"]), device="cuda", generator=gen).to(torch.bfloat16) if with_res else None)
    ws = torch.empty(max(i["workspace_bytes"], 16), dtype=torch.uint8, device="cuda")
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        for j in range(nsets):                                 # encodes the tensor maps of every buffer set
            cp.cprune_task_run(plan, xs[j], wp, bp, rs[j], ys[j], ws)
        torch.cuda.synchronize()
        with torch.cuda.graph(graph, stream=side):
            for j in range(launches):
                k = j % nsets
                cp.cprune_task_run(plan, xs[k], wp, bp, rs[k], ys[k], ws)
    for _ in range(warmup):
        graph.replay()
    torch.cuda.synchronize()
    best = 1e9
    stream = torch.cuda.current_stream()
    for _ in range(reps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        graph.replay()
        e1.record(stream)
        torch.cuda.synchronize()
        best = min(best, e0.elapsed_time(e1) / launches)
    return best, nsets


def net_task_times(cp, net, table):
    """Times every distinct conv task of the network alone, cold (see time_task_cold), with its own packed weights."""
    out, seen = [], {}
    for l in table["layers"]:
        if l["kind"] != "conv" or l["name"] not in net.plans:
            continue
        plan = net.plans[l["name"]]
        key = plan.handle.value
        if key not in seen:
            wp, bp = net.packed[l["name"]]
            seen[key] = time_task_cold(cp, plan, wp, bp, l.get("res") is not None)
        ms, nsets = seen[key]
        i = plan.info
        out.append({"name": l["name"], "kernel": cp.KERNEL_NAMES[i["kernel"]], "C": i["C"], "K": i["K"],
                    "HW": [i["H"], i["W"]], "R": i["R"], "stride": i["stride"], "ms": ms, "flops": i["flops"],
                    "variant": i["variant"], "bytes": i["algorithmic_bytes"], "tflops": i["flops"] / ms / 1e9,
                    "gbs": i["algorithmic_bytes"] / ms / 1e6, "tile_n": i["tile_n"], "tiles": i["tiles_m"] * i["tiles_n"],
                    "buffer_sets": nsets, "timing": "8 launches per event pair, rotating buffers (cold)"})
    return out


if __name__ == "__main__":
    main()

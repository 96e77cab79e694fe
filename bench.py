#!/usr/bin/env python
"""Benchmark of the partitioned, micro-batch pipelined training step on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload r1001|r110|r11|r152|r1001k] [--impl reference]

One step = forward + backward + gradient average of the whole batch (all partitions, all
micro-batches).  Prints ONE JSON line.  N > 1 (under torchrun) runs N independent replicas, one per
GPU, with no data-path collective (weak scaling); the timing is the max over ranks.
`--impl reference` times the fp64 CPU oracle on the host cores instead (rank 0 only).
"""
import argparse
import json
import os
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import workloads as wl  # noqa: E402

METRIC = "images/sec fwd+bwd (1 B200) ResNet-1001 v2 32x32 b128; conv tensor-pipe % of peak"
UNIT = "images/s"
NAMES = {"r1001": "ResNet-1001 v2 (n=111, widths 16/32/64 x4), 32x32x3, batch 128, 8 partitions x 8 micro-batches",
         "r110": "ResNet-110 v2 (n=12), 32x32x3, batch 128, 4 partitions x 4 micro-batches",
         "r11": "ResNet-11 v2 (n=1), 32x32x3, batch 8, 2 partitions x 2 micro-batches",
         "r152": "ResNet-152 v2 ImageNet layout, 224x224x3, batch 64, 4 partitions x 4 micro-batches",
         "r1001k": "ResNet-1001 v2 with the Keras example's widths (16/64/128 -> 64/128/256, 30.25 M parameters), 32x32x3, batch 128, "
                   "8 partitions x 8 micro-batches",
         "r20k": "ResNet-20 v2 with the Keras example's widths, 32x32x3, batch 16, 2 partitions x 2 micro-batches",
         "r110v1": "ResNet-110 v1 (post-activation basic blocks, n=18), 32x32x3, batch 128, 4 partitions x 4 micro-batches",
         "r8v1": "ResNet-8 v1, 32x32x3, batch 8, 2 partitions x 2 micro-batches",
         "vgg16": "VGG-16 for 32x32 inputs (13 conv + 2 hidden FC + classifier, no biases), batch 128, 4 partitions x 4 micro-batches",
         "vgg16s": "VGG-16 layout at reduced width, 32x32x3, batch 8, 2 partitions x 2 micro-batches"}


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm_gbs=p["hbm_gbs"], bf16_tflops=p["bf16_tflops"], bf16_tflops_sustained=p.get("bf16_tflops_sustained"),
                    source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


def measure_tf32_peak(torch, seconds=2.0):
    """Dense TF32 tensor throughput of this GPU, measured in this run: torch.matmul (a library GEMM: a probe for the
    roofline's denominator, not a product path) on 8192^3 fp32 operands with TF32 allowed; best of 10 single calls
    (burst: for a kernel timed alone) and back to back for `seconds` (sustained, under the power cap)."""
    old = torch.backends.cuda.matmul.allow_tf32
    torch.backends.cuda.matmul.allow_tf32 = True
    try:
        n = 8192
        a = torch.randn(n, n, device="cuda"); b = torch.randn(n, n, device="cuda"); c = torch.empty(n, n, device="cuda")
        for _ in range(3):
            torch.matmul(a, b, out=c)
        torch.cuda.synchronize()
        flop = 2.0 * n ** 3
        best = 0.0
        for _ in range(10):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(); torch.matmul(a, b, out=c); e1.record(); torch.cuda.synchronize()
            best = max(best, flop / (e0.elapsed_time(e1) * 1e-3) / 1e12)
        reps = max(10, int(seconds * best * 1e12 / flop))
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            torch.matmul(a, b, out=c)
        e1.record(); torch.cuda.synchronize()
        sustained = reps * flop / (e0.elapsed_time(e1) * 1e-3) / 1e12
        del a, b, c
        return {"burst_tflops": best, "sustained_tflops": sustained, "how": "torch.matmul fp32 operands, TF32 allowed, 8192^3: best of 10 "
                "(burst) and %d back to back (sustained); measured in this run" % reps}
    finally:
        torch.backends.cuda.matmul.allow_tf32 = old


def dram_traffic_table():
    """DRAM bytes of the convolution kernel per launch as ncu counted them, from the tracked summary
    profiles/conv_tc_fwd_dram_traffic.txt: rows `ksize stride c_in c_out H batch read_bytes write_bytes`."""
    table = {}
    path = os.path.join(ROOT, "profiles", "conv_tc_fwd_dram_traffic.txt")
    if os.path.exists(path):
        for line in open(path):
            f = line.split("#")[0].split()
            if len(f) >= 8:
                table[tuple(int(v) for v in f[:5])] = (int(f[5]), float(f[6]) + float(f[7]))
    return table


# ----------------------------------------------------------------------------------------------------
# algorithmic byte / flop model of one step (unfused op model: every op reads its inputs and writes
# its outputs once; conv counted for forward, data gradient and weight gradient)
# ----------------------------------------------------------------------------------------------------
def step_model(ops, in_hwc, B):
    shapes = wl.tensor_shapes(ops, in_hwc)
    by = dict(conv=0.0, bn=0.0, add=0.0, other=0.0)
    flops = 0.0
    for i, o in enumerate(ops):
        H, W, C = shapes[i]
        iH, iW, iC = in_hwc if o.src0 < 0 else shapes[o.src0]
        out_el = B * H * W * C
        if o.kind == wl.CONV:
            in_el = B * H * W * iC if o.stride > 1 else B * iH * iW * iC     # only the sampled pixels of a strided 1x1
            wts = o.c_out * o.ksize * o.ksize * o.c_in
            passes = 3 if o.src0 >= 0 else 2
            by["conv"] += 4.0 * (in_el + out_el + wts) * passes
            flops += 2.0 * out_el * o.ksize * o.ksize * o.c_in * passes
        elif o.kind == wl.BNRELU:
            by["bn"] += 8.0 * out_el + 12.0 * out_el
        elif o.kind == wl.ADD:
            by["add"] += 12.0 * out_el
        else:
            by["other"] += 8.0 * out_el
    return by, flops


class ClockSampler:
    """nvidia-smi sampling of SM clock and throttle reasons while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.proc, self.path = index, None, "/tmp/hpf_clocks_%d_%d.csv" % (os.getpid(), index)

    def start(self):
        try:
            self.out = open(self.path, "w")
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "200"], stdout=self.out,
                                         stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unavailable"]}
        time.sleep(0.25)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.out.close()
        sm, mx, reasons, power = [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in open(self.path):
            f = [t.strip() for t in line.split(",")]
            if len(f) < 8:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1])); power.append(float(f[2]))
            except ValueError:
                continue
            for k, name in enumerate(names):
                if f[4 + k].lower().startswith("active"):
                    reasons.add(name)
        try:
            os.remove(self.path)
        except OSError:
            pass
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        return {"sm_mhz": float(np.median(sm)), "sm_max_mhz": float(max(mx)), "power_w_max": float(max(power)),
                "samples": len(sm), "reasons": sorted(reasons)}


# ----------------------------------------------------------------------------------------------------
def oracle_sample(cfg, images, threads=None):
    """Times the oracle (forward + reverse sweep) on `images` samples of the workload."""
    from oracle import reference as ora
    ops, hwc = cfg["ops"], cfg["in_hwc"]
    x, labels = wl.draw_inputs(images, hwc, ops[-1].c_out)
    theta = wl.draw_params(ops)
    t0 = time.perf_counter()
    ora.microbatch(ops, hwc, theta, x, labels, want=[])
    return time.perf_counter() - t0


def run_reference(args, cfg):
    """The reference arm: the oracle as it stands on the host cores, bounded sample per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cores = os.cpu_count()
    b = cfg["B"] // cfg["M"]
    t1 = oracle_sample(cfg, 1)                               # calibration, untimed
    per_step_s = 150.0 / max(1, args.steps + args.warmup)
    images = int(max(1, min(b, per_step_s / max(t1, 1e-3))))
    for _ in range(args.warmup):
        oracle_sample(cfg, images)
    ts = [oracle_sample(cfg, images) for _ in range(args.steps)]
    total = sum(ts)
    value = images * args.steps / total
    sample = "forward+backward of one micro-batch of %d image(s) of the workload per step (fp64, OpenMP)" % images
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": 1e3 * total / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": NAMES[args.workload], "sample": sample},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def max_over_ranks(dist, values, device):
    """Step times of a multi-rank run: the slowest rank counts (all_reduce MAX; no data-path collective)."""
    import torch
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def replica_inputs(cfg, rank):
    """Rank r's replica: its own batch (seeded by rank), the same parameters on every rank."""
    x, labels = wl.draw_inputs(cfg["B"], cfg["in_hwc"], cfg["ops"][-1].c_out, seed_x=wl.inputs.SEED_X + rank,
                               seed_labels=wl.inputs.SEED_LABELS + rank)
    return x, labels, wl.draw_params(cfg["ops"])


def aggregate_throughput(world, batch_per_rank, ms_per_step):
    """Whole-job images/s of `world` replicas that each finish a batch every ms_per_step (weak scaling)."""
    return world * batch_per_rank / (ms_per_step * 1e-3)


def kernel_roofline(torch, hpf, cfg, pk):
    """The dominant kernel of the step (the tensor-core convolution forward / data-gradient kernel: a third of the
    summed kernel time in the ncu launch list, profiles/) timed alone through the C ABI on the workload's heaviest
    convolution shape at the micro-batch size, cycling through operand sets that together exceed L2.  The calls are
    captured once into a CUDA graph and the replay is timed with CUDA events on the launching stream, so that the
    figure is the kernel's launch-to-launch duration and not the host's call overhead."""
    b = cfg["B"] // cfg["M"]
    shapes = wl.tensor_shapes(cfg["ops"], cfg["in_hwc"])
    weight = {}
    for i, o in enumerate(cfg["ops"]):
        if o.kind == wl.CONV and o.src0 >= 0 and o.c_in % 16 == 0 and o.c_out % 16 == 0:
            H, W, C = shapes[o.src0]
            P, Q, K = shapes[i]
            in_el = b * P * Q * C if o.stride > 1 else b * H * W * C
            key = (o.ksize, o.stride, o.pad, C, K, H)
            weight[key] = weight.get(key, 0) + 4.0 * (in_el + b * P * Q * K + K * o.ksize * o.ksize * C)
    (ks, st, pad, ci, co, H), _ = max(weight.items(), key=lambda kv: (kv[1], kv[0][3]))      # ties: the wider input
    P = (H + 2 * pad - ks) // st + 1
    in_el = b * P * P * ci if st > 1 else b * H * H * ci
    alg = 4.0 * (in_el + b * P * P * co + co * ks * ks * ci)
    nset = max(3, int(260e6 // (4 * (b * H * H * ci + b * P * P * co))) + 1)
    dev = "cuda"
    xs = [torch.randn(b, H, H, ci, device=dev) for _ in range(nset)]
    ys = [torch.empty(b, P, P, co, device=dev) for _ in range(nset)]
    w = torch.randn(co, ks, ks, ci, device=dev) * (2.0 / (ci * ks * ks)) ** 0.5
    wprep = torch.empty(4 * w.numel(), device=dev)
    scratch = torch.zeros(hpf.conv_scratch_bytes(b, H, H, ci, co, ks, st, pad), dtype=torch.uint8, device=dev)
    hpf.conv_prepare_weights(w, wprep, ci, co, ks)
    geo = (b, H, H, ci, co, ks, st, pad, 0)
    for k in range(nset):
        hpf.conv_fwd(xs[k], w, wprep, ys[k], *geo, scratch)
    torch.cuda.synchronize()
    reps = 3 * nset
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        for i in range(reps):
            hpf.conv_fwd(xs[i % nset], w, wprep, ys[i % nset], *geo, scratch)
    graph.replay()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    st_cur = torch.cuda.current_stream()
    e0.record(st_cur)
    for _ in range(3):
        graph.replay()
    e1.record(st_cur)
    torch.cuda.synchronize()
    sec = e0.elapsed_time(e1) * 1e-3 / (3 * reps)
    achieved = alg / sec / 1e9
    cap = dram_traffic_table().get((ks, st, ci, co, H))
    traffic = cap[1] * b / cap[0] if cap else None
    return {"bound": "hbm", "achieved": achieved, "peak": pk["hbm_gbs"], "unit": "GB/s", "frac": achieved / pk["hbm_gbs"],
            # dram__bytes_read + dram__bytes_write of this kernel in the ncu capture of the same shape (tracked table under
            # profiles/, captured at a batch whose operands exceed L2), scaled by the pixels per launch: traffic grows in
            # proportion to the pixels (the input is read once, nothing is re-read); null when no capture covers the shape
            "traffic": traffic,
            "peak_source": pk["source"],
            "kernel": "conv_tc_fwd_kernel (tcgen05 implicit GEMM, three-pass TF32), %dx%d stride %d, %d->%d channels, %dx%d "
                      "pixels, micro-batch %d; %d rotating operand sets, kernel nodes only, launched with programmatic dependent launch as in the step"
                      % (ks, ks, st, ci, co, H, H, b, nset),
            "algorithmic_bytes_per_launch": alg, "us_per_launch": sec * 1e6,
            "note": "at the micro-batch size the kernel is latency bound (one 128-pixel tile per CTA, %d CTAs); "
                    "the batch-128 sweep (--workload conv_sweep) gives the bandwidth-bound figures" % ((b * P * P + 127) // 128)}


def run_hybrid(args, cfg, torch, hpf, dist, rank, local, world, dev):
    """Hybrid parallelism across the GPUs of the job: rank = replica * P + partition.  One step = every rank's cells of its
    partition for all micro-batches, the hand-offs, the micro-batch average and the per-partition allreduce over replicas."""
    from paper_1911_05146_b200.hybrid import HybridLayout, Stage, TorchDistComm, SingleRankComm, run_step
    P = args.hybrid_partitions
    layout = HybridLayout(world, P)
    replica, part = layout.coords(rank)
    ops, hwc, B, M = cfg["ops"], cfg["in_hwc"], cfg["B"], cfg["M"]
    x, labels, theta = replica_inputs(cfg, replica)
    cuts = wl.default_cuts(len(ops), P)
    stage = Stage(ops, (B,) + tuple(hwc), cuts, M, torch.from_numpy(theta), part, dev)
    comm = TorchDistComm(layout, rank) if world > 1 else SingleRankComm()
    dx, dl = torch.from_numpy(x).to(dev), torch.from_numpy(labels).to(dev)

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        run_step(stage, layout, rank, comm, dx, dl)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record()
    for _ in range(args.steps):
        run_step(stage, layout, rank, comm, dx, dl)          # ends with a host wait for this rank's slice
    e1.record()
    barrier()
    ms = e0.elapsed_time(e1)
    if dist is not None:
        ms, = max_over_ranks(dist, [ms], dev)
    if rank == 0:
        ms_step = ms / args.steps
        print(json.dumps({"metric": METRIC, "value": layout.R * B / (ms_step * 1e-3), "unit": UNIT, "n_gpus": world, "steps": args.steps,
                          "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
                          "dtype": "tf32", "data": "synthetic",
                          "config": {"workload": NAMES[args.workload], "global_batch": layout.R * B, "micro_batches": M, "partitions": P,
                                     "parallelism": "hybrid: %d replica(s) x %d partitions, one partition per GPU; NCCL send / recv across "
                                                    "cuts, one allreduce group per partition" % (layout.R, P),
                                     "cut_points": list(cuts), "graph": False}}), flush=True)
    if dist is not None:
        dist.barrier(); dist.destroy_process_group()


def conv_sweep(args):
    """Configuration 2: the bottleneck convolution shapes at batch 128, forward / data gradient / weight
    gradient each, through the C ABI on rotating operand sets that together exceed L2.  One JSON line with
    a row per (shape, pass): microseconds, achieved TFLOP/s and GB/s (algorithmic), and the fraction of
    min(TF32 peak, arithmetic intensity x HBM bandwidth)."""
    import torch
    import paper_1911_05146_b200 as hpf
    torch.cuda.set_device(0)
    pk = peaks()
    N, rows_out = 128, []
    dev = "cuda"
    for (ks, st, ci, co, H) in wl.conv_sweep_shapes():
        if args.sweep_filter and args.sweep_filter not in "%dx%d s%d %d->%d @%d" % (ks, ks, st, ci, co, H):
            continue
        pad = 1 if ks == 3 else 0
        P = (H + 2 * pad - ks) // st + 1
        x_el, y_el, w_el = N * H * H * ci, N * P * P * co, co * ks * ks * ci
        in_el = N * P * P * ci if st > 1 else x_el
        nset = max(2, int(260e6 // (4 * (x_el + y_el))) + 1)
        xs = [torch.randn(N, H, H, ci, device=dev) for _ in range(nset)]
        ys = [torch.randn(N, P, P, co, device=dev) for _ in range(nset)]
        w = torch.randn(co, ks, ks, ci, device=dev) * (2.0 / (ci * ks * ks)) ** 0.5
        dw = torch.empty_like(w)
        wprep = torch.empty(4 * w_el, device=dev)
        scratch = torch.zeros(hpf.conv_scratch_bytes(N, H, H, ci, co, ks, st, pad), dtype=torch.uint8, device=dev)
        hpf.conv_prepare_weights(w, wprep, ci, co, ks)
        geo = (N, H, H, ci, co, ks, st, pad, args.conv_path)
        calls = {
            "fwd": lambda k: hpf.conv_fwd(xs[k], w, wprep, ys[k], *geo, scratch),
            "dgrad": lambda k: hpf.conv_dgrad(ys[k], w, wprep, xs[k], *geo, scratch),
            "wgrad": lambda k: hpf.conv_wgrad(xs[k], ys[k], dw, *geo, scratch),
        }
        if args.conv_path == 0:
            # what the training step runs: the weight gradient with ONE TF32 pass (its error does not compound with depth)
            geo1 = geo[:-1] + (2,)
            calls["wgrad, one pass"] = lambda k: hpf.conv_wgrad(xs[k], ys[k], dw, *geo1, scratch)
        flops = 2.0 * N * P * P * ci * co * ks * ks
        nbytes = 4.0 * (in_el + y_el + w_el)
        for name, fn in calls.items():
            for k in range(nset):
                fn(k)
            reps = 2 if args.profile else max(10, 3 * nset)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            if args.profile:
                e0.record()
                for i in range(reps):
                    fn(i % nset)
                e1.record()
                torch.cuda.synchronize()
                sec = e0.elapsed_time(e1) * 1e-3 / reps
            else:
                # the calls are captured once into a CUDA graph and the replay is timed: the figure is the kernels'
                # launch-to-launch duration, not the host's call overhead (about 5 us per launch through ctypes)
                graph = torch.cuda.CUDAGraph()
                with torch.cuda.graph(graph):
                    for i in range(reps):
                        fn(i % nset)
                graph.replay()
                torch.cuda.synchronize()
                cur = torch.cuda.current_stream()
                e0.record(cur)
                for _ in range(3):
                    graph.replay()
                e1.record(cur)
                torch.cuda.synchronize()
                sec = e0.elapsed_time(e1) * 1e-3 / (3 * reps)
                del graph
            rows_out.append({"shape": "%dx%d s%d %d->%d @%d" % (ks, ks, st, ci, co, H), "pass": name, "us": sec * 1e6,
                             "tflops": flops / sec / 1e12, "gbs": nbytes / sec / 1e9, "ai": flops / nbytes})
        del xs, ys
    # the TF32 denominator is measured last: seconds of back-to-back GEMMs heat the part and would colour the rows above
    tf32 = measure_tf32_peak(torch)
    tf32_peak = tf32["burst_tflops"]               # the kernels of the sweep are timed alone: the burst figure
    for r in rows_out:
        ceiling = min(tf32_peak, r["ai"] * pk["hbm_gbs"] / 1e3)     # TFLOP/s
        r["ceiling_tflops"] = ceiling
        r["frac_of_ceiling"] = r["tflops"] / ceiling
    best = max(r["tflops"] for r in rows_out)
    print(json.dumps({"metric": "conv sweep (configuration 2), batch 128", "unit": "TFLOP/s", "value": best, "n_gpus": 1,
                      "dtype": "tf32", "data": "synthetic", "config": {"workload": "28 bottleneck conv shapes x {fwd, dgrad, wgrad}",
                      "conv_path": args.conv_path, "tf32_peak_tflops": tf32_peak, "tf32_peak": tf32,
                      "tf32_from_bf16_over_2_tflops": pk["bf16_tflops"] / 2.0, "hbm_gbs": pk["hbm_gbs"], "peak_source": pk["source"]},
                      "rows": rows_out}), flush=True)


def membound_sweep(args):
    """The memory-bound kernels alone, through the C ABI: fused BN+ReLU forward / backward at batch 128 and at the
    headline micro-batch size (16) on the bottleneck tensor shapes, and the gradient average at the parameter
    counts of configurations 4 and 5.  Rotating operand sets larger than L2; CUDA events on the launching stream."""
    import torch
    import paper_1911_05146_b200 as hpf
    torch.cuda.set_device(0)
    pk = peaks()
    dev, out = "cuda", []

    def timed(fn, nset, reps):
        """Seconds per call: the calls are captured once into a CUDA graph and the replay is timed with CUDA events on
        the launching stream, so that the figure is the kernels' launch-to-launch duration, not the host's call overhead."""
        for k in range(nset):
            fn(k)
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            for i in range(reps):
                fn(i % nset)
        graph.replay()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        cur = torch.cuda.current_stream()
        e0.record(cur)
        for _ in range(3):
            graph.replay()
        e1.record(cur)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) * 1e-3 / (3 * reps)

    # Latency floor of each kernel: the same entry point on a tensor of a few rows of the same width, where nothing but the
    # launch, the statistics exchange (block reduction, cluster or ticket hand-off) and the dependent second phase is left.
    floors = {}
    for C in (16, 64, 128, 256):
        rows0 = 512
        x0 = torch.randn(rows0, C, device=dev); y0 = torch.empty_like(x0); d0 = torch.randn_like(x0)
        g0 = torch.ones(C, device=dev); b0 = torch.zeros(C, device=dev); st0 = torch.empty(2 * C, device=dev)
        dg0 = torch.empty(C, device=dev); db0 = torch.empty(C, device=dev)
        sc0 = torch.zeros(hpf.bnrelu_scratch_bytes(rows0, C), dtype=torch.uint8, device=dev)
        floors[("bnrelu_fwd", C)] = timed(lambda k: hpf.bnrelu_fwd(x0, g0, b0, 1e-5, y0, st0, rows0, C, sc0), 1, 50)
        floors[("bnrelu_bwd", C)] = timed(lambda k: hpf.bnrelu_bwd(x0, d0, g0, b0, st0, y0, None, 0, dg0, db0, rows0, C, sc0), 1, 50)
    l2_mb = 126.0
    shapes = [(N, H, C) for N in (128, 16) for (H, C) in ((32, 64), (16, 128), (8, 256), (32, 16))] + [(64, 56, 256)]
    for (N, H, C) in shapes:
        rows = N * H * H
        nset = max(3, int(300e6 // (rows * C * 4 * 3)) + 1)
        xs = [torch.randn(rows, C, device=dev) for _ in range(nset)]
        dys = [torch.randn(rows, C, device=dev) for _ in range(nset)]
        outs = [torch.empty(rows, C, device=dev) for _ in range(nset)]
        g = torch.ones(C, device=dev); b = torch.zeros(C, device=dev)
        stats = torch.empty(2 * C, device=dev); dg = torch.empty(C, device=dev); db = torch.empty(C, device=dev)
        scratch = torch.zeros(hpf.bnrelu_scratch_bytes(rows, C), dtype=torch.uint8, device=dev)
        reps = max(20, 3 * nset)
        tf = timed(lambda k: hpf.bnrelu_fwd(xs[k], g, b, 1e-5, outs[k], stats, rows, C, scratch), nset, reps)
        tb = timed(lambda k: hpf.bnrelu_bwd(xs[k], dys[k], g, b, stats, outs[k], None, 0, dg, db, rows, C, scratch), nset, reps)
        # context, not ours: a library one-pass element-wise kernel (read once, write once) on the same tensor - what
        # 8 B/element costs at this size when nothing has to be known about the whole tensor before the first store
        tc = timed(lambda k: torch.relu_(xs[k]), nset, reps)
        for name, t, bpe in (("bnrelu_fwd", tf, 8.0), ("bnrelu_bwd", tb, 12.0), ("one-pass elementwise (torch.relu_, context)", tc, 8.0)):
            gbs = bpe * rows * C / t / 1e9
            row = {"kernel": name, "shape": "N=%d %dx%d C=%d" % (N, H, H, C), "mb": rows * C * 4 / 1e6, "us": t * 1e6,
                   "gbs": gbs, "frac_hbm": gbs / pk["hbm_gbs"]}
            if name.startswith("bnrelu"):
                # beyond L2 the statistics pass and the apply pass both read the input from HBM: 12 B (forward) / 16 B
                # (backward) per element is what such a tensor has to move, the 8 / 12 B model is unreachable there
                mb = rows * C * 4 / 1e6
                bpe2 = bpe + 4.0 if mb > l2_mb else bpe
                t_hbm = bpe2 * rows * C / (pk["hbm_gbs"] * 1e9)
                t_lat = floors[(name, C)]
                row.update({"bytes_per_element_model": bpe2, "frac_hbm_model": bpe2 * rows * C / t / 1e9 / pk["hbm_gbs"],
                            "latency_floor_us": t_lat * 1e6, "hbm_floor_us": t_hbm * 1e6,
                            "bound": "latency" if t_lat > t_hbm else "hbm", "frac_of_floor": max(t_lat, t_hbm) / t})
            out.append(row)
        del xs, dys, outs
    for (M, G) in ((8, 10327706), (4, 60185128)):
        nset = 2
        slots = [torch.randn(M, G, device=dev) for _ in range(nset)]
        avg = torch.empty(G, device=dev)
        t = timed(lambda k: hpf.grad_average_flat(slots[k], avg, M, G), nset, 20)
        gbs = 4.0 * (M + 1) * G / t / 1e9
        out.append({"kernel": "grad_average", "shape": "M=%d G=%d" % (M, G), "mb": 4.0 * M * G / 1e6, "us": t * 1e6, "gbs": gbs,
                    "frac_hbm": gbs / pk["hbm_gbs"]})
        del slots
    print(json.dumps({"metric": "memory-bound kernels alone (algorithmic GB/s)", "unit": "GB/s", "value": max(r["gbs"] for r in out),
                      "n_gpus": 1, "dtype": "f32", "data": "synthetic", "config": {"workload": "BN+ReLU fwd/bwd, gradient average",
                      "hbm_gbs": pk["hbm_gbs"], "peak_source": pk["source"]}, "rows": out}), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="hpf", choices=["hpf", "reference"])
    ap.add_argument("--workload", default="r1001", choices=sorted(wl.CONFIGS) + ["conv_sweep", "membound_sweep"])
    ap.add_argument("--no-graph", action="store_true")
    ap.add_argument("--cuts", default="equal", choices=["balanced", "equal", "measured"],
                    help="partition cut points: balanced = the library's load balancer on its modelled op costs; "
                         "measured = the load balancer on per-op costs apportioned from the measured, loaded cell times "
                         "(tuner.balance_by_measurement; its history, equal cuts first, goes into the line); "
                         "equal = the same number of ops in every partition")
    ap.add_argument("--conv-path", type=int, default=0)
    ap.add_argument("--lanes", type=int, default=1,
                    help="stage lanes (HPF_OPT_STAGE_LANES): micro-batches a stage keeps under way at once; 1 = the paper's schedule")
    ap.add_argument("--cell-ctas", type=int, default=-1,
                    help="CTAs of the persistent forward cell kernels (HPF_OPT_CELL_CTAS); 0: one launch per convolution; -1: the library's default")
    ap.add_argument("--hybrid-partitions", type=int, default=0,
                    help="N GPUs as N / P replicas of a P-stage pipeline, one partition per GPU (paper_1911_05146_b200.hybrid): "
                         "activations and partial errors by NCCL send / recv, one allreduce group per partition.  Not the default "
                         "(the default for N > 1 is independent replicas) and not yet measured on hardware.")
    ap.add_argument("--two-phases", action="store_true",
                    help="hpf_forward then hpf_backward (backward after the forward drain) instead of hpf_forward_backward")
    ap.add_argument("--opt", action="append", default=[], help="library option as NUMBER=VALUE (hpf_set_option), repeatable")
    ap.add_argument("--skip-cpu-baseline", action="store_true")
    ap.add_argument("--skip-kernel-roofline", action="store_true")
    ap.add_argument("--skip-e2e", action="store_true")
    ap.add_argument("--sweep-filter", default="", help="conv_sweep: only shapes whose label contains this text")
    ap.add_argument("--profile", action="store_true",
                    help="for runs under a profiler: honour --warmup below 3 and skip the side measurements")
    args = ap.parse_args()
    if args.profile:
        args.skip_e2e = args.skip_cpu_baseline = args.skip_kernel_roofline = True
    elif args.impl == "hpf":
        args.warmup = max(args.warmup, 3)
    if args.workload == "conv_sweep":
        conv_sweep(args)
        return
    if args.workload == "membound_sweep":
        membound_sweep(args)
        return
    cfg = wl.config(args.workload)
    if args.impl == "reference":
        run_reference(args, cfg)
        return

    import torch
    import paper_1911_05146_b200 as hpf

    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    dev = torch.device("cuda", local)
    pk = peaks()

    if args.hybrid_partitions > 0:
        run_hybrid(args, cfg, torch, hpf, dist, rank, local, world, dev)
        return
    ops, hwc, B, M = cfg["ops"], cfg["in_hwc"], cfg["B"], cfg["M"]
    x, labels, theta = replica_inputs(cfg, rank)          # each replica its own batch, shared parameters
    cuts = cfg["cuts"]
    balance_history = None
    if args.cuts == "balanced":
        cuts = hpf.balance_cuts(hpf.estimate_op_costs(ops, (B // M,) + tuple(hwc)), cfg["P"])
    elif args.cuts == "measured":
        # the load balancer by measurement (outside the timed region): loaded per-cell times -> per-op costs -> cuts
        from paper_1911_05146_b200.tuner import balance_by_measurement
        opts = {hpf.OPT_CONV_PATH: args.conv_path}
        if args.cell_ctas >= 0:
            opts[hpf.OPT_CELL_CTAS] = args.cell_ctas
        cuts, balance_history = balance_by_measurement(ops, (B,) + tuple(hwc), cfg["P"], M, torch.from_numpy(theta), cfg["cuts"], options=opts)
    model = hpf.Model(ops, (B,) + tuple(hwc), cuts, M)
    model.set_option(hpf.OPT_GRAPH, 0 if args.no_graph else 1)
    model.set_option(hpf.OPT_CONV_PATH, args.conv_path)
    if args.cell_ctas >= 0:
        model.set_option(hpf.OPT_CELL_CTAS, args.cell_ctas)
    if args.lanes != 1:
        model.set_option(hpf.OPT_STAGE_LANES, args.lanes)
    for kv in args.opt:
        k, v = kv.split("=")
        model.set_option(int(k), int(v))
    G = model.num_params()
    params = torch.from_numpy(theta).to(dev)
    slots = torch.empty((M, G), device=dev)
    avg = torch.empty(G, device=dev)
    ws_bytes = model.workspace_bytes()
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device=dev)
    # stage streams + weight-gradient side streams + backward streams (the one-graph schedule)
    streams = [torch.cuda.Stream(device=dev) for _ in range((2 if args.two_phases else 3) * model.num_stream_slots())]
    torch.cuda.synchronize()
    model.bind(params, slots, avg, ws, streams)
    dx, dl = torch.from_numpy(x).to(dev), torch.from_numpy(labels).to(dev)
    hx, hl = torch.from_numpy(x).pin_memory(), torch.from_numpy(labels).pin_memory()
    s0 = streams[0]

    def step():
        if args.two_phases:
            model.forward(dx, dl)
            model.backward()
        else:
            model.forward_backward(dx, dl)
        model.grad_average()

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        step()
    model.synchronize(0)
    l0 = model.launch_count()
    sampler = ClockSampler(local)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    sampler.start()
    e0.record(s0)
    for _ in range(args.steps):
        step()
    e1.record(s0)
    barrier()
    clocks = sampler.stop()
    ms = e0.elapsed_time(e1)
    launches = model.launch_count() - l0
    loss = model.loss()
    model.synchronize(0)

    # where the step's time goes: the three phases timed apart (a diagnostic; events on stream 0, which every phase joins)
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
    phase_ms = [0.0, 0.0, 0.0]
    if not args.profile:
        model.forward(dx, dl); model.backward(); model.grad_average()          # untimed: the two-phase graphs may not exist yet
        barrier()
    for _ in range(0 if args.profile else 3):
        ev[0].record(s0); model.forward(dx, dl); ev[1].record(s0); model.backward(); ev[2].record(s0); model.grad_average(); ev[3].record(s0)
        barrier()
        for k in range(3):
            phase_ms[k] += ev[k].elapsed_time(ev[k + 1]) / 3

    # end to end: host buffers in, loss out, every step
    ms_e2e = float("nan")
    if not args.skip_e2e:
        for _ in range(2):
            model.step_host(hx, hl)
        barrier()
        e0.record(s0)
        for _ in range(args.steps):
            model.step_host(hx, hl)
        e1.record(s0)
        barrier()
        ms_e2e = e0.elapsed_time(e1)

    if dist is not None:
        ms, ms_e2e = max_over_ranks(dist, [ms, ms_e2e], dev)
    if rank != 0:
        if dist is not None:
            dist.barrier(); dist.destroy_process_group()
        return

    ms_step = ms / args.steps
    value = aggregate_throughput(world, B, ms_step)
    by, flops = step_model(ops, hwc, B)
    step_bytes = sum(by.values())
    n_tc, n_cc = model.conv_path_counts()
    fused_bytes = model.step_bytes()
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "tf32" if n_tc else "f32", "data": "synthetic",
        "config": {"workload": NAMES[args.workload], "global_batch": world * B, "micro_batches": M,
                   "partitions": model.num_partitions(), "parallelism": "replicas x%d, no data-path collective" % world,
                   "l2": "working set %.1f GB per step exceeds the 126 MB L2; no explicit flush" % (ws_bytes / 1e9),
                   "cuts": args.cuts, "cut_points": list(cuts), "balance_history": balance_history, "graph": not args.no_graph, "cell_ctas": args.cell_ctas, "stage_lanes": args.lanes, "options": args.opt,
                   "schedule": "forward then backward, two graphs (fill / drain twice)" if args.two_phases else
                               "hpf_forward_backward: one graph, a backward cell starts when the cell that feeds it is done",
                   "phase_ms": {"forward": phase_ms[0], "backward": phase_ms[1], "average": phase_ms[2]}, "conv_sites_tensor_core": n_tc, "conv_sites_cuda_core": n_cc,
                   "loss": loss},
        "e2e": {"value": world * B / (ms_e2e / args.steps * 1e-3), "unit": UNIT,
                "h2d_bytes_per_step": int(hx.numel() * 4 + hl.numel() * 4), "d2h_bytes_per_step": 4},
        "gpu_launches": int(launches),
        "clocks": clocks,
        "step_roofline": {"bound": "hbm", "algorithmic_bytes_per_step": step_bytes, "bytes_by_class": by,
                          "conv_flops_per_step": flops, "achieved": step_bytes / (ms_step * 1e-3) / 1e9,
                          "peak": pk["hbm_gbs"], "unit": "GB/s", "frac": step_bytes / (ms_step * 1e-3) / 1e9 / pk["hbm_gbs"],
                          "peak_source": pk["source"],
                          # what the step has to move with the fusions it runs with (BN+ReLU applied by the reading convolution,
                          # residual adds in the write-out): fewer bytes for the same time, so a lower fraction of the roof
                          "fused_algorithmic_bytes_per_step": fused_bytes,
                          "fused_achieved": fused_bytes / (ms_step * 1e-3) / 1e9,
                          "fused_frac": fused_bytes / (ms_step * 1e-3) / 1e9 / pk["hbm_gbs"],
                          "hbm_floor_ms": {"unfused_model": step_bytes / (pk["hbm_gbs"] * 1e9) * 1e3, "fused_model": fused_bytes / (pk["hbm_gbs"] * 1e9) * 1e3},
                          "conv_tflops": flops / (ms_step * 1e-3) / 1e12},
    }
    if not args.skip_kernel_roofline:
        line["roofline"] = kernel_roofline(torch, hpf, cfg, pk)
    if not args.skip_cpu_baseline:
        b = B // M
        t1 = oracle_sample(cfg, 1)
        images = int(max(1, min(b, 20.0 / max(t1, 1e-3))))
        t = oracle_sample(cfg, images)
        line["cpu_baseline"] = {"value": images / t, "unit": UNIT, "cores": os.cpu_count(), "kind": "oracle",
                                "sample": "forward+backward of one micro-batch of %d image(s) of the workload, %.1f s "
                                          "(fp64, OpenMP on all host cores)" % (images, t)}
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.barrier(); dist.destroy_process_group()


if __name__ == "__main__":
    main()

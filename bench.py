#!/usr/bin/env python
"""Benchmark of the int8 quantized-convolution hot path on the ResNet-50 bottleneck workload.

    python bench.py --gpus N --steps K --warmup W [--impl reference]

One step = one int8 forward of the bottleneck block (1x1 256->64, 3x3 64->64, 1x1 64->256 with fused
bias, requantisation, ReLU and residual sum) over a batch of 32 56x56x256 u8 images: two launches
through the C ABI (the 1x1, then the 3x3 and the expanding 1x1 as one tcgen05 kernel whose 8-bit tensor
between the two layers stays in shared memory).  Prints ONE JSON line (rank 0).

* value      : int8 conv TOPS (2 * MACs / time), inputs resident in HBM, the K steps captured as one CUDA
               graph over rotating buffer sets whose total size exceeds L2; the graph is replayed until the
               timed region lasts at least 0.25 s and the median time of a replay counts (timed_repeats).  The
               steps are independent batches and alternate between --step-streams streams (default 2).
* e2e        : same metric with the u8 input of every step copied from pinned host memory and its u8 output
               copied back inside the timed region (three streams: the copies overlap the kernels).
* roofline   : dominant kernel, algorithmic bytes / CUDA-event duration against the measured copy peak.
* cpu_baseline: the CPU oracle timed on a bounded sample of the same workload on the host cores.
* int8_mma_peak: issue rate of tcgen05.mma.kind::i8 128x256x32 measured on all SMs (q8_int8_mma_rate), the
               int8 tensor peak every roofline below uses, at the SM clock sampled during the run.
* config1    : latency of the single 14x14x64 3x3 layer (configs[0]) in microseconds.
* resnet50_layers: every launch of ResNet-50 at batch 64 alone, cold L2: us, TOPS, bytes, bound, fraction of
               its roofline max(2 MACs / int8 peak, bytes / copy bandwidth).
* bandwidth_kernels: the memory-bound kernels (max-abs, quantize, dequantize, concat, pooling) against the measured
               copy bandwidth; networks: int8 forward of ResNet-50, Inception-v3 and SSD-300 (images/s), with the
               paper's Xeon figures beside them as context.  ssd_tail: L2 normalisation, detection output, and the
               projection blocks of ResNet-50 through the int8 route and through the paper's FP32 route for signed
               tensors.  All only at N = 1; --skip-networks leaves them out.
* --impl reference: the oracle alone (there is no reference implementation to install for this paper).
With N > 1 every rank runs its own batch (weak scaling, replicated weights, no data-path collective).
"""
import argparse
import hashlib
import json
import os
import statistics
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

BATCH, H, W, C, MID = 32, 56, 56, 256, 64
MACS_PER_IMAGE = H * W * (C * MID + 9 * MID * MID + MID * C)
METRIC = "int8_conv_tops_resnet50_bottleneck_b32"
UNIT = "TOPS"
CONFIG = {"workload": "configs[1]: ResNet-50 bottleneck, batch 32, 56x56x256 u8 in, 1x1 256->64 / 3x3 64->64 / "
                      "1x1 64->256 + identity residual, BN folded, ReLU fused, max-abs factors from 4 seeded batches",
          "global_batch_per_gpu": BATCH, "parallelism": "replicas"}

# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) of one launch of a kernel, from one ncu capture of
# this workload, with the hash of the kernel sources the capture was taken with: the figure is reported only while
# the sources still have that hash (a changed kernel has unknown traffic: null).  Traffic can lie below the
# algorithmic bytes: the output of a launch stays in the 126 MB L2 until later launches evict it.
NCU_TRAFFIC = {"source_sha256": "a71461ea12db545a249197980523119b30f28e9f626a4343958cbe874a1062a3",
               "bytes": {"conv_fused 3x3 64->64 + 1x1 64->256 +res": 32.34e6, "conv_umma 1x1 256->64": 26.11e6}}
KERNEL_SOURCES = ["q8_umma_common.cuh", "q8_conv_umma.cu", "q8_conv_fused.cu"]


def kernel_source_hash():
    h = hashlib.sha256()
    for f in KERNEL_SOURCES:
        with open(os.path.join(ROOT, "paper_1805_08691_b200", "csrc", f), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()


def ncu_traffic(kernel):
    if NCU_TRAFFIC["source_sha256"] and NCU_TRAFFIC["source_sha256"] == kernel_source_hash():
        return NCU_TRAFFIC["bytes"].get(kernel)
    return None


def layer_bytes(M, Cin, K, R, S, out_bytes=1, residual=False):
    """Algorithmic bytes of one conv launch: input once, weights, bias, output, residual."""
    return M * Cin + K * R * S * Cin + 4 * K + M * K * out_bytes + (M * K if residual else 0)


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return dict(hbm_gbs=d["hbm_gbs"], bf16_tflops=d["bf16_tflops"], sm_max_mhz=d.get("sm_max_mhz", 1965.0), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, sm_max_mhz=1965.0, source="fallback")


class ClockMonitor:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.proc = None
        self.index = index

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.strip().splitlines():
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                smax.append(float(parts[1]))
            except ValueError:
                continue
            for n, v in zip(names, parts[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ------------------------------------------------------------------------------------------ CPU oracle legs
def oracle_setup(n_images, seed=2000):
    """Oracle-side preparation of the block on a reduced calibration set; returns (factors, x_q)."""
    import oracle as o
    import workloads as wl
    from oracle import net as oracle_net
    cfg = wl.config2(seed=seed, batch=n_images, calib_batches=4, calib_batch=2)
    folded = [o.fold_bn(sp.w, sp.b, sp.gamma, sp.beta, sp.mean, sp.var, 1e-5) for sp in cfg["convs"]]
    per_batch = []
    for xb in cfg["calib"]:
        s = wl.bottleneck_fp32(xb, folded)
        per_batch.append({k: s[k] for k in ("x", "a", "b", "c")})
    f = oracle_net.bottleneck_prepare(folded, oracle_net.calib_maxima(per_batch))
    return f, o.quantize(cfg["x"], f["q_x"], o.U8)


def oracle_time_steps(steps, warmup, budget_s=150.0):
    """Times the oracle's bottleneck forward.  A step is a bounded sample of the batch, sized so that
    steps + warmup of them fit the time budget: one image per host thread, else a single image, else a square
    crop of a single image (the bottleneck is fully convolutional; throughput counts the MACs of the sample)."""
    from oracle import net as oracle_net
    cores = os.cpu_count() or 1
    threads = min(cores, BATCH)
    f, xq = oracle_setup(threads)
    t0 = time.perf_counter()
    oracle_net.bottleneck_forward(f, xq[:1], threads=1)
    t1 = time.perf_counter() - t0
    total = steps + warmup
    n, hw = threads, H
    if t1 * 1.5 * total > budget_s:
        n = 1
        while hw > 7 and t1 * (hw * hw) / float(H * W) * total > budget_s:
            hw //= 2
    xq = np.ascontiguousarray(xq[:n, :hw, :hw, :])
    times = []
    for i in range(total):
        t0 = time.perf_counter()
        oracle_net.bottleneck_forward(f, xq, threads=n)
        dt = time.perf_counter() - t0
        if i >= warmup:
            times.append(dt)
    per_step = sum(times) / len(times)
    frac = (hw * hw) / float(H * W)
    tops = 2.0 * MACS_PER_IMAGE * frac * n / per_step / 1e12
    what = f"{n} of {BATCH} images per step" + ("" if hw == H else f", cropped to {hw}x{hw} pixels")
    return dict(value=tops, per_step_s=per_step, images=n, threads=n, total_cores=cores, what=what)


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    r = oracle_time_steps(args.steps, args.warmup)
    sample = f"{r['what']}, one image per thread, oracle loop nest unchanged"
    line = {"impl": "reference", "metric": METRIC, "value": r["value"], "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": r["per_step_s"] * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "s32", "data": "synthetic",
            "config": CONFIG,
            "cpu_baseline": {"value": r["value"], "unit": UNIT, "cores": r["threads"], "kind": "oracle", "sample": sample},
            "e2e": {"value": r["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------------ GPU arm
def bandwidth_kernel_numbers(dev, peak_gbs, reps=20):
    """The memory-bound kernels of the path on tensors larger than L2: algorithmic bytes (max-abs 4 B/elem,
    quantize and dequantize 5, concat 2, pooling input + output) over the CUDA-event time, against the measured
    copy bandwidth."""
    import torch
    import paper_1805_08691_b200 as q8

    def timed(fn):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / reps * 1e-3

    out = {}

    def report(name, nbytes, fn):
        t = timed(fn)
        out[name] = {"GB/s": nbytes / t / 1e9, "frac": nbytes / t / 1e9 / peak_gbs, "us": t * 1e6}

    n = 64 * 112 * 112 * 64 * 2                      # 102.8 M elements: conv1 output of two ResNet-50 batches
    x = torch.randn(n, device=dev)
    slot = torch.zeros(1, device=dev)
    z = torch.empty(n, dtype=torch.uint8, device=dev)
    r = torch.empty(n, dtype=torch.float32, device=dev)
    report("maxabs", n * 4, lambda: q8.q8_calibrate_maxabs(x, slot))
    report("quantize_u8", n * 5, lambda: q8.q8_quantize(x, 0.02, q8.Q8_U8, z))
    report("dequantize_u8", n * 5, lambda: q8.q8_dequantize(z, 0.02, r))
    del r
    img = torch.randn((4 * 64, 224, 224, 3), device=dev)   # 154 MB fp32 in, 206 MB s8 out
    zi = torch.empty((4 * 64, 224, 224, 16), dtype=torch.int8, device=dev)
    report("quantize_pad_3_to_16", img.numel() * 4 + zi.numel(), lambda: q8.q8_quantize_pad_channels(img, 16, 0.02, q8.Q8_S8, out=zi))
    del img, zi
    rows = n // 2 // 192
    a = z[:rows * 192].view(rows, 192)
    b = z[n // 2:n // 2 + rows * 192].view(rows, 192)
    cat = torch.empty((rows, 384), dtype=torch.uint8, device=dev)
    report("concat_requant", rows * 384 * 2, lambda: q8.q8_concat([a, b], [0.01, 0.02], 0.02, out=cat))
    xp = z.view(2 * 64, 112, 112, 64)
    yp = torch.empty((2 * 64, 56, 56, 64), dtype=torch.uint8, device=dev)
    report("maxpool_3x3_s2", xp.numel() + yp.numel(), lambda: q8.q8_maxpool2d(xp, (3, 3), (2, 2), (1, 1), out=yp))
    xa = z[:4 * 64 * 35 * 35 * 288].view(4 * 64, 35, 35, 288)
    ya = torch.empty_like(xa)
    report("avgpool_3x3_s1", xa.numel() * 2, lambda: q8.q8_avgpool2d(xa, (3, 3), (1, 1), (1, 1), out=ya))
    return out


# The paper's own whole-network int8 figures (Tables 1 and 2: one 18-core Xeon socket; throughput at this
# batch, latency at batch 1).  Another machine: context beside the numbers below, not a target.
NETWORKS = {
    "resnet50": dict(fn="resnet50", hw=224, batch=64, seed=3000, paper_xeon={"images_per_s": 462, "latency_ms": 3.5}),
    "inception_v3": dict(fn="inception_v3", hw=299, batch=64, seed=4000, paper_xeon={"images_per_s": 282, "latency_ms": 5.9}),
    "ssd300": dict(fn="ssd300", hw=300, batch=32, seed=5000, paper_xeon={"images_per_s": 43, "latency_ms": 24.8}),
}


def network_numbers(dev, name, reps=20):
    """One whole network (configs[2..4]) through the library: int8 forward of seeded synthetic images as one
    CUDA graph replay per batch (input quantization included), He-init weights, BN folded, factors from a
    short seeded calibration run (timing does not depend on the factors)."""
    import torch
    import paper_1805_08691_b200 as q8
    from paper_1805_08691_b200 import network, pipeline
    from workloads import nets

    def cuda(a):
        return torch.from_numpy(np.ascontiguousarray(a)).to(dev)

    cfg = NETWORKS[name]
    hw = cfg["hw"]
    layers = getattr(nets, cfg["fn"])()

    def fold(ls):
        f = {}
        for L in ls:
            if L.op != "conv":
                continue
            sp = L.conv
            f[L.name] = (q8.q8_fold_bn(cuda(sp.w), None, cuda(sp.gamma), cuda(sp.beta), cuda(sp.mean), cuda(sp.var), 1e-5)
                         if sp.bn else (cuda(sp.w), cuda(sp.b)))
        return f, {k: (w.cpu().numpy(), b.cpu().numpy()) for k, (w, b) in f.items()}

    folded, folded_np = fold(layers)
    acts = nets.fp32_forward(layers, nets.images(cfg["seed"] + 10, 2, hw), folded_np, device=dev)
    cal = pipeline.Calibrator(sorted(acts), device=dev)
    for k, v in acts.items():
        cal.observe(k, cuda(v))
    maxima = cal.maxima()
    del acts
    out = {"macs_per_image": nets.macs(layers, hw), "paper_xeon": cfg["paper_xeon"]}
    # int8 against FP32 on two seeded images (the stand-in for the paper's accuracy table, which needs trained
    # weights and data sets): relative L2 error of the dequantized outputs (logits / all detection heads) for one
    # weight factor per tensor (the paper) or per output channel, and for the factor of a fused residual sum from
    # the "+" rule on its summands or calibrated on the sum itself
    xt = nets.images(cfg["seed"] + 2, 2, hw)
    ref = nets.fp32_forward(layers, xt, folded_np, device=dev)
    heads = [L.name for L in layers if L.f32_out]
    rel = {}
    for per_channel in (False, True):
        for policy in ("max", "post_sum"):
            net = network.QuantNetwork(layers, folded, maxima, (2, hw, hw, 3), device=dev, per_channel=per_channel,
                                       sum_policy=policy)
            got = net.forward(cuda(xt))
            num = sum(float(((got[h].cpu().numpy().astype(np.float64) - ref[h]) ** 2).sum()) for h in heads)
            den = sum(float((ref[h].astype(np.float64) ** 2).sum()) for h in heads)
            rel[("per_channel" if per_channel else "per_tensor") + "/" + policy] = (num / den) ** 0.5
            del net, got
    out["rel_l2_int8_vs_fp32"] = rel
    del ref
    variants = [("batch%d" % cfg["batch"], cfg["batch"], layers), ("batch1", 1, layers)]
    if name == "resnet50":
        # the paper's "remove sparsity" graph rewrite: same FP32 function, 3 % fewer MACs (throughput is still
        # quoted on the MACs of the original network)
        from paper_1805_08691_b200 import graph
        variants.append(("batch%d_sparsity_removed" % cfg["batch"], cfg["batch"], graph.remove_sparsity(layers)))
    if name == "ssd300":
        # the detector as the paper ran it: conv4_3 L2-normalised for its heads, detection output on the heads
        variants.append(("batch%d_with_l2norm_and_detection_output" % cfg["batch"], cfg["batch"], nets.ssd300(l2norm=True)))
    for key, batch, net_layers in variants:
        folded_v = folded
        if net_layers is not layers:
            folded_v, folded_np_v = fold(net_layers)
            acts = nets.fp32_forward(net_layers, nets.images(cfg["seed"] + 10, 2, hw), folded_np_v, device=dev)
            cal = pipeline.Calibrator(sorted(acts), device=dev)
            for k, v in acts.items():
                cal.observe(k, cuda(v))
            maxima = cal.maxima()
            del acts
        net = network.QuantNetwork(net_layers, folded_v, maxima, (batch, hw, hw, 3), device=dev,
                                   streams=int(os.environ.get("Q8_BENCH_STREAMS", "4")))
        x = cuda(nets.images(cfg["seed"] + 1, batch, hw))
        tail = None
        if key.endswith("detection_output"):
            srcs = [L.src[0] for L in net_layers if L.name.endswith("_mbox_loc")]
            heads = [(net.outputs[s_ + "_mbox_loc"], net.outputs[s_ + "_mbox_conf"], net.by_name[s_ + "_mbox_loc"].conv.K // 4) for s_ in srcs]
            priors = cuda(nets.ssd300_priors())
            ws = torch.empty(q8.q8_detection_output_workspace_bytes(batch, 8732, 21, 0, 400, 200), dtype=torch.uint8, device=dev)
            rows, counts = torch.empty((batch, 200, 6), device=dev), torch.empty(batch, dtype=torch.int32, device=dev)

            def tail():
                q8.q8_detection_output(heads, priors, nets.SSD300_VARIANCES, 21, workspace=ws, out=rows, counts=counts)

        def run():
            net.forward(x)
            if tail is not None:
                tail()

        run()
        torch.cuda.synchronize()
        q8.q8_read_status()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            run()
        for _ in range(3):
            g.replay()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            g.replay()
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / reps
        out[key] = {"ms_per_forward": ms, "images_per_s": batch / ms * 1e3,
                                "TOPS": 2.0 * out["macs_per_image"] * batch / ms / 1e9}
        del net, g, x
    torch.cuda.empty_cache()
    return out


def int8_mma_peak(dev, sms):
    """Issue rate of tcgen05.mma.kind::i8 (128 x 256 x 32, two alternating accumulators) on every SM: cycles per
    instruction (slowest CTA, median of five launches) and the MACs per clock and SM that follow."""
    import torch
    import paper_1805_08691_b200 as q8
    n = 8192
    cyc = torch.zeros(sms, dtype=torch.int64, device=dev)
    per, tops = [], []
    for i in range(6):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        q8.q8_int8_mma_rate(256, 2, n, sms, cyc)
        e1.record()
        torch.cuda.synchronize()
        if i:
            per.append(cyc.max().item() / n)
            tops.append(2.0 * 128 * 256 * 32 * n * sms / e0.elapsed_time(e1) / 1e9)
    q8.q8_read_status()
    c = statistics.median(per)
    return {"instruction": "tcgen05.mma.cta_group::1.kind::i8 128x256x32", "instructions_per_sm": n, "sms": sms,
            "cycles_per_instruction": c, "macs_per_clk_per_sm": 128 * 256 * 32 / c,
            "TOPS_whole_launch": statistics.median(tops)}


def config1_numbers(dev):
    """configs[0]: the single 1x14x14x64 3x3 layer, launch-latency bound: microseconds per launch from a CUDA graph of
    200 back-to-back launches, and the single-thread oracle beside it."""
    import torch
    import paper_1805_08691_b200 as q8
    import oracle as o
    g = np.random.default_rng(0)
    x = g.integers(0, 256, (1, 14, 14, 64), dtype=np.uint8)
    w = g.integers(-128, 128, (64, 3, 3, 64)).astype(np.int8)
    b = g.integers(-2000, 2000, 64).astype(np.int32)
    d = q8.make_conv_desc(1, 14, 14, 64, 64, 3, 3, (1, 1), (1, 1), (1, 1), relu=True)
    xt, wt, bt = (torch.from_numpy(a).to(dev) for a in (x, w, b))
    sc = torch.tensor([2e-4], device=dev)
    y = torch.empty((1, 14, 14, 64), dtype=torch.uint8, device=dev)
    q8.q8_conv2d(d, xt, wt, bt, sc, None, 0.0, y)
    torch.cuda.synchronize()
    gr = torch.cuda.CUDAGraph()
    n = 200
    with torch.cuda.graph(gr):
        for _ in range(n):
            q8.q8_conv2d(d, xt, wt, bt, sc, None, 0.0, y)
    gr.replay()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(5):
        gr.replay()
    e1.record()
    torch.cuda.synchronize()
    us = e0.elapsed_time(e1) * 1e3 / (5 * n)
    t0 = time.perf_counter()
    for _ in range(5):
        o.conv2d(x, w, b, np.float32(2e-4), pad=(1, 1), relu=True, threads=1)
    cpu_us = (time.perf_counter() - t0) / 5 * 1e6
    macs = 14 * 14 * 64 * 9 * 64
    return {"workload": "configs[0]: 1x14x14x64 u8, 3x3 pad 1, 64 output channels, bias + requantize + ReLU",
            "us_per_launch": us, "launches_in_graph": n, "TOPS": 2.0 * macs / us / 1e6,
            "oracle_single_thread_us": cpu_us}


def resnet50_layer_table(dev, peak_gbs, int8_peak_tops, batch=64, reps=10):
    """Every launch of ResNet-50 at `batch`, alone: CUDA graph of reps x [evict L2, launch] minus a graph of the
    evictions alone.  Roofline of a launch: max(2 MACs / int8 peak, algorithmic bytes / copy bandwidth)."""
    import torch
    import paper_1805_08691_b200 as q8
    from paper_1805_08691_b200 import network, pipeline
    from workloads import nets

    def cuda(a):
        return torch.from_numpy(np.ascontiguousarray(a)).to(dev)

    layers = nets.resnet50()
    folded = {}
    for L in layers:
        if L.op == "conv":
            sp = L.conv
            folded[L.name] = (q8.q8_fold_bn(cuda(sp.w), None, cuda(sp.gamma), cuda(sp.beta), cuda(sp.mean), cuda(sp.var), 1e-5)
                              if sp.bn else (cuda(sp.w), cuda(sp.b)))
    folded_np = {k: (w.cpu().numpy(), b.cpu().numpy()) for k, (w, b) in folded.items()}
    acts = nets.fp32_forward(layers, nets.images(3010, 2, 224), folded_np, device=dev)
    cal = pipeline.Calibrator(sorted(acts), device=dev)
    for k, v in acts.items():
        cal.observe(k, cuda(v))
    maxima = cal.maxima()
    del acts
    net = network.QuantNetwork(layers, folded, maxima, (batch, 224, 224, 3), device=dev, streams=1)
    net.forward(cuda(nets.images(3001, batch, 224)))
    torch.cuda.synchronize()
    q8.q8_read_status()
    evict = torch.empty(256 << 20, dtype=torch.uint8, device=dev)

    def timed_graph(fn):
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            for _ in range(reps):
                evict.zero_()
                if fn is not None:
                    fn()
        g.replay()
        torch.cuda.synchronize()
        ts = []
        for _ in range(3):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            g.replay()
            e1.record()
            torch.cuda.synchronize()
            ts.append(e0.elapsed_time(e1))
        return statistics.median(ts) * 1e3 / reps   # us per [evict, launch]

    base_us = timed_graph(None)
    rows = []
    ws = net.workspaces[0]
    for L in layers:
        if L.op != "conv" or L.name in net.fused_with or L.name in net.skip:
            continue
        parts = [L]
        if L.name in net.fused_second:
            parts = [net.by_name[L.src[0]], L]
        macs, nbytes = 0, 0
        for i, P in enumerate(parts):
            d = net.convs[P.name].desc
            pq = q8.conv_out_shape(d)
            m = d.N * pq[0] * pq[1]
            macs += m * P.conv.K * P.conv.R * P.conv.S * P.conv.C       # true channel counts
            nbytes += d.K * d.R * d.S * d.C + 4 * d.K
            if i == 0:
                nbytes += d.N * d.H * d.W * d.C
            if i == len(parts) - 1:
                nbytes += m * d.K * (4 if P.f32_out else 1) + (m * d.K if P.residual else 0)
        us = timed_graph(lambda: net._launch(L, ws)) - base_us
        t_mma, t_hbm = 2.0 * macs / int8_peak_tops / 1e6, nbytes / peak_gbs / 1e3     # us
        sp = parts[0].conv
        rows.append({"layer": "+".join(P.name for P in parts),
                     "shape": "%dx%d %d->%d %dx%d/%d" % (net.convs[parts[0].name].desc.H, net.convs[parts[0].name].desc.W,
                                                         sp.C, parts[-1].conv.K, sp.R, sp.S, sp.stride[0]) + (" + 1x1" if len(parts) > 1 else ""),
                     "us": us, "TOPS": 2.0 * macs / us / 1e6, "bytes": nbytes, "GB/s": nbytes / us / 1e3,
                     "bound": "tensor" if t_mma >= t_hbm else "hbm", "roofline_us": max(t_mma, t_hbm),
                     "frac": max(t_mma, t_hbm) / us})
    del net
    torch.cuda.empty_cache()
    return {"batch": batch, "l2": "256 MB written between launches (cold inputs)", "evict_us": base_us, "layers": rows,
            "sum_us": sum(r["us"] for r in rows), "sum_roofline_us": sum(r["roofline_us"] for r in rows)}


def run_ours(args):
    import torch
    import torch.distributed as dist
    import paper_1805_08691_b200 as q8
    from paper_1805_08691_b200 import pipeline
    import workloads as wl
    from workloads import synth

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the q8 library has no CPU path")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    sms = torch.cuda.get_device_properties(dev).multi_processor_count

    def cuda(a):
        return torch.from_numpy(np.ascontiguousarray(a)).to(dev)

    # ---- preparation (untimed): fold BN, calibrate on 4 seeded batches, quantize weights/bias.  Weights and
    # calibration batches are the same on every rank (replicas); only the images of a rank's batch differ.
    cfg = wl.config2(seed=2000, batch=BATCH, calib_batches=4, calib_batch=8)
    folded = []
    for sp in cfg["convs"]:
        folded.append(q8.q8_fold_bn(cuda(sp.w), None, cuda(sp.gamma), cuda(sp.beta), cuda(sp.mean), cuda(sp.var), 1e-5))
    names = ["x", "a", "b", "c"]
    cal = pipeline.Calibrator(names, device=dev)
    folded_np = [(w.cpu().numpy(), b.cpu().numpy()) for w, b in folded]
    for xb in cfg["calib"]:
        s = wl.bottleneck_fp32(xb, folded_np, device=dev)
        for k in names:
            cal.observe(k, cuda(s[k]))
    maxima = pipeline.sync_maxima(cal.maxima(), dev if world > 1 else None)
    shape = (BATCH, H, W, C)
    x_np = cfg["x"] if rank == 0 else synth.relu_normal(synth.rng(2001 + 100 * rank), shape)
    x_f32 = cuda(x_np)
    n_sets = max(2, args.sets)
    blocks = [pipeline.Bottleneck(folded, maxima, shape) for _ in range(n_sets)]
    fused = blocks[0].fused
    xs = [q8.q8_quantize(x_f32.roll(i, dims=0), blocks[0].q_x, q8.Q8_U8) for i in range(n_sets)]
    ys = [torch.empty(shape, dtype=torch.uint8, device=dev) for _ in range(n_sets)]
    del x_f32
    set_bytes = 2 * BATCH * H * W * C + 2 * BATCH * H * W * MID
    for lay in (blocks[0].a, blocks[0].b, blocks[0].c):
        assert q8.q8_conv2d_query_algo(lay.desc) == q8.Q8_ALGO_UMMA

    # eager warm-up (loads kernels, sets attributes) then one CUDA graph per buffer set
    for i in range(n_sets):
        blocks[i](xs[i], out=ys[i])
    torch.cuda.synchronize()
    q8.q8_read_status()
    graphs = []
    for i in range(n_sets):
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            blocks[i](xs[i], out=ys[i])
        graphs.append(g)
    # the timed region replays ONE graph holding the K steps (step i works on buffer set i % n_sets), so that no
    # host launch gap sits between steps (K > 240: a graph of the largest divisor of K up to 240, replayed K / chunk
    # times per repeat)
    chunk = args.steps
    if chunk > 240:
        divs = [d for d in range(240, 0, -1) if args.steps % d == 0]
        chunk = next((d for d in divs if d % n_sets == 0), divs[0])
    replays_per_repeat = args.steps // chunk
    # Steps work on different batches and are independent, so they may be in flight together: with
    # --step-streams S step i is enqueued on stream i % S (every buffer set stays on one stream).  A step is still
    # the whole block over one batch; the next batch's first kernel fills the SMs that the last kernel of this one
    # leaves idle while it drains.
    n_step_streams = max(1, min(args.step_streams, n_sets))
    while n_sets % n_step_streams:
        n_step_streams -= 1
    side = [torch.cuda.Stream(device=dev) for _ in range(n_step_streams - 1)]
    timed = torch.cuda.CUDAGraph()
    with torch.cuda.graph(timed):
        main = torch.cuda.current_stream()
        for st in side:
            st.wait_stream(main)
        for i in range(chunk):
            st = main if i % n_step_streams == 0 else side[i % n_step_streams - 1]
            with torch.cuda.stream(st):
                blocks[i % n_sets](xs[i % n_sets], out=ys[i % n_sets])
        for st in side:
            main.wait_stream(st)
    # one graph per launch kind for the per-kernel durations: the same launch repeated over all buffer sets
    kreps = 8
    kinds = ["a", "bc"] if fused else ["a", "b", "c"]
    kgraphs = []
    for kind in kinds:
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            for _ in range(kreps):
                for i in range(n_sets):
                    blk = blocks[i]
                    if kind == "a":
                        blk.a(xs[i], out=blk.ya)
                    elif kind == "b":
                        blk.b(blk.ya, out=blk.yb)
                    elif kind == "c":
                        blk.c(blk.yb, residual=xs[i], out=ys[i])
                    else:
                        pipeline.fused_pair(blk.b, blk.c, blk.ya, residual=xs[i], out=ys[i])
        kgraphs.append(g)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(max(3, args.warmup)):
        graphs[i % n_sets].replay()
    barrier()
    mon = ClockMonitor(local)
    if rank == 0:
        mon.start()
    # keep the monitor sampling for a moment under load before the timed region; the step time seen here sizes
    # the number of repeats
    t_end = time.time() + 0.3
    i = 0
    while time.time() < t_end:
        graphs[i % n_sets].replay()
        i += 1
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    timed.replay()  # untimed: first replay of a graph uploads it
    e1.record()
    barrier()
    est_ms = max(e0.elapsed_time(e1) * replays_per_repeat, 1e-3)
    repeats = int(min(2000, max(3, -(-250.0 // est_ms))))
    if world > 1:
        r_t = torch.tensor([repeats], dtype=torch.int64, device=dev)
        dist.all_reduce(r_t, op=dist.ReduceOp.MAX)
        repeats = int(r_t.item())
    evs = [torch.cuda.Event(enable_timing=True) for _ in range(repeats + 1)]
    barrier()
    evs[0].record()
    for r in range(repeats):
        for _ in range(replays_per_repeat):
            timed.replay()
        evs[r + 1].record()
    barrier()
    rep_ms = [evs[r].elapsed_time(evs[r + 1]) for r in range(repeats)]
    ms_total = statistics.median(rep_ms)          # K steps
    ms_min, ms_region = min(rep_ms), evs[0].elapsed_time(evs[repeats])

    # ---- per-kernel durations: CUDA events around a graph of kreps * n_sets launches of one kind
    kms = []
    for g in kgraphs:
        g.replay()
        torch.cuda.synchronize()
        e0.record()
        g.replay()
        e1.record()
        torch.cuda.synchronize()
        kms.append(e0.elapsed_time(e1) / (kreps * n_sets))
    mma_peak = int8_mma_peak(dev, sms) if rank == 0 else None
    barrier()
    clocks = mon.stop() if rank == 0 else None

    # ---- end to end: u8 input from pinned host memory, u8 result back to pinned host memory, every step.
    # Three streams (H2D, compute through the public API, D2H) linked by events, so that the copies of neighbouring
    # steps overlap the kernels and each other (PCIe is full duplex); buffer sets rotate as in the timed region.
    hx = [torch.from_numpy(np.ascontiguousarray(xs[0].cpu().numpy())).pin_memory() for _ in range(2)]
    hy = [torch.empty(shape, dtype=torch.uint8).pin_memory() for _ in range(2)]
    esteps = max(3, min(args.steps, 400))
    s_in, s_cmp, s_out = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()
    ev_in = [torch.cuda.Event() for _ in range(n_sets)]
    ev_cmp = [torch.cuda.Event() for _ in range(n_sets)]
    ev_out = [torch.cuda.Event() for _ in range(n_sets)]

    def e2e_step(i):
        k, j = i % n_sets, i % 2
        with torch.cuda.stream(s_in):
            if i >= n_sets:
                s_in.wait_event(ev_cmp[k])      # the kernels that last read this input set are done
            xs[k].copy_(hx[j], non_blocking=True)
            ev_in[k].record(s_in)
        with torch.cuda.stream(s_cmp):
            s_cmp.wait_event(ev_in[k])
            if i >= n_sets:
                s_cmp.wait_event(ev_out[k])     # the previous result in this output set has left the device
            blocks[k](xs[k], out=ys[k])
            ev_cmp[k].record(s_cmp)
        with torch.cuda.stream(s_out):
            s_out.wait_event(ev_cmp[k])
            hy[j].copy_(ys[k], non_blocking=True)
            ev_out[k].record(s_out)

    torch.cuda.synchronize()
    for i in range(n_sets):
        e2e_step(i)
    torch.cuda.synchronize()
    barrier()
    e0.record()
    for st in (s_in, s_cmp, s_out):
        st.wait_event(e0)
    for i in range(n_sets, n_sets + esteps):
        e2e_step(i)
    cur = torch.cuda.current_stream()
    for st in (s_in, s_cmp, s_out):
        done = torch.cuda.Event()
        done.record(st)
        cur.wait_event(done)
    e1.record()
    barrier()
    ms_e2e = e0.elapsed_time(e1) / esteps
    q8.q8_read_status()

    t = torch.tensor([ms_total, ms_e2e, ms_min, ms_region], dtype=torch.float64, device=dev)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    ms_total, ms_e2e, ms_min, ms_region = t.tolist()
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    ms_step = ms_total / args.steps
    ops_step = 2.0 * MACS_PER_IMAGE * BATCH * world
    peaks = measured_peaks()
    # int8 tensor peak: the measured issue rate (MACs per clock and SM) at the SM clock sampled during this run
    sm_mhz = (clocks or {}).get("sm_mhz") or peaks["sm_max_mhz"]
    int8_peak = sms * mma_peak["macs_per_clk_per_sm"] * 2.0 * sm_mhz * 1e6 / 1e12
    mma_peak.update({"sm_mhz_used": sm_mhz, "peak_TOPS_at_sampled_clock": int8_peak,
                     "peak_TOPS_at_max_clock": sms * mma_peak["macs_per_clk_per_sm"] * 2.0 * peaks["sm_max_mhz"] * 1e6 / 1e12,
                     "for_context_2x_bf16_burst_TOPS": 2.0 * peaks["bf16_tflops"]})
    M = BATCH * H * W
    if fused:
        kinfo = [("conv_umma 1x1 256->64", layer_bytes(M, C, MID, 1, 1), 2.0 * M * C * MID),
                 ("conv_fused 3x3 64->64 + 1x1 64->256 +res",
                  M * MID + 9 * MID * MID + 4 * MID + MID * C + 4 * C + 2 * M * C, 2.0 * M * (9 * MID * MID + MID * C))]
    else:
        kinfo = [("conv_umma 1x1 256->64", layer_bytes(M, C, MID, 1, 1), 2.0 * M * C * MID),
                 ("conv_umma 3x3 64->64", layer_bytes(M, MID, MID, 3, 3), 2.0 * M * 9 * MID * MID),
                 ("conv_umma 1x1 64->256 +res", layer_bytes(M, MID, C, 1, 1, residual=True), 2.0 * M * MID * C)]
    kernels = []
    for (name, nbytes, ops), ms in zip(kinfo, kms):
        kernels.append({"kernel": name, "ms": ms, "GB/s": nbytes / ms / 1e6, "TOPS": ops / ms / 1e9,
                        "roofline_ms": max(nbytes / peaks["hbm_gbs"] / 1e6, ops / int8_peak / 1e9)})
    dom = max(range(len(kms)), key=lambda j: kms[j])
    achieved = kinfo[dom][1] / kms[dom] / 1e6
    roofline = {"bound": "hbm", "kernel": kinfo[dom][0], "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": achieved / peaks["hbm_gbs"], "peak_source": peaks["source"],
                "algorithmic_bytes_per_launch": kinfo[dom][1], "traffic": ncu_traffic(kinfo[dom][0])}
    line = {"metric": METRIC, "value": ops_step / ms_step / 1e9, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(3, args.warmup), "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "s32", "data": "synthetic",
            "config": CONFIG,
            "timing": {"l2": "rotating %d buffer sets of %.0f MB (> 126 MB L2)" % (n_sets, set_bytes / 1e6),
                       "launch": "CUDA graph of %d steps on %d stream(s), %d replays per repeat" % (chunk, n_step_streams, replays_per_repeat),
                       "timed_repeats": repeats, "statistic": "median over the repeats of the time of K steps",
                       "ms_per_step_min": ms_min / args.steps, "timed_region_ms": ms_region},
            "clocks": clocks,
            "e2e": {"value": ops_step / ms_e2e / 1e9, "unit": UNIT, "ms_per_step": ms_e2e,
                    "h2d_bytes_per_step": BATCH * H * W * C, "d2h_bytes_per_step": BATCH * H * W * C,
                    "pipeline": "H2D, kernels and D2H of neighbouring steps overlap on three streams"},
            "gpu_launches": len(kinds) * args.steps * repeats,
            "launches_per_step": len(kinds),
            "roofline": roofline, "kernels": kernels, "int8_mma_peak": mma_peak,
            "images_per_s": BATCH * world / ms_step * 1e3}
    if world == 1:
        line["config1"] = config1_numbers(dev)
    if world == 1 and not args.skip_networks:
        line["bandwidth_kernels"] = bandwidth_kernel_numbers(dev, peaks["hbm_gbs"])
        line["resnet50_layers"] = resnet50_layer_table(dev, peaks["hbm_gbs"], int8_peak)
        line["ssd_tail"] = ssd_tail_numbers(dev, peaks["hbm_gbs"])
        line["networks"] = {name: network_numbers(dev, name) for name in NETWORKS}
    if world == 1 and not args.skip_cpu_baseline:
        r = oracle_time_steps(steps=2, warmup=1)
        line["cpu_baseline"] = {"value": r["value"], "unit": UNIT, "cores": r["threads"], "kind": "oracle",
                                "sample": f"{r['what']} x 2 steps, one image per thread"}
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def ssd_tail_numbers(dev, peak_gbs, reps=20):
    """The SSD tail and the FP32 route (all at N = 1, CUDA-event times of back-to-back launches):
    * l2norm: L2 normalisation of a conv4_3-shaped tensor (128 x 38 x 38 x 512 u8, in + out larger than L2) against
      the measured copy bandwidth;
    * detection_output: 8732 boxes x 21 classes per image at batch 32, seeded head outputs (2 % confident boxes);
    * fp32_route: the four projection blocks of ResNet-50 at batch 64, the shortcut convolution (no ReLU, signed
      output) and the block's last 1x1 convolution, (a) as the library runs them: s8 shortcut, residual sum fused
      into the last convolution's epilogue; (b) the paper's FP32 route for signed tensors: both convolutions write
      fp32, one more kernel adds, applies the ReLU and quantizes."""
    import torch
    import paper_1805_08691_b200 as q8
    from workloads import nets

    def timed(fn):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / reps * 1e-3

    g = torch.Generator(device=dev).manual_seed(0)

    def rnd(shape, lo=0, hi=256, dt=torch.uint8):
        return torch.randint(lo, hi, shape, dtype=dt, device=dev, generator=g)

    out = {}
    x = rnd((128, 38, 38, 512))
    y = torch.empty_like(x)
    mult = torch.full((512,), 20.0 * 0.03 / 0.08, device=dev)
    t = timed(lambda: q8.q8_l2norm(x, 0.03, 1e-10, mult, out=y))
    out["l2norm"] = {"us": t * 1e6, "GB/s": 2 * x.numel() / t / 1e9, "frac": 2 * x.numel() / t / 1e9 / peak_gbs}
    del x, y
    N = 32
    loc_np, conf_np = nets.detection_inputs(77, N)
    priors = torch.from_numpy(nets.ssd300_priors()).to(dev)
    loc, conf = torch.from_numpy(loc_np).to(dev), torch.from_numpy(conf_np).to(dev)
    ws = torch.empty(q8.q8_detection_output_workspace_bytes(N, 8732, 21, 0, 400, 200), dtype=torch.uint8, device=dev)
    rows = torch.empty((N, 200, 6), device=dev)
    counts = torch.empty(N, dtype=torch.int32, device=dev)
    src = [(loc, conf, 1)]
    t = timed(lambda: q8.q8_detection_output(src, priors, nets.SSD300_VARIANCES, 21, workspace=ws, out=rows, counts=counts))
    out["detection_output"] = {"batch": N, "us": t * 1e6, "images_per_s": N / t, "detections_per_image": float(counts.float().mean()),
                               "launches": 3}
    # the worst case for the per-class sort: flat logits, every box a candidate of every class
    gen = np.random.default_rng(78)
    conf = torch.from_numpy(gen.normal(0, 0.3, (N, 8732, 21)).astype(np.float32)).to(dev)
    src = [(loc, conf, 1)]
    t = timed(lambda: q8.q8_detection_output(src, priors, nets.SSD300_VARIANCES, 21, workspace=ws, out=rows, counts=counts))
    out["detection_output_every_box_a_candidate"] = {"batch": N, "us": t * 1e6, "images_per_s": N / t}
    del loc, conf, ws
    blocks = {}
    B = 64
    for name, (H, Cin, Cmid, K, st) in {"res2a": (56, 64, 64, 256, 1), "res3a": (56, 256, 128, 512, 2), "res4a": (28, 512, 256, 1024, 2),
                                        "res5a": (14, 1024, 512, 2048, 2)}.items():
        Ho = H // st
        xin, xmid = rnd((B, H, H, Cin)), rnd((B, Ho, Ho, Cmid))
        w1, w2 = rnd((K, 1, 1, Cin), -128, 128, torch.int8), rnd((K, 1, 1, Cmid), -128, 128, torch.int8)
        b1, b2 = rnd((K,), -1000, 1000, torch.int32), rnd((K,), -1000, 1000, torch.int32)
        s = torch.tensor([1e-4], device=dev)
        U8, S8, F32 = q8.Q8_U8, q8.Q8_S8, q8.Q8_F32
        d1s = q8.make_conv_desc(B, H, H, Cin, K, 1, 1, (st, st), (0, 0), (1, 1), U8, U8, S8, False)
        d2s = q8.make_conv_desc(B, Ho, Ho, Cmid, K, 1, 1, (1, 1), (0, 0), (1, 1), U8, S8, U8, True)
        d1f = q8.make_conv_desc(B, H, H, Cin, K, 1, 1, (st, st), (0, 0), (1, 1), U8, U8, F32, False)
        d2f = q8.make_conv_desc(B, Ho, Ho, Cmid, K, 1, 1, (1, 1), (0, 0), (1, 1), U8, U8, F32, False)
        sc = torch.empty((B, Ho, Ho, K), dtype=torch.int8, device=dev)
        yo = torch.empty((B, Ho, Ho, K), dtype=torch.uint8, device=dev)
        fa, fb = torch.empty((B, Ho, Ho, K), device=dev), torch.empty((B, Ho, Ho, K), device=dev)

        def int8_route():
            q8.q8_conv2d(d1s, xin, w1, b1, s, None, 0.0, sc)
            q8.q8_conv2d(d2s, xmid, w2, b2, s, sc, 0.5, yo)

        def fp32_route():
            q8.q8_conv2d(d1f, xin, w1, b1, s, None, 0.0, fa)
            q8.q8_conv2d(d2f, xmid, w2, b2, s, None, 0.0, fb)
            q8.q8_add_relu_quantize(fa, fb, 0.05, out=yo)

        ti, tf = timed(int8_route), timed(fp32_route)
        blocks[name] = {"int8_us": ti * 1e6, "fp32_route_us": tf * 1e6, "ratio": tf / ti,
                        "int8_bytes": xin.numel() + xmid.numel() + 3 * yo.numel(),
                        "fp32_route_bytes": xin.numel() + xmid.numel() + 17 * yo.numel()}
        del xin, xmid, sc, yo, fa, fb
    q8.q8_read_status()
    out["fp32_route"] = {"batch": B, "blocks": blocks,
                         "int8_us": sum(v["int8_us"] for v in blocks.values()),
                         "fp32_route_us": sum(v["fp32_route_us"] for v in blocks.values())}
    torch.cuda.empty_cache()
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None, help="timed steps (default 12000; 3 for --impl reference)")
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--sets", type=int, default=6, help="rotating buffer sets (working set must exceed L2)")
    ap.add_argument("--step-streams", type=int, default=2,
                    help="streams the steps of the timed region alternate between (steps are independent batches)")
    ap.add_argument("--skip-cpu-baseline", action="store_true")
    ap.add_argument("--bandwidth-only", type=int, default=0, metavar="REPS",
                    help="run only the memory-bound kernels, REPS timed launches each, print their JSON and exit "
                         "(the command the ncu summary of these kernels is taken with)")
    ap.add_argument("--ssd-tail-only", action="store_true",
                    help="run only the SSD tail and the FP32-route comparison, print their JSON and exit")
    ap.add_argument("--skip-networks", "--skip-resnet50", dest="skip_networks", action="store_true",
                    help="leave out the whole-network numbers (ResNet-50, Inception-v3, SSD-300)")
    args = ap.parse_args()
    if args.steps is None:
        args.steps = 3 if args.impl == "reference" else 12000
    if args.bandwidth_only:
        import torch
        print(json.dumps({"bandwidth_kernels": bandwidth_kernel_numbers(torch.device("cuda", 0), measured_peaks()["hbm_gbs"],
                                                                        reps=args.bandwidth_only)}), flush=True)
        return
    if args.ssd_tail_only:
        import torch
        print(json.dumps({"ssd_tail": ssd_tail_numbers(torch.device("cuda", 0), measured_peaks()["hbm_gbs"])}), flush=True)
        return
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()

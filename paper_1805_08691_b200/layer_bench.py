"""Time one quantized convolution layer (or a fused pair) through the C ABI.

    python -m paper_1805_08691_b200.layer_bench --layer 64,28,28,128,128,3,3,1,1 [--then-1x1 512] [--residual] [--reps 20]

--layer N,H,W,C,K,R,S,stride,pad.  --then-1x1 K2 appends a 1x1 layer with K2 output channels and runs the pair as
one launch where the library supports it.  --residual adds a fused u8 residual sum to the (last) layer.
Inputs are uniform random 8-bit payloads; the launch is replayed from a CUDA graph over rotating buffer sets larger
than L2 ("cold") and over one set ("warm").  Prints microseconds, algorithmic GB/s and TOPS.  Also the small
command the ncu summaries under profiles/ were taken with (--launches N: plain launches, no graph).
"""
import argparse

import torch

from . import binding as q8

U8 = q8.Q8_U8


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--layer", required=True)
    ap.add_argument("--then-1x1", type=int, default=0)
    ap.add_argument("--residual", action="store_true")
    ap.add_argument("--reps", type=int, default=20)
    ap.add_argument("--l2-mb", type=int, default=400)
    ap.add_argument("--launches", type=int, default=0, help="only run this many plain launches (for profilers)")
    a = ap.parse_args()
    N, H, W, C, K, R, S, st, pad = (int(v) for v in a.layer.split(","))
    pads = (pad, pad) if R == S else ((R // 2) if pad else 0, (S // 2) if pad else 0)
    d1 = q8.make_conv_desc(N, H, W, C, K, R, S, (st, st), pads, (1, 1), U8, U8, U8, True)
    P, Q = q8.conv_out_shape(d1)
    K_out = a.then_1x1 or K
    d2 = q8.make_conv_desc(N, P, Q, K, K_out, 1, 1, (1, 1), (0, 0), (1, 1), U8, U8, U8, True) if a.then_1x1 else None
    fused = bool(d2) and q8.q8_conv2d_then_1x1_supported(d1, d2)
    M = N * P * Q
    per_set = N * H * W * C + M * K_out * (2 if a.residual else 1) + (M * K if d2 and not fused else 0)
    sets = 1 if a.launches else min(max(2, int(a.l2_mb * 1e6 / per_set) + 1), 64)
    g = torch.Generator(device="cuda").manual_seed(0)

    def rnd(shape, lo=0, hi=256, dt=torch.uint8):
        return torch.randint(lo, hi, shape, dtype=dt, device="cuda", generator=g)

    xs = [rnd((N, H, W, C)) for _ in range(sets)]
    rs = [rnd((N, P, Q, K_out)) for _ in range(sets)] if a.residual else [None] * sets
    ms = [torch.empty((N, P, Q, K), dtype=torch.uint8, device="cuda") for _ in range(sets)] if d2 and not fused else None
    ys = [torch.empty((N, P, Q, K_out), dtype=torch.uint8, device="cuda") for _ in range(sets)]
    w1, b1 = rnd((K, R, S, C), -128, 128, torch.int8), rnd((K,), -1000, 1000, torch.int32)
    s1 = torch.tensor([1e-4], device="cuda")
    w2 = b2 = s2 = None
    if d2:
        w2, b2 = rnd((K_out, 1, 1, K), -128, 128, torch.int8), rnd((K_out,), -1000, 1000, torch.int32)
        s2 = torch.tensor([1e-4], device="cuda")
    nws = q8.q8_conv2d_workspace_bytes(d1)
    ws = torch.empty(max(nws, 16), dtype=torch.uint8, device="cuda") if nws else None

    def launch(i):
        if fused:
            q8.q8_conv2d_then_1x1(d1, d2, xs[i], w1, b1, s1, w2, b2, s2, rs[i], 0.5, ys[i])
        elif d2:
            q8.q8_conv2d(d1, xs[i], w1, b1, s1, None, 0.0, ms[i], ws)
            q8.q8_conv2d(d2, ms[i], w2, b2, s2, rs[i], 0.5, ys[i])
        else:
            q8.q8_conv2d(d1, xs[i], w1, b1, s1, rs[i], 0.5, ys[i], ws)

    if a.launches:
        for _ in range(a.launches):
            launch(0)
        torch.cuda.synchronize()
        q8.q8_read_status()
        print("ran", a.launches, "launches" + (" (fused pair)" if fused else ""))
        return
    for i in range(sets):
        launch(i)
    torch.cuda.synchronize()
    q8.q8_read_status()
    out = {}
    for mode in ("cold", "warm"):
        gr = torch.cuda.CUDAGraph()
        with torch.cuda.graph(gr):
            for i in range(sets):
                launch(i if mode == "cold" else 0)
        for _ in range(3):
            gr.replay()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(a.reps):
            gr.replay()
        e1.record()
        torch.cuda.synchronize()
        out[mode] = e0.elapsed_time(e1) * 1e3 / (a.reps * sets)
    nbytes = N * H * W * C + K * R * S * C + 4 * K + M * K_out * (2 if a.residual else 1) + (K_out * K + 4 * K_out if d2 else 0)
    ops = 2.0 * M * K * R * S * C + (2.0 * M * K * K_out if d2 else 0)
    us = out["cold"]
    print(f"{a.layer}{' -> 1x1 %d' % K_out if d2 else ''}{' (one launch)' if fused else ''}: cold {us:.2f} us, warm {out['warm']:.2f} us, "
          f"{nbytes / us / 1e3:.0f} GB/s, {ops / us / 1e6:.0f} TOPS, {sets} buffer sets")


if __name__ == "__main__":
    main()

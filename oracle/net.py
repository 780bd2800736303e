"""Oracle-side assembly of quantized layers: the paper's workflow (fold, calibrate, quantize, run) with oracle calls only.

TEST INFRASTRUCTURE like the rest of this package.
"""
import numpy as np

from . import q8_oracle as o


def prepare_conv(w, b, q_x, q_y, y_type=o.U8, q_res=None):
    q_w = o.factor(o.maxabs(w), 7)
    w_q = o.quantize(w, q_w, o.S8)
    b_q = o.quantize(b, o.bias_factor(q_x, q_w), o.S32) if b is not None else None
    if y_type == o.F32:
        q_y = 1.0
    scale = o.requant_scale(q_x, q_w, q_y)
    res_scale = o.requant_scale(q_res, 1.0, q_y) if q_res is not None else 0.0
    return dict(w_q=w_q, b_q=b_q, scale=scale, q_w=q_w, res_scale=res_scale)


def bottleneck_prepare(folded, maxima):
    (wa, ba), (wb, bb), (wc, bc) = folded
    f = dict(q_x=o.factor(maxima["x"], 8), q_a=o.factor(maxima["a"], 8), q_b=o.factor(maxima["b"], 8),
             q_y=o.factor(max(maxima["c"], maxima["x"]), 8))
    f["a"] = prepare_conv(wa, ba, f["q_x"], f["q_a"])
    f["b"] = prepare_conv(wb, bb, f["q_a"], f["q_b"])
    f["c"] = prepare_conv(wc, bc, f["q_b"], f["q_y"], q_res=f["q_x"])
    return f


def bottleneck_forward(f, x_q, threads=1):
    a, b, c = f["a"], f["b"], f["c"]
    ya = o.conv2d(x_q, a["w_q"], a["b_q"], a["scale"], relu=True, threads=threads)
    yb = o.conv2d(ya, b["w_q"], b["b_q"], b["scale"], pad=(1, 1), relu=True, threads=threads)
    y = o.conv2d(yb, c["w_q"], c["b_q"], c["scale"], residual=x_q, res_scale=c["res_scale"], relu=True,
                 threads=threads)
    return ya, yb, y


def calib_maxima(samples_per_batch):
    """samples_per_batch: list of dict name -> fp32 array; running max over batches."""
    m = {}
    for batch in samples_per_batch:
        for k, v in batch.items():
            m[k] = o.maxabs(v, init=m.get(k, 0.0))
    return m

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


# --------------------------------------------------------------------------------------------------
# Whole networks (layer lists from workloads.nets), oracle calls only.
#
# Factor rules (calibration paragraph of Sec. "8-bit Low Precision Inference", Eq. arithmetics):
#   network input (signed)            : s8, q = max|x| / 127
#   conv + ReLU                       : u8, q = max / 255
#   conv without ReLU                 : s8, q = max|y| / 127
#   conv + residual sum + ReLU        : u8, q = max(max|conv|, max|residual|) / 255   ("+" rule on a common footing)
#   dequantized output (logits, heads): fp32, the accumulator is only multiplied by q_x * q_w
#   pooling                           : type and factor of its input
#   concat                            : ONE factor for the whole output: the largest branch factor.  A conv + ReLU
#                                       whose only reader is a concat (or a concat nested in one) is quantized
#                                       straight at that shared factor (one rounding); any other branch (a pooled
#                                       tensor) is re-expressed at it by the concat.  A nested concat shares the
#                                       factor of the outermost one.
# A 3-channel input is zero padded to 16 channels (weights too): zeros are exact under a symmetric quantizer.
# --------------------------------------------------------------------------------------------------
def _pad_c(a, c_pad):
    if a.shape[-1] == c_pad:
        return a
    out = np.zeros(a.shape[:-1] + (c_pad,), dtype=a.dtype)
    out[..., :a.shape[-1]] = a
    return out


def _concat_groups(layers):
    """For every tensor that ends in a concat: the outermost concat it belongs to.  Returns (root of each
    concat, shared-factor convs -> root, leaves of each root)."""
    readers = {}
    for L in layers:
        for s in L.src + ([L.residual] if L.residual else []):
            readers.setdefault(s, []).append(L)
    by_name = {L.name: L for L in layers}

    def root_of(name):
        r = readers.get(name, [])
        while len(r) == 1 and r[0].op == "concat":
            name = r[0].name
            r = readers.get(name, [])
        return name

    root, shared, leaves = {}, {}, {}
    for L in layers:
        if L.op != "concat":
            continue
        root[L.name] = root_of(L.name)
        for s in L.src:
            if by_name[s].op == "concat":
                continue
            leaves.setdefault(root[L.name], []).append(s)
            Ls = by_name[s]
            if (Ls.op == "conv" and Ls.conv.relu and not Ls.f32_out and Ls.residual is None
                    and len(readers[s]) == 1):
                shared[s] = root[L.name]
    return root, shared, leaves


def network_prepare(layers, folded, maxima, per_channel=False, sum_policy="max"):
    """Returns {layer name: dict} with the quantized parameters and the (type, factor) of every tensor.
    per_channel: one weight factor per output channel, max|w[k]| / 127 (the paper takes one per tensor); bias
    and requantisation multiplier of channel k then use q_w[k].
    sum_policy: factor of a fused residual sum.  "max": the "+" rule of Eq. arithmetics on the two summands,
    max(max|conv|, max|residual|) / 255.  "post_sum": the calibration rule applied to the tensor the layer
    actually emits, max|ReLU(conv + residual)| / 255 (never larger than twice the first, often smaller)."""
    assert sum_policy in ("max", "post_sum")
    root, shared, leaves = _concat_groups(layers)
    by_name = {L.name: L for L in layers}
    own = {}

    def own_factor(name):
        """Factor a tensor has before any sharing: its calibrated maximum, or its input's factor for a pool."""
        if name not in own:
            L = by_name.get(name)
            if name == "input":
                own[name] = o.factor(maxima["input"], 7)
            elif L.op in ("maxpool", "avgpool"):
                own[name] = final_factor(L.src[0])
            elif L.op == "concat":
                own[name] = group_factor(root[name])
            elif L.op == "l2norm":
                own[name] = o.factor(maxima[name], 8)
            elif L.residual is not None and sum_policy == "post_sum":
                own[name] = o.factor(maxima[name], 8)
            elif L.residual is not None:
                own[name] = o.factor(max(maxima[name + ":pre"], maxima[L.residual]), 8)
            else:
                own[name] = o.factor(maxima[name], 8 if L.conv.relu else 7)
        return own[name]

    def group_factor(r):
        return max(own_factor(s) for s in leaves[r])

    def final_factor(name):
        return group_factor(shared[name]) if name in shared else own_factor(name)

    info = {"input": (o.S8, own_factor("input"))}
    prep = {}
    for L in layers:
        t_in, q_in = info[L.src[0]]
        if L.op == "conv":
            w, b = folded[L.name]
            c_pad = -(-w.shape[-1] // 16) * 16
            if per_channel:
                q_w = [o.factor(o.maxabs(w[k]), 7) for k in range(w.shape[0])]
                w_q = _pad_c(np.stack([o.quantize(w[k], q_w[k], o.S8) for k in range(w.shape[0])]), c_pad)
                b_q = np.concatenate([o.quantize(b[k:k + 1], o.bias_factor(q_in, q_w[k]), o.S32) for k in range(w.shape[0])])
            else:
                q_w = o.factor(o.maxabs(w), 7)
                w_q = _pad_c(o.quantize(w, q_w, o.S8), c_pad)
                b_q = o.quantize(b, o.bias_factor(q_in, q_w), o.S32)
            d = dict(w_q=w_q, b_q=b_q, q_w=q_w, res_scale=0.0, c_pad=c_pad)
            if L.f32_out:
                d.update(y_type=o.F32, q_y=1.0)
            elif L.residual is not None:
                q_y = final_factor(L.name)
                d.update(y_type=o.U8, q_y=q_y, res_scale=o.requant_scale(info[L.residual][1], 1.0, q_y))
            elif L.conv.relu:
                d.update(y_type=o.U8, q_y=final_factor(L.name))
            else:
                d.update(y_type=o.S8, q_y=final_factor(L.name))
            if per_channel:
                d["scale"] = np.array([o.requant_scale(q_in, qk, d["q_y"]) for qk in q_w], dtype=np.float32)
            else:
                d["scale"] = o.requant_scale(q_in, q_w, d["q_y"])
            prep[L.name] = d
            info[L.name] = (d["y_type"], d["q_y"])
        elif L.op in ("maxpool", "avgpool"):
            info[L.name] = (t_in, q_in)
        elif L.op == "concat":
            info[L.name] = (t_in, group_factor(root[L.name]))
        elif L.op == "l2norm":
            assert t_in == o.U8, "L2 normalisation follows a ReLU"
            q_y = final_factor(L.name)
            prep[L.name] = {"mult": o.l2norm_mult(L.gamma, q_in, q_y), "eps": L.eps, "q_in": q_in}
            info[L.name] = (o.U8, q_y)
        else:
            raise ValueError(L.op)
    return prep, info


def network_forward(layers, prep, info, x_f32, threads=1):
    """Quantized run; returns every tensor (quantized payloads, fp32 for dequantized outputs)."""
    first = next(L for L in layers if L.op == "conv")
    xq = o.quantize(x_f32, info["input"][1], o.S8)
    out = {"input": _pad_c(xq, prep[first.name]["c_pad"])}
    for L in layers:
        x = out[L.src[0]]
        if L.op == "conv":
            d, sp = prep[L.name], L.conv
            res = out[L.residual] if L.residual is not None else None
            out[L.name] = o.conv2d(x, d["w_q"], d["b_q"], d["scale"], sp.stride, sp.pad, sp.dil, res, d["res_scale"],
                                   sp.relu, d["y_type"], threads=threads)
        elif L.op == "maxpool":
            out[L.name] = o.pool(x, "max", L.k, L.stride, L.pad, L.ceil_mode)
        elif L.op == "avgpool":
            out[L.name] = o.pool(x, "avg", L.k, L.stride, L.pad, L.ceil_mode)
        elif L.op == "concat":
            out[L.name] = o.concat([out[s] for s in L.src], [info[s][1] for s in L.src], info[L.name][1])
        elif L.op == "l2norm":
            d = prep[L.name]
            out[L.name] = o.l2norm(x, d["q_in"], d["eps"], d["mult"])
    return out

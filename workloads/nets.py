"""Layer lists of the paper's benchmark networks with seeded random parameters, and their FP32 run.

Structure and random numbers only: none of the quantization method's arithmetic lives here.  A network
is a list of `Layer`s in execution order; every layer names its input tensor(s) and produces the tensor
called like the layer.  The FP32 run (library convolutions through torch) yields the tensors that the
calibration step samples.

Layouts: activations NHWC float32, weights KRSC float32.
"""
from dataclasses import dataclass, field
from typing import Dict, List, Optional, Tuple

import numpy as np
import torch
import torch.nn.functional as F

from .synth import ConvSpec, make_conv, normal, rng


@dataclass
class Layer:
    name: str
    op: str                      # "conv", "maxpool", "avgpool", "concat", "l2norm"
    src: List[str]               # input tensor names ("input" = network input)
    conv: Optional[ConvSpec] = None
    residual: Optional[str] = None   # tensor added to the conv output before the ReLU (fused eltwise sum)
    f32_out: bool = False        # dequantized output (logits, detection heads)
    k: Tuple[int, int] = (1, 1)  # pooling window
    stride: Tuple[int, int] = (1, 1)
    pad: Tuple[int, int] = (0, 0)
    ceil_mode: bool = False
    gamma: Optional[np.ndarray] = None   # "l2norm": per-channel scale of the normalised vector
    eps: float = 1e-10                   # "l2norm": added to the sum of squares


def _pair(v):
    return tuple(v) if isinstance(v, (tuple, list)) else (v, v)


def _conv(g, layers, name, src, C, K, R=1, S=None, stride=1, pad=0, dil=1, relu=True, bn=True, bias=False,
          residual=None, f32_out=False):
    S = R if S is None else S
    sp = make_conv(g, name, C, K, R, S, 1, 0, 1, relu, bn, bias)
    sp.stride, sp.pad, sp.dil = _pair(stride), _pair(pad), _pair(dil)
    layers.append(Layer(name, "conv", [src], conv=sp, residual=residual, f32_out=f32_out))
    return name


def resnet50(seed: int = 3000, classes: int = 1000) -> List[Layer]:
    """ResNet-50 v1 as in the original Caffe model: stride 2 sits on the first 1x1 convolution of a stage's
    first block and on its projection shortcut; 3.86 GMAC per 224x224 image."""
    g = rng(seed)
    L: List[Layer] = []
    x = _conv(g, L, "conv1", "input", 3, 64, 7, stride=2, pad=3)
    L.append(Layer("pool1", "maxpool", [x], k=(3, 3), stride=(2, 2), pad=(1, 1)))
    x, c_in = "pool1", 64
    for stage, (blocks, mid) in enumerate(zip((3, 4, 6, 3), (64, 128, 256, 512)), start=2):
        for b in range(blocks):
            tag = f"res{stage}{chr(ord('a') + b)}"
            st = 2 if (b == 0 and stage > 2) else 1
            short = x
            if b == 0:
                short = _conv(g, L, tag + "_branch1", x, c_in, mid * 4, 1, stride=st, relu=False)
            a = _conv(g, L, tag + "_branch2a", x, c_in, mid, 1, stride=st)
            bb = _conv(g, L, tag + "_branch2b", a, mid, mid, 3, pad=1)
            x = _conv(g, L, tag + "_branch2c", bb, mid, mid * 4, 1, relu=True, residual=short)
            c_in = mid * 4
    L.append(Layer("pool5", "avgpool", [x], k=(7, 7), stride=(1, 1)))
    _conv(g, L, "fc1000", "pool5", 2048, classes, 1, relu=False, bn=False, bias=True, f32_out=True)
    return L


def bottleneck_stack(seed: int = 3100, C: int = 64, blocks: int = 2) -> List[Layer]:
    """A short ResNet-like stack for quick checks: stem conv, pool, `blocks` bottlenecks (first with a
    strided projection shortcut), global pool, classifier."""
    g = rng(seed)
    L: List[Layer] = []
    x = _conv(g, L, "conv1", "input", 3, C, 3, stride=1, pad=1)
    L.append(Layer("pool1", "maxpool", [x], k=(3, 3), stride=(2, 2), pad=(1, 1)))
    x, c_in = "pool1", C
    for b in range(blocks):
        tag = f"blk{b}"
        st = 2 if b == 0 else 1
        short = x
        if b == 0:
            short = _conv(g, L, tag + "_branch1", x, c_in, C * 4, 1, stride=st, relu=False)
        a = _conv(g, L, tag + "_branch2a", x, c_in, C, 1, stride=st)
        bb = _conv(g, L, tag + "_branch2b", a, C, C, 3, pad=1)
        x = _conv(g, L, tag + "_branch2c", bb, C, C * 4, 1, relu=True, residual=short)
        c_in = C * 4
    return L


def inception_v3(seed: int = 4000, classes: int = 1000) -> List[Layer]:
    """Inception-v3 for 299x299 inputs: stem, 3 modules at 35x35, grid reduction, 4 modules with factorized
    7x7 filters at 17x17, grid reduction, 2 expanded modules at 8x8, global pool, classifier.  Every convolution
    is conv + BN + ReLU; branches meet in channel concatenations; 95 affine layers, 5.71 GMAC per image."""
    g = rng(seed)
    L: List[Layer] = []

    def cat(name, srcs):
        L.append(Layer(name, "concat", list(srcs)))
        return name

    def pool(name, src, kind, k, stride, pad=0):
        L.append(Layer(name, kind, [src], k=(k, k), stride=(stride, stride), pad=(pad, pad)))
        return name

    x = _conv(g, L, "conv1_3x3_s2", "input", 3, 32, 3, stride=2)
    x = _conv(g, L, "conv2_3x3", x, 32, 32, 3)
    x = _conv(g, L, "conv3_3x3", x, 32, 64, 3, pad=1)
    x = pool("pool1", x, "maxpool", 3, 2)
    x = _conv(g, L, "conv4_1x1", x, 64, 80, 1)
    x = _conv(g, L, "conv5_3x3", x, 80, 192, 3)
    x = pool("pool2", x, "maxpool", 3, 2)
    c = 192
    for i, pf in enumerate((32, 64, 64)):                      # 35x35 modules
        t = f"mixed{i}"
        b1 = _conv(g, L, t + "_1x1", x, c, 64, 1)
        b2 = _conv(g, L, t + "_5x5_reduce", x, c, 48, 1)
        b2 = _conv(g, L, t + "_5x5", b2, 48, 64, 5, pad=2)
        b3 = _conv(g, L, t + "_3x3_reduce", x, c, 64, 1)
        b3 = _conv(g, L, t + "_3x3_1", b3, 64, 96, 3, pad=1)
        b3 = _conv(g, L, t + "_3x3_2", b3, 96, 96, 3, pad=1)
        b4 = pool(t + "_pool", x, "avgpool", 3, 1, 1)
        b4 = _conv(g, L, t + "_pool_proj", b4, c, pf, 1)
        x, c = cat(t, (b1, b2, b3, b4)), 64 + 64 + 96 + pf
    t = "mixed3"                                                # 35 -> 17
    b1 = _conv(g, L, t + "_3x3_s2", x, c, 384, 3, stride=2)
    b2 = _conv(g, L, t + "_dbl_reduce", x, c, 64, 1)
    b2 = _conv(g, L, t + "_dbl_1", b2, 64, 96, 3, pad=1)
    b2 = _conv(g, L, t + "_dbl_2_s2", b2, 96, 96, 3, stride=2)
    b3 = pool(t + "_pool", x, "maxpool", 3, 2)
    x, c = cat(t, (b1, b2, b3)), 384 + 96 + c
    for i, c7 in enumerate((128, 160, 160, 192), start=4):     # 17x17 modules
        t = f"mixed{i}"
        b1 = _conv(g, L, t + "_1x1", x, c, 192, 1)
        b2 = _conv(g, L, t + "_7x7_reduce", x, c, c7, 1)
        b2 = _conv(g, L, t + "_1x7", b2, c7, c7, 1, 7, pad=(0, 3))
        b2 = _conv(g, L, t + "_7x1", b2, c7, 192, 7, 1, pad=(3, 0))
        b3 = _conv(g, L, t + "_dbl_reduce", x, c, c7, 1)
        b3 = _conv(g, L, t + "_dbl_7x1_1", b3, c7, c7, 7, 1, pad=(3, 0))
        b3 = _conv(g, L, t + "_dbl_1x7_1", b3, c7, c7, 1, 7, pad=(0, 3))
        b3 = _conv(g, L, t + "_dbl_7x1_2", b3, c7, c7, 7, 1, pad=(3, 0))
        b3 = _conv(g, L, t + "_dbl_1x7_2", b3, c7, 192, 1, 7, pad=(0, 3))
        b4 = pool(t + "_pool", x, "avgpool", 3, 1, 1)
        b4 = _conv(g, L, t + "_pool_proj", b4, c, 192, 1)
        x, c = cat(t, (b1, b2, b3, b4)), 768
    t = "mixed8"                                                # 17 -> 8
    b1 = _conv(g, L, t + "_3x3_reduce", x, c, 192, 1)
    b1 = _conv(g, L, t + "_3x3_s2", b1, 192, 320, 3, stride=2)
    b2 = _conv(g, L, t + "_7x7x3_reduce", x, c, 192, 1)
    b2 = _conv(g, L, t + "_7x7x3_1x7", b2, 192, 192, 1, 7, pad=(0, 3))
    b2 = _conv(g, L, t + "_7x7x3_7x1", b2, 192, 192, 7, 1, pad=(3, 0))
    b2 = _conv(g, L, t + "_7x7x3_3x3_s2", b2, 192, 192, 3, stride=2)
    b3 = pool(t + "_pool", x, "maxpool", 3, 2)
    x, c = cat(t, (b1, b2, b3)), 320 + 192 + c
    for i in (9, 10):                                           # 8x8 modules
        t = f"mixed{i}"
        b1 = _conv(g, L, t + "_1x1", x, c, 320, 1)
        r = _conv(g, L, t + "_3x3_reduce", x, c, 384, 1)
        b2 = cat(t + "_3x3", (_conv(g, L, t + "_3x3_1x3", r, 384, 384, 1, 3, pad=(0, 1)),
                              _conv(g, L, t + "_3x3_3x1", r, 384, 384, 3, 1, pad=(1, 0))))
        r = _conv(g, L, t + "_dbl_reduce", x, c, 448, 1)
        r = _conv(g, L, t + "_dbl_3x3", r, 448, 384, 3, pad=1)
        b3 = cat(t + "_dbl", (_conv(g, L, t + "_dbl_1x3", r, 384, 384, 1, 3, pad=(0, 1)),
                              _conv(g, L, t + "_dbl_3x1", r, 384, 384, 3, 1, pad=(1, 0))))
        b4 = pool(t + "_pool", x, "avgpool", 3, 1, 1)
        b4 = _conv(g, L, t + "_pool_proj", b4, c, 192, 1)
        x, c = cat(t, (b1, b2, b3, b4)), 2048
    L.append(Layer("pool3", "avgpool", [x], k=(8, 8), stride=(1, 1)))
    _conv(g, L, "fc", "pool3", 2048, classes, 1, relu=False, bn=False, bias=True, f32_out=True)
    return L


def ssd300(seed: int = 5000, classes: int = 21, l2norm: bool = False) -> List[Layer]:
    """SSD-300 on VGG-16: the base network through conv5_3 (pool3 in ceil mode, pool5 3x3 stride 1), fc6 as
    a dilated 3x3 (dilation 6), fc7 as 1x1, four extra stages, and a 3x3 localisation and confidence head on
    each of the six source maps (38, 19, 10, 5, 3, 1; 4/6/6/6/4/4 boxes per cell, 8732 boxes).  Convolutions
    carry a bias and no BN; head outputs are dequantized FP32.  l2norm: the heads of conv4_3 read its L2-normalised
    copy (scale initialised around 20, as the detector's definition has it) instead of conv4_3 itself."""
    g = rng(seed)
    L: List[Layer] = []

    def conv(name, src, C, K, R=3, **kw):
        kw.setdefault("pad", 1 if R == 3 else 0)
        return _conv(g, L, name, src, C, K, R, bn=False, bias=True, **kw)

    def pool(name, src, k, stride, pad=0, ceil_mode=False):
        L.append(Layer(name, "maxpool", [src], k=(k, k), stride=(stride, stride), pad=(pad, pad), ceil_mode=ceil_mode))
        return name

    x, c = "input", 3
    for stage, (n, k) in enumerate(((2, 64), (2, 128), (3, 256), (3, 512), (3, 512)), start=1):
        for i in range(1, n + 1):
            x, c = conv(f"conv{stage}_{i}", x, c, k), k
        if stage < 5:
            x = pool(f"pool{stage}", x, 2, 2, ceil_mode=(stage == 3))
    sources = [("conv4_3", 512, 4)]
    if l2norm:
        L.append(Layer("conv4_3_norm", "l2norm", ["conv4_3"], gamma=g.uniform(15.0, 25.0, 512).astype(np.float32)))
        sources = [("conv4_3_norm", 512, 4)]
    x = pool("pool5", x, 3, 1, 1)
    x = conv("fc6", x, 512, 1024, 3, pad=6, dil=6)
    x = conv("fc7", x, 1024, 1024, 1)
    sources.append((x, 1024, 6))
    x = conv("conv6_1", x, 1024, 256, 1)
    x = conv("conv6_2", x, 256, 512, 3, stride=2)
    sources.append((x, 512, 6))
    x = conv("conv7_1", x, 512, 128, 1)
    x = conv("conv7_2", x, 128, 256, 3, stride=2)
    sources.append((x, 256, 6))
    x = conv("conv8_1", x, 256, 128, 1)
    x = conv("conv8_2", x, 128, 256, 3, pad=0)
    sources.append((x, 256, 4))
    x = conv("conv9_1", x, 256, 128, 1)
    x = conv("conv9_2", x, 128, 256, 3, pad=0)
    sources.append((x, 256, 4))
    for src, c, boxes in sources:
        conv(src + "_mbox_loc", src, c, boxes * 4, relu=False, f32_out=True)
        conv(src + "_mbox_conf", src, c, boxes * classes, relu=False, f32_out=True)
    return L


def images(seed: int, batch: int, hw: int = 224) -> np.ndarray:
    """Seeded N(0,1) stand-ins for preprocessed images, NHWC with 3 channels."""
    return normal(rng(seed), (batch, hw, hw, 3))


def _t(a, device):
    return torch.from_numpy(np.ascontiguousarray(a)).to(device)


def fp32_forward(layers: List[Layer], x: np.ndarray, folded: Dict[str, Tuple[np.ndarray, np.ndarray]], device="cpu",
                 keep: bool = True) -> Dict[str, np.ndarray]:
    """FP32 run with BN already folded (`folded[name] = (w KRSC, b K)`).  Returns every layer output
    (NHWC); for a convolution with a fused residual also `<name>:pre`, the convolution output before the sum."""
    out: Dict[str, torch.Tensor] = {"input": _t(x, device).permute(0, 3, 1, 2)}
    res: Dict[str, np.ndarray] = {}

    def save(name, t):
        res[name] = t.permute(0, 2, 3, 1).contiguous().cpu().numpy()

    save("input", out["input"])
    with torch.no_grad():
        for L in layers:
            xin = out[L.src[0]]
            if L.op == "conv":
                sp = L.conv
                w, b = folded[L.name]
                y = F.conv2d(xin, _t(w, device).permute(0, 3, 1, 2), _t(b, device), stride=sp.stride, padding=sp.pad,
                             dilation=sp.dil)
                if L.residual is not None:
                    save(L.name + ":pre", y)
                    y = y + out[L.residual]
                if sp.relu:
                    y = torch.relu(y)
            elif L.op == "maxpool":
                y = F.max_pool2d(xin, L.k, L.stride, L.pad, ceil_mode=L.ceil_mode)
            elif L.op == "avgpool":
                y = F.avg_pool2d(xin, L.k, L.stride, L.pad, ceil_mode=L.ceil_mode, count_include_pad=True)
            elif L.op == "concat":
                y = torch.cat([out[s] for s in L.src], dim=1)
            elif L.op == "l2norm":
                y = xin / torch.sqrt((xin * xin).sum(1, keepdim=True) + L.eps) * _t(L.gamma, device).view(1, -1, 1, 1)
            else:
                raise ValueError(L.op)
            out[L.name] = y
            save(L.name, y)
    return res


def macs(layers: List[Layer], hw: int) -> int:
    """Multiply-accumulates of one image (true channel counts)."""
    size = {"input": (hw, hw)}
    total = 0
    for L in layers:
        H, W = size[L.src[0]]
        if L.op == "conv":
            sp = L.conv
            P = (H + 2 * sp.pad[0] - sp.dil[0] * (sp.R - 1) - 1) // sp.stride[0] + 1
            Q = (W + 2 * sp.pad[1] - sp.dil[1] * (sp.S - 1) - 1) // sp.stride[1] + 1
            total += P * Q * sp.K * sp.R * sp.S * sp.C
        elif L.op in ("maxpool", "avgpool"):
            def ext(h, k, s, p):
                num = h + 2 * p - k
                o = (-(-num // s) if L.ceil_mode else num // s) + 1
                if L.ceil_mode and (o - 1) * s >= h + p:
                    o -= 1
                return o
            P, Q = ext(H, L.k[0], L.stride[0], L.pad[0]), ext(W, L.k[1], L.stride[1], L.pad[1])
        else:
            P, Q = H, W
        size[L.name] = (P, Q)
    return total


# SSD-300 prior boxes (inputs of the detection output step, fixed by the detector's published configuration, not by
# the quantization method): six source maps, per cell one box of the minimum size, one of sqrt(min * max), and two
# per extra aspect ratio; centres at (cell + 0.5) * step / 300.
SSD300_MAPS = (38, 19, 10, 5, 3, 1)
SSD300_STEPS = (8, 16, 32, 64, 100, 300)
SSD300_MIN = (30, 60, 111, 162, 213, 264)
SSD300_MAX = (60, 111, 162, 213, 264, 315)
SSD300_RATIOS = ((2,), (2, 3), (2, 3), (2, 3), (2,), (2,))
SSD300_VARIANCES = (0.1, 0.1, 0.2, 0.2)


def ssd300_priors() -> np.ndarray:
    """[8732, 4] fp32 (cx, cy, w, h) in units of the image side, in the order of the head outputs: source map,
    row, column, box."""
    rows = []
    for fm, step, smin, smax, ratios in zip(SSD300_MAPS, SSD300_STEPS, SSD300_MIN, SSD300_MAX, SSD300_RATIOS):
        sizes = [(smin / 300.0, smin / 300.0), ((smin * smax) ** 0.5 / 300.0,) * 2]
        for r in ratios:
            sizes.append((smin / 300.0 * r ** 0.5, smin / 300.0 / r ** 0.5))
            sizes.append((smin / 300.0 / r ** 0.5, smin / 300.0 * r ** 0.5))
        for i in range(fm):
            for j in range(fm):
                cx, cy = (j + 0.5) * step / 300.0, (i + 0.5) * step / 300.0
                rows.extend((cx, cy, w, h) for w, h in sizes)
    return np.asarray(rows, dtype=np.float32)


def detection_inputs(seed: int, batch: int, priors: int = 8732, classes: int = 21, peaked: float = 0.02):
    """Seeded stand-ins for the head outputs of a detector: localisation offsets N(0, 1) and class logits N(0, 1)
    with a fraction `peaked` of the boxes given one strongly preferred class (confident detections), the rest
    mostly background.  Returns (loc [N, P, 4], conf [N, P, classes])."""
    g = rng(seed)
    loc = normal(g, (batch, priors, 4))
    conf = normal(g, (batch, priors, classes))
    conf[..., 0] += 8.0                                         # background dominates, as in a trained detector:
    #                                                             a few boxes per class and image pass a 0.01 threshold
    hot = g.random((batch, priors)) < peaked
    cls = g.integers(1, classes, (batch, priors))
    n_idx, p_idx = np.nonzero(hot)
    conf[n_idx, p_idx, cls[n_idx, p_idx]] += g.uniform(4.0, 9.0, n_idx.size).astype(np.float32)
    return loc.astype(np.float32), conf.astype(np.float32)

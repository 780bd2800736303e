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
    op: str                      # "conv", "maxpool", "avgpool", "concat"
    src: List[str]               # input tensor names ("input" = network input)
    conv: Optional[ConvSpec] = None
    residual: Optional[str] = None   # tensor added to the conv output before the ReLU (fused eltwise sum)
    f32_out: bool = False        # dequantized output (logits, detection heads)
    k: Tuple[int, int] = (1, 1)  # pooling window
    stride: Tuple[int, int] = (1, 1)
    pad: Tuple[int, int] = (0, 0)
    ceil_mode: bool = False


def _conv(g, layers, name, src, C, K, R=1, S=None, stride=1, pad=0, dil=1, relu=True, bn=True, bias=False,
          residual=None, f32_out=False):
    S = R if S is None else S
    sp = make_conv(g, name, C, K, R, S, stride, pad, dil, relu, bn, bias)
    if isinstance(pad, tuple):
        sp.pad = pad
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

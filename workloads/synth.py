"""Seeded generators for the benchmark configurations and the FP32 model run.

Layouts: activations NHWC, weights KRSC (Cout, R, S, Cin), all float32.
The paper measures throughput on fake random data and calibrates on dataset
images; here seeded normal tensors of the same shapes stand in for both.
"""
from dataclasses import dataclass, field
from typing import List, Optional, Tuple

import numpy as np
import torch
import torch.nn.functional as F


def rng(seed: int) -> np.random.Generator:
    return np.random.default_rng(seed)


def normal(g, shape, std=1.0, mean=0.0):
    return (g.standard_normal(shape, dtype=np.float32) * np.float32(std) + np.float32(mean)).astype(np.float32)


def uniform(g, shape, lo, hi):
    return (g.random(shape, dtype=np.float32) * np.float32(hi - lo) + np.float32(lo)).astype(np.float32)


def relu_normal(g, shape):
    return np.maximum(normal(g, shape), np.float32(0))


@dataclass
class ConvSpec:
    """One affine layer of the FP32 model (before BN folding)."""
    name: str
    C: int
    K: int
    R: int = 1
    S: int = 1
    stride: Tuple[int, int] = (1, 1)
    pad: Tuple[int, int] = (0, 0)
    dil: Tuple[int, int] = (1, 1)
    relu: bool = True
    bn: bool = True
    w: Optional[np.ndarray] = None       # KRSC fp32
    b: Optional[np.ndarray] = None       # K fp32 (conv bias, may be None when bn)
    gamma: Optional[np.ndarray] = None
    beta: Optional[np.ndarray] = None
    mean: Optional[np.ndarray] = None
    var: Optional[np.ndarray] = None


def he_weights(g, K, R, S, C):
    return normal(g, (K, R, S, C), std=float(np.sqrt(2.0 / (R * S * C))))


def bn_params(g, K):
    """gamma ~ U(0.5,1.5), beta ~ N(0,0.1), running mean ~ N(0,0.1), var ~ U(0.5,1.5)."""
    return dict(gamma=uniform(g, (K,), 0.5, 1.5), beta=normal(g, (K,), 0.1),
                mean=normal(g, (K,), 0.1), var=uniform(g, (K,), 0.5, 1.5))


def make_conv(g, name, C, K, R=1, S=1, stride=1, pad=0, dil=1, relu=True, bn=True, bias=False):
    sp = ConvSpec(name, C, K, R, S, (stride, stride), (pad, pad), (dil, dil), relu, bn)
    sp.w = he_weights(g, K, R, S, C)
    if bias:
        sp.b = normal(g, (K,), 0.01)
    if bn:
        for k, v in bn_params(g, K).items():
            setattr(sp, k, v)
    return sp


# --------------------------------------------------------------------------------------
# FP32 model run (library convolution).  Takes FOLDED weights: calibration follows
# the model optimisation steps, as in the paper's workflow figure.
# --------------------------------------------------------------------------------------
def fp32_conv(x_nhwc: np.ndarray, w_krsc: np.ndarray, b: Optional[np.ndarray], stride=(1, 1), pad=(0, 0),
              dil=(1, 1), device="cpu") -> np.ndarray:
    xt = torch.from_numpy(np.ascontiguousarray(x_nhwc)).to(device).permute(0, 3, 1, 2)
    wt = torch.from_numpy(np.ascontiguousarray(w_krsc)).to(device).permute(0, 3, 1, 2)
    bt = torch.from_numpy(b).to(device) if b is not None else None
    with torch.no_grad():
        y = F.conv2d(xt, wt, bt, stride=stride, padding=pad, dilation=dil)
    return y.permute(0, 2, 3, 1).contiguous().cpu().numpy()


# --------------------------------------------------------------------------------------
# Config 1: a single 3x3 layer, 1x14x14x64 -> 64, seed 0.
# --------------------------------------------------------------------------------------
def config1(seed: int = 0, N=1, H=14, W=14, C=64, K=64):
    g = rng(seed)
    x = relu_normal(g, (N, H, W, C))
    sp = ConvSpec("conv", C, K, 3, 3, (1, 1), (1, 1), (1, 1), relu=True, bn=False)
    sp.w = normal(g, (K, 3, 3, C), std=0.05)
    sp.b = normal(g, (K,), std=0.01)
    return dict(x=x, conv=sp)


# --------------------------------------------------------------------------------------
# Config 2: ResNet-50 bottleneck, 56x56x256 input, 1x1 256->64, 3x3 64->64, 1x1 64->256,
# BN on each, identity residual.  `calib` seeded calibration batches + one test batch.
# --------------------------------------------------------------------------------------
def config2(seed: int = 2000, batch: int = 32, H: int = 56, W: int = 56, C: int = 256, mid: int = 64,
            calib_batches: int = 4, calib_batch: Optional[int] = None):
    g = rng(seed)
    a = make_conv(g, "branch2a", C, mid, 1, 1, relu=True)
    b = make_conv(g, "branch2b", mid, mid, 3, 3, pad=1, relu=True)
    c = make_conv(g, "branch2c", mid, C, 1, 1, relu=False)
    cb = calib_batch or batch
    calib = [relu_normal(rng(seed + 10 + i), (cb, H, W, C)) for i in range(calib_batches)]
    x = relu_normal(rng(seed + 1), (batch, H, W, C))
    return dict(convs=[a, b, c], calib=calib, x=x)


def bottleneck_fp32(x, folded, device="cpu"):
    """FP32 run of the (BN-folded) bottleneck.  folded = [(w,b)]*3.  Returns every tensor that calibration samples."""
    (wa, ba), (wb, bb), (wc, bc) = folded
    a = np.maximum(fp32_conv(x, wa, ba, device=device), 0)
    b = np.maximum(fp32_conv(a, wb, bb, pad=(1, 1), device=device), 0)
    c = fp32_conv(b, wc, bc, device=device)
    y = np.maximum(c + x, 0)
    return dict(x=x, a=a, b=b, c=c, y=y)

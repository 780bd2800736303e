"""Host-side preparation of quantized layers on top of the C ABI.

Follows the paper's workflow: fold BN into the FP32 weights, calibrate max-abs factors on sample
tensors, quantize weights (p = 7, s8) and bias (int32 at q_x * q_w), and derive the single
requantisation multiplier of each layer.  All tensor arithmetic happens in the library's kernels;
this module only sequences calls and keeps the per-tensor factors (host floats).
"""
from dataclasses import dataclass
from typing import Dict, Optional, Tuple

import torch

from . import binding as q8


class Calibrator:
    """Running max-abs of named tensors over calibration batches; one device->host copy at the end."""

    def __init__(self, names, device="cuda"):
        self.names = list(names)
        self.slots = torch.zeros(len(self.names), dtype=torch.float32, device=device)
        self.index = {n: i for i, n in enumerate(self.names)}

    def observe(self, name, x):
        i = self.index[name]
        q8.q8_calibrate_maxabs(x, self.slots[i:i + 1])

    def maxima(self) -> Dict[str, float]:
        host = self.slots.cpu().tolist()
        return {n: host[i] for n, i in self.index.items()}


def tensor_maxabs(x) -> float:
    slot = torch.zeros(1, dtype=torch.float32, device=x.device)
    q8.q8_calibrate_maxabs(x, slot)
    return float(slot.item())


@dataclass
class QuantConv:
    """One quantized affine layer ready to run: s8 weights, s32 bias, device scale, descriptor."""
    desc: q8.q8_conv_desc
    w_q: torch.Tensor
    b_q: Optional[torch.Tensor]
    scale: torch.Tensor
    q_w: object  # float, or a list of K floats with per-channel factors
    q_x: float
    q_y: float
    res_scale: float = 0.0

    def __call__(self, x_q, residual=None, out=None):
        return q8.q8_conv2d(self.desc, x_q, self.w_q, self.b_q, self.scale, residual, self.res_scale, out)


def prepare_conv(w, b, in_shape, q_x, q_y, x_type=q8.Q8_U8, y_type=q8.Q8_U8, relu=True, stride=(1, 1), pad=(0, 0),
                 dil=(1, 1), q_res=None, res_type=q8.Q8_U8, y_ldc=0, y_c_offset=0, algo=q8.Q8_ALGO_AUTO,
                 per_channel=False) -> QuantConv:
    """w: folded FP32 weights KRSC on the device, b: folded FP32 bias [K] or None.

    q_y is the output factor; for y_type F32 the layer dequantizes (q_y is taken as 1).
    per_channel: one weight factor per output channel (max|w[k]| / 127) instead of the paper's one per tensor;
    the bias and the requantisation multiplier then carry the factor of their channel.
    """
    N, H, W, Cin = in_shape
    K, R, S, C2 = w.shape
    assert C2 == Cin
    if y_type == q8.Q8_F32:
        q_y = 1.0
    b_q = None
    if per_channel:
        slots = torch.zeros(K, dtype=torch.float32, device=w.device)
        q8.q8_calibrate_maxabs_rows(w, slots)
        q_w = [q8.q8_factor(m, 7) for m in slots.cpu().tolist()]
        w_q = q8.q8_quantize_rows(w, torch.tensor(q_w, dtype=torch.float32, device=w.device), q8.Q8_S8)
        if b is not None:
            q_b = torch.tensor([q8.q8_bias_factor(q_x, qk) for qk in q_w], dtype=torch.float32, device=w.device)
            b_q = q8.q8_quantize_rows(b.reshape(K, 1).contiguous(), q_b, q8.Q8_S32).reshape(K)
        scale = torch.tensor([q8.q8_requant_scale(q_x, qk, q_y) for qk in q_w], dtype=torch.float32, device=w.device)
    else:
        q_w = q8.q8_factor(tensor_maxabs(w), 7)
        w_q = q8.q8_quantize(w, q_w, q8.Q8_S8)
        if b is not None:
            b_q = q8.q8_quantize(b, q8.q8_bias_factor(q_x, q_w), q8.Q8_S32)
        scale = torch.tensor([q8.q8_requant_scale(q_x, q_w, q_y)], dtype=torch.float32, device=w.device)
    res_scale = q8.q8_requant_scale(q_res, 1.0, q_y) if q_res is not None else 0.0
    desc = q8.make_conv_desc(N, H, W, Cin, K, R, S, stride, pad, dil, x_type, res_type, y_type, relu,
                             K if per_channel else 1, y_ldc, y_c_offset, algo)
    return QuantConv(desc, w_q, b_q, scale, q_w, q_x, q_y, res_scale)


def fused_pair(first: QuantConv, second: QuantConv, x_q, residual=None, out=None):
    """`first` followed by the 1x1 layer `second` in one launch; the tensor between them is never written."""
    return q8.q8_conv2d_then_1x1(first.desc, second.desc, x_q, first.w_q, first.b_q, first.scale, second.w_q, second.b_q,
                                 second.scale, residual, second.res_scale, out)


class Bottleneck:
    """ResNet bottleneck (1x1 -> 3x3 -> 1x1 + identity residual, ReLU fused everywhere) in int8.

    folded: [(w,b)] * 3 FP32 device tensors; maxima: calibrated max-abs of x, a, b, c (pre-sum conv
    output).  The output factor follows the "+" rule on a common p = 8 footing:
    q_y = max(max|c|, max|x|) / 255.
    """

    def __init__(self, folded, maxima, in_shape, algo=q8.Q8_ALGO_AUTO, fuse=True):
        """fuse: run the 3x3 and the expanding 1x1 as one launch (q8_conv2d_then_1x1) when the library supports the
        pair; the result is the same bit for bit, the 3x3 output is then never written (self.yb stays unused)."""
        N, H, W, C = in_shape
        (wa, ba), (wb, bb), (wc, bc) = folded
        mid = wa.shape[0]
        self.q_x = q8.q8_factor(maxima["x"], 8)
        self.q_a = q8.q8_factor(maxima["a"], 8)
        self.q_b = q8.q8_factor(maxima["b"], 8)
        self.q_y = q8.q8_factor(max(maxima["c"], maxima["x"]), 8)
        self.a = prepare_conv(wa, ba, (N, H, W, C), self.q_x, self.q_a, relu=True, algo=algo)
        self.b = prepare_conv(wb, bb, (N, H, W, mid), self.q_a, self.q_b, relu=True, pad=(1, 1), algo=algo)
        self.c = prepare_conv(wc, bc, (N, H, W, mid), self.q_b, self.q_y, relu=True, q_res=self.q_x, algo=algo)
        self.ya = torch.empty((N, H, W, mid), dtype=torch.uint8, device=wa.device)
        self.yb = torch.empty((N, H, W, mid), dtype=torch.uint8, device=wa.device)
        self.fused = bool(fuse) and algo == q8.Q8_ALGO_AUTO and q8.q8_conv2d_then_1x1_supported(self.b.desc, self.c.desc)

    def __call__(self, x_q, out=None):
        self.a(x_q, out=self.ya)
        if self.fused:
            return fused_pair(self.b, self.c, self.ya, residual=x_q, out=out)
        self.b(self.ya, out=self.yb)
        return self.c(self.yb, residual=x_q, out=out)


def sync_maxima(maxima: Dict[str, float], device=None) -> Dict[str, float]:
    """Element-wise MAX of the calibration maxima over all ranks of the default process group.

    The only exchange the data-parallel path needs: with replicated weights and images sharded over
    GPUs, equal factors on every rank keep the outputs independent of the GPU count.  Returns the
    input unchanged when no process group is initialised.  `device`: CUDA device for NCCL, None for
    a CPU (gloo) group.
    """
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return dict(maxima)
    names = sorted(maxima)
    t = torch.tensor([maxima[n] for n in names], dtype=torch.float32, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    vals = t.cpu().tolist()
    return {n: v for n, v in zip(names, vals)}


def shard_batch(n_images: int, rank: int, world: int) -> Tuple[int, int]:
    """Contiguous [begin, end) slice of a batch owned by `rank` (images are independent units)."""
    base, extra = divmod(n_images, world)
    begin = rank * base + min(rank, extra)
    return begin, begin + base + (1 if rank < extra else 0)

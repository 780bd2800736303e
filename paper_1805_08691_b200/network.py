"""Whole quantized networks on top of the C ABI: a layer list (workloads.nets) becomes a sequence of
q8_conv2d / pooling / concat calls on preallocated device tensors.

Host logic only: per-tensor factors follow the paper's calibration rule (max-abs / (2^p - 1)) and its "+" rule
for the fused residual sum; all tensor arithmetic runs in the library's kernels.

  network input (signed)            : s8, q = max|x| / 127, 3 channels zero padded to 16
  conv + ReLU                       : u8, q = max / 255
  conv without ReLU                 : s8, q = max|y| / 127
  conv + residual sum + ReLU        : u8, q = max(max|conv|, max|residual|) / 255
  dequantized output (logits, heads): fp32
  pooling                           : type and factor of its input;  concat: largest branch factor
"""
from typing import Dict, List

import torch
import torch.nn.functional as F

from . import binding as q8
from . import pipeline


class QuantNetwork:
    def __init__(self, layers, folded: Dict[str, tuple], maxima: Dict[str, float], in_shape, device="cuda"):
        """folded[name] = (w KRSC, b K) FP32 device tensors; maxima: calibrated max-abs of "input", every layer
        output and "<name>:pre" of residual convolutions; in_shape = (N, H, W, 3)."""
        self.layers = layers
        self.info = {"input": (q8.Q8_S8, q8.q8_factor(maxima["input"], 7))}
        self.shape = {}
        self.convs: Dict[str, pipeline.QuantConv] = {}
        self.bufs: Dict[str, torch.Tensor] = {}
        N, H, W, _ = in_shape
        first = next(L for L in layers if L.op == "conv")
        self.c_pad_in = -(-first.conv.C // 16) * 16
        self.shape["input"] = (N, H, W, self.c_pad_in)
        self.bufs["input"] = torch.empty(self.shape["input"], dtype=torch.int8, device=device)
        ws_bytes = 0
        for L in layers:
            t_in, q_in = self.info[L.src[0]]
            n, h, w_, c = self.shape[L.src[0]]
            if L.op == "conv":
                sp = L.conv
                wf, bf = folded[L.name]
                if wf.shape[-1] != c:  # zero padded input channels: exact under a symmetric quantizer
                    wf = F.pad(wf, (0, c - wf.shape[-1]))
                if L.f32_out:
                    y_type, q_y = q8.Q8_F32, 1.0
                elif L.residual is not None:
                    y_type = q8.Q8_U8
                    q_y = q8.q8_factor(max(maxima[L.name + ":pre"], maxima[L.residual]), 8)
                elif sp.relu:
                    y_type, q_y = q8.Q8_U8, q8.q8_factor(maxima[L.name], 8)
                else:
                    y_type, q_y = q8.Q8_S8, q8.q8_factor(maxima[L.name], 7)
                q_res, res_type = None, q8.Q8_U8
                if L.residual is not None:
                    res_type, q_res = self.info[L.residual]
                qc = pipeline.prepare_conv(wf.contiguous(), bf, (n, h, w_, c), q_in, q_y, t_in, y_type, sp.relu, sp.stride,
                                           sp.pad, sp.dil, q_res, res_type)
                self.convs[L.name] = qc
                P, Q = q8.conv_out_shape(qc.desc)
                self.shape[L.name] = (n, P, Q, sp.K)
                self.info[L.name] = (y_type, qc.q_y)
                ws_bytes = max(ws_bytes, q8.q8_conv2d_workspace_bytes(qc.desc))
            elif L.op in ("maxpool", "avgpool"):
                P = q8.q8_pool_out_extent(h, L.k[0], L.stride[0], L.pad[0], L.ceil_mode)
                Q = q8.q8_pool_out_extent(w_, L.k[1], L.stride[1], L.pad[1], L.ceil_mode)
                self.shape[L.name] = (n, P, Q, c)
                self.info[L.name] = (t_in, q_in)
            elif L.op == "concat":
                self.shape[L.name] = (n, h, w_, sum(self.shape[s][3] for s in L.src))
                self.info[L.name] = (t_in, max(self.info[s][1] for s in L.src))
            else:
                raise ValueError(L.op)
            self.bufs[L.name] = torch.empty(self.shape[L.name], dtype=q8.TORCH_DTYPES[self.info[L.name][0]], device=device)
        self.workspace = torch.empty(max(ws_bytes, 16), dtype=torch.uint8, device=device) if ws_bytes else None

    def forward(self, x_f32: torch.Tensor) -> Dict[str, torch.Tensor]:
        """Enqueues the whole network on the current stream; returns the tensors (views of preallocated buffers)."""
        q8.q8_quantize_pad_channels(x_f32, self.c_pad_in, self.info["input"][1], q8.Q8_S8, out=self.bufs["input"])
        self.run_quantized()
        return self.bufs

    def run_quantized(self):
        """Everything after the input quantization (the part a CUDA graph replays)."""
        b = self.bufs
        for L in self.layers:
            x = b[L.src[0]]
            if L.op == "conv":
                qc = self.convs[L.name]
                res = b[L.residual] if L.residual is not None else None
                q8.q8_conv2d(qc.desc, x, qc.w_q, qc.b_q, qc.scale, res, qc.res_scale, b[L.name], self.workspace)
            elif L.op == "maxpool":
                q8.q8_maxpool2d(x, L.k, L.stride, L.pad, L.ceil_mode, out=b[L.name])
            elif L.op == "avgpool":
                q8.q8_avgpool2d(x, L.k, L.stride, L.pad, L.ceil_mode, out=b[L.name])
            elif L.op == "concat":
                q8.q8_concat([b[s] for s in L.src], [self.info[s][1] for s in L.src], self.info[L.name][1], out=b[L.name])

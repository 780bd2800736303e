"""Whole quantized networks on top of the C ABI: a layer list (workloads.nets) becomes a sequence of
q8_conv2d / pooling / concat calls on preallocated device tensors.

Host logic only: per-tensor factors follow the paper's calibration rule (max-abs / (2^p - 1)) and its "+" rule
for the fused residual sum; all tensor arithmetic runs in the library's kernels.

  network input (signed)            : s8, q = max|x| / 127, 3 channels zero padded to 16; an odd image width is
                                      padded with one zero column when the first layer has stride 2 and the column
                                      adds no output (the kernel reads stride-2 inputs as pixel pairs)
  conv + ReLU                       : u8, q = max / 255
  conv without ReLU                 : s8, q = max|y| / 127
  conv + residual sum + ReLU        : u8, q = max(max|conv|, max|residual|) / 255 (the paper's "+" rule), or with
                                      sum_policy="post_sum" the calibrated maximum of the sum itself / 255
  dequantized output (logits, heads): fp32
  sibling heads                     : dequantized convolutions that read the same tensor with the same filter
                                      geometry (the localisation and confidence heads of an SSD source map) run as
                                      ONE convolution over the concatenated output channels with per-channel
                                      multipliers and biases (each channel keeps its own layer's factors, so
                                      every value is the one the separate layers give); the layers' outputs are
                                      channel slices of its result
  channel padding                   : a convolution output with a channel count that is not a multiple of 32 and is
                                      read only by convolutions lives in a buffer padded with zero channels (to 64,
                                      128 or the next multiple of 32), and its readers get zero weights there: exact,
                                      and the readers' TMA rows start on 32-byte boundaries (48- and 80-byte rows
                                      load up to 2.5x slower)
  pooling                           : type and factor of its input
  concat                            : one factor for the whole output, the largest factor among its branches.  A
                                      conv + ReLU read by nothing but the concat writes its channel slice of the
                                      concat buffer itself, quantized at that factor; other branches (pooled
                                      tensors) are re-expressed and copied in by q8_concat_branch; a concat nested
                                      in another is a slice of the outer buffer and shares its factor
"""
from typing import Dict, List

import numpy as np
import torch
import torch.nn.functional as F

from . import binding as q8
from . import pipeline


class QuantNetwork:
    def __init__(self, layers, folded: Dict[str, tuple], maxima: Dict[str, float], in_shape, device="cuda",
                 per_channel=False, streams=1, fuse=True, sum_policy="max"):
        """folded[name] = (w KRSC, b K) FP32 device tensors; maxima: calibrated max-abs of "input", every layer
        output and "<name>:pre" of residual convolutions; in_shape = (N, H, W, 3); per_channel: one weight
        factor per output channel instead of one per tensor; streams: independent branches (the
        branches of an Inception module, a projection shortcut beside its residual branch, detection heads beside
        the trunk) are enqueued on up to this many CUDA streams, so that one branch's kernels start on SMs that
        another branch's kernel has already left.  fuse: a convolution whose only reader is a 1x1 convolution runs
        with it in one launch where the library supports the pair (q8_conv2d_then_1x1: same bytes, the tensor between
        them is not written, so it is absent from the returned tensors)."""
        assert sum_policy in ("max", "post_sum")
        self.sum_policy = sum_policy
        self.layers = layers
        self.maxima = maxima
        self.by_name = {L.name: L for L in layers}
        self.convs: Dict[str, pipeline.QuantConv] = {}
        self.l2: Dict[str, tuple] = {}   # L2 normalisation layers: (input factor, eps, per-channel multipliers)
        self.bufs: Dict[str, torch.Tensor] = {}
        N, H, W, _ = in_shape
        first = next(L for L in layers if L.op == "conv")
        self.c_pad_in = -(-first.conv.C // 16) * 16
        self.uses: Dict[str, List] = {}
        for L in layers:
            for s in L.src + ([L.residual] if L.residual else []):
                self.uses.setdefault(s, []).append(L)
        self.w_pad_in = W
        sp0 = first.conv
        if first.src == ["input"] and sp0.stride[1] == 2 and W % 2 == 1 and sp0.dil[1] == 1:
            q_of = lambda w: (w + 2 * sp0.pad[1] - (sp0.S - 1) - 1) // 2 + 1
            if q_of(W + 1) == q_of(W) and all(L is first or "input" not in L.src for L in layers):
                self.w_pad_in = W + 1
        self._shapes((N, H, self.w_pad_in, self.c_pad_in))
        self._place_concats()
        self._factors = {}
        self.info = {"input": (q8.Q8_S8, self._factor("input"))}
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
                else:
                    y_type, q_y = (q8.Q8_U8 if (sp.relu or L.residual is not None) else q8.Q8_S8), self._factor(L.name)
                q_res, res_type = None, q8.Q8_U8
                if L.residual is not None:
                    res_type, q_res = self.info[L.residual]
                ldc, off = 0, 0
                if L.name in self.in_place:
                    root, off = self.slot[L.name]
                    ldc = self.shape[root][3]
                elif self.shape[L.name][3] != sp.K:
                    ldc = self.shape[L.name][3]  # padded with zero channels
                qc = pipeline.prepare_conv(wf.contiguous(), bf, (n, h, w_, c), q_in, q_y, t_in, y_type, sp.relu, sp.stride,
                                           sp.pad, sp.dil, q_res, res_type, ldc, off, per_channel=per_channel)
                self.convs[L.name] = qc
                self.info[L.name] = (y_type, qc.q_y)
                ws_bytes = max(ws_bytes, q8.q8_conv2d_workspace_bytes(qc.desc))
            elif L.op in ("maxpool", "avgpool"):
                self.info[L.name] = (t_in, q_in)
            elif L.op == "concat":
                self.info[L.name] = (t_in, self._factor(L.name))
            elif L.op == "l2norm":
                if t_in != q8.Q8_U8:
                    raise ValueError("L2 normalisation needs unsigned codes (it follows a ReLU)")
                q_y = self._factor(L.name)
                # gamma q_x / q_y formed in fp64 (a multiply, a division) and rounded once, per channel
                mult = ((np.asarray(L.gamma, dtype=np.float64) * np.float64(q_in)) / np.float64(q_y)).astype(np.float32)
                self.l2[L.name] = (float(q_in), float(L.eps), torch.from_numpy(mult).to(device))
                self.info[L.name] = (q8.Q8_U8, q_y)
            else:
                raise ValueError(L.op)
            dt = q8.TORCH_DTYPES[self.info[L.name][0]]
            if L.name in self.in_place or (L.op == "concat" and self.slot[L.name][0] != L.name):
                continue  # a slice of the outermost concat's buffer, bound below
            padded = L.op == "conv" and self.shape[L.name][3] != L.conv.K
            self.bufs[L.name] = (torch.zeros if padded else torch.empty)(self.shape[L.name], dtype=dt, device=device)
        for name, (root, off) in self.slot.items():
            if name in self.in_place or (self.by_name[name].op == "concat" and root != name):
                self.bufs[name] = self.bufs[root][..., off:off + self.shape[name][3]]
        ws_bytes = max(ws_bytes, self._merge_sibling_heads(device))
        self._pair_layers(bool(fuse))
        self._assign_streams(max(1, int(streams)))
        # split-K scratch: one per stream, layers on different streams may run at the same time
        self.workspaces = [torch.empty(max(ws_bytes, 16), dtype=torch.uint8, device=device) if ws_bytes else None
                           for _ in range(self.n_streams)]
        self.side_streams = [torch.cuda.Stream(device=device) for _ in range(self.n_streams - 1)]
        # what a caller sees: every tensor with its own channel count (padding channels cut off)
        self.outputs = {k: v for k, v in self.bufs.items()}
        for L in layers:
            if L.op == "conv" and L.name in self.bufs and self.bufs[L.name].shape[-1] != L.conv.K and L.name not in self.slot:
                self.outputs[L.name] = self.bufs[L.name][..., :L.conv.K]
        for first in self.fused_with:   # the tensor between two layers of one launch is never written
            self.outputs.pop(first, None)

    # ---- host bookkeeping ---------------------------------------------------------------------------
    def _shapes(self, in_shape):
        self.shape = {"input": in_shape}
        for L in self.layers:
            n, h, w_, c = self.shape[L.src[0]]
            if L.op == "conv":
                sp = L.conv
                P = (h + 2 * sp.pad[0] - sp.dil[0] * (sp.R - 1) - 1) // sp.stride[0] + 1
                Q = (w_ + 2 * sp.pad[1] - sp.dil[1] * (sp.S - 1) - 1) // sp.stride[1] + 1
                k_out = sp.K
                readers = self.uses.get(L.name, [])
                if (sp.K > 32 and sp.K % 32 and not L.f32_out and readers
                        and all(r.op == "conv" and r.src == [L.name] and r.residual != L.name for r in readers)):
                    k_out = 64 if sp.K <= 64 else (128 if sp.K <= 128 else -(-sp.K // 32) * 32)
                self.shape[L.name] = (n, P, Q, k_out)
            elif L.op in ("maxpool", "avgpool"):
                P = q8.q8_pool_out_extent(h, L.k[0], L.stride[0], L.pad[0], L.ceil_mode)
                Q = q8.q8_pool_out_extent(w_, L.k[1], L.stride[1], L.pad[1], L.ceil_mode)
                self.shape[L.name] = (n, P, Q, c)
            elif L.op == "concat":
                self.shape[L.name] = (n, h, w_, sum(self.shape[s][3] for s in L.src))
            elif L.op == "l2norm":
                self.shape[L.name] = (n, h, w_, c)
            else:
                raise ValueError(L.op)

    def _place_concats(self):
        """slot[name] = (outermost concat, channel offset) for every tensor that is part of a concat;
        in_place = the convolutions that write their slice themselves; members[root] = all non-concat parts."""
        uses = self.uses
        self.slot, self.in_place, self.members = {}, set(), {}

        def place(cat, root, base):
            self.slot[cat.name] = (root, base)
            for s in cat.src:
                Ls = self.by_name[s]
                self.slot[s] = (root, base)
                if Ls.op == "concat":
                    place(Ls, root, base)
                else:
                    self.members.setdefault(root, []).append(s)
                    if (Ls.op == "conv" and Ls.conv.relu and Ls.residual is None and not Ls.f32_out
                            and len(uses[s]) == 1):
                        self.in_place.add(s)
                base += self.shape[s][3]

        for L in self.layers:
            u = uses.get(L.name, [])
            if L.op == "concat" and not (len(u) == 1 and u[0].op == "concat"):
                place(L, L.name, 0)

    def _factor(self, name):
        """Output factor of a tensor under the rules in the module docstring."""
        if name in self._factors:
            return self._factors[name]
        if name in self.in_place or (name in self.slot and self.by_name[name].op == "concat"):
            q = max(self._own_factor(m) for m in self.members[self.slot[name][0]])
        else:
            q = self._own_factor(name)
        self._factors[name] = q
        return q

    def _own_factor(self, name):
        m = self.maxima
        if name == "input":
            return q8.q8_factor(m["input"], 7)
        L = self.by_name[name]
        if L.op in ("maxpool", "avgpool"):
            return self._factor(L.src[0])
        if L.op == "concat":
            return self._factor(name)
        if L.op == "l2norm":
            return q8.q8_factor(m[name], 8)
        if L.residual is not None and self.sum_policy == "post_sum":
            return q8.q8_factor(m[name], 8)       # calibrated on the tensor the layer emits
        if L.residual is not None:
            return q8.q8_factor(max(m[name + ":pre"], m[L.residual]), 8)
        return q8.q8_factor(m[name], 8 if L.conv.relu else 7)

    def _merge_sibling_heads(self, device):
        """Groups of FP32-output convolutions on one input with one geometry become one launch (see the module
        docstring).  merged[leader] = member names; self.skip = the members that no longer launch."""
        self.merged, self.skip = {}, set()
        ws_bytes = 0
        groups = {}
        for L in self.layers:
            if L.op == "conv" and L.f32_out and L.residual is None and L.name not in self.slot and not self.uses.get(L.name):
                sp = L.conv
                key = (L.src[0], sp.R, sp.S, tuple(sp.stride), tuple(sp.pad), tuple(sp.dil), bool(sp.relu))
                groups.setdefault(key, []).append(L.name)
        for names in groups.values():
            if len(names) < 2:
                continue
            parts = [self.convs[n] for n in names]
            ks = [int(qc.w_q.shape[0]) for qc in parts]
            K = sum(ks)
            d0 = parts[0].desc
            w_q = torch.cat([qc.w_q for qc in parts], dim=0).contiguous()
            b_q = torch.cat([qc.b_q if qc.b_q is not None else torch.zeros(k, dtype=torch.int32, device=device)
                             for qc, k in zip(parts, ks)]).contiguous()
            scale = torch.cat([qc.scale if qc.scale.numel() == k else qc.scale.expand(k) for qc, k in zip(parts, ks)]).contiguous()
            desc = q8.make_conv_desc(d0.N, d0.H, d0.W, d0.C, K, d0.R, d0.S, (d0.stride_h, d0.stride_w), (d0.pad_h, d0.pad_w),
                                     (d0.dil_h, d0.dil_w), d0.x_type, d0.res_type, q8.Q8_F32, bool(d0.relu), K, 0, 0)
            leader = names[0]
            self.convs[leader] = pipeline.QuantConv(desc, w_q, b_q, scale, None, parts[0].q_x, 1.0, 0.0)
            n, P, Q, _ = self.shape[leader]
            buf = torch.empty((n, P, Q, K), dtype=torch.float32, device=device)
            off = 0
            for name, k in zip(names, ks):
                self.bufs[name] = buf[..., off:off + k]
                off += k
            self.bufs[leader + ":merged"] = buf
            self.merged[leader] = names
            self.skip.update(names[1:])
            ws_bytes = max(ws_bytes, q8.q8_conv2d_workspace_bytes(desc))
        return ws_bytes

    def _pair_layers(self, fuse):
        """fused_with[first] = second for every convolution pair that runs as one launch: `second` is a 1x1
        convolution, the only reader of `first`, neither writes a concat slice or a padded tensor, `second` does not
        take `first` as its residual, and the library accepts the pair."""
        self.fused_with, self.fused_second = {}, set()
        if not fuse:
            return
        for L in self.layers:
            if L.op != "conv" or L.name in self.skip or L.name in self.merged or L.name in self.in_place or L.f32_out:
                continue
            readers = self.uses.get(L.name, [])
            if len(readers) != 1 or L.residual is not None or self.shape[L.name][3] != L.conv.K:
                continue
            R = readers[0]
            if (R.op != "conv" or R.src != [L.name] or R.residual == L.name or R.name in self.skip or R.name in self.merged
                    or R.name in self.in_place or R.f32_out or self.shape[R.name][3] != R.conv.K
                    or L.name in self.fused_second):
                continue
            if q8.q8_conv2d_then_1x1_supported(self.convs[L.name].desc, self.convs[R.name].desc):
                self.fused_with[L.name] = R.name
                self.fused_second.add(R.name)

    def _assign_streams(self, limit):
        """stream_of[layer]: a layer continues on the stream of its first input if it is that tensor's first
        reader, otherwise it opens the least recently used other stream.  deps[layer]: the tensors it must wait
        for (concat members count through their leaves)."""
        self.stream_of, self.deps = {"input": 0}, {}
        first_reader_done = set()
        next_side = 0

        def leaves(name):
            L = self.by_name.get(name)
            if L is not None and L.op == "concat":
                out = []
                for s in L.src:
                    out += leaves(s)
                return out + [name]   # the concat layer itself (copies of pooled branches)
            return [name]

        used = 1
        for L in self.layers:
            ins = list(L.src) + ([L.residual] if L.residual else [])
            deps = []
            for t in ins:
                deps += leaves(t)
            self.deps[L.name] = deps
            src0 = L.src[0]
            if limit == 1:
                sid = 0
            elif src0 not in first_reader_done:
                sid = self.stream_of[src0]
                first_reader_done.add(src0)
            else:
                next_side = next_side % (limit - 1) + 1
                sid = next_side
                used = max(used, sid + 1)
            self.stream_of[L.name] = sid
        self.n_streams = used if limit > 1 else 1

    # ---- device work --------------------------------------------------------------------------------
    def forward(self, x_f32: torch.Tensor) -> Dict[str, torch.Tensor]:
        """Enqueues the whole network on the current stream; returns the tensors (preallocated buffers, or
        channel slices of a concat buffer)."""
        q8.q8_quantize_pad_image(x_f32, self.w_pad_in, self.c_pad_in, self.info["input"][1], q8.Q8_S8, out=self.bufs["input"])
        self.run_quantized()
        return self.outputs

    def run_quantized(self):
        """Everything after the input quantization (the part a CUDA graph replays)."""
        if self.n_streams == 1:
            for L in self.layers:
                self._launch(L, self.workspaces[0])
            return
        main = torch.cuda.current_stream()
        streams = [main] + self.side_streams
        fork = torch.cuda.Event()
        fork.record(main)
        for st in self.side_streams:
            st.wait_event(fork)
        done: Dict[str, torch.cuda.Event] = {}
        for L in self.layers:
            sid = self.stream_of[L.name]
            st = streams[sid]
            for t in self.deps[L.name]:
                if t in done and self.stream_of[t] != sid:
                    st.wait_event(done[t])
            with torch.cuda.stream(st):
                self._launch(L, self.workspaces[sid])
            ev = torch.cuda.Event()
            ev.record(st)
            done[L.name] = ev
        for st in self.side_streams:
            join = torch.cuda.Event()
            join.record(st)
            main.wait_event(join)

    def _launch(self, L, workspace):
        b = self.bufs
        x = b[L.src[0]]
        if L.op == "conv":
            qc = self.convs[L.name]
            res = b[L.residual] if L.residual is not None else None
            if L.name in self.skip:
                return  # computed by the merged launch of its first sibling
            if L.name in self.fused_with:
                return  # runs together with its reader, below
            if L.name in self.fused_second:
                first = self.by_name[L.src[0]]
                pipeline.fused_pair(self.convs[first.name], qc, b[first.src[0]], res, b[L.name])
                return
            y = b[self.slot[L.name][0]] if L.name in self.in_place else b[L.name]
            if L.name in self.merged:
                y = b[L.name + ":merged"]
            q8.q8_conv2d(qc.desc, x, qc.w_q, qc.b_q, qc.scale, res, qc.res_scale, y, workspace)
        elif L.op == "maxpool":
            q8.q8_maxpool2d(x, L.k, L.stride, L.pad, L.ceil_mode, out=b[L.name])
        elif L.op == "avgpool":
            q8.q8_avgpool2d(x, L.k, L.stride, L.pad, L.ceil_mode, out=b[L.name])
        elif L.op == "l2norm":
            q_in, eps, mult = self.l2[L.name]
            q8.q8_l2norm(x, q_in, eps, mult, out=b[L.name])
        elif L.op == "concat":
            for s in L.src:
                if s in self.in_place or self.by_name[s].op == "concat":
                    continue
                root, off = self.slot[s]
                q8.q8_concat_branch(b[s], self.info[s][1], self.info[L.name][1], b[root], off)

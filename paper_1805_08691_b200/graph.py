"""Graph rewrites of the paper's model-optimisation step that change what is computed, not how.

`remove_sparsity` (Sec. "Model Optimization", residual-structure figure): when every reader of a tensor is a
1x1 convolution with stride 2, three quarters of that tensor are never used.  The producing convolution is
given the stride instead (it computes only the pixels that are read), a 1x1 stride-2 pooling layer subsamples
the skip branch that is summed into it, and the readers become stride-1 convolutions.  The FP32 network
computes the same function; the quantized one differs only through the calibration maxima of the smaller
tensor.

Works on a layer list as in `workloads.nets` (objects with name, op, src, conv, residual, f32_out, k, stride,
pad): returns a new list, the input is not modified.
"""
import copy
from typing import List


def remove_sparsity(layers: List) -> List:
    readers = {}
    for L in layers:
        for s in list(L.src) + ([L.residual] if L.residual else []):
            readers.setdefault(s, []).append(L)
    by_name = {L.name: L for L in layers}

    def is_strided_1x1(L, t):
        return (L.op == "conv" and L.src == [t] and L.residual != t and L.conv.R == 1 and L.conv.S == 1
                and tuple(L.conv.stride) == (2, 2) and tuple(L.conv.pad) == (0, 0))

    moved = {}      # producer name -> True
    relaxed = set() # readers whose stride moves into the producer
    for t, rs in readers.items():
        P = by_name.get(t)
        if P is None or P.op != "conv" or P.f32_out or not rs:
            continue
        if all(is_strided_1x1(L, t) for L in rs):
            moved[t] = True
            relaxed.update(L.name for L in rs)
    out = []
    layer_cls = type(layers[0])
    for L in layers:
        if L.name in moved:
            N = copy.copy(L)
            N.conv = copy.copy(L.conv)
            N.conv.stride = (L.conv.stride[0] * 2, L.conv.stride[1] * 2)
            if L.residual is not None:
                sub = layer_cls(L.name + "_skip_s2", "maxpool", [L.residual], k=(1, 1), stride=(2, 2), pad=(0, 0))
                out.append(sub)
                N.residual = sub.name
            out.append(N)
        elif L.name in relaxed:
            N = copy.copy(L)
            N.conv = copy.copy(L.conv)
            N.conv.stride = (1, 1)
            out.append(N)
        else:
            out.append(L)
    return out

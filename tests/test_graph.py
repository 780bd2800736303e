"""The "remove sparsity" rewrite (Sec. "Model Optimization"): same FP32 function, fewer MACs."""
import numpy as np

import oracle as o
from paper_1805_08691_b200 import graph
from workloads import nets


def _fold(layers):
    return {L.name: (o.fold_bn(L.conv.w, L.conv.b, L.conv.gamma, L.conv.beta, L.conv.mean, L.conv.var, 1e-5)
                     if L.conv.bn else (L.conv.w, L.conv.b)) for L in layers if L.op == "conv"}


def test_remove_sparsity_keeps_the_function_and_drops_the_unused_pixels():
    layers = nets.resnet50()
    rewritten = graph.remove_sparsity(layers)
    # three stage transitions: the last 1x1 of res2c / res3d / res4f takes the stride, its skip branch a 1x1 stride-2 pool
    added = [L.name for L in rewritten if L.name not in {x.name for x in layers}]
    assert added == ["res2c_branch2c_skip_s2", "res3d_branch2c_skip_s2", "res4f_branch2c_skip_s2"]
    by = {L.name: L for L in rewritten}
    for blk, nxt in (("res2c", "res3a"), ("res3d", "res4a"), ("res4f", "res5a")):
        assert by[blk + "_branch2c"].conv.stride == (2, 2) and by[blk + "_branch2c"].residual == blk + "_branch2c_skip_s2"
        assert by[nxt + "_branch1"].conv.stride == (1, 1) and by[nxt + "_branch2a"].conv.stride == (1, 1)
    assert by["res2a_branch1"].conv.stride == (1, 1) and by["conv1"].conv.stride == (2, 2)   # untouched
    assert {L.name: L.conv.stride for L in layers if L.op == "conv"}["res3a_branch1"] == (2, 2)  # input list not modified
    # saved: 3/4 of the three expanding 1x1 convolutions
    saved = sum(3 * (hw * hw // 4) * cin * cout for hw, cin, cout in ((56, 64, 256), (28, 128, 512), (14, 256, 1024)))
    assert nets.macs(layers, 224) - nets.macs(rewritten, 224) == saved
    folded = _fold(layers)
    x = nets.images(7, 1, 224)
    a, b = nets.fp32_forward(layers, x, folded), nets.fp32_forward(rewritten, x, folded)
    assert np.array_equal(a["res2c_branch2c"][:, ::2, ::2], b["res2c_branch2c"])
    assert np.array_equal(a["res3a_branch2a"], b["res3a_branch2a"])
    assert np.allclose(a["fc1000"], b["fc1000"], rtol=1e-5, atol=1e-5 * np.abs(a["fc1000"]).max())


def test_remove_sparsity_leaves_other_networks_alone():
    for layers in (nets.bottleneck_stack(C=16), nets.ssd300()):
        assert [L.name for L in graph.remove_sparsity(layers)] == [L.name for L in layers]

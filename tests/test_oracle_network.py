"""CPU pins of the oracle's whole-network assembly (factor rules, residual sum, concat under one factor) and of
the layer lists: the quantized run must track the FP32 run of the same seeded network, and the structural
rules must hold on the tensors it returns."""
import numpy as np

import oracle as o
from oracle import net as oracle_net
from workloads import nets
from workloads.nets import Layer, _conv
from workloads.synth import rng


def _fold(layers):
    folded = {}
    for L in layers:
        if L.op != "conv":
            continue
        sp = L.conv
        if sp.bn:
            folded[L.name] = o.fold_bn(sp.w, sp.b, sp.gamma, sp.beta, sp.mean, sp.var, 1e-5)
        else:
            folded[L.name] = (sp.w, sp.b if sp.b is not None else np.zeros(sp.K, np.float32))
    return folded


def _calibrate(layers, folded, seed, batch, hw, batches=2):
    maxima = {}
    for i in range(batches):
        acts = nets.fp32_forward(layers, nets.images(seed + 10 + i, batch, hw), folded)
        for k, v in acts.items():
            maxima[k] = o.maxabs(v, init=maxima.get(k, 0.0))
    return maxima


def _mini_inception(seed=77):
    """Stem, one module with conv / avg-pool branches and a nested concat, one reduction module with a max-pool
    branch, classifier."""
    g = rng(seed)
    L = []
    x = _conv(g, L, "stem", "input", 3, 32, 3, pad=1)
    b1 = _conv(g, L, "m0_1x1", x, 32, 16, 1)
    r = _conv(g, L, "m0_reduce", x, 32, 16, 1)
    L.append(Layer("m0_pair", "concat", [_conv(g, L, "m0_1x3", r, 16, 16, 1, 3, pad=(0, 1)),
                                         _conv(g, L, "m0_3x1", r, 16, 16, 3, 1, pad=(1, 0))]))
    L.append(Layer("m0_pool", "avgpool", [x], k=(3, 3), stride=(1, 1), pad=(1, 1)))
    b4 = _conv(g, L, "m0_proj", "m0_pool", 32, 16, 1)
    L.append(Layer("m0", "concat", [b1, "m0_pair", b4]))
    c1 = _conv(g, L, "m1_3x3_s2", "m0", 64, 32, 3, stride=2)
    L.append(Layer("m1_pool", "maxpool", ["m0"], k=(3, 3), stride=(2, 2)))
    L.append(Layer("m1", "concat", [c1, "m1_pool"]))
    L.append(Layer("gap", "avgpool", ["m1"], k=(5, 5), stride=(1, 1)))
    _conv(g, L, "fc", "gap", 96, 10, 1, relu=False, bn=False, bias=True, f32_out=True)
    return L


def _rel(a, b):
    return float(np.linalg.norm(a.astype(np.float64) - b) / np.linalg.norm(b))


def test_concat_groups_share_one_factor_and_copy_their_conv_branches():
    layers = _mini_inception()
    folded = _fold(layers)
    maxima = _calibrate(layers, folded, 77, 2, 12)
    prep, info = oracle_net.network_prepare(layers, folded, maxima)
    # module 0: every leaf is a conv + ReLU read only by the concat tree -> all five tensors carry one factor,
    # the largest of the leaves' own max/255
    leaves0 = ["m0_1x1", "m0_1x3", "m0_3x1", "m0_proj"]
    q0 = max(o.factor(maxima[n], 8) for n in leaves0)
    for n in leaves0 + ["m0_pair", "m0"]:
        assert info[n] == (o.U8, q0), n
    # module 1: the pooled branch keeps the factor of its input (q0) and is re-expressed by the concat
    q1 = max(o.factor(maxima["m1_3x3_s2"], 8), q0)
    assert info["m1_pool"] == (o.U8, q0) and info["m1"][1] == q1 and info["m1_3x3_s2"][1] == q1
    # a tensor with a second reader keeps its own factor
    assert info["stem"][1] == o.factor(maxima["stem"], 8) and info["m0_reduce"][1] == o.factor(maxima["m0_reduce"], 8)

    x = nets.images(78, 2, 12)
    out = oracle_net.network_forward(layers, prep, info, x)
    assert np.array_equal(out["m0"], np.concatenate([out["m0_1x1"], out["m0_1x3"], out["m0_3x1"], out["m0_proj"]], -1))
    assert np.array_equal(out["m1"][..., :32], out["m1_3x3_s2"])
    assert np.array_equal(out["m1"][..., 32:], o.concat([out["m1_pool"]], [q0], q1))
    # the quantized tensors follow the FP32 run
    ref = nets.fp32_forward(layers, x, folded)
    for n in ("stem", "m0", "m1"):
        assert _rel(o.dequantize(out[n], info[n][1]), ref[n]) < 0.06, n
    assert _rel(out["fc"], ref["fc"]) < 0.1


def test_residual_stack_follows_fp32_and_uses_the_plus_rule():
    layers = nets.bottleneck_stack(C=16, blocks=2)
    folded = _fold(layers)
    maxima = _calibrate(layers, folded, 31, 2, 16)
    prep, info = oracle_net.network_prepare(layers, folded, maxima)
    assert info["input"] == (o.S8, o.factor(maxima["input"], 7))
    assert info["blk0_branch1"] == (o.S8, o.factor(maxima["blk0_branch1"], 7))        # no ReLU: signed, p = 7
    assert info["blk0_branch2c"][1] == o.factor(max(maxima["blk0_branch2c:pre"], maxima["blk0_branch1"]), 8)
    assert info["blk1_branch2c"][1] == o.factor(max(maxima["blk1_branch2c:pre"], maxima["blk0_branch2c"]), 8)
    assert info["pool1"] == info["conv1"]
    x = nets.images(32, 2, 16)
    out = oracle_net.network_forward(layers, prep, info, x)
    ref = nets.fp32_forward(layers, x, folded)
    for L in layers:
        assert _rel(o.dequantize(out[L.name], info[L.name][1]), ref[L.name]) < 0.12, L.name
    # the fused sum equals the literal "+" of the two quantized summands up to one output code
    pre = oracle_net.network_forward([L for L in layers if L.name != "blk1_branch2c"], prep, info, x)
    d = prep["blk1_branch2c"]
    sp = layers[-1].conv
    unfused = o.conv2d(pre["blk1_branch2b"], d["w_q"], d["b_q"], d["scale"], sp.stride, sp.pad, sp.dil, None, 0.0, False, o.F32)
    want = np.clip(np.rint(np.maximum(unfused + out["blk0_branch2c"].astype(np.float32) * np.float32(d["res_scale"]), 0)), 0, 255)
    assert np.array_equal(out["blk1_branch2c"], want.astype(np.uint8))


def test_post_sum_policy_calibrates_the_emitted_tensor():
    """sum_policy="post_sum": the factor of a fused residual sum is the calibrated maximum of the sum itself; every
    other factor is untouched; on a calibration batch the sum then reaches the top code, which the "+" rule on the
    two summands only does when the maxima of conv and residual do not add up."""
    layers = nets.bottleneck_stack(C=16, blocks=2)
    folded = _fold(layers)
    x = nets.images(41, 2, 16)
    acts = nets.fp32_forward(layers, x, folded)
    maxima = {k: o.maxabs(v) for k, v in acts.items()}
    prep_m, info_m = oracle_net.network_prepare(layers, folded, maxima)
    prep_s, info_s = oracle_net.network_prepare(layers, folded, maxima, sum_policy="post_sum")
    sums = [L.name for L in layers if L.residual is not None]
    assert sums == ["blk0_branch2c", "blk1_branch2c"]
    for L in layers:
        if L.name in sums:
            assert info_s[L.name][1] == o.factor(maxima[L.name], 8)
            # |a + b| <= |a| + |b| <= 2 max(|a|, |b|): the post-sum factor is at most twice the "+" rule's
            assert info_s[L.name][1] <= 2 * info_m[L.name][1]
    assert info_s["conv1"] == info_m["conv1"] and info_s["blk0_branch2a"] == info_m["blk0_branch2a"]
    out_s = oracle_net.network_forward(layers, prep_s, info_s, x)
    # calibrated on this very batch: the largest FP32 value of the sum maps to 255 (quantization noise of the
    # layers before it moves the largest code by a few steps at most)
    assert out_s["blk0_branch2c"].max() >= 250
    ref = acts
    for name in sums:
        assert _rel(o.dequantize(out_s[name], info_s[name][1]), ref[name]) < 0.12, name


def test_layer_lists_match_the_published_architectures():
    r50, inc, ssd = nets.resnet50(), nets.inception_v3(), nets.ssd300()
    assert sum(L.op == "conv" for L in r50) == 54 and nets.macs(r50, 224) == 3857973248
    assert sum(L.op == "conv" for L in inc) == 95 and nets.macs(inc, 299) == 5713216096
    assert sum(L.op == "conv" for L in ssd) == 35 and nets.macs(ssd, 300) == 31373537792
    assert sum(L.op == "concat" for L in inc) == 15
    heads = [L for L in ssd if L.f32_out]
    assert len(heads) == 12 and sorted({L.conv.K for L in heads}) == [16, 24, 84, 126]
    fc6 = next(L for L in ssd if L.name == "fc6").conv
    assert (fc6.R, fc6.dil, fc6.pad) == (3, (6, 6), (6, 6))
    assert next(L for L in ssd if L.name == "pool3").ceil_mode


def test_per_channel_weight_factors():
    """One factor per output channel: every channel uses its full code range, the multiplier and the bias follow
    the channel's factor, and the quantized run tracks FP32 at least as well as with one factor per tensor."""
    layers = nets.bottleneck_stack(C=16, blocks=2)
    folded = _fold(layers)
    maxima = _calibrate(layers, folded, 31, 2, 16)
    pt, info_t = oracle_net.network_prepare(layers, folded, maxima)
    pc, info_c = oracle_net.network_prepare(layers, folded, maxima, per_channel=True)
    assert info_t == info_c                              # activation factors do not depend on the weight factors
    name = "blk0_branch2b"
    w, b = folded[name]
    d = pc[name]
    K = w.shape[0]
    assert len(d["q_w"]) == K and d["scale"].shape == (K,)
    q_in = info_c["blk0_branch2a"][1]
    for k in range(K):
        assert d["q_w"][k] == o.factor(o.maxabs(w[k]), 7)
        assert np.abs(d["w_q"][k].astype(np.int32)).max() == 127
        assert d["scale"][k] == o.requant_scale(q_in, d["q_w"][k], d["q_y"])
        assert d["b_q"][k] == o.quantize(b[k:k + 1], o.bias_factor(q_in, d["q_w"][k]), o.S32)[0]
    assert max(d["q_w"]) == pt[name]["q_w"]              # the per-tensor factor is the largest channel factor
    x = nets.images(32, 2, 16)
    ref = nets.fp32_forward(layers, x, folded)
    out_t = oracle_net.network_forward(layers, pt, info_t, x)
    out_c = oracle_net.network_forward(layers, pc, info_c, x)
    last = layers[-1].name
    err_t = _rel(o.dequantize(out_t[last], info_t[last][1]), ref[last])
    err_c = _rel(o.dequantize(out_c[last], info_c[last][1]), ref[last])
    assert err_c < 0.12 and err_c <= err_t * 1.05


def test_l2norm_layer_in_a_network_follows_fp32_and_keeps_its_structure():
    """conv -> L2 normalisation -> two heads: the quantized run tracks the FP32 run, the normalised tensor is u8 at
    its own calibrated factor, and dequantized it has per-pixel norms of about gamma (all channels equal here)."""
    g = rng(91)
    L = []
    x = _conv(g, L, "c1", "input", 3, 32, 3, pad=1)
    x = _conv(g, L, "c2", x, 32, 64, 3, pad=1)
    L.append(Layer("c2_norm", "l2norm", [x], gamma=np.full(64, 20.0, np.float32)))
    _conv(g, L, "head_a", "c2_norm", 64, 8, 3, pad=1, relu=False, bn=False, bias=True, f32_out=True)
    _conv(g, L, "head_b", "c2_norm", 64, 12, 3, pad=1, relu=False, bn=False, bias=True, f32_out=True)
    folded = _fold(L)
    maxima = _calibrate(L, folded, 91, 2, 24)
    prep, info = oracle_net.network_prepare(L, folded, maxima)
    xin = nets.images(92, 2, 24)
    got = oracle_net.network_forward(L, prep, info, xin, threads=2)
    ref = nets.fp32_forward(L, xin, folded)
    t, q = info["c2_norm"]
    assert t == o.U8 and q == o.factor(maxima["c2_norm"], 8) and got["c2_norm"].dtype == np.uint8
    deq = got["c2_norm"].astype(np.float64) * float(q)
    norms = np.sqrt((deq ** 2).sum(-1))
    live = np.sqrt((ref["c2"].astype(np.float64) ** 2).sum(-1)) > 1e-3
    assert np.allclose(norms[live], 20.0, rtol=0.03)
    assert _rel(deq, ref["c2_norm"]) < 0.05
    for h in ("head_a", "head_b"):
        assert _rel(got[h], ref[h]) < 0.1
    # the SSD layer list with the option: one more layer, the conv4_3 heads read it
    ssd = nets.ssd300(l2norm=True)
    by = {x.name: x for x in ssd}
    assert by["conv4_3_norm"].op == "l2norm" and by["conv4_3_norm_mbox_loc"].src == ["conv4_3_norm"] and by["pool4"].src == ["conv4_3"]
    assert len(ssd) == len(nets.ssd300()) + 1 and nets.macs(ssd, 300) == nets.macs(nets.ssd300(), 300)

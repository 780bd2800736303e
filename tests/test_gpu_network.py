"""Whole networks: the library's quantized run must equal the oracle's bit for bit, layer by layer.

Both sides start from the same seeded FP32 parameters and the same FP32 calibration samples (one FP32 run
on the GPU shared by both), then fold BN, derive factors, quantize and run on their own.
"""
import numpy as np
import pytest
import torch

import oracle as o
import workloads as wl
from oracle import net as oracle_net
from workloads import nets

pytestmark = pytest.mark.gpu


def _cuda(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def _compare(layers, got, want, net, info, rows=None, check_layers=None):
    """Every tensor the network exposes against the oracle's, bit for bit (rows: the images of the batch the oracle
    ran).  A tensor is absent only if its layer runs in one launch with its reader."""
    for L in layers:
        if check_layers is not None and L.name not in check_layers:
            continue
        if L.name not in got:
            assert L.name in net.fused_with, L.name
            continue
        a, e = got[L.name].cpu().numpy(), want[L.name]
        if rows is not None:
            a = a[rows]
        if a.dtype == np.float32:
            a, e = a.view(np.uint32), e.view(np.uint32)
        assert a.shape == e.shape and np.array_equal(a, e), L.name
        assert net.info[L.name][1] == info[L.name][1], L.name


def _run_both(q8, layers, hw, batch, calib_batches, seed, check_layers=None, per_channel=False, streams=1, fuse=False,
              calib_batch=None, rows=None, sum_policy="max"):
    """rows: run the library on the whole batch but the oracle only on these images of it (images are independent)."""
    from paper_1805_08691_b200 import network, pipeline
    # fold BN on both sides, must agree bit for bit
    folded_o, folded_g = {}, {}
    for L in layers:
        if L.op != "conv":
            continue
        sp = L.conv
        if sp.bn:
            wo, bo = o.fold_bn(sp.w, sp.b, sp.gamma, sp.beta, sp.mean, sp.var, 1e-5)
            wg, bg = q8.q8_fold_bn(_cuda(sp.w), _cuda(sp.b) if sp.b is not None else None, _cuda(sp.gamma), _cuda(sp.beta),
                                   _cuda(sp.mean), _cuda(sp.var), 1e-5)
            assert np.array_equal(wg.cpu().numpy(), wo) and np.array_equal(bg.cpu().numpy(), bo)
        else:
            wo, bo = sp.w, (sp.b if sp.b is not None else np.zeros(sp.K, np.float32))
            wg, bg = _cuda(wo), _cuda(bo)
        folded_o[L.name], folded_g[L.name] = (wo, bo), (wg, bg)
    # calibration: FP32 run on seeded batches, running max-abs on both sides
    names = None
    cal = None
    max_o = {}
    for i in range(calib_batches):
        acts = nets.fp32_forward(layers, nets.images(seed + 10 + i, calib_batch or batch, hw), folded_o, device="cuda")
        if cal is None:
            names = sorted(acts)
            cal = pipeline.Calibrator(names)
        for k in names:
            cal.observe(k, _cuda(acts[k]))
            max_o[k] = o.maxabs(acts[k], init=max_o.get(k, 0.0))
    max_g = cal.maxima()
    assert max_g == max_o
    # prepare and run
    x = nets.images(seed + 1, batch, hw)
    prep, info = oracle_net.network_prepare(layers, folded_o, max_o, per_channel, sum_policy)
    xo = x if rows is None else np.ascontiguousarray(x[rows])
    want = oracle_net.network_forward(layers, prep, info, xo, threads=min(len(xo), o.hw_threads()))
    net = network.QuantNetwork(layers, folded_g, max_g, x.shape, per_channel=per_channel, streams=streams, fuse=fuse,
                               sum_policy=sum_policy)
    got = net.forward(_cuda(x))
    q8.q8_read_status()
    _compare(layers, got, want, net, info, rows, check_layers)
    ref = nets.fp32_forward(layers, xo, folded_o, device="cuda")
    return got, want, ref, net


def test_bottleneck_stack_every_layer(q8):
    layers = nets.bottleneck_stack(C=64, blocks=2)
    _run_both(q8, layers, hw=32, batch=3, calib_batches=2, seed=3100)
    _run_both(q8, layers, hw=32, batch=3, calib_batches=2, seed=3100, streams=2)
    got, want, ref, net = _run_both(q8, layers, hw=32, batch=3, calib_batches=2, seed=3100, streams=2, fuse=True)
    assert len(net.fused_with) == 2     # the 3x3 of each block runs in one launch with the 1x1 after it
    # factor of a fused sum calibrated on the sum itself instead of the "+" rule on its summands
    _run_both(q8, layers, hw=32, batch=3, calib_batches=2, seed=3100, fuse=True, sum_policy="post_sum")


# ---- the benchmarked launch configurations: whole batch on the GPU (pair mode, tile widths and reduction splits
# depend on the batch), every layer of three sampled images against the oracle run on just those images
FULL = [("resnet50", 224, 64, 3000, False), ("resnet50", 224, 1, 3000, False), ("resnet50_sparsity_removed", 224, 64, 3000, False),
        ("resnet50", 224, 64, 3000, True), ("inception_v3", 299, 64, 4000, True), ("ssd300", 300, 32, 5000, True)]


@pytest.mark.parametrize("name,hw,batch,seed,fuse", FULL, ids=[f"{n}_b{b}{'_fused' if f else ''}" for n, _, b, _, f in FULL])
def test_full_batch_sampled_images_bit_exact(q8, name, hw, batch, seed, fuse):
    """Configs 3-5 at the batch sizes bench.py times (64 / 64 / 32, ResNet-50 also at 1), four streams, with and
    without layer pairs in one launch: every tensor of the first, middle and last image equals the oracle's."""
    if name == "resnet50_sparsity_removed":
        from paper_1805_08691_b200 import graph
        layers = graph.remove_sparsity(nets.resnet50())
    else:
        layers = getattr(nets, name)()
    rows = sorted({0, batch // 2, batch - 1})
    got, want, ref, net = _run_both(q8, layers, hw=hw, batch=batch, calib_batches=1, seed=seed, streams=4, fuse=fuse,
                                    calib_batch=2, rows=rows)
    if fuse and name == "resnet50":
        assert len(net.fused_with) >= 7


def test_per_channel_weight_factors_every_layer(q8):
    """One weight factor per output channel (scale_count = K) through residual blocks and concat modules."""
    from tests.test_oracle_network import _mini_inception
    _run_both(q8, nets.bottleneck_stack(C=64, blocks=2), hw=32, batch=2, calib_batches=2, seed=3100, per_channel=True)
    got, want, ref, net = _run_both(q8, _mini_inception(), hw=12, batch=2, calib_batches=2, seed=77, per_channel=True)
    assert net.convs["m0_1x3"].scale.numel() == 16


def test_resnet50_logits_bit_exact_and_close_to_fp32(q8):
    """Config 3 at a batch the oracle finishes in seconds: all 54 affine layers, pools, dequantized logits."""
    layers = nets.resnet50()
    assert nets.macs(layers, 224) == 3857973248  # 3.858 GMAC per image
    got, want, ref, net = _run_both(q8, layers, hw=224, batch=2, calib_batches=2, seed=3000)
    logits, fp32 = got["fc1000"].cpu().numpy().reshape(2, -1), ref["fc1000"].reshape(2, -1)
    rel = float(np.linalg.norm(logits - fp32) / np.linalg.norm(fp32))
    print(f"ResNet-50 int8 vs FP32 logits: relative L2 error {rel:.4f}")
    assert rel < 0.5


def test_concat_modules_write_in_place_and_match_the_oracle(q8):
    """Conv / pooled / nested-concat branches under one factor: every tensor of a small Inception-like net."""
    from tests.test_oracle_network import _mini_inception
    layers = _mini_inception()
    got, want, ref, net = _run_both(q8, layers, hw=12, batch=3, calib_batches=2, seed=77)
    assert {"m0_1x1", "m0_1x3", "m0_3x1", "m0_proj", "m1_3x3_s2"} == net.in_place
    assert got["m0_1x3"].data_ptr() == got["m0"].data_ptr() + 16      # a slice of the concat buffer, not a copy


def test_inception_v3_bit_exact_and_close_to_fp32(q8):
    """Config 4 at batch 2: 95 affine layers, 15 concatenations (11 modules, 4 nested), 1x7 / 7x1 / 5x5 filters,
    stride-2 reductions with a pooled branch, 3x3 average pools, dequantized logits."""
    layers = nets.inception_v3()
    got, want, ref, net = _run_both(q8, layers, hw=299, batch=2, calib_batches=2, seed=4000, streams=4)
    assert net.n_streams == 4       # module branches on their own streams, joined at the concatenations
    logits, fp32 = got["fc"].cpu().numpy().reshape(2, -1), ref["fc"].reshape(2, -1)
    rel = float(np.linalg.norm(logits - fp32) / np.linalg.norm(fp32))
    print(f"Inception-v3 int8 vs FP32 logits: relative L2 error {rel:.4f}")
    assert rel < 0.5


def test_ssd300_heads_bit_exact_and_close_to_fp32(q8):
    """Config 5 at batch 1: VGG-16 base with ceil-mode pool3, dilation-6 fc6, extra stages, and the twelve
    dequantized 3x3 heads (16/24 and 84/126 output channels) over 8732 boxes."""
    layers = nets.ssd300()
    got, want, ref, net = _run_both(q8, layers, hw=300, batch=1, calib_batches=1, seed=5000, streams=3)
    boxes = 0
    num = den = 0.0
    for L in layers:
        if not L.f32_out:
            continue
        a, f = got[L.name].cpu().numpy().astype(np.float64), ref[L.name]
        num, den = num + float(((a - f) ** 2).sum()), den + float((f.astype(np.float64) ** 2).sum())
        if L.name.endswith("_loc"):
            boxes += a.size // 4
    assert boxes == 8732
    rel = (num / den) ** 0.5
    print(f"SSD-300 int8 vs FP32 head outputs: relative L2 error {rel:.4f}")
    assert rel < 0.5


def test_resnet50_with_sparsity_removed_bit_exact(q8):
    """The rewritten ResNet-50 (stride moved into the producing 1x1, 1x1 stride-2 pooling on the skip branch)."""
    from paper_1805_08691_b200 import graph
    layers = graph.remove_sparsity(nets.resnet50())
    got, want, ref, net = _run_both(q8, layers, hw=224, batch=2, calib_batches=2, seed=3000)
    logits, fp32 = got["fc1000"].cpu().numpy().reshape(2, -1), ref["fc1000"].reshape(2, -1)
    assert float(np.linalg.norm(logits - fp32) / np.linalg.norm(fp32)) < 0.5


def test_ssd300_with_normalisation_and_detection_output(q8):
    """SSD-300 as the detector defines it: the heads of conv4_3 read its L2-normalised copy, and the twelve head
    tensors (merged per source map on the GPU) go through the detection output.  Every layer and every kept
    detection bit-exact against the oracle at batch 2."""
    layers = nets.ssd300(l2norm=True)
    got, want, ref, net = _run_both(q8, layers, hw=300, batch=2, calib_batches=1, seed=5100, streams=3)
    assert np.array_equal(got["conv4_3_norm"].cpu().numpy(), want["conv4_3_norm"])
    srcs = [L.src[0] for L in layers if L.name.endswith("_mbox_loc")]
    boxes = [L.conv.K // 4 for L in layers if L.name.endswith("_mbox_loc")]
    classes = 21
    loc = np.concatenate([want[s + "_mbox_loc"].reshape(2, -1, 4) for s in srcs], 1)
    conf = np.concatenate([want[s + "_mbox_conf"].reshape(2, -1, classes) for s in srcs], 1)
    assert loc.shape == (2, 8732, 4) and conf.shape == (2, 8732, classes)
    priors = nets.ssd300_priors()
    # random-init heads are nearly flat: a low threshold on purpose, so that suppression has work to do
    kw = dict(conf_thresh=0.02, nms_thresh=0.45, nms_top_k=400, keep_top_k=200)
    want_rows, want_counts = o.detection_output(loc, conf, priors, nets.SSD300_VARIANCES, **kw)
    rows, counts = q8.q8_detection_output([(got[s + "_mbox_loc"], got[s + "_mbox_conf"], b) for s, b in zip(srcs, boxes)],
                                          _cuda(priors), nets.SSD300_VARIANCES, classes, **kw)
    q8.q8_read_status()
    assert np.array_equal(counts.cpu().numpy(), want_counts) and want_counts.min() > 0
    assert np.array_equal(rows.cpu().numpy(), want_rows)

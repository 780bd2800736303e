"""Config 2 (ResNet-50 bottleneck) end to end: fold BN, calibrate, quantize, three fused convs.

Both sides start from the same seeded FP32 parameters and the same FP32 calibration samples; every
intermediate (folded weights, factors, quantized weights/bias, scales, activations) must agree
bit for bit.
"""
import numpy as np
import pytest
import torch

import oracle as o
import workloads as wl
from oracle import net as oracle_net

pytestmark = pytest.mark.gpu


def _cuda(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def _run_both(q8, cfg, check_images):
    from paper_1805_08691_b200 import pipeline
    convs = cfg["convs"]
    # --- fold BN on both sides
    folded_o, folded_g = [], []
    for sp in convs:
        wo, bo = o.fold_bn(sp.w, sp.b, sp.gamma, sp.beta, sp.mean, sp.var, 1e-5)
        wg, bg = q8.q8_fold_bn(_cuda(sp.w), None, _cuda(sp.gamma), _cuda(sp.beta), _cuda(sp.mean), _cuda(sp.var), 1e-5)
        assert np.array_equal(wg.cpu().numpy(), wo) and np.array_equal(bg.cpu().numpy(), bo)
        folded_o.append((wo, bo))
        folded_g.append((wg, bg))
    # --- calibration samples from the FP32 model (shared input), max-abs on both sides
    names = ["x", "a", "b", "c"]
    cal = pipeline.Calibrator(names)
    per_batch = []
    for xb in cfg["calib"]:
        s = wl.bottleneck_fp32(xb, folded_o, device="cuda")
        per_batch.append({k: s[k] for k in names})
        for k in names:
            cal.observe(k, _cuda(s[k]))
    max_o = oracle_net.calib_maxima(per_batch)
    max_g = cal.maxima()
    assert max_o == max_g
    # --- prepare and run
    fo = oracle_net.bottleneck_prepare(folded_o, max_o)
    x = cfg["x"]
    block = pipeline.Bottleneck(folded_g, max_g, x.shape)
    for k in ("q_x", "q_a", "q_b", "q_y"):
        assert getattr(block, k) == fo[k]
    for name in "abc":
        lay = getattr(block, name)
        assert lay.q_w == fo[name]["q_w"] and lay.scale.item() == fo[name]["scale"]
        assert np.array_equal(lay.w_q.cpu().numpy(), fo[name]["w_q"])
        assert np.array_equal(lay.b_q.cpu().numpy(), fo[name]["b_q"])
        assert q8.q8_conv2d_query_algo(lay.desc) == q8.Q8_ALGO_UMMA
    xq_o = o.quantize(x, fo["q_x"], o.U8)
    xq_g = q8.q8_quantize(_cuda(x), block.q_x, q8.Q8_U8)
    assert np.array_equal(xq_g.cpu().numpy(), xq_o)
    assert block.fused          # the 3x3 and the expanding 1x1 run as one launch; its 3x3 output is never written
    y = block(xq_g)
    q8.q8_read_status()
    plain = pipeline.Bottleneck(folded_g, max_g, x.shape, fuse=False)   # three launches, every tensor written
    y3 = plain(xq_g)
    q8.q8_read_status()
    ya_g, yb_g, y_g = plain.ya.cpu().numpy(), plain.yb.cpu().numpy(), y.cpu().numpy()
    assert torch.equal(y, y3) and torch.equal(block.ya, plain.ya)
    for n in check_images:
        ya, yb, yo = oracle_net.bottleneck_forward(fo, xq_o[n:n + 1])
        assert np.array_equal(ya_g[n:n + 1], ya)
        assert np.array_equal(yb_g[n:n + 1], yb)
        assert np.array_equal(y_g[n:n + 1], yo)
    # dequantized output against the oracle's, and sanity of the quantized range
    deq = q8.q8_dequantize(y, block.q_y).cpu().numpy()
    n0 = check_images[0]
    assert np.array_equal(deq[n0], o.dequantize(y_g[n0], fo["q_y"]))
    assert y_g.max() > 100  # the output uses the 8-bit range


def test_bottleneck_small(q8):
    cfg = wl.config2(batch=3, H=30, W=30, calib_batches=2)
    _run_both(q8, cfg, check_images=[0, 1, 2])


def test_bottleneck_full_size_sampled(q8):
    """Batch 32, 56x56x256 as benchmarked; the oracle checks whole images sampled from the batch."""
    cfg = wl.config2(batch=32, calib_batches=4, calib_batch=8)
    _run_both(q8, cfg, check_images=[0, 17, 31])

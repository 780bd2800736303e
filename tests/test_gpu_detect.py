"""GPU parity of the SSD tail (L2 normalisation, FP32 route of a signed sum, detection output) against the CPU
oracle, through the C ABI.  8-bit results and kept detections bit-exact: both sides take every floating-point step
as the same IEEE fp32 operation in the same order.
"""
import numpy as np
import pytest
import torch

import oracle as o
from workloads import nets

pytestmark = pytest.mark.gpu


def _cuda(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


@pytest.mark.parametrize("shape", [(2, 38, 38, 512), (1, 5, 7, 2048), (3, 9, 9, 36), (2, 4, 4, 1156), (5, 3, 3, 7)])
def test_l2norm_bit_exact(q8, shape):
    g = np.random.default_rng(sum(shape))
    C = shape[-1]
    x = g.integers(0, 256, shape, dtype=np.uint8)
    x[g.random(shape) < 0.5] = 0
    x[0, 0, 0, :] = 0                                                  # an all-zero pixel
    x[0, 0, 1, :] = 255                                                # the largest sum of squares
    gamma = g.uniform(-5, 25, C).astype(np.float32)                    # a few negative scales clamp to 0
    qx, qy = np.float32(0.031), np.float32(0.0625)
    mult = o.l2norm_mult(gamma, qx, qy)
    for eps in (1e-10, 0.0):
        got = q8.q8_l2norm(_cuda(x), float(qx), eps, _cuda(mult)).cpu().numpy()
        assert np.array_equal(got, o.l2norm(x, qx, eps, mult))


def test_l2norm_unaligned_rows_take_the_scalar_kernel(q8):
    g = np.random.default_rng(5)
    x = g.integers(0, 256, (37, 10), dtype=np.uint8)
    mult = g.uniform(1, 60, 10).astype(np.float32)
    buf = torch.zeros(37 * 10 + 1, dtype=torch.uint8, device="cuda")
    view = buf[1:].view(37, 10)
    view.copy_(_cuda(x))
    got = q8.q8_l2norm(view, 0.02, 1e-10, _cuda(mult)).cpu().numpy()
    assert np.array_equal(got, o.l2norm(x, 0.02, 1e-10, mult))


@pytest.mark.parametrize("n", [1, 3, 4, 1027, 64 * 56 * 56 + 5])
def test_add_relu_quantize_bit_exact(q8, n):
    g = np.random.default_rng(n)
    a, b = g.normal(0, 3, n).astype(np.float32), g.normal(0, 3, n).astype(np.float32)
    a[:1] = np.float32(1e9)                                            # saturates
    got = q8.q8_add_relu_quantize(_cuda(a), _cuda(b), 0.037).cpu().numpy()
    assert np.array_equal(got, o.add_relu_quantize(a, b, 0.037))


def _heads(loc, conf, splits, boxes_per_cell, merged):
    """Cut dense [N, P, 4] / [N, P, classes] arrays into per-source head tensors [N, cells, boxes * 4] and
    [N, cells, boxes * classes]; merged: one tensor per source holding both, as a network with merged sibling heads
    produces them."""
    N, _, classes = conf.shape
    out, first = [], 0
    for cells, b in zip(splits, boxes_per_cell):
        l = loc[:, first:first + cells * b].reshape(N, cells, b * 4)
        c = conf[:, first:first + cells * b].reshape(N, cells, b * classes)
        first += cells * b
        if merged:
            both = _cuda(np.concatenate([l, c], 2))
            out.append((both[..., :b * 4], both[..., b * 4:], b))
        else:
            out.append((_cuda(l), _cuda(c), b))
    return out


def _compare(q8, loc, conf, priors, splits, boxes_per_cell, merged=False, **kw):
    var = nets.SSD300_VARIANCES
    classes = conf.shape[-1]
    want_rows, want_counts = o.detection_output(loc, conf, priors, var, **kw)
    rows, counts = q8.q8_detection_output(_heads(loc, conf, splits, boxes_per_cell, merged), _cuda(priors), var, classes, **kw)
    q8.q8_read_status()
    assert np.array_equal(counts.cpu().numpy(), want_counts)
    assert np.array_equal(rows.cpu().numpy(), want_rows)
    return want_counts


def test_detection_output_ssd300_bit_exact(q8):
    """The full SSD-300 shape: 8732 boxes from six head tensors, 21 classes, the published thresholds and limits."""
    priors = nets.ssd300_priors()
    splits = [m * m for m in nets.SSD300_MAPS]
    boxes = [2 + 2 * len(r) for r in nets.SSD300_RATIOS]
    loc, conf = nets.detection_inputs(7, 3)
    counts = _compare(q8, loc, conf, priors, splits, boxes)
    assert counts.min() > 20                                           # the scene is not trivial
    _compare(q8, loc, conf, priors, splits, boxes, merged=True)


def test_detection_output_every_box_a_candidate(q8):
    """Flat logits: every box passes the confidence threshold for every class, so each class sorts all 8732 boxes,
    the suppression sees nms_top_k of them, and the per-image limit cuts the result."""
    priors = nets.ssd300_priors()
    splits = [m * m for m in nets.SSD300_MAPS]
    boxes = [2 + 2 * len(r) for r in nets.SSD300_RATIOS]
    g = np.random.default_rng(9)
    loc = g.normal(0, 1, (2, 8732, 4)).astype(np.float32)
    conf = g.normal(0, 0.3, (2, 8732, 21)).astype(np.float32)
    counts = _compare(q8, loc, conf, priors, splits, boxes)
    assert (counts == 200).all()


@pytest.mark.parametrize("case", ["tiny", "ties", "no_background", "small_limits", "nothing_passes"])
def test_detection_output_edge_cases(q8, case):
    g = np.random.default_rng(len(case))
    P, classes = 300, 5
    x0, y0 = g.integers(0, 12, P) / 16.0, g.integers(0, 12, P) / 16.0
    w, h = g.integers(2, 5, P) / 16.0, g.integers(2, 5, P) / 16.0
    priors = np.stack([x0 + w / 2, y0 + h / 2, w, h], 1).astype(np.float32)
    loc = np.zeros((2, P, 4), np.float32)
    conf = g.normal(0, 2, (2, P, classes)).astype(np.float32)
    kw = dict(conf_thresh=0.05, nms_top_k=60, keep_top_k=40)
    if case == "tiny":
        P = 3
        priors, loc, conf = priors[:3], loc[:, :3], conf[:, :3]
    elif case == "ties":
        conf[:] = np.round(conf)                                       # many equal probabilities and duplicate boxes
        priors[1::2] = priors[0::2]
    elif case == "no_background":
        kw["background"] = -1
    elif case == "small_limits":
        kw.update(nms_top_k=1, keep_top_k=1)
    elif case == "nothing_passes":
        kw["conf_thresh"] = 0.999
        conf[:] = 0.0
    _compare(q8, loc, conf, priors, [P], [1], **kw)


@pytest.mark.parametrize("spread", [0.0, 1e-3, 0.5])
def test_detection_output_many_candidates_with_equal_leading_bits(q8, spread):
    """More candidates than the pre-selection hands to the sort: identical probabilities (the selection cannot
    separate them and everything is sorted), probabilities that differ in their last bits only, and well spread
    ones."""
    g = np.random.default_rng(17)
    P, classes = 4000, 3
    x0, y0 = g.integers(0, 28, P) / 32.0, g.integers(0, 28, P) / 32.0
    w, h = g.integers(1, 5, P) / 32.0, g.integers(1, 5, P) / 32.0
    priors = np.stack([x0 + w / 2, y0 + h / 2, w, h], 1).astype(np.float32)
    conf = (g.normal(0, 1, (2, P, classes)) * spread).astype(np.float32)
    _compare(q8, np.zeros((2, P, 4), np.float32), conf, priors, [P], [1], conf_thresh=0.05, nms_top_k=300, keep_top_k=150)


def test_detection_output_refuses_what_it_cannot_hold(q8):
    loc = torch.zeros((1, 20000, 4), device="cuda")
    conf = torch.zeros((1, 20000, 3), device="cuda")
    pri = torch.zeros((20000, 4), device="cuda")
    with pytest.raises(q8.Q8Error) as e:
        q8.q8_detection_output([(loc, conf, 1)], pri, nets.SSD300_VARIANCES, 3)
    assert e.value.code == 2
    with pytest.raises(q8.Q8Error) as e:
        q8.q8_detection_output([(loc[:, :100], conf[:, :100], 1)], pri[:100], nets.SSD300_VARIANCES, 3, nms_top_k=600)
    assert e.value.code == 2

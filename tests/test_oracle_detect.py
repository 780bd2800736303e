"""Pins of the SSD-tail oracle (oracle/q8_oracle_detect.cpp) against things other than itself: closed forms,
library routines in fp64, hand-built cases whose answer is known by construction, and an independent brute-force
statement of the suppression rule.  CPU only.
"""
import numpy as np
import torch

import oracle as o
from workloads import nets


# ------------------------------------------------------------------------------------------------ exp / softmax
def test_exp_is_close_to_the_exponential_and_exact_where_it_must_be():
    assert o.exp(np.float32(0.0)) == 1.0
    x = np.linspace(-87.0, 88.0, 20001).astype(np.float32)
    got = o.exp(x).astype(np.float64)
    want = np.exp(x.astype(np.float64))
    ulp = np.spacing(want.astype(np.float32)).astype(np.float64)
    assert np.max(np.abs(got - want) / ulp) <= 2.0
    assert np.all(np.diff(got) >= 0)                                  # monotone on the grid
    assert o.exp(np.float32(-1000.0)) == o.exp(np.float32(-87.0))     # clamped, finite, positive
    assert np.isfinite(o.exp(np.float32(1000.0)))
    # exp(k ln2) = 2^k to within the error of the reduction
    for k in (-100, -3, 1, 7, 100):
        assert abs(o.exp(np.float32(k * np.log(2.0))).item() / 2.0 ** k - 1.0) < 1e-5


def test_softmax_against_fp64_and_its_invariants():
    g = np.random.default_rng(3)
    x = g.normal(0, 3, (500, 21)).astype(np.float32)
    p = o.softmax(x)
    e = np.exp(x.astype(np.float64) - x.max(1, keepdims=True))
    want = e / e.sum(1, keepdims=True)
    assert np.max(np.abs(p - want)) < 5e-7
    assert np.max(np.abs(p.sum(1) - 1.0)) < 1e-6
    assert np.array_equal(p.argmax(1), x.argmax(1))
    assert np.max(np.abs(o.softmax(x + np.float32(8.0)) - p)) < 1e-6  # a common shift of the logits changes nothing
    assert np.allclose(o.softmax(np.zeros((1, 4), np.float32)), 0.25)


# ------------------------------------------------------------------------------------------------ L2 normalisation
def test_l2norm_closed_forms():
    qx, qy = np.float32(0.05), np.float32(0.1)
    C = 64
    mult = o.l2norm_mult(np.full(C, 20.0, np.float32), qx, qy)
    assert np.allclose(mult, 20.0 * 0.05 / 0.1, rtol=1e-6)
    # one non-zero channel: v = gamma exactly (up to eps), whatever the code
    x = np.zeros((3, C), np.uint8)
    x[0, 5], x[1, 9], x[2, 0] = 1, 77, 255
    y = o.l2norm(x, qx, 1e-10, mult)
    assert y[0, 5] == y[1, 9] == y[2, 0] == 200 and y.sum() == 600   # gamma / q_y = 200
    # a constant vector: v = gamma / sqrt(C) = 20 / 8 = 2.5 -> code 25
    y = o.l2norm(np.full((1, C), 33, np.uint8), qx, 1e-10, mult)
    assert np.all(y == 25)
    # an all-zero pixel stays zero (eps keeps the divisor positive)
    assert not o.l2norm(np.zeros((1, C), np.uint8), qx, 1e-10, mult).any()
    # saturation: gamma / q_y above 255 clamps
    big = o.l2norm_mult(np.full(C, 40.0, np.float32), qx, qy)
    assert o.l2norm(x, qx, 1e-10, big)[2, 0] == 255


def test_l2norm_against_the_library_normalisation_in_fp64():
    g = np.random.default_rng(8)
    C = 512
    x = g.integers(0, 256, (300, C), dtype=np.uint8)
    x[g.random((300, C)) < 0.5] = 0                                   # post-ReLU sparsity
    gamma = g.uniform(5, 25, C).astype(np.float32)
    qx, qy = np.float32(0.031), np.float32(0.004)
    mult = o.l2norm_mult(gamma, qx, qy)
    got = o.l2norm(x, qx, 1e-10, mult).astype(np.float64)
    r = torch.from_numpy(x.astype(np.float64) * float(qx))
    v = torch.nn.functional.normalize(r, p=2.0, dim=1, eps=1e-12).numpy() * gamma.astype(np.float64)
    want = np.clip(v / float(qy), 0, 255)
    assert np.max(np.abs(got - want)) <= 0.5 + 1e-3                   # the nearest code, up to fp32 rounding near ties
    assert np.mean(got == np.rint(want)) > 0.999
    # direction only: doubling every code of a pixel changes nothing
    half = (x // 2).astype(np.uint8)
    assert np.array_equal(o.l2norm((half * 2).astype(np.uint8), qx, 0.0, mult)[half.any(1)],
                          o.l2norm(half, qx, 0.0, mult)[half.any(1)])


# ------------------------------------------------------------------------------------------------ boxes
def test_prior_boxes_of_ssd300():
    p = nets.ssd300_priors()
    assert p.shape == (8732, 4) and p.dtype == np.float32
    assert np.allclose(p[0], [4 / 300, 4 / 300, 0.1, 0.1])
    assert np.allclose(p[1, 2:], (30 * 60) ** 0.5 / 300)
    assert np.allclose(p[-4], [0.5, 0.5, 0.88, 0.88])                 # the 1x1 map: min size 264
    assert np.all(p[:, :2] > 0) and np.all(p[:, :2] < 1.02)          # 10 cells of 32 pixels overshoot the 300-pixel side
    # two boxes per extra ratio are transposes of each other
    assert np.allclose(p[2, 2:], p[3, 2:][::-1])


def test_decode_boxes_known_cases():
    var = np.array(nets.SSD300_VARIANCES, np.float32)
    dy = np.array([[0.5, 0.25, 0.25, 0.375]], np.float32)             # dyadic: every step is exact
    z = o.decode_boxes(np.zeros((1, 1, 4), np.float32), dy, var)[0, 0]
    assert np.array_equal(z, np.array([0.375, 0.0625, 0.625, 0.4375], np.float32))   # the prior's own corners
    pr = np.array([[0.5, 0.25, 0.2, 0.4]], np.float32)
    # l0 = 10 with variance 0.1 moves the centre by one prior width; l3 = ln(2) / 0.2 doubles the height
    loc = np.array([[[10.0, 0.0, 0.0, np.log(2.0) / 0.2]]], np.float32)
    b = o.decode_boxes(loc, pr, var)[0, 0].astype(np.float64)
    assert np.allclose(b, [0.6, 0.25 - 0.4, 0.8, 0.25 + 0.4], atol=1e-6)
    g = np.random.default_rng(2)
    P = 200
    priors = np.concatenate([g.uniform(0.1, 0.9, (P, 2)), g.uniform(0.05, 0.5, (P, 2))], 1).astype(np.float32)
    loc = g.normal(0, 1, (2, P, 4)).astype(np.float32)
    got = o.decode_boxes(loc, priors, var).astype(np.float64)
    l, q, v = loc.astype(np.float64), priors.astype(np.float64), var.astype(np.float64)
    cx, cy = v[0] * l[..., 0] * q[:, 2] + q[:, 0], v[1] * l[..., 1] * q[:, 3] + q[:, 1]
    w, h = np.exp(v[2] * l[..., 2]) * q[:, 2], np.exp(v[3] * l[..., 3]) * q[:, 3]
    want = np.stack([cx - w / 2, cy - h / 2, cx + w / 2, cy + h / 2], -1)
    assert np.max(np.abs(got - want)) < 2e-6


def test_iou_known_values():
    a = [0.0, 0.0, 2.0, 2.0]
    assert o.iou(a, a) == 1.0
    assert o.iou(a, [2.0, 0.0, 4.0, 2.0]) == 0.0                      # touching edges do not intersect
    assert o.iou(a, [3.0, 3.0, 4.0, 4.0]) == 0.0
    assert o.iou(a, [1.0, 0.0, 3.0, 2.0]) == np.float32(2.0) / np.float32(6.0)   # half overlap: 2 / (4 + 4 - 2)
    assert o.iou(a, [0.5, 0.5, 1.5, 1.5]) == 0.25                     # contained
    assert o.iou([1.0, 0.0, 3.0, 2.0], a) == o.iou(a, [1.0, 0.0, 3.0, 2.0])


# ------------------------------------------------------------------------------------------------ detection output
def _logits_for(prob_rows):
    """Logits whose softmax is the given probability rows (log p; the rows sum to 1)."""
    return np.log(np.asarray(prob_rows, np.float64)).astype(np.float32)


def _unit_priors(boxes):
    """Priors equal to the wanted corner boxes, to be decoded with zero offsets."""
    b = np.asarray(boxes, np.float32)
    return np.stack([(b[:, 0] + b[:, 2]) / 2, (b[:, 1] + b[:, 3]) / 2, b[:, 2] - b[:, 0], b[:, 3] - b[:, 1]], 1)


def test_detection_output_hand_built_scene():
    # dyadic coordinates: every decoded corner and every overlap is exact
    boxes = [[0.0, 0.0, 0.5, 0.5],       # 0: class 1, p 0.9
             [0.0, 0.0, 0.5, 0.375],     # 1: class 1, p 0.8, overlap with 0 = 0.75 -> suppressed
             [0.5, 0.5, 1.0, 1.0],       # 2: class 1, p 0.7, disjoint -> kept
             [0.0, 0.0, 0.5, 0.5],       # 3: class 2, p 0.6, same place as 0 but another class -> kept
             [0.25, 0.25, 0.75, 0.75],   # 4: class 1, p 0.5, overlap with 0 and 2 = 1/7 -> kept
             [0.0, 0.5, 0.5, 1.0]]       # 5: everything below the threshold
    probs = [[0.05, 0.9, 0.05], [0.1, 0.8, 0.1], [0.2, 0.7, 0.1], [0.3, 0.1, 0.6], [0.4, 0.5, 0.1], [0.99, 0.005, 0.005]]
    pri = _unit_priors(boxes)
    var = np.array(nets.SSD300_VARIANCES, np.float32)
    rows, counts = o.detection_output(np.zeros((1, 6, 4), np.float32), _logits_for(probs)[None], pri, var,
                                      conf_thresh=0.01, nms_thresh=0.45, nms_top_k=400, keep_top_k=10)
    # class-2 probabilities above 0.01 also exist for boxes 0, 1, 2, 4 (0.05, 0.1, 0.1, 0.1): box 3 (0.6) suppresses
    # box 0 and box 1 of class 2 (overlaps 1 and 0.75); boxes 2 and 4 of class 2 survive
    assert counts[0] == 6
    got = [(int(r[0]), round(float(r[1]), 4), [float(v) for v in r[2:]]) for r in rows[0, :6]]
    assert [(c, s) for c, s, _ in got] == [(1, 0.9), (1, 0.7), (2, 0.6), (1, 0.5), (2, 0.1), (2, 0.1)]
    assert got[0][2] == boxes[0] and got[1][2] == boxes[2] and got[2][2] == boxes[3] and got[3][2] == boxes[4]
    assert got[4][2] == boxes[2] and got[5][2] == boxes[4]           # equal scores: lower box index first
    assert not rows[0, 6:].any()
    # limits: one candidate per class before suppression, then two detections per image
    rows, counts = o.detection_output(np.zeros((1, 6, 4), np.float32), _logits_for(probs)[None], pri, var,
                                      nms_top_k=1, keep_top_k=10)
    assert counts[0] == 2 and [int(r[0]) for r in rows[0, :2]] == [1, 2]
    rows, counts = o.detection_output(np.zeros((1, 6, 4), np.float32), _logits_for(probs)[None], pri, var, keep_top_k=2)
    assert counts[0] == 2 and [round(float(r[1]), 4) for r in rows[0]] == [0.9, 0.7]
    # a threshold above every probability: nothing
    _, counts = o.detection_output(np.zeros((1, 6, 4), np.float32), _logits_for(probs)[None], pri, var, conf_thresh=0.95)
    assert counts[0] == 0


def _brute_force(boxes, prob, background, conf_thresh, nms_thresh, nms_top_k, keep_top_k):
    """The suppression rule stated over the whole overlap matrix (fp64): box i of a class is kept iff no kept box
    earlier in the order overlaps it beyond the threshold."""
    P, classes = prob.shape
    b = boxes.astype(np.float64)
    area = (b[:, 2] - b[:, 0]) * (b[:, 3] - b[:, 1])
    iw = np.minimum(b[:, None, 2], b[None, :, 2]) - np.maximum(b[:, None, 0], b[None, :, 0])
    ih = np.minimum(b[:, None, 3], b[None, :, 3]) - np.maximum(b[:, None, 1], b[None, :, 1])
    inter = np.where((iw > 0) & (ih > 0), iw * ih, 0.0)
    iou = inter / (area[:, None] + area[None, :] - inter)
    kept_all = []
    for c in range(classes):
        if c == background:
            continue
        order = [p for p in np.lexsort((np.arange(P), -prob[:, c].astype(np.float64))) if prob[p, c] > conf_thresh][:nms_top_k]
        kept = []
        for p in order:
            if all(iou[p, k] <= nms_thresh for k in kept):
                kept.append(p)
        kept_all += [(-float(prob[p, c]), c, p) for p in kept]
    kept_all.sort()
    return [(c, p) for _, c, p in kept_all[:keep_top_k]]


def test_detection_output_against_brute_force_on_random_scenes():
    g = np.random.default_rng(21)
    var = np.array(nets.SSD300_VARIANCES, np.float32)
    for trial in range(4):
        P, classes = 300, 5
        # boxes on a coarse dyadic lattice: overlaps are ratios of small integers, far from the threshold's rounding
        x0, y0 = g.integers(0, 12, P) / 16.0, g.integers(0, 12, P) / 16.0
        w, h = g.integers(2, 5, P) / 16.0, g.integers(2, 5, P) / 16.0
        boxes = np.stack([x0, y0, x0 + w, y0 + h], 1).astype(np.float32)
        conf = g.normal(0, 2, (1, P, classes)).astype(np.float32)
        rows, counts = o.detection_output(np.zeros((1, P, 4), np.float32), conf, _unit_priors(boxes), var,
                                          conf_thresh=0.05, nms_thresh=0.45, nms_top_k=60, keep_top_k=40)
        prob = o.softmax(conf)[0]
        want = _brute_force(boxes, prob, 0, np.float32(0.05), 0.45, 60, 40)
        assert counts[0] == len(want)
        for r, (c, p) in zip(rows[0], want):
            assert int(r[0]) == c and r[1] == prob[p, c] and np.array_equal(r[2:], boxes[p])


# ------------------------------------------------------------------------------------------------ FP32 route
def test_add_relu_quantize_is_the_pinned_quantizer_applied_to_the_fp32_sum():
    g = np.random.default_rng(4)
    a, b = g.normal(0, 3, 5000).astype(np.float32), g.normal(0, 3, 5000).astype(np.float32)
    q = np.float32(0.037)
    want = o.quantize(np.maximum(a + b, np.float32(0)), q, o.U8)
    assert np.array_equal(o.add_relu_quantize(a, b, q), want)
    # powers of two: exact by hand
    assert list(o.add_relu_quantize(np.float32([1.0, -3.0, 0.75, 100.0]), np.float32([0.5, 1.0, 0.5, 100.0]), 0.5)) == [3, 0, 2, 255]

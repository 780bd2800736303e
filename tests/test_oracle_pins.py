"""Pins of the CPU oracle against things other than itself.

The paper prints no worked numeric example, so each oracle function is held to
closed forms, hand-evaluated cases (tests/golden), invariants, special cases
that reduce to a library routine, and an independent brute-force formulation.
Each pin is chosen so that a plausible slip (dropped term, wrong sign or
index, transposed operand, wrong rounding mode) fails at least one of them.
"""
import os
from fractions import Fraction

import numpy as np
import pytest
import torch
import torch.nn.functional as F

import oracle as o

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ----------------------------------------------------------------------------- quantizer, Eq. (Q)
def _golden_cases():
    rows = []
    with open(os.path.join(GOLDEN, "quantizer_cases.txt")) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                r, q, lo, hi, z = line.split()
                rows.append((float(r), float(q), float(lo), float(hi), int(z)))
    return rows


@pytest.mark.parametrize("r,q,lo,hi,z", _golden_cases())
def test_quantize_hand_cases(r, q, lo, hi, z):
    assert int(o.quantize(np.array([r]), q, lo=lo, hi=hi)[0]) == z


def test_quantize_literal_bounds_of_eq_Q():
    assert o.bounds_p(8) == (-256.0, 255.0) and o.bounds_p(7) == (-128.0, 127.0)
    lo, hi = o.bounds_p(31)
    z = o.quantize(np.array([1e20, -1e20, 3.0]), 1.0, lo=lo, hi=hi)
    assert z.tolist() == [2 ** 31 - 1, -2 ** 31, 3]


def test_factor_maps_max_to_top_code():
    g = np.random.default_rng(1)
    for _ in range(200):
        m = float(np.float32(g.uniform(1e-3, 1e3)))
        q8 = o.factor(m, 8)
        q7 = o.factor(m, 7)
        assert o.quantize(np.array([m]), q8, o.U8)[0] == 255
        assert o.quantize(np.array([m, -m]), q7, o.S8).tolist() == [127, -127]
    assert o.factor(255.0, 8) == 1.0 and o.factor(127.0, 7) == 1.0
    assert o.factor(0.0, 8) == 1.0  # all-zero tensor: factor 1 keeps Q defined
    assert o.factor(2.0 ** 31 - 1, 31) == 1.0


def test_quantize_roundtrip_error_bound_and_saturation():
    g = np.random.default_rng(2)
    r = g.standard_normal(200000).astype(np.float32) * 3
    m = o.maxabs(r)
    q = o.factor(m, 7)
    z = o.quantize(r, q, o.S8)
    back = o.dequantize(z, q)
    # inside the clamp range the error is at most half a step (plus the fp32 rounding of r/q and q*z)
    assert np.all(np.abs(back.astype(np.float64) - r) <= 0.5 * q * (1 + 2.0 ** -20))
    # outside: exact saturation
    big = np.array([3 * m, -3 * m, 1e30, -1e30, np.inf, -np.inf], dtype=np.float32)
    assert o.quantize(big, q, o.S8).tolist() == [127, -128, 127, -128, 127, -128]
    assert o.quantize(big, q, o.U8).tolist() == [255, 0, 255, 0, 255, 0]


def test_quantize_matches_exact_rational_rounding():
    """Independent formulation: fp32 quotient (numpy), then exact half-even rounding with rationals."""
    g = np.random.default_rng(3)
    r = (g.standard_normal(5000) * 40).astype(np.float32)
    # add exact ties: (k + 0.5) * q with q a power of two
    q = np.float32(0.25)
    ties = ((np.arange(-300, 300) + 0.5) * q).astype(np.float32)
    r = np.concatenate([r, ties])
    z = o.quantize(r, q, lo=-256.0, hi=255.0)
    for ri, zi in zip(r, z):
        t = Fraction(float(np.float32(ri) / q))  # fp32 division, exact value of the result
        fl = t.numerator // t.denominator
        frac = t - fl
        if frac > Fraction(1, 2) or (frac == Fraction(1, 2) and fl % 2 == 1):
            fl += 1
        assert zi == min(max(fl, -256), 255)


def test_quantize_uses_division_not_reciprocal():
    # r/q and r*(1/q) differ for some fp32 pairs; the oracle must take the quotient.
    g = np.random.default_rng(4)
    r = g.uniform(0, 1000, 400000).astype(np.float32)
    q = np.float32(0.0437)
    want = np.rint(r / q).astype(np.int64)
    got = o.quantize(r, q, lo=-2.0 ** 31, hi=2.0 ** 31 - 1)
    assert np.array_equal(got, want)
    assert np.any(np.rint(r * (np.float32(1) / q)).astype(np.int64) != want)


# ----------------------------------------------------------------------------- D, max-abs
def test_dequantize_is_q_times_z():
    z = np.arange(-128, 128, dtype=np.int32)
    q = np.float32(0.0371)
    assert np.array_equal(o.dequantize(z, q), q * z.astype(np.float32))
    assert o.dequantize(np.array([3]), 0.5)[0] == 1.5


def test_maxabs_sequential_and_running():
    g = np.random.default_rng(5)
    r = g.standard_normal(100001).astype(np.float32)
    r[777] = -9.5
    assert o.maxabs(r) == 9.5
    assert o.maxabs(r, init=11.0) == 11.0
    assert o.maxabs(np.zeros(5, np.float32)) == 0.0
    assert o.maxabs(r[:10]) == float(np.max(np.abs(r[:10])))


# ----------------------------------------------------------------------------- "+" of Eq. (arithmetics)
def test_eltwise_add_uses_max_factor():
    # D: 10*0.5 + 3*0.25 = 5.75; factor max(0.5,0.25)=0.5 -> 11.5 -> even -> 12  (min would give 23)
    z, qo = o.eltwise_add(np.array([10]), 0.5, np.array([3]), 0.25, *o.bounds_p(8))
    assert qo == 0.5 and z.tolist() == [12]
    z2, qo2 = o.eltwise_add(np.array([3]), 0.25, np.array([10]), 0.5, *o.bounds_p(8))
    assert qo2 == 0.5 and z2.tolist() == [12]  # commutative
    # saturation at 2^p - 1 and at -2^p
    z3, _ = o.eltwise_add(np.array([200, -200]), 1.0, np.array([200, -200]), 1.0, *o.bounds_p(8))
    assert z3.tolist() == [255, -256]
    # equal factors: plain integer addition
    a = np.arange(-50, 50)
    z4, _ = o.eltwise_add(a, 0.125, a[::-1].copy(), 0.125, *o.bounds_p(8))
    assert np.array_equal(z4, a + a[::-1])


# ----------------------------------------------------------------------------- BN folding closed form
def test_fold_bn_equals_conv_then_bn_fp64():
    g = np.random.default_rng(6)
    K, R, S, C = 8, 3, 3, 5
    w = g.standard_normal((K, R, S, C)).astype(np.float32)
    b = g.standard_normal(K).astype(np.float32)
    gamma = g.uniform(0.5, 1.5, K).astype(np.float32)
    beta = g.standard_normal(K).astype(np.float32)
    mean = g.standard_normal(K).astype(np.float32)
    var = g.uniform(0.5, 1.5, K).astype(np.float32)
    eps = 1e-5
    x = torch.from_numpy(g.standard_normal((2, C, 9, 9)))
    for bias in (b, None):
        wf, bf = o.fold_bn(w, bias, gamma, beta, mean, var, eps, f64=True)
        # library routine: conv then batch_norm in eval mode, all fp64
        y = F.conv2d(x, torch.from_numpy(w).double().permute(0, 3, 1, 2),
                     torch.from_numpy(bias).double() if bias is not None else None, padding=1)
        y = F.batch_norm(y, torch.from_numpy(mean).double(), torch.from_numpy(var).double(),
                         torch.from_numpy(gamma).double(), torch.from_numpy(beta).double(), False, 0.0, eps)
        yf = F.conv2d(x, torch.from_numpy(wf).permute(0, 3, 1, 2), torch.from_numpy(bf), padding=1)
        rel = (y - yf).abs().max() / y.abs().max()
        assert rel < 1e-12
        # fp32 parameters are those values rounded once
        w32, b32 = o.fold_bn(w, bias, gamma, beta, mean, var, eps)
        assert np.array_equal(w32, wf.astype(np.float32)) and np.array_equal(b32, bf.astype(np.float32))


# ----------------------------------------------------------------------------- integer convolution
def _im2col_reference(x, w, bias, stride, pad, dil):
    """Second formulation: explicit patch matrix and an int64 matrix product."""
    N, H, W, C = x.shape
    K, R, S, _ = w.shape
    P = (H + 2 * pad[0] - dil[0] * (R - 1) - 1) // stride[0] + 1
    Q = (W + 2 * pad[1] - dil[1] * (S - 1) - 1) // stride[1] + 1
    xp = np.zeros((N, H + 2 * pad[0], W + 2 * pad[1], C), dtype=np.int64)
    xp[:, pad[0]:pad[0] + H, pad[1]:pad[1] + W] = x.astype(np.int64)
    cols = np.empty((N, P, Q, R, S, C), dtype=np.int64)
    for r in range(R):
        for s in range(S):
            cols[:, :, :, r, s] = xp[:, r * dil[0]: r * dil[0] + (P - 1) * stride[0] + 1: stride[0],
                                     s * dil[1]: s * dil[1] + (Q - 1) * stride[1] + 1: stride[1]]
    out = cols.reshape(N * P * Q, R * S * C) @ w.astype(np.int64).reshape(K, -1).T
    if bias is not None:
        out = out + bias.astype(np.int64)
    return out.reshape(N, P, Q, K)


def test_conv_hand_cases():
    # 1x1x1: a single product, u8 vs s8 reading of the same byte
    x = np.array([[[[200]]]], dtype=np.uint8)
    w = np.array([[[[-3]]]], dtype=np.int8)
    assert o.conv_acc(x, w)[0, 0, 0, 0] == -600
    assert o.conv_acc(x.view(np.int8), w)[0, 0, 0, 0] == 168  # 200 as s8 is -56
    assert o.conv_acc(x, w, bias=np.array([-7]))[0, 0, 0, 0] == -607
    # all-ones 3x3 over all-ones 3x3 image with zero padding: counts of in-image taps
    ones = o.conv_acc(np.ones((1, 3, 3, 1), np.uint8), np.ones((1, 3, 3, 1), np.int8), pad=(1, 1))
    assert ones[0, :, :, 0].tolist() == [[4, 6, 4], [6, 9, 6], [4, 6, 4]]
    # identity 1x1 weights copy the input
    g = np.random.default_rng(7)
    xi = g.integers(0, 256, (2, 5, 4, 6), dtype=np.uint8)
    assert np.array_equal(o.conv_acc(xi, np.eye(6, dtype=np.int8).reshape(6, 1, 1, 6)), xi.astype(np.int32))
    # a one-hot 3x3 tap shifts the image: tap (r=0,s=2) reads x[p-1, q+1]
    wshift = np.zeros((1, 3, 3, 1), np.int8)
    wshift[0, 0, 2, 0] = 1
    img = np.arange(1, 13, dtype=np.uint8).reshape(1, 3, 4, 1)
    got = o.conv_acc(img, wshift, pad=(1, 1))[0, :, :, 0]
    want = np.zeros((3, 4), np.int32)
    want[1:, :3] = img[0, :2, 1:, 0]
    assert np.array_equal(got, want)


CONV_CASES = [
    # N  H   W   C   K  R  S  stride  pad     dil
    (2, 9, 7, 5, 4, 3, 3, (1, 1), (1, 1), (1, 1)),
    (1, 12, 10, 3, 6, 7, 7, (2, 2), (3, 3), (1, 1)),
    (2, 8, 8, 16, 8, 1, 1, (2, 2), (0, 0), (1, 1)),
    (1, 11, 9, 4, 5, 1, 7, (1, 1), (0, 3), (1, 1)),
    (1, 9, 11, 4, 5, 7, 1, (1, 1), (3, 0), (1, 1)),
    (1, 19, 19, 8, 4, 3, 3, (1, 1), (6, 6), (6, 6)),
    (1, 10, 13, 2, 3, 3, 2, (2, 1), (1, 0), (1, 2)),
    (3, 5, 5, 7, 9, 5, 5, (1, 1), (2, 2), (1, 1)),
]


@pytest.mark.parametrize("case", CONV_CASES)
@pytest.mark.parametrize("signed", [False, True])
def test_conv_against_im2col_and_library(case, signed):
    N, H, W, C, K, R, S, stride, pad, dil = case
    g = np.random.default_rng(hash(case) % 2 ** 31)
    x = g.integers(-128, 128, (N, H, W, C)).astype(np.int8) if signed else g.integers(0, 256, (N, H, W, C), dtype=np.uint8)
    w = g.integers(-128, 128, (K, R, S, C)).astype(np.int8)
    bias = g.integers(-10000, 10000, K).astype(np.int32)
    got = o.conv_acc(x, w, bias, stride, pad, dil)
    assert np.array_equal(got, _im2col_reference(x, w, bias, stride, pad, dil))
    # third witness: the library's fp64 convolution is exact on these integers
    yt = F.conv2d(torch.from_numpy(x.astype(np.float64)).permute(0, 3, 1, 2),
                  torch.from_numpy(w.astype(np.float64)).permute(0, 3, 1, 2),
                  torch.from_numpy(bias.astype(np.float64)), stride=stride, padding=pad, dilation=dil)
    assert np.array_equal(got, yt.permute(0, 2, 3, 1).numpy().astype(np.int64))
    # threads only split the batch
    assert np.array_equal(got, o.conv_acc(x, w, bias, stride, pad, dil, threads=3))


# ----------------------------------------------------------------------------- epilogue
def test_epilogue_identity_clamp_and_relu():
    acc = np.array([[-300, -128, -1, 0, 1, 127, 128, 255, 256, 100000]], dtype=np.int32)
    assert o.epilogue(acc, 1.0, y_type=o.U8).tolist() == [[0, 0, 0, 0, 1, 127, 128, 255, 255, 255]]
    assert o.epilogue(acc, 1.0, y_type=o.S8).tolist() == [[-128, -128, -1, 0, 1, 127, 127, 127, 127, 127]]
    # ReLU before a u8 clamp changes nothing; before s8 it removes negatives
    assert np.array_equal(o.epilogue(acc, 1.0, relu=True, y_type=o.U8), o.epilogue(acc, 1.0, y_type=o.U8))
    assert o.epilogue(acc, 1.0, relu=True, y_type=o.S8).tolist() == [[0, 0, 0, 0, 1, 127, 127, 127, 127, 127]]
    assert np.array_equal(o.epilogue(acc, 1.0, y_type=o.S32), acc)


def test_epilogue_ties_and_scale():
    acc = np.array([[1, 3, 5, 7, -1, -3, -5]], dtype=np.int32)
    assert o.epilogue(acc, 0.5, y_type=o.S8).tolist() == [[0, 2, 2, 4, 0, -2, -2]]
    # per-channel scales
    acc2 = np.array([[10, 10, 10], [20, 20, 20]], dtype=np.int32)
    assert o.epilogue(acc2, np.array([0.5, 1.0, 2.0]), y_type=o.U8).tolist() == [[5, 10, 20], [10, 20, 40]]
    # fp32 output is float(acc) * s
    f = o.epilogue(acc, 0.3, y_type=o.F32)
    assert np.array_equal(f, acc.astype(np.float32) * np.float32(0.3))


def test_epilogue_residual():
    acc = np.array([[10, -20, 30, 250]], dtype=np.int32)
    res = np.array([[5, 7, 9, 11]], dtype=np.uint8)
    assert o.epilogue(acc, 1.0, residual=res, res_scale=1.0, y_type=o.U8).tolist() == [[15, 0, 39, 255]]
    assert o.epilogue(acc, 1.0, residual=res.view(np.int8), res_scale=-1.0, y_type=o.S8).tolist() == [[5, -27, 21, 127]]
    # signed residual bytes
    sres = np.array([[-5, -7, 100, -128]], dtype=np.int8)
    assert o.epilogue(acc, 1.0, residual=sres, res_scale=1.0, y_type=o.S8).tolist() == [[5, -27, 127, 122]]
    # product and sum are rounded separately (numpy fp32 ops as the independent witness)
    g = np.random.default_rng(8)
    a = g.integers(-2 ** 20, 2 ** 20, (64, 32)).astype(np.int32)
    r = g.integers(0, 256, (64, 32), dtype=np.uint8)
    s, sr = np.float32(1.1920929e-3), np.float32(0.7310586)
    want = a.astype(np.float32) * s
    want = want + r.astype(np.float32) * sr
    got = o.epilogue(a, s, residual=r, res_scale=sr, y_type=o.F32)
    assert np.array_equal(got, want)
    fused = (a.astype(np.float64) * np.float64(s) + r.astype(np.float64) * np.float64(sr)).astype(np.float32)
    assert np.any(fused != want)  # the case set does distinguish single from double rounding
    assert np.array_equal(o.epilogue(a, s, residual=r, res_scale=sr, relu=True, y_type=o.U8),
                          np.clip(np.rint(np.maximum(want, 0)), 0, 255).astype(np.uint8))


def test_epilogue_writes_channel_slice():
    acc = np.arange(12, dtype=np.int32).reshape(4, 3)
    out = np.full((4, 8), 99, dtype=np.uint8)
    o.epilogue(acc, 1.0, y_type=o.U8, out=out, c_off=2)
    assert np.array_equal(out[:, 2:5], acc.astype(np.uint8))
    assert np.all(out[:, :2] == 99) and np.all(out[:, 5:] == 99)


def test_requant_scale_and_bias_factor():
    qx, qw, qy = np.float32(0.0123), np.float32(0.00371), np.float32(0.0456)
    assert o.requant_scale(qx, qw, qy) == float(np.float32(np.float64(qx) * np.float64(qw) / np.float64(qy)))
    assert o.bias_factor(qx, qw) == float(qx * qw)
    assert o.requant_scale(2.0, 3.0, 4.0) == 1.5 and o.bias_factor(0.5, 0.25) == 0.125


def test_affine_layer_matches_real_arithmetic_within_quantization_error():
    """Eq. (int8_affine) end to end: the quantized layer approximates ReLU(Wx+b) to within the
    error budget implied by the factors (a dropped bias or a wrong scale breaks this)."""
    g = np.random.default_rng(9)
    x = np.maximum(g.standard_normal((1, 6, 6, 32)), 0).astype(np.float32)
    w = (g.standard_normal((16, 3, 3, 32)) * 0.05).astype(np.float32)
    b = (g.standard_normal(16) * 0.5).astype(np.float32)
    ref = F.conv2d(torch.from_numpy(x).double().permute(0, 3, 1, 2), torch.from_numpy(w).double().permute(0, 3, 1, 2),
                   torch.from_numpy(b).double(), padding=1).clamp(min=0).permute(0, 2, 3, 1).numpy()
    qx, qw = o.factor(o.maxabs(x), 8), o.factor(o.maxabs(w), 7)
    qy = o.factor(float(ref.max()), 8)
    xq, wq = o.quantize(x, qx, o.U8), o.quantize(w, qw, o.S8)
    bq = o.quantize(b, o.bias_factor(qx, qw), o.S32)
    y = o.conv2d(xq, wq, bq, o.requant_scale(qx, qw, qy), pad=(1, 1), relu=True, y_type=o.U8)
    err = np.abs(o.dequantize(y, qy) - ref)
    # per-output bound: sum over taps of (|x| qw/2 + |w| qx/2 + qx qw/4) + qy/2
    bound = 288 * (x.max() * qw / 2 + np.abs(w).max() * qx / 2 + qx * qw / 4) + qy / 2
    assert err.max() < bound and err.mean() < 0.05 * ref.max()
    assert y.max() == 255


# ----------------------------------------------------------------------------- concat, pools
def test_concat_shared_factor():
    g = np.random.default_rng(10)
    a = g.integers(0, 256, (2, 3, 3, 4), dtype=np.uint8)
    b = g.integers(0, 256, (2, 3, 3, 6), dtype=np.uint8)
    assert np.array_equal(o.concat([a, b], [0.5, 0.5], 0.5), np.concatenate([a, b], axis=-1))
    y = o.concat([a, b], [0.25, 0.5], 0.5)
    assert np.array_equal(y[..., 4:], b)
    assert np.array_equal(y[..., :4], np.rint(a.astype(np.float32) * np.float32(0.5)).astype(np.uint8))
    s = g.integers(-128, 128, (1, 2, 2, 3)).astype(np.int8)
    ys = o.concat([s], [1.0], 0.75)
    sc = np.float32(np.float64(np.float32(1.0)) / np.float64(np.float32(0.75)))
    assert np.array_equal(ys, np.clip(np.rint(s.astype(np.float32) * sc), -128, 127).astype(np.int8))


@pytest.mark.parametrize("k,st,pad,ceil", [(3, 2, 1, False), (2, 2, 0, True), (3, 1, 1, False), (3, 2, 0, False)])
def test_pools_against_library(k, st, pad, ceil):
    g = np.random.default_rng(11)
    x = g.integers(0, 256, (2, 9, 11, 5), dtype=np.uint8)
    xt = torch.from_numpy(x.astype(np.float64)).permute(0, 3, 1, 2)
    mp = F.max_pool2d(xt, k, st, pad, ceil_mode=ceil).permute(0, 2, 3, 1).numpy()
    assert np.array_equal(o.pool(x, "max", (k, k), (st, st), (pad, pad), ceil), mp.astype(np.uint8))
    if not ceil:
        sums = F.avg_pool2d(xt, k, st, pad, count_include_pad=True, divisor_override=1).permute(0, 2, 3, 1).numpy()
        want = np.rint(sums.astype(np.float32) * (np.float32(1) / np.float32(k * k))).astype(np.uint8)
        assert np.array_equal(o.pool(x, "avg", (k, k), (st, st), (pad, pad), ceil), want)
    # average pooling in both modes, signed input too, against window sums taken by slicing a zero-embedded copy
    # (cells outside the image count as zeros, the divisor is the full window; ceil mode only adds windows)
    for arr in (x, x.view(np.int8)):
        N, H, W, C = arr.shape
        P, Q = o.pool_out(H, k, st, pad, ceil), o.pool_out(W, k, st, pad, ceil)
        big = np.zeros((N, pad + (P - 1) * st + k + pad, pad + (Q - 1) * st + k + pad, C), dtype=np.int64)
        big[:, pad:pad + H, pad:pad + W, :] = arr
        want = np.empty((N, P, Q, C), dtype=arr.dtype)
        for pi in range(P):
            for qi in range(Q):
                sums = big[:, pi * st:pi * st + k, qi * st:qi * st + k, :].sum(axis=(1, 2))
                want[:, pi, qi, :] = np.rint(sums.astype(np.float32) * (np.float32(1) / np.float32(k * k))).astype(arr.dtype)
        assert np.array_equal(o.pool(arr, "avg", (k, k), (st, st), (pad, pad), ceil), want)


def test_pool_ceil_mode_extent():
    assert o.pool_out(75, 2, 2, 0, True) == 38 and o.pool_out(75, 2, 2, 0, False) == 37
    assert o.pool_out(112, 3, 2, 1, False) == 56 and o.pool_out(147, 3, 2, 0, False) == 73


# ----------------------------------------------------------------------------- multiplier and dequantizer, by properties
def test_requant_scale_exact_on_powers_of_two_and_single_rounding():
    """s = q_x q_w / q_y: with powers of two every step is exact, so the value is known without any formula of the
    test's own; for general factors the result is the fp32 nearest to the exact rational (one rounding), which the
    rational arithmetic of Python's fractions decides."""
    from fractions import Fraction
    assert o.requant_scale(0.5, 0.25, 0.125) == 1.0
    assert o.requant_scale(2.0 ** -7, 2.0 ** -9, 2.0 ** -3) == 2.0 ** -13
    assert o.requant_scale(0.5, 0.25, 0.25) == 2 * o.requant_scale(0.5, 0.25, 0.5)
    g = np.random.default_rng(12)
    for _ in range(200):
        qx, qw, qy = (float(np.float32(v)) for v in g.uniform(1e-4, 2.0, 3))
        exact = Fraction(qx) * Fraction(qw) / Fraction(qy)
        s = float(o.requant_scale(qx, qw, qy))
        lo, hi = float(np.nextafter(np.float32(s), np.float32(-np.inf))), float(np.nextafter(np.float32(s), np.float32(np.inf)))
        assert abs(Fraction(s) - exact) <= abs(Fraction(lo) - exact) and abs(Fraction(s) - exact) <= abs(Fraction(hi) - exact)


def test_dequantize_is_one_fp32_product():
    """r' = q z: exact for power-of-two factors, odd in z, and the fp32 nearest to the exact product otherwise."""
    from fractions import Fraction
    z = np.arange(-128, 128, dtype=np.int8)
    assert np.array_equal(o.dequantize(z, 0.25), z.astype(np.float32) / 4)
    assert np.array_equal(o.dequantize(z[1:], 0.3), -o.dequantize((-z[1:].astype(np.int16)).astype(np.int8), 0.3))
    q = float(np.float32(0.0123))
    got = o.dequantize(np.array([77, 255], dtype=np.uint8), q)
    for v, zz in zip(got, (77, 255)):
        exact = Fraction(q) * zz
        near = [float(v), float(np.nextafter(v, np.float32(-np.inf))), float(np.nextafter(v, np.float32(np.inf)))]
        assert min(near, key=lambda c: abs(Fraction(c) - exact)) == float(v)
    big = o.dequantize(np.array([2 ** 30 + 12345, -(2 ** 31)], dtype=np.int32), 0.5)    # int32 -> fp32 rounds first
    assert big[0] == np.float32(2 ** 30 + 12345) * np.float32(0.5) and big[1] == -(2.0 ** 30)


def test_avgpool_3x3_is_nearest_integer_division_for_every_window_sum():
    """A 3x3 window sum n is never half-way between multiples of 9, so clamp(Round(float(n) * fp32(1/9))) must be
    the integer nearest to n / 9 (Python integers decide) for every sum a window of u8 or s8 codes can have.  The
    images hold one window each, chosen so that all sums 0..2295 and -1152..1143 occur."""
    for dt, lo, hi in ((np.uint8, 0, 255), (np.int8, -128, 127)):
        sums = np.arange(9 * lo, 9 * hi + 1)
        base, extra = np.divmod(sums - 9 * lo, 9)                     # nine cells: base each, `extra` of them one more
        cells = lo + base[:, None] + (np.arange(9)[None, :] < extra[:, None])
        assert np.array_equal(cells.sum(1), sums) and cells.min() >= lo and cells.max() <= hi
        x = cells.astype(dt).reshape(-1, 3, 3, 1)
        got = o.pool(x, "avg", (3, 3), (1, 1), (0, 0)).reshape(-1).astype(np.int64)
        want = np.array([(2 * int(n) + 9) // 18 for n in sums])       # floor(n/9 + 1/2); no ties exist
        assert np.array_equal(got, want)


def test_single_fused_multiply_add_form_of_the_3x3_average():
    """Host check of the arithmetic the strip pooling kernels use: with B = 9 * 2^20, fma(float(B + n), fp32(1/9),
    1.5 * 2^23 - 2^20) rounds once at unit spacing and leaves Round(n / 9) in the low mantissa bits.  The fused
    operation is evaluated exactly here (a 24 x 24 bit product fits a double; the sum with an integer below 2^24 is
    then rounded half to even to an integer), for every n a window can produce (signed sums shifted by 9 * 128)."""
    inv = np.float32(1.0) / np.float32(9.0)
    B = 9 * 2 ** 20
    for n in range(0, 9 * 255 + 1):
        x = np.float32(B + n)
        assert int(x) == B + n                                        # representable: below 2^24
        exact = float(np.float64(x) * np.float64(inv))                # exact product
        assert 2 ** 23 <= exact + (1.5 * 2 ** 23 - 2 ** 20) < 2 ** 24 # the sum lands where fp32 spacing is 1
        z = int(np.rint(exact)) - 2 ** 20                             # the integer constant only shifts the result
        assert z == (2 * n + 9) // 18

"""GPU parity of the bandwidth-bound kernels against the CPU oracle (bit-exact)."""
import numpy as np
import pytest
import torch

import oracle as o

pytestmark = pytest.mark.gpu


def _cuda(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


@pytest.mark.parametrize("n", [0, 1, 5, 16, 1000, 4099, 1 << 20, (1 << 22) + 13])
def test_maxabs_matches_sequential_scan(q8, n):
    g = np.random.default_rng(n)
    r = (g.standard_normal(n) * 3).astype(np.float32)
    slot = torch.zeros(1, dtype=torch.float32, device="cuda")
    q8.q8_calibrate_maxabs(_cuda(r), slot)
    assert slot.item() == o.maxabs(r)
    # running maximum over a second batch, and an unaligned view
    r2 = (g.standard_normal(n + 3) * 2).astype(np.float32)
    t2 = _cuda(r2)
    q8.q8_calibrate_maxabs(t2[1:], slot)
    assert slot.item() == o.maxabs(r2[1:], init=o.maxabs(r))


@pytest.mark.parametrize("out_type,otype", [(0, o.U8), (1, o.S8), (2, o.S32)])
@pytest.mark.parametrize("n", [1, 15, 16, 17, 4099, (1 << 20) + 7])
def test_quantize_bit_exact(q8, out_type, otype, n):
    g = np.random.default_rng(n + out_type)
    r = (g.standard_normal(n) * 50).astype(np.float32)
    r[: min(n, 8)] = np.array([0.5, 1.5, 2.5, -0.5, -1.5, 1e30, -1e30, 254.5], dtype=np.float32)[: min(n, 8)]
    for qf in (1.0, 0.0437, 0.25):
        got = q8.q8_quantize(_cuda(r), qf, out_type).cpu().numpy()
        assert np.array_equal(got, o.quantize(r, qf, otype))
    # unaligned input view takes the scalar path
    t = _cuda(np.concatenate([[0], r]).astype(np.float32))
    got = q8.q8_quantize(t[1:], 0.0437, out_type).cpu().numpy()
    assert np.array_equal(got, o.quantize(r, 0.0437, otype))


def test_quantize_calibrated_extremes(q8):
    g = np.random.default_rng(3)
    r = np.maximum(g.standard_normal(100000), 0).astype(np.float32)
    slot = torch.zeros(1, dtype=torch.float32, device="cuda")
    q8.q8_calibrate_maxabs(_cuda(r), slot)
    qf = q8.q8_factor(slot.item(), 8)
    assert qf == o.factor(o.maxabs(r), 8)
    z = q8.q8_quantize(_cuda(r), qf, 0)
    assert int(z.max()) == 255 and np.array_equal(z.cpu().numpy(), o.quantize(r, qf, o.U8))


@pytest.mark.parametrize("C,C_pad,out", [(3, 16, 1), (3, 16, 0), (20, 32, 1), (5, 8, 1), (16, 16, 0)])
def test_quantize_pad_channels(q8, C, C_pad, out):
    g = np.random.default_rng(4 + C)
    x = (g.standard_normal((2, 37, 41, C)) * 2).astype(np.float32)
    got = q8.q8_quantize_pad_channels(_cuda(x), C_pad, 0.02, out).cpu().numpy()
    assert got.shape == (2, 37, 41, C_pad)
    assert np.array_equal(got[..., :C], o.quantize(x, 0.02, o.S8 if out else o.U8)) and np.all(got[..., C:] == 0)


@pytest.mark.parametrize("dt", [np.uint8, np.int8, np.int32])
@pytest.mark.parametrize("n", [1, 16, 33, 100003])
def test_dequantize_bit_exact(q8, dt, n):
    g = np.random.default_rng(n)
    info = np.iinfo(dt)
    z = g.integers(max(info.min, -10 ** 6), min(info.max, 10 ** 6) + 1, n).astype(dt)
    got = q8.q8_dequantize(_cuda(z), 0.0371).cpu().numpy()
    assert np.array_equal(got, o.dequantize(z, 0.0371))


def test_fold_bn_bit_exact(q8):
    g = np.random.default_rng(5)
    K, R, S, C = 37, 3, 3, 20
    w = g.standard_normal((K, R, S, C)).astype(np.float32)
    b = g.standard_normal(K).astype(np.float32)
    gamma = g.uniform(0.5, 1.5, K).astype(np.float32)
    beta = g.standard_normal(K).astype(np.float32)
    mean = g.standard_normal(K).astype(np.float32)
    var = g.uniform(0.5, 1.5, K).astype(np.float32)
    for bias in (b, None):
        wf, bf = q8.q8_fold_bn(_cuda(w), _cuda(bias) if bias is not None else None, _cuda(gamma), _cuda(beta),
                               _cuda(mean), _cuda(var), 1e-5)
        wo, bo = o.fold_bn(w, bias, gamma, beta, mean, var, 1e-5)
        assert np.array_equal(wf.cpu().numpy(), wo) and np.array_equal(bf.cpu().numpy(), bo)


@pytest.mark.parametrize("chans", [(16, 32), (64, 96, 32), (5, 7), (48,)])
@pytest.mark.parametrize("signed", [False, True])
def test_concat_bit_exact(q8, chans, signed):
    g = np.random.default_rng(sum(chans))
    dt = np.int8 if signed else np.uint8
    lo, hi = (-128, 128) if signed else (0, 256)
    xs = [g.integers(lo, hi, (2, 5, 6, c)).astype(dt) for c in chans]
    fac = [float(np.float32(0.01 * (i + 1))) for i in range(len(chans))]
    # the shared factor as the rule gives it (multipliers <= 1, no clamp can act), and a smaller one (multipliers
    # > 1: codes saturate)
    for out_f in (max(fac), min(fac) * 0.75):
        got = q8.q8_concat([_cuda(a) for a in xs], fac, out_f).cpu().numpy()
        assert np.array_equal(got, o.concat(xs, fac, out_f))


@pytest.mark.parametrize("signed", [False, True])
def test_concat_one_launch_many_blocks_per_branch(q8, signed):
    """All branches 16-byte aligned: one launch whose blocks are split between the branches; a copied branch, one
    with a multiplier below one, one above one, and a single-group branch, over enough pixels for many blocks each."""
    g = np.random.default_rng(77)
    dt = np.int8 if signed else np.uint8
    lo, hi = (-128, 128) if signed else (0, 256)
    chans = (192, 16, 64, 128)
    fac = [0.02, 0.013, 0.031, 0.0071]
    xs = [g.integers(lo, hi, (3, 71, 53, c)).astype(dt) for c in chans]
    got = q8.q8_concat([_cuda(a) for a in xs], fac, 0.02).cpu().numpy()
    assert np.array_equal(got, o.concat(xs, fac, 0.02))


@pytest.mark.parametrize("k,st,pad,ceil", [(3, 2, 1, False), (2, 2, 0, True), (3, 1, 1, False), (3, 2, 0, False), (7, 1, 0, False)])
@pytest.mark.parametrize("C", [64, 48, 12, 5])
def test_pools_bit_exact(q8, k, st, pad, ceil, C):
    g = np.random.default_rng(k * 10 + C)
    x = g.integers(0, 256, (2, 15, 13, C), dtype=np.uint8)
    got = q8.q8_maxpool2d(_cuda(x), (k, k), (st, st), (pad, pad), ceil).cpu().numpy()
    assert np.array_equal(got, o.pool(x, "max", (k, k), (st, st), (pad, pad), ceil))
    got = q8.q8_avgpool2d(_cuda(x), (k, k), (st, st), (pad, pad), ceil).cpu().numpy()
    assert np.array_equal(got, o.pool(x, "avg", (k, k), (st, st), (pad, pad), ceil))
    xs = x.view(np.int8)
    got = q8.q8_maxpool2d(_cuda(xs), (k, k), (st, st), (pad, pad), ceil).cpu().numpy()
    assert np.array_equal(got, o.pool(xs, "max", (k, k), (st, st), (pad, pad), ceil))
    got = q8.q8_avgpool2d(_cuda(xs), (k, k), (st, st), (pad, pad), ceil).cpu().numpy()
    assert np.array_equal(got, o.pool(xs, "avg", (k, k), (st, st), (pad, pad), ceil))


@pytest.mark.parametrize("st,pad,ceil", [(1, 1, False), (2, 1, False), (2, 0, True), (1, 0, False), (2, 2, False)])
def test_3x3_pools_in_row_strips_bit_exact(q8, st, pad, ceil):
    """Tensors large enough for the strip kernel (eight output rows per thread): ragged last strip, both strides,
    padding 0 to 2, extreme codes in the corners, u8 and s8."""
    g = np.random.default_rng(31 * st + pad)
    x = g.integers(0, 256, (16, 61, 52, 128), dtype=np.uint8)
    x[:, :2, :2, :] = 255
    x[:, -2:, -2:, :] = 0
    for arr in (x, x.view(np.int8)):
        for kind, fn in (("max", q8.q8_maxpool2d), ("avg", q8.q8_avgpool2d)):
            got = fn(_cuda(arr), (3, 3), (st, st), (pad, pad), ceil).cpu().numpy()
            assert np.array_equal(got, o.pool(arr, kind, (3, 3), (st, st), (pad, pad), ceil)), (kind, arr.dtype)


@pytest.mark.parametrize("value,dt", [(255, np.uint8), (-128, np.int8), (127, np.int8)])
def test_avgpool_extreme_codes_largest_window(q8, value, dt):
    """A 16 x 16 window of one extreme code: the packed 16-bit lane sums may not carry into their neighbours."""
    x = np.full((1, 17, 18, 32), value, dtype=dt)
    x[0, 3, 4, 5] = 0
    got = q8.q8_avgpool2d(_cuda(x), (16, 16), (1, 1), (0, 0), False).cpu().numpy()
    assert np.array_equal(got, o.pool(x, "avg", (16, 16), (1, 1), (0, 0), False))


@pytest.mark.parametrize("signed", [False, True])
@pytest.mark.parametrize("ch,ldc,off", [(32, 96, 48), (20, 50, 7)])
def test_concat_branch_writes_only_its_slice(q8, signed, ch, ldc, off):
    g = np.random.default_rng(ch + ldc)
    dt, lo, hi = (np.int8, -128, 128) if signed else (np.uint8, 0, 256)
    x = g.integers(lo, hi, (3, 7, 5, ch)).astype(dt)
    y0 = g.integers(lo, hi, (3, 7, 5, ldc)).astype(dt)
    for q_in, q_out in ((0.02, 0.05), (0.05, 0.05)):
        y = _cuda(y0.copy())
        q8.q8_concat_branch(_cuda(x), q_in, q_out, y, off)
        want = y0.copy()
        want[..., off:off + ch] = o.concat([x], [q_in], q_out)
        assert np.array_equal(y.cpu().numpy(), want)


@pytest.mark.parametrize("rows,cols", [(1, 1), (7, 33), (300, 1153), (2048, 64)])
def test_per_row_maxabs_and_quantize(q8, rows, cols):
    g = np.random.default_rng(rows + cols)
    x = (g.standard_normal((rows, cols)) * g.uniform(0.01, 3.0, (rows, 1))).astype(np.float32)
    running = torch.full((rows,), 0.001, dtype=torch.float32, device="cuda")
    q8.q8_calibrate_maxabs_rows(_cuda(x), running)
    want = np.array([o.maxabs(x[r], init=0.001) for r in range(rows)], dtype=np.float32)
    assert np.array_equal(running.cpu().numpy(), want)
    q = np.array([o.factor(m, 7) for m in want], dtype=np.float32)
    for t, ot in ((1, o.S8), (0, o.U8), (2, o.S32)):
        qq = q if t != 2 else (q * np.float32(1e-3)).astype(np.float32)
        got = q8.q8_quantize_rows(_cuda(x), _cuda(qq), t).cpu().numpy()
        assert np.array_equal(got, np.stack([o.quantize(x[r], float(qq[r]), ot) for r in range(rows)]))


@pytest.mark.parametrize("W,W_pad,C,C_pad", [(41, 42, 3, 16), (40, 40, 3, 16), (7, 9, 20, 32)])
def test_quantize_pad_image(q8, W, W_pad, C, C_pad):
    g = np.random.default_rng(W + C)
    x = (g.standard_normal((2, 5, W, C)) * 2).astype(np.float32)
    got = q8.q8_quantize_pad_image(_cuda(x), W_pad, C_pad, 0.02, 1).cpu().numpy()
    assert got.shape == (2, 5, W_pad, C_pad)
    assert np.array_equal(got[:, :, :W, :C], o.quantize(x, 0.02, o.S8))
    assert np.all(got[:, :, W:, :] == 0) and np.all(got[..., C:] == 0)


@pytest.mark.parametrize("H,W,C,dt", [(7, 7, 2048, np.uint8), (8, 8, 2048, np.uint8), (5, 3, 20, np.int8), (1, 1, 4, np.int8)])
def test_global_average_pool(q8, H, W, C, dt):
    g = np.random.default_rng(H * W + C)
    lo, hi = (0, 256) if dt == np.uint8 else (-128, 128)
    x = g.integers(lo, hi, (3, H, W, C)).astype(dt)
    got = q8.q8_avgpool2d(_cuda(x), (H, W), (1, 1), (0, 0), False).cpu().numpy()
    assert np.array_equal(got, o.pool(x, "avg", (H, W), (1, 1), (0, 0), False))

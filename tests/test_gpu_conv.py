"""GPU parity of q8_conv2d (tensor-core and direct kernels) against the CPU oracle, bit-exact.

Sizes are small enough for the oracle to finish in seconds yet span several 128-row tiles and a
ragged tail in both GEMM dimensions.
"""
import numpy as np
import pytest
import torch

import oracle as o

pytestmark = pytest.mark.gpu

U8, S8, S32, F32 = 0, 1, 2, 3
OT = {U8: o.U8, S8: o.S8, S32: o.S32, F32: o.F32}


def _pair(v):
    return v if isinstance(v, tuple) else (v, v)


def _cuda(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def _bits(a):
    return a.view(np.uint32) if a.dtype == np.float32 else a


CASES = [
    # name, N,H,W,C,K,R,S,stride,pad,dil, x signed, y type, residual, relu
    ("1x1_c64_k64_raw", 2, 15, 15, 64, 64, 1, 1, 1, 0, 1, False, S32, None, False),
    ("1x1_c256_k64", 2, 15, 15, 256, 64, 1, 1, 1, 0, 1, False, U8, None, True),
    ("1x1_c64_k256_res", 2, 15, 15, 64, 256, 1, 1, 1, 0, 1, False, U8, "u8", True),
    ("1x1_c384_k64_three_blocks", 3, 21, 21, 384, 64, 1, 1, 1, 0, 1, False, U8, None, True),   # stages of 2 + 1 channel blocks
    ("1x1_c512_k128_res", 3, 21, 21, 512, 128, 1, 1, 1, 0, 1, False, U8, "u8", True),
    ("1x1_c128_k128_s8", 2, 15, 15, 128, 128, 1, 1, 1, 0, 1, True, S8, "s8", False),
    ("1x1_c32_k16", 2, 15, 15, 32, 16, 1, 1, 1, 0, 1, False, U8, None, True),
    ("1x1_c16_k24_f32", 2, 15, 15, 16, 24, 1, 1, 1, 0, 1, False, F32, None, False),
    ("3x3_c64_k64", 3, 31, 31, 64, 64, 3, 3, 1, 1, 1, False, U8, None, True),
    ("3x3_c128_k128_raw", 2, 28, 28, 128, 128, 3, 3, 1, 1, 1, False, S32, None, False),
    ("1x1s2_c256_k512", 2, 28, 28, 256, 512, 1, 1, 2, 0, 1, False, S8, None, False),
    ("3x3s2_c64_k64", 2, 33, 35, 64, 64, 3, 3, 2, 1, 1, False, U8, None, True),
    ("7x7s2_c16_k64", 2, 64, 64, 16, 64, 7, 7, 2, 3, 1, True, U8, None, True),
    ("1x7_c64_k64", 2, 33, 33, 64, 64, 1, 7, 1, (0, 3), 1, False, U8, None, True),
    ("7x1_c64_k64", 2, 33, 33, 64, 64, 7, 1, 1, (3, 0), 1, False, U8, None, True),
    ("3x3d6_c64_k64", 2, 40, 40, 64, 64, 3, 3, 1, 6, 6, False, U8, None, True),
    ("3x3_c80_k96", 2, 35, 35, 80, 96, 3, 3, 1, 1, 1, False, U8, None, True),
    ("3x3_c48_k84_f32", 2, 38, 38, 48, 84, 3, 3, 1, 1, 1, False, F32, None, False),
    ("fc_c2048_k1000", 64, 1, 1, 2048, 1000, 1, 1, 1, 0, 1, False, F32, None, False),
    ("3x3_c512_k512", 1, 16, 16, 512, 512, 3, 3, 1, 1, 1, False, U8, "u8", True),
    ("3x3_c3_k8_direct", 2, 17, 19, 3, 8, 3, 3, 2, 1, 1, True, U8, None, True),
    ("config1_shape", 1, 14, 14, 64, 64, 3, 3, 1, 1, 1, False, U8, None, True),
    # stride 2 read as pixel pairs (even W, C in 16/32/64): odd and even padding, odd and even S
    ("7x7s2_c16_k64_conv1", 2, 112, 112, 16, 64, 7, 7, 2, 3, 1, True, U8, None, True),
    ("3x3s2_c64_k96_pad1", 2, 30, 36, 64, 96, 3, 3, 2, 1, 1, False, U8, None, True),
    ("3x3s2_c32_k32_pad0", 3, 31, 34, 32, 32, 3, 3, 2, 0, 1, False, S8, None, False),
    ("2x2s2_c64_k64", 2, 20, 24, 64, 64, 2, 2, 2, 0, 1, False, U8, None, True),
    ("5x4s2_c16_k48_pad2", 2, 25, 26, 16, 48, 5, 4, 2, 2, 1, True, F32, None, False),
    # tile widths that are not a power of two times 16/32/64, channel counts padded to a 128-wide block
    ("1x1_c64_k80", 2, 37, 37, 64, 80, 1, 1, 1, 0, 1, False, U8, None, True),
    ("1x7_c160_k160", 2, 17, 17, 160, 160, 1, 7, 1, (0, 3), 1, False, U8, None, True),
    ("7x1_c160_k192_res", 2, 17, 17, 160, 192, 7, 1, 1, (3, 0), 1, False, U8, "u8", True),
    ("1x1_c768_k320_s8", 2, 17, 17, 768, 320, 1, 1, 1, 0, 1, False, S8, "s8", False),
    ("1x1_c1280_k448", 4, 8, 8, 1280, 448, 1, 1, 1, 0, 1, False, U8, None, True),
    ("3x3_c448_k384", 4, 8, 8, 448, 384, 3, 3, 1, 1, 1, False, U8, None, True),
    ("3x3_c80_k192_pad0", 2, 25, 25, 80, 192, 3, 3, 1, 0, 1, False, U8, None, True),
    ("1x1_c96_k112_f32", 2, 20, 20, 96, 112, 1, 1, 1, 0, 1, False, F32, None, False),
    ("1x1_c320_k144_raw", 2, 20, 20, 320, 144, 1, 1, 1, 0, 1, False, S32, None, False),
    ("3x3_c192_k176", 2, 20, 20, 192, 176, 3, 3, 1, 1, 1, False, U8, "u8", True),
    ("3x3_c128_k208", 2, 20, 20, 128, 208, 3, 3, 1, 1, 1, True, S8, None, False),
    ("3x3_c128_k240", 2, 20, 20, 128, 240, 3, 3, 1, 1, 1, False, U8, None, True),
    # images smaller than an accumulator tile: halo tiles with mostly empty rows instead of the fallback
    ("3x3_5x5_pad0_c128_k256", 8, 5, 5, 128, 256, 3, 3, 1, 0, 1, False, U8, None, True),
    ("3x3_3x3_pad0_c128_k256", 8, 3, 3, 128, 256, 3, 3, 1, 0, 1, False, U8, None, True),
    ("3x3_3x3_pad1_c256_k84_f32", 8, 3, 3, 256, 84, 3, 3, 1, 1, 1, False, F32, None, False),
    ("3x3_1x1_pad1_c256_k16_f32", 8, 1, 1, 256, 16, 3, 3, 1, 1, 1, False, F32, None, False),
    ("3x3_1x1_pad1_c256_k126_f32", 32, 1, 1, 256, 126, 3, 3, 1, 1, 1, False, F32, None, False),
]


def _make(case):
    name, N, H, W, C, K, R, S, st, pad, dil, xs8, ytype, res, relu = case
    st, pad, dil = _pair(st), _pair(pad), _pair(dil)
    g = np.random.default_rng(sum(map(ord, name)))
    x = g.integers(-128, 128, (N, H, W, C)).astype(np.int8) if xs8 else g.integers(0, 256, (N, H, W, C), dtype=np.uint8)
    w = g.integers(-128, 128, (K, R, S, C)).astype(np.int8)
    bias = g.integers(-5000, 5000, K).astype(np.int32)
    acc = o.conv_acc(x, w, bias, st, pad, dil, threads=8)
    P, Q = acc.shape[1:3]
    resid = None
    if res == "u8":
        resid = g.integers(0, 256, (N, P, Q, K), dtype=np.uint8)
    elif res == "s8":
        resid = g.integers(-128, 128, (N, P, Q, K)).astype(np.int8)
    return x, w, bias, acc, resid, (st, pad, dil)


@pytest.mark.parametrize("algo", [0, 2], ids=["auto", "direct"])
@pytest.mark.parametrize("case", CASES, ids=[c[0] for c in CASES])
def test_conv_matches_oracle(q8, case, algo):
    name, N, H, W, C, K, R, S, _, _, _, xs8, ytype, res, relu = case
    x, w, bias, acc, resid, (st, pad, dil) = _make(case)
    scale = np.float32(100.0 / max(1, np.abs(acc).max()))
    rs = 0.37 if resid is not None else 0.0
    want = o.epilogue(acc, scale, resid, rs, relu, OT[ytype])
    d = q8.make_conv_desc(N, H, W, C, K, R, S, st, pad, dil, S8 if xs8 else U8, S8 if res == "s8" else U8, ytype, relu,
                          1, 0, 0, algo)
    y = q8.q8_conv2d(d, _cuda(x), _cuda(w), _cuda(bias), torch.tensor([scale], device="cuda"),
                     _cuda(resid) if resid is not None else None, rs)
    q8.q8_read_status()
    assert np.array_equal(_bits(y.cpu().numpy()), _bits(want))


@pytest.mark.parametrize("xs8", [False, True])
@pytest.mark.parametrize("extra", [0, 1, 1 << 29])
def test_short_reduction_extreme_accumulators(q8, xs8, extra):
    """1x1, C = 64: accumulators at their bound (all-extreme inputs and weights) with biases that bring
    |acc + bias| to 2^22 - 1, to 2^22 and to ~2^29: int -> float conversion and scaling of extreme values."""
    N, H, W, C, K = 2, 12, 12, 64, 128
    g = np.random.default_rng(5 + extra % 7)
    x = g.integers(-128, 128, (N, H, W, C)).astype(np.int8) if xs8 else g.integers(0, 256, (N, H, W, C), dtype=np.uint8)
    w = g.integers(-128, 128, (K, 1, 1, C)).astype(np.int8)
    xmax = 128 if xs8 else 255
    x[0, 0, 0, :] = -128 if xs8 else 255          # pixel 0 with filters 0 / 1 reaches -bound / +bound (s8: +bound - 64*128)
    w[0], w[1] = -128, (-128 if xs8 else 127)
    bound = C * xmax * 128
    margin = (1 << 22) - 1 - bound + extra
    bias = g.integers(-margin, margin + 1, K).astype(np.int64)
    bias[0], bias[1], bias[2], bias[3] = (-margin if not xs8 else margin), margin, -margin, margin
    bias = bias.astype(np.int32)
    acc = o.conv_acc(x, w, bias, (1, 1), (0, 0), (1, 1), threads=4)
    assert extra or np.abs(acc.astype(np.int64)).max() == (1 << 22) - 1
    scale = np.float32(127.0 / (1 << 22)) if extra < 2 else np.float32(127.0 / (1 << 30))
    resid = g.integers(0, 256, (N, H, W, K), dtype=np.uint8)
    for ytype, res, relu in ((S8, None, False), (U8, resid, True), (F32, None, False)):
        want = o.epilogue(acc, scale, res, 0.21 if res is not None else 0.0, relu, OT[ytype])
        d = q8.make_conv_desc(N, H, W, C, K, 1, 1, (1, 1), (0, 0), (1, 1), S8 if xs8 else U8, U8, ytype, relu)
        y = q8.q8_conv2d(d, _cuda(x), _cuda(w), _cuda(bias), torch.tensor([scale], device="cuda"),
                         _cuda(res) if res is not None else None, 0.21 if res is not None else 0.0)
        q8.q8_read_status()
        assert np.array_equal(_bits(y.cpu().numpy()), _bits(want))


PAIR_CASES = [
    # enough 128 x 256 tiles for every SM pair: these run as clusters of two CTAs (tcgen05.mma.cta_group::2);
    # an odd number of m tiles leaves the last pair with a phantom second tile
    ("pair_3x3_c256_k256", 7, 75, 75, 256, 256, 3, 3, 1, 1, 1, False, U8, None, True),
    ("pair_3x3_c128_k512_res", 10, 38, 38, 128, 512, 3, 3, 1, 1, 1, False, U8, "u8", True),
    ("pair_3x3_c256_k256_s8", 7, 75, 75, 256, 256, 3, 3, 1, 1, 1, True, S8, "s8", False),
    ("pair_3x3_c128_k128", 7, 150, 150, 128, 128, 3, 3, 1, 1, 1, False, U8, None, True),   # 128-wide tiles, four groups
    # 160-, 192- and 96-wide tiles whose halves are 80, 96 and 48 weight rows, ragged tap groups (7 taps in
    # stages of 4 + 3)
    ("pair_1x7_c160_k160", 100, 17, 17, 160, 160, 1, 7, 1, (0, 3), 1, False, U8, None, True),
    ("pair_7x1_c192_k192_res", 100, 17, 17, 192, 192, 7, 1, 1, (3, 0), 1, False, U8, "u8", True),
    ("pair_3x3_c96_k96_s8", 16, 35, 35, 96, 96, 3, 3, 1, 1, 1, True, S8, None, False),
    # long launches with resident weights (single CTAs, three MMA lanes)
    ("long_3x3_c64_k64_resident", 24, 112, 112, 64, 64, 3, 3, 1, 1, 1, False, U8, None, True),
    ("long_5x5_c64_k64_resident_res", 100, 35, 35, 64, 64, 5, 5, 1, 2, 1, False, U8, "u8", True),
]


@pytest.mark.parametrize("case", PAIR_CASES, ids=[c[0] for c in PAIR_CASES])
def test_cta_pair_layers_match_oracle(q8, case):
    name, N, H, W, C, K, R, S, _, _, _, xs8, ytype, res, relu = case
    x, w, bias, acc, resid, (st, pad, dil) = _make(case)
    scale = np.float32(100.0 / max(1, np.abs(acc).max()))
    rs = 0.37 if resid is not None else 0.0
    want = o.epilogue(acc, scale, resid, rs, relu, OT[ytype])
    d = q8.make_conv_desc(N, H, W, C, K, R, S, st, pad, dil, S8 if xs8 else U8, S8 if res == "s8" else U8, ytype, relu)
    for _ in range(2):   # twice: the second launch follows a cluster launch in the stream
        y = q8.q8_conv2d(d, _cuda(x), _cuda(w), _cuda(bias), torch.tensor([scale], device="cuda"),
                         _cuda(resid) if resid is not None else None, rs)
    q8.q8_read_status()
    assert np.array_equal(y.cpu().numpy(), want)


def test_tensor_core_kernel_is_selected(q8):
    """The shapes of the paper's networks must run on tcgen05, not on the fallback."""
    for (N, H, W, C, K, R, S, st, pad) in [(32, 56, 56, 256, 64, 1, 1, 1, 0), (32, 56, 56, 64, 64, 3, 3, 1, 1),
                                            (32, 56, 56, 64, 256, 1, 1, 1, 0), (64, 28, 28, 256, 512, 1, 1, 2, 0),
                                            (64, 7, 7, 512, 512, 3, 3, 1, 1), (64, 224, 224, 16, 64, 7, 7, 2, 3)]:
        d = q8.make_conv_desc(N, H, W, C, K, R, S, (st, st), (pad, pad))
        assert q8.q8_conv2d_query_algo(d) == q8.Q8_ALGO_UMMA


@pytest.mark.parametrize("algo", [0, 2], ids=["auto", "direct"])
def test_per_channel_scale_and_concat_slice(q8, algo):
    g = np.random.default_rng(77)
    N, H, W, C, K = 2, 13, 11, 64, 48
    x = g.integers(0, 256, (N, H, W, C), dtype=np.uint8)
    w = g.integers(-128, 128, (K, 1, 1, C)).astype(np.int8)
    bias = g.integers(-100, 100, K).astype(np.int32)
    scales = (g.uniform(0.5, 1.5, K) * 1e-3).astype(np.float32)
    ldc, c_off = 112, 32
    want = np.full((N, H, W, ldc), 0xAB, dtype=np.uint8)
    o.conv2d(x, w, bias, scales, relu=True, y_type=o.U8, out=want, c_off=c_off)
    y = torch.full((N, H, W, ldc), 0xAB, dtype=torch.uint8, device="cuda")
    d = q8.make_conv_desc(N, H, W, C, K, 1, 1, y_type=U8, relu=True, scale_count=K, y_ldc=ldc, y_c_offset=c_off, algo=algo)
    q8.q8_conv2d(d, _cuda(x), _cuda(w), _cuda(bias), _cuda(scales), y=y)
    q8.q8_read_status()
    assert np.array_equal(y.cpu().numpy(), want)  # neighbours of the slice untouched


def test_output_canaries_untouched(q8):
    """Rows before and after the output tensor keep their sentinel (tile tails must be masked)."""
    g = np.random.default_rng(78)
    N, H, W, C, K = 1, 9, 9, 64, 40  # M = 81 (< one tile), Cout with a ragged 16-column chunk
    x = g.integers(0, 256, (N, H, W, C), dtype=np.uint8)
    w = g.integers(-128, 128, (K, 1, 1, C)).astype(np.int8)
    M = N * H * W
    for ytype, tdt in ((U8, torch.uint8), (F32, torch.float32), (S32, torch.int32)):
        buf = torch.full((M + 256, K), 7, dtype=tdt, device="cuda")
        y = buf[128:128 + M]
        d = q8.make_conv_desc(N, H, W, C, K, 1, 1, y_type=ytype)
        q8.q8_conv2d(d, _cuda(x), _cuda(w), None, torch.tensor([1e-3], device="cuda"), y=y)
        q8.q8_read_status()
        want = o.conv2d(x, w, None, np.float32(1e-3), y_type=OT[ytype]).reshape(M, K)
        assert np.array_equal(_bits(y.cpu().numpy()), _bits(want))
        assert bool((buf[:128] == 7).all()) and bool((buf[128 + M:] == 7).all())


def test_forced_umma_rejects_ineligible_shapes(q8):
    d = q8.make_conv_desc(1, 8, 8, 3, 8, 3, 3, pad=(1, 1), algo=q8.Q8_ALGO_UMMA)
    x = torch.zeros((1, 8, 8, 3), dtype=torch.uint8, device="cuda")
    w = torch.zeros((8, 3, 3, 3), dtype=torch.int8, device="cuda")
    with pytest.raises(q8.Q8Error) as e:
        q8.q8_conv2d(d, x, w, None, torch.ones(1, device="cuda"))
    assert e.value.code == 2


SPLITK_CASES = [
    # name, N,H,W,C,K,R,S,stride,pad, y type, residual, relu
    ("fc_c2048_k1000_f32", 64, 1, 1, 2048, 1000, 1, 1, 1, 0, F32, None, False),
    ("3x3_7x7_c512_k512_res", 8, 7, 7, 512, 512, 3, 3, 1, 1, U8, "u8", True),
    ("1x1_c2048_k512", 8, 7, 7, 2048, 512, 1, 1, 1, 0, U8, None, True),
    ("3x3s2_c256_k256_s8", 4, 15, 15, 256, 256, 3, 3, 2, 1, S8, None, False),
    ("1x1_c1024_k24_slice", 2, 10, 10, 1024, 24, 1, 1, 1, 0, F32, None, True),
]


@pytest.mark.parametrize("case", SPLITK_CASES, ids=[c[0] for c in SPLITK_CASES])
def test_split_k_matches_oracle_and_unsplit(q8, case):
    """Layers with few output tiles split the reduction when given a workspace; the result must not change."""
    name, N, H, W, C, K, R, S, st, pad, ytype, res, relu = case
    g = np.random.default_rng(sum(map(ord, name)))
    x = g.integers(0, 256, (N, H, W, C), dtype=np.uint8)
    w = g.integers(-128, 128, (K, R, S, C)).astype(np.int8)
    bias = g.integers(-5000, 5000, K).astype(np.int32)
    acc = o.conv_acc(x, w, bias, (st, st), (pad, pad), (1, 1), threads=8)
    P, Q = acc.shape[1:3]
    resid = g.integers(0, 256, (N, P, Q, K), dtype=np.uint8) if res else None
    scale = np.float32(100.0 / max(1, np.abs(acc).max()))
    rs = 0.37 if resid is not None else 0.0
    want = o.epilogue(acc, scale, resid, rs, relu, OT[ytype])
    d = q8.make_conv_desc(N, H, W, C, K, R, S, (st, st), (pad, pad), (1, 1), U8, U8, ytype, relu)
    nbytes = q8.q8_conv2d_workspace_bytes(d)
    assert nbytes > 0, "this shape is expected to split"
    ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    args = (_cuda(x), _cuda(w), _cuda(bias), torch.tensor([scale], device="cuda"), _cuda(resid) if res else None, rs)
    y_split = q8.q8_conv2d(d, *args, workspace=ws)
    y_plain = q8.q8_conv2d(d, *args)
    q8.q8_read_status()
    assert np.array_equal(_bits(y_split.cpu().numpy()), _bits(want))
    assert np.array_equal(_bits(y_plain.cpu().numpy()), _bits(want))

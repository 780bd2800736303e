"""GPU parity of q8_conv2d_then_1x1 (two convolutions in one launch, the tensor between them kept in shared
memory) against the CPU oracle applied twice, bit-exact, and against the two-launch path of the library.

Sizes span several tiles per CTA, ragged image edges, resident and ring-fed first-layer weights, one and several
output chunks, ragged last chunks, signed tensors, and an output slice of a wider tensor.
"""
import numpy as np
import pytest
import torch

import oracle as o

pytestmark = pytest.mark.gpu

U8, S8 = 0, 1
OT = {U8: o.U8, S8: o.S8}


def _cuda(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


CASES = [
    # name, N,H,W, C1, K1, R,S, pad, dil, K2, x signed, relu1 (u8 between) / s8, out type, residual, relu2
    ("bottleneck_56_64_64_256_res", 3, 56, 56, 64, 64, 3, 3, 1, 1, 256, False, True, U8, "u8", True),
    ("bottleneck_28_128_128_512_res", 3, 28, 28, 128, 128, 3, 3, 1, 1, 512, False, True, U8, "u8", True),
    ("many_tiles_per_cta", 40, 30, 30, 64, 64, 3, 3, 1, 1, 128, False, True, U8, "u8", True),
    ("ragged_edges_37x41", 2, 37, 41, 64, 64, 3, 3, 1, 1, 256, False, True, U8, None, True),
    ("k1_32_k2_64", 2, 33, 33, 32, 32, 3, 3, 1, 1, 64, False, True, U8, None, True),
    ("ragged_chunk_k2_192", 2, 28, 28, 64, 64, 3, 3, 1, 1, 192, False, True, U8, "u8", True),
    ("small_k2_80", 2, 28, 28, 64, 128, 3, 3, 1, 1, 80, False, True, U8, None, True),
    ("signed_everything", 2, 28, 28, 64, 64, 3, 3, 1, 1, 256, True, False, S8, "s8", False),
    ("c1_256_ring", 2, 20, 20, 256, 128, 3, 3, 1, 1, 256, False, True, U8, "u8", True),
    ("5x5_pad2", 2, 35, 35, 48, 64, 5, 5, 2, 1, 96, False, True, U8, None, True),
    ("1x7", 2, 17, 17, 128, 128, 1, 7, (0, 3), 1, 192, False, True, U8, None, True),
    ("dilated", 2, 40, 40, 64, 64, 3, 3, 2, 2, 128, False, True, U8, "u8", True),
    ("pad0_valid", 2, 30, 30, 64, 64, 3, 3, 0, 1, 128, False, True, U8, None, True),
    ("one_tile_total", 1, 8, 8, 64, 64, 3, 3, 1, 1, 256, False, True, U8, "u8", True),
]


def _pair(v):
    return v if isinstance(v, tuple) else (v, v)


@pytest.mark.parametrize("case", CASES, ids=[c[0] for c in CASES])
def test_fused_pair_matches_oracle(q8, case):
    name, N, H, W, C1, K1, R, S, pad, dil, K2, xs8, relu1, ytype, res, relu2 = case
    pad, dil = _pair(pad), _pair(dil)
    g = np.random.default_rng(sum(map(ord, name)))
    x = g.integers(-128, 128, (N, H, W, C1)).astype(np.int8) if xs8 else g.integers(0, 256, (N, H, W, C1), dtype=np.uint8)
    w1 = g.integers(-128, 128, (K1, R, S, C1)).astype(np.int8)
    b1 = g.integers(-5000, 5000, K1).astype(np.int32)
    acc1 = o.conv_acc(x, w1, b1, (1, 1), pad, dil, threads=8)
    s1 = (np.float32(200.0) / np.float32(max(1, np.abs(acc1).max()))).astype(np.float32)
    t_type = U8 if relu1 else S8
    mid = o.epilogue(acc1, s1, None, 0.0, relu1, OT[t_type])
    P, Q = mid.shape[1:3]
    w2 = g.integers(-128, 128, (K2, 1, 1, K1)).astype(np.int8)
    b2 = g.integers(-5000, 5000, K2).astype(np.int32)
    acc2 = o.conv_acc(mid, w2, b2, (1, 1), (0, 0), (1, 1), threads=8)
    s2 = g.uniform(0.5, 1.5, K2).astype(np.float32) * np.float32(150.0 / max(1, np.abs(acc2).max()))  # per channel
    resid = None
    if res == "u8":
        resid = g.integers(0, 256, (N, P, Q, K2), dtype=np.uint8)
    elif res == "s8":
        resid = g.integers(-128, 128, (N, P, Q, K2)).astype(np.int8)
    rs = 0.37 if resid is not None else 0.0
    want = o.epilogue(acc2, s2, resid, rs, relu2, OT[ytype])

    d1 = q8.make_conv_desc(N, H, W, C1, K1, R, S, (1, 1), pad, dil, S8 if xs8 else U8, U8, t_type, relu1)
    d2 = q8.make_conv_desc(N, P, Q, K1, K2, 1, 1, (1, 1), (0, 0), (1, 1), t_type, S8 if res == "s8" else U8, ytype, relu2, K2)
    assert q8.q8_conv2d_then_1x1_supported(d1, d2)
    args = (_cuda(x), _cuda(w1), _cuda(b1), torch.tensor([s1], device="cuda"), _cuda(w2), _cuda(b2), _cuda(s2))
    r = _cuda(resid) if resid is not None else None
    y = q8.q8_conv2d_then_1x1(d1, d2, *args, r, rs)
    q8.q8_read_status()
    assert np.array_equal(y.cpu().numpy(), want)
    # the two-launch path of the library gives the same bytes
    mid_gpu = q8.q8_conv2d(d1, args[0], args[1], args[2], args[3])
    y2 = q8.q8_conv2d(d2, mid_gpu, args[4], args[5], args[6], r, rs)
    q8.q8_read_status()
    assert torch.equal(y, y2)


def test_fused_pair_writes_a_channel_slice_and_leaves_the_rest(q8):
    N, H, W, C1, K1, K2, ldc, off = 2, 28, 28, 64, 64, 128, 320, 64
    g = np.random.default_rng(11)
    x = g.integers(0, 256, (N, H, W, C1), dtype=np.uint8)
    w1 = g.integers(-128, 128, (K1, 3, 3, C1)).astype(np.int8)
    w2 = g.integers(-128, 128, (K2, 1, 1, K1)).astype(np.int8)
    b2 = g.integers(-3000, 3000, K2).astype(np.int32)
    s1, s2 = np.float32(3e-4), np.float32(2e-4)
    mid = o.conv2d(x, w1, None, s1, pad=(1, 1), relu=True, threads=8)
    want = o.conv2d(mid, w2, b2, s2, relu=True, threads=8)
    d1 = q8.make_conv_desc(N, H, W, C1, K1, 3, 3, (1, 1), (1, 1), (1, 1), U8, U8, U8, True)
    d2 = q8.make_conv_desc(N, H, W, K1, K2, 1, 1, (1, 1), (0, 0), (1, 1), U8, U8, U8, True, 1, ldc, off)
    y = torch.full((N, H, W, ldc), 0xA5, dtype=torch.uint8, device="cuda")
    q8.q8_conv2d_then_1x1(d1, d2, _cuda(x), _cuda(w1), None, torch.tensor([s1], device="cuda"), _cuda(w2), _cuda(b2),
                          torch.tensor([s2], device="cuda"), y=y)
    q8.q8_read_status()
    got = y.cpu().numpy()
    assert np.array_equal(got[..., off:off + K2], want)
    assert (got[..., :off] == 0xA5).all() and (got[..., off + K2:] == 0xA5).all()


def test_ineligible_pairs_are_refused_with_a_reason(q8):
    d1 = q8.make_conv_desc(2, 28, 28, 64, 64, 3, 3, (2, 2), (1, 1), (1, 1), U8, U8, U8, True)      # stride 2
    d2 = q8.make_conv_desc(2, 14, 14, 64, 256, 1, 1, (1, 1), (0, 0), (1, 1), U8, U8, U8, True)
    assert not q8.q8_conv2d_then_1x1_supported(d1, d2)
    d1 = q8.make_conv_desc(2, 28, 28, 64, 256, 3, 3, (1, 1), (1, 1), (1, 1), U8, U8, U8, True)     # 256 channels between
    d2 = q8.make_conv_desc(2, 28, 28, 256, 256, 1, 1, (1, 1), (0, 0), (1, 1), U8, U8, U8, True)
    assert not q8.q8_conv2d_then_1x1_supported(d1, d2)
    x = torch.zeros((2, 28, 28, 64), dtype=torch.uint8, device="cuda")
    w1 = torch.zeros((256, 3, 3, 64), dtype=torch.int8, device="cuda")
    w2 = torch.zeros((256, 1, 1, 256), dtype=torch.int8, device="cuda")
    s = torch.ones(1, device="cuda")
    with pytest.raises(q8.Q8Error) as e:
        q8.q8_conv2d_then_1x1(d1, d2, x, w1, None, s, w2, None, s)
    assert e.value.code == 2 and "32, 64 or 128" in str(e.value)

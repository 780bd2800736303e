"""The no-allocation convolution entry point, q8_conv2d_static_workspace.

It exists for hosts that must not allocate device memory while they call this library (all memory handed
out up front, or cudaMalloc forbidden because it stalls the device): the scratch of the split reduction is a
fixed array inside the library.  This file is named to be collected last, so that a failure here cannot hide
the result of any other test.  Every check goes through the C ABI and compares with q8_conv2d given an
ordinary workspace and with the CPU oracle: same bits, on two calls in a row (the array keeps the previous
call's contents).  A call after the first must also leave the amount of free device memory unchanged.
"""
import numpy as np
import pytest
import torch

import oracle as o

pytestmark = pytest.mark.gpu

U8, S8, S32, F32 = 0, 1, 2, 3


def _case(q8, N, H, W, C, K, R, pad, ytype, with_res, seed):
    g = torch.Generator(device="cuda").manual_seed(seed)
    d = q8.make_conv_desc(N, H, W, C, K, R, R, (1, 1), (pad, pad), (1, 1), U8, U8, ytype, True)
    P, Q = q8.conv_out_shape(d)
    x = torch.randint(0, 256, (N, H, W, C), dtype=torch.uint8, device="cuda", generator=g)
    w = torch.randint(-128, 128, (K, R, R, C), dtype=torch.int8, device="cuda", generator=g)
    b = torch.randint(-3000, 3000, (K,), dtype=torch.int32, device="cuda", generator=g)
    res = torch.randint(0, 256, (N, P, Q, K), dtype=torch.uint8, device="cuda", generator=g) if with_res else None
    scale = torch.tensor([3e-5], dtype=torch.float32, device="cuda")
    return d, x, w, b, scale, res


@pytest.mark.parametrize("shape", [(64, 1, 1, 2048, 1000, 1, 0, F32, False), (8, 7, 7, 512, 512, 3, 1, U8, True)],
                         ids=["fc_2048_1000_f32", "3x3_7x7_512_res_u8"])
def test_static_workspace_matches_caller_workspace_twice(q8, shape):
    N, H, W, C, K, R, pad, ytype, with_res = shape
    for call in range(2):  # second call: the built-in array still holds the first call's partial sums
        d, x, w, b, scale, res = _case(q8, N, H, W, C, K, R, pad, ytype, with_res, seed=100 + call)
        need = q8.q8_conv2d_workspace_bytes(d)
        assert 0 < need <= q8.q8_static_workspace_bytes(), "the case must exercise the scratch array"
        ws = torch.empty(need, dtype=torch.uint8, device="cuda")
        want = q8.q8_conv2d(d, x, w, b, scale, res, 0.41, workspace=ws)
        got = q8.q8_conv2d_static_workspace(d, x, w, b, scale, res, 0.41)
        q8.q8_read_status()
        ref = o.conv2d(x.cpu().numpy(), w.cpu().numpy(), b.cpu().numpy(), np.float32(3e-5), pad=(pad, pad),
                       residual=None if res is None else res.cpu().numpy(), res_scale=np.float32(0.41), relu=True,
                       y_type={U8: o.U8, F32: o.F32}[ytype], threads=o.hw_threads())
        a, e = got.cpu().numpy(), want.cpu().numpy()
        if a.dtype == np.float32:
            a, e, ref = a.view(np.uint32), e.view(np.uint32), ref.view(np.uint32)
        assert np.array_equal(a, e)
        assert np.array_equal(a, ref)
        # the entry point allocates nothing: with the output preallocated, free device memory does not move
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        q8.q8_conv2d_static_workspace(d, x, w, b, scale, res, 0.41, y=got)
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] == free_before


def test_static_workspace_refuses_oversized_layers_and_runs_unsplit_ones(q8):
    # 20 images of 7x7x512, 3x3: nine splits of 980 x 512 int32 exceed 16 MiB -> refused, nothing launched
    d, x, w, b, scale, res = _case(q8, 20, 7, 7, 512, 512, 3, 1, U8, False, seed=7)
    assert q8.q8_conv2d_workspace_bytes(d) > q8.q8_static_workspace_bytes()
    with pytest.raises(q8.Q8Error) as e:
        q8.q8_conv2d_static_workspace(d, x, w, b, scale)
    assert e.value.code == 4 and "built-in" in str(e.value)
    # a layer that needs no scratch simply runs
    d, x, w, b, scale, res = _case(q8, 2, 16, 16, 64, 64, 3, 1, U8, False, seed=8)
    assert q8.q8_conv2d_workspace_bytes(d) == 0
    got = q8.q8_conv2d_static_workspace(d, x, w, b, scale)
    want = q8.q8_conv2d(d, x, w, b, scale)
    q8.q8_read_status()
    assert torch.equal(got, want)

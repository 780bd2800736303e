"""The bounded-wait path of the tensor-core kernels, exercised without any fault: a wait that nothing satisfies runs
out after its limit, the status word reports it once, the other role of the CTA drains through the abort flag, and
the library keeps working."""
import time

import numpy as np
import pytest
import torch

import oracle as o

pytestmark = pytest.mark.gpu


def test_wait_runs_out_sets_status_once_and_library_stays_usable(q8):
    q8.q8_read_status()                      # healthy before
    t0 = time.perf_counter()
    q8.q8_selftest_bounded_wait(2000)        # first warp gives up after 2 ms
    with pytest.raises(q8.Q8Error) as e:
        q8.q8_read_status()
    elapsed = time.perf_counter() - t0
    assert e.value.code == 6 and "0x5" in str(e.value)       # Q8_ERR_TIMEOUT, both sites recorded
    assert elapsed < 1.0                     # the second warp (2 s limit) left through the abort flag
    q8.q8_read_status()                      # reading the status cleared it
    # the next convolution runs and is bit-exact
    g = np.random.default_rng(3)
    x = g.integers(0, 256, (2, 20, 20, 64), dtype=np.uint8)
    w = g.integers(-128, 128, (64, 3, 3, 64)).astype(np.int8)
    d = q8.make_conv_desc(2, 20, 20, 64, 64, 3, 3, pad=(1, 1), relu=True)
    y = q8.q8_conv2d(d, torch.from_numpy(x).cuda(), torch.from_numpy(w).cuda(), None, torch.tensor([2e-4], device="cuda"))
    q8.q8_read_status()
    assert np.array_equal(y.cpu().numpy(), o.conv2d(x, w, None, np.float32(2e-4), pad=(1, 1), relu=True, threads=4))


def test_selftest_rejects_limits_out_of_range(q8):
    for bad in (0, 2000000):
        with pytest.raises(q8.Q8Error) as e:
            q8.q8_selftest_bounded_wait(bad)
        assert e.value.code == 1

"""CPU checks of the C ABI: the library loads, exports what include/q8.h declares, and its host-side
validation turns bad requests into documented error codes without launching anything."""
import ctypes as C
import os
import re

import numpy as np
import pytest

import oracle as o
import paper_1805_08691_b200 as q8

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "q8.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(q8_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported_and_bound():
    names = _declared()
    assert len(names) >= 18
    for n in names:
        assert hasattr(q8.lib, n), n
        assert n in q8.EXPORTS, n
        assert callable(getattr(q8, n)), n  # the Python binding carries the same name


def test_struct_layout_matches_header():
    text = open(os.path.join(ROOT, "include", "q8.h")).read()
    body = re.search(r"typedef struct q8_conv_desc \{(.*?)\} q8_conv_desc;", text, flags=re.S).group(1)
    body = re.sub(r"/\*.*?\*/", "", body, flags=re.S)
    fields = []
    for decl in body.split(";"):
        decl = decl.strip()
        if decl.startswith("int32_t"):
            fields += [f.strip() for f in decl[len("int32_t"):].split(",")]
    assert fields == [f[0] for f in q8.q8_conv_desc._fields_]
    assert C.sizeof(q8.q8_conv_desc) == 4 * len(fields)


def test_host_helpers_agree_with_oracle():
    g = np.random.default_rng(0)
    for _ in range(2000):
        m = float(np.float32(g.uniform(1e-4, 1e4)))
        for p in (7, 8):
            assert q8.q8_factor(m, p) == o.factor(m, p)
        a, b, c = (float(np.float32(v)) for v in g.uniform(1e-4, 1.0, 3))
        assert q8.q8_requant_scale(a, b, c) == o.requant_scale(a, b, c)
        assert q8.q8_bias_factor(a, b) == o.bias_factor(a, b)
    assert q8.q8_factor(0.0, 8) == 1.0
    for H, k, st, pad, ceil in [(75, 2, 2, 0, True), (75, 2, 2, 0, False), (112, 3, 2, 1, False), (147, 3, 2, 0, False),
                                (8, 8, 1, 0, False), (19, 3, 1, 1, False)]:
        assert q8.q8_pool_out_extent(H, k, st, pad, ceil) == o.pool_out(H, k, st, pad, ceil)


def _code(fn, *a, **k):
    with pytest.raises(q8.Q8Error) as e:
        fn(*a, **k)
    return e.value.code


def test_bad_requests_are_rejected_on_the_host():
    assert _code(q8.q8_factor, float("nan"), 8) == 7
    assert _code(q8.q8_factor, float("inf"), 8) == 7
    assert _code(q8.q8_factor, 1.0, 0) == 1
    assert _code(q8.q8_requant_scale, 0.0, 1.0, 1.0) == 7
    d = q8.make_conv_desc(1, 8, 8, 16, 16, 3, 3)
    assert q8.q8_conv2d_workspace_bytes(d) == 0
    for field, bad in [("N", 0), ("C", -1), ("stride_h", 0), ("pad_w", -1), ("x_type", 3), ("y_type", 9),
                       ("scale_count", 2), ("algo", 5), ("y_ldc", 8), ("y_c_offset", -16)]:
        d = q8.make_conv_desc(1, 8, 8, 16, 16, 3, 3)
        setattr(d, field, bad)
        assert _code(q8.q8_conv2d_query_algo, d) == 1, field
    # filter larger than the padded image -> empty output
    assert _code(q8.q8_conv2d_query_algo, q8.make_conv_desc(1, 2, 2, 16, 16, 3, 3)) == 1
    # accumulator overflow guard
    assert _code(q8.q8_conv2d_query_algo, q8.make_conv_desc(1, 16, 16, 8192, 16, 3, 3)) == 1
    # null pointers never reach a launch
    d = q8.make_conv_desc(1, 8, 8, 16, 16, 3, 3)
    rc = q8.lib.q8_conv2d(C.byref(d), None, None, None, None, None, 0.0, None, None, 0, None)
    assert rc == 1 and b"null" in q8.lib.q8_last_error()
    assert q8.lib.q8_quantize(None, 10, 1.0, 0, None, None) == 1
    assert q8.lib.q8_quantize(None, 0, 0.0, 0, None, None) == 7
    assert q8.lib.q8_calibrate_maxabs(None, 4, None, None) == 1
    assert q8.lib.q8_dequantize(None, 3, 4, 1.0, None, None) == 1
    assert q8.lib.q8_fold_bn(None, None, None, None, None, None, 1e-5, 4, 4, None, None, None) == 1


def test_kernel_selection_rules():
    U = q8.Q8_ALGO_UMMA
    assert q8.q8_conv2d_query_algo(q8.make_conv_desc(32, 56, 56, 256, 64, 1, 1)) == U
    assert q8.q8_conv2d_query_algo(q8.make_conv_desc(32, 56, 56, 64, 64, 3, 3, pad=(1, 1))) == U
    assert q8.q8_conv2d_query_algo(q8.make_conv_desc(1, 8, 8, 3, 8, 3, 3, pad=(1, 1))) == q8.Q8_ALGO_DIRECT
    assert q8.q8_conv2d_query_algo(q8.make_conv_desc(32, 56, 56, 64, 64, 3, 3, pad=(1, 1), algo=q8.Q8_ALGO_DIRECT)) == q8.Q8_ALGO_DIRECT

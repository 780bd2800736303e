"""ctypes binding of libq8.so: argument marshalling only.

Every function has the name and meaning of the C entry point declared in include/q8.h; tensors
are torch CUDA tensors used purely as device memory, and work is enqueued on torch's current
stream.  There is no CPU path: importing this module without the compiled library raises.
"""
import ctypes as C
import os
import shutil

import torch

from . import build as _build

Q8_U8, Q8_S8, Q8_S32, Q8_F32 = 0, 1, 2, 3
Q8_ALGO_AUTO, Q8_ALGO_UMMA, Q8_ALGO_DIRECT = 0, 1, 2
Q8_OK = 0
STATUS_NAMES = {0: "Q8_OK", 1: "Q8_ERR_INVALID_ARG", 2: "Q8_ERR_UNSUPPORTED", 3: "Q8_ERR_ALIGNMENT",
                4: "Q8_ERR_WORKSPACE", 5: "Q8_ERR_CUDA", 6: "Q8_ERR_TIMEOUT", 7: "Q8_ERR_NONFINITE"}
TORCH_DTYPES = {Q8_U8: torch.uint8, Q8_S8: torch.int8, Q8_S32: torch.int32, Q8_F32: torch.float32}
EXPORTS = ["q8_version", "q8_last_error", "q8_read_status", "q8_calibrate_maxabs", "q8_factor", "q8_requant_scale",
           "q8_bias_factor", "q8_quantize", "q8_quantize_pad_channels", "q8_dequantize", "q8_fold_bn",
           "q8_conv2d_workspace_bytes", "q8_conv2d_query_algo", "q8_conv2d", "q8_static_workspace_bytes",
           "q8_conv2d_static_workspace", "q8_conv2d_then_1x1_supported", "q8_conv2d_then_1x1", "q8_int8_mma_rate", "q8_selftest_bounded_wait", "q8_concat", "q8_concat_branch", "q8_calibrate_maxabs_rows", "q8_quantize_rows", "q8_quantize_pad_image", "q8_pool_out_extent",
           "q8_maxpool2d", "q8_avgpool2d", "q8_l2norm", "q8_add_relu_quantize", "q8_detection_output_workspace_bytes",
           "q8_detection_output"]


class Q8Error(RuntimeError):
    def __init__(self, code, text):
        super().__init__(f"{STATUS_NAMES.get(code, code)}: {text}")
        self.code = code


class q8_conv_desc(C.Structure):
    _fields_ = [(n, C.c_int32) for n in (
        "N", "H", "W", "C", "K", "R", "S", "stride_h", "stride_w", "pad_h", "pad_w", "dil_h", "dil_w",
        "x_type", "res_type", "y_type", "relu", "scale_count", "y_ldc", "y_c_offset", "algo")]


def _load():
    path = _build.LIB
    if shutil.which("nvcc") is not None:
        path = _build.build()
    if not os.path.exists(path):
        raise ImportError(f"{path} is missing and nvcc is not available to build it; "
                          "run `python -m paper_1805_08691_b200.build` on a machine with CUDA 12.9")
    return C.CDLL(path)


lib = _load()

_vp, _sz, _i, _f = C.c_void_p, C.c_size_t, C.c_int, C.c_float
_fp, _ip = C.POINTER(C.c_float), C.POINTER(C.c_int)
lib.q8_version.restype = C.c_char_p
lib.q8_last_error.restype = C.c_char_p
lib.q8_read_status.argtypes = [_vp]
lib.q8_calibrate_maxabs.argtypes = [_vp, _sz, _vp, _vp]
lib.q8_factor.argtypes = [_f, _i, _fp]
lib.q8_requant_scale.argtypes = [_f, _f, _f, _fp]
lib.q8_bias_factor.argtypes = [_f, _f, _fp]
lib.q8_quantize.argtypes = [_vp, _sz, _f, _i, _vp, _vp]
lib.q8_quantize_pad_channels.argtypes = [_vp, _sz, _i, _i, _f, _i, _vp, _vp]
lib.q8_dequantize.argtypes = [_vp, _i, _sz, _f, _vp, _vp]
lib.q8_fold_bn.argtypes = [_vp] * 6 + [C.c_double, _i, _sz, _vp, _vp, _vp]
lib.q8_conv2d_workspace_bytes.argtypes = [C.POINTER(q8_conv_desc), C.POINTER(_sz)]
lib.q8_conv2d_query_algo.argtypes = [C.POINTER(q8_conv_desc), _ip]
lib.q8_conv2d.argtypes = [C.POINTER(q8_conv_desc), _vp, _vp, _vp, _vp, _vp, _f, _vp, _vp, _sz, _vp]
lib.q8_static_workspace_bytes.argtypes = []
lib.q8_selftest_bounded_wait.argtypes = [C.c_uint, _vp]
lib.q8_int8_mma_rate.argtypes = [_i, _i, _i, _i, _vp, _vp]
lib.q8_conv2d_then_1x1_supported.argtypes = [C.POINTER(q8_conv_desc), C.POINTER(q8_conv_desc), _ip]
lib.q8_conv2d_then_1x1.argtypes = [C.POINTER(q8_conv_desc), C.POINTER(q8_conv_desc), _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _f, _vp, _vp]
lib.q8_conv2d_static_workspace.argtypes = [C.POINTER(q8_conv_desc), _vp, _vp, _vp, _vp, _vp, _f, _vp, _vp]
lib.q8_concat.argtypes = [_i, C.POINTER(_vp), _ip, _fp, _f, _i, _sz, _vp, _vp]
lib.q8_calibrate_maxabs_rows.argtypes = [_vp, _sz, _sz, _vp, _vp]
lib.q8_quantize_pad_image.argtypes = [_vp, _i, _i, _i, _i, _i, _i, _f, _i, _vp, _vp]
lib.q8_quantize_rows.argtypes = [_vp, _sz, _sz, _vp, _i, _vp, _vp]
lib.q8_concat_branch.argtypes = [_vp, _i, _f, _f, _i, _sz, _vp, _i, _i, _vp]
lib.q8_pool_out_extent.argtypes = [_i] * 5 + [_ip]
lib.q8_maxpool2d.argtypes = [_vp, _i] + [_i] * 11 + [_vp, _vp]
lib.q8_avgpool2d.argtypes = [_vp, _i] + [_i] * 11 + [_vp, _vp]
lib.q8_l2norm.argtypes = [_vp, _sz, _i, _f, _f, _vp, _vp, _vp]
lib.q8_add_relu_quantize.argtypes = [_vp, _vp, _sz, _f, _vp, _vp]
lib.q8_detection_output_workspace_bytes.argtypes = [_i] * 6 + [C.POINTER(_sz)]
lib.q8_detection_output.argtypes = [_i, C.POINTER(_vp), _ip, C.POINTER(_vp), _ip, _ip, _ip, _vp, _fp, _i, _i, _i, _f, _f, _i, _i,
                                    _vp, _sz, _vp, _vp, _vp]
for _n in EXPORTS[2:]:
    getattr(lib, _n).restype = C.c_int
lib.q8_static_workspace_bytes.restype = C.c_size_t


def _check(rc):
    if rc != Q8_OK:
        raise Q8Error(rc, lib.q8_last_error().decode())


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _dev(t, what):
    if t is None:
        return None
    if not (isinstance(t, torch.Tensor) and t.is_cuda and t.is_contiguous()):
        raise TypeError(f"{what}: expected a contiguous CUDA tensor")
    return C.c_void_p(t.data_ptr())


def q8_version():
    return lib.q8_version().decode()


def q8_last_error():
    return lib.q8_last_error().decode()


def q8_read_status():
    _check(lib.q8_read_status(_stream()))


def q8_calibrate_maxabs(x, running_max):
    assert x.dtype == torch.float32 and running_max.dtype == torch.float32 and running_max.numel() == 1
    _check(lib.q8_calibrate_maxabs(_dev(x, "x"), x.numel(), _dev(running_max, "running_max"), _stream()))


def q8_factor(maxabs, p):
    q = C.c_float()
    _check(lib.q8_factor(maxabs, p, C.byref(q)))
    return q.value


def q8_requant_scale(q_x, q_w, q_y):
    s = C.c_float()
    _check(lib.q8_requant_scale(q_x, q_w, q_y, C.byref(s)))
    return s.value


def q8_bias_factor(q_x, q_w):
    s = C.c_float()
    _check(lib.q8_bias_factor(q_x, q_w, C.byref(s)))
    return s.value


def q8_quantize(x, q, out_type, out=None):
    assert x.dtype == torch.float32
    if out is None:
        out = torch.empty(x.shape, dtype=TORCH_DTYPES[out_type], device=x.device)
    assert out.dtype == TORCH_DTYPES[out_type] and out.numel() == x.numel()
    _check(lib.q8_quantize(_dev(x, "x"), x.numel(), q, out_type, _dev(out, "out"), _stream()))
    return out


def q8_quantize_pad_channels(x, C_pad, q, out_type, out=None):
    assert x.dtype == torch.float32
    Cc = x.shape[-1]
    pixels = x.numel() // Cc
    if out is None:
        out = torch.empty(x.shape[:-1] + (C_pad,), dtype=TORCH_DTYPES[out_type], device=x.device)
    _check(lib.q8_quantize_pad_channels(_dev(x, "x"), pixels, Cc, C_pad, q, out_type, _dev(out, "out"), _stream()))
    return out


def q8_quantize_pad_image(x, W_pad, C_pad, q, out_type, out=None):
    """x: [N, H, W, C] fp32 -> [N, H, W_pad, C_pad] codes, zero beyond W and C."""
    assert x.dtype == torch.float32 and x.dim() == 4
    N, H, W, Cc = (int(v) for v in x.shape)
    if out is None:
        out = torch.empty((N, H, W_pad, C_pad), dtype=TORCH_DTYPES[out_type], device=x.device)
    _check(lib.q8_quantize_pad_image(_dev(x, "x"), N, H, W, Cc, W_pad, C_pad, q, out_type, _dev(out, "out"), _stream()))
    return out


def q8_dequantize(z, q, out=None):
    in_type = {torch.uint8: Q8_U8, torch.int8: Q8_S8, torch.int32: Q8_S32}[z.dtype]
    if out is None:
        out = torch.empty(z.shape, dtype=torch.float32, device=z.device)
    _check(lib.q8_dequantize(_dev(z, "z"), in_type, z.numel(), q, _dev(out, "out"), _stream()))
    return out


def q8_fold_bn(w, b, gamma, beta, mean, var, eps=1e-5):
    K = w.shape[0]
    w_out = torch.empty_like(w)
    b_out = torch.empty(K, dtype=torch.float32, device=w.device)
    _check(lib.q8_fold_bn(_dev(w, "w"), _dev(b, "b"), _dev(gamma, "gamma"), _dev(beta, "beta"), _dev(mean, "mean"),
                          _dev(var, "var"), float(eps), K, w.numel() // K, _dev(w_out, "w_out"), _dev(b_out, "b_out"),
                          _stream()))
    return w_out, b_out


def make_conv_desc(N, H, W, Cin, K, R, S, stride=(1, 1), pad=(0, 0), dil=(1, 1), x_type=Q8_U8, res_type=Q8_U8,
                   y_type=Q8_U8, relu=False, scale_count=1, y_ldc=0, y_c_offset=0, algo=Q8_ALGO_AUTO):
    return q8_conv_desc(N, H, W, Cin, K, R, S, stride[0], stride[1], pad[0], pad[1], dil[0], dil[1], x_type, res_type,
                        y_type, int(relu), scale_count, y_ldc, y_c_offset, algo)


def conv_out_shape(d):
    P = (d.H + 2 * d.pad_h - d.dil_h * (d.R - 1) - 1) // d.stride_h + 1
    Q = (d.W + 2 * d.pad_w - d.dil_w * (d.S - 1) - 1) // d.stride_w + 1
    return P, Q


def q8_conv2d_workspace_bytes(d):
    n = C.c_size_t()
    _check(lib.q8_conv2d_workspace_bytes(C.byref(d), C.byref(n)))
    return n.value


def q8_conv2d_query_algo(d):
    a = C.c_int()
    _check(lib.q8_conv2d_query_algo(C.byref(d), C.byref(a)))
    return a.value


def q8_conv2d(d, x, w, bias, scale, residual=None, residual_scale=0.0, y=None, workspace=None):
    if y is None:
        P, Q = conv_out_shape(d)
        y = torch.empty((d.N, P, Q, d.y_ldc or d.K), dtype=TORCH_DTYPES[d.y_type], device=x.device)
    ws_bytes = workspace.numel() * workspace.element_size() if workspace is not None else 0
    _check(lib.q8_conv2d(C.byref(d), _dev(x, "x"), _dev(w, "w"), _dev(bias, "bias"), _dev(scale, "scale"),
                         _dev(residual, "residual"), residual_scale, _dev(y, "y"), _dev(workspace, "workspace"),
                         ws_bytes, _stream()))
    return y


def q8_conv2d_then_1x1_supported(d1, d2):
    ok = C.c_int(0)
    _check(lib.q8_conv2d_then_1x1_supported(C.byref(d1), C.byref(d2), C.byref(ok)))
    return bool(ok.value)


def q8_conv2d_then_1x1(d1, d2, x, w1, bias1, scale1, w2, bias2, scale2, residual=None, residual_scale=0.0, y=None):
    """Layer d1 followed by the 1x1 layer d2 in one launch; the tensor between them is never written."""
    if y is None:
        P, Q = conv_out_shape(d2)
        y = torch.empty((d2.N, P, Q, d2.y_ldc or d2.K), dtype=TORCH_DTYPES[d2.y_type], device=x.device)
    _check(lib.q8_conv2d_then_1x1(C.byref(d1), C.byref(d2), _dev(x, "x"), _dev(w1, "w1"), _dev(bias1, "bias1"),
                                  _dev(scale1, "scale1"), _dev(w2, "w2"), _dev(bias2, "bias2"), _dev(scale2, "scale2"),
                                  _dev(residual, "residual"), residual_scale, _dev(y, "y"), _stream()))
    return y


def q8_int8_mma_rate(bn, chains, instructions, ctas, cycles):
    """cycles: int64 CUDA tensor of `ctas` entries, filled with the SM cycles each CTA needed."""
    _check(lib.q8_int8_mma_rate(bn, chains, instructions, ctas, _dev(cycles, "cycles"), _stream()))
    return cycles


def q8_selftest_bounded_wait(limit_us):
    _check(lib.q8_selftest_bounded_wait(int(limit_us), _stream()))


def q8_static_workspace_bytes():
    return int(lib.q8_static_workspace_bytes())


def q8_conv2d_static_workspace(d, x, w, bias, scale, residual=None, residual_scale=0.0, y=None):
    """q8_conv2d with the library's built-in scratch array instead of a caller workspace; allocates nothing
    (pass `y`; it is only created here, by torch, when omitted)."""
    if y is None:
        P, Q = conv_out_shape(d)
        y = torch.empty((d.N, P, Q, d.y_ldc or d.K), dtype=TORCH_DTYPES[d.y_type], device=x.device)
    _check(lib.q8_conv2d_static_workspace(C.byref(d), _dev(x, "x"), _dev(w, "w"), _dev(bias, "bias"), _dev(scale, "scale"),
                                          _dev(residual, "residual"), residual_scale, _dev(y, "y"), _stream()))
    return y


def q8_concat(xs, in_factors, out_factor, out=None):
    t = {torch.uint8: Q8_U8, torch.int8: Q8_S8}[xs[0].dtype]
    chans = [int(a.shape[-1]) for a in xs]
    pixels = xs[0].numel() // chans[0]
    if out is None:
        out = torch.empty(xs[0].shape[:-1] + (sum(chans),), dtype=xs[0].dtype, device=xs[0].device)
    ptrs = (C.c_void_p * len(xs))(*[a.data_ptr() for a in xs])
    for a in xs:
        _dev(a, "branch")
    _check(lib.q8_concat(len(xs), ptrs, (C.c_int * len(xs))(*chans), (C.c_float * len(xs))(*in_factors), out_factor, t,
                         pixels, _dev(out, "out"), _stream()))
    return out


def q8_calibrate_maxabs_rows(x, running):
    """running[r] = max(running[r], max|x[r, ...]|) for a tensor whose first dimension indexes the rows."""
    rows = int(x.shape[0])
    _check(lib.q8_calibrate_maxabs_rows(_dev(x, "x"), rows, x.numel() // max(rows, 1), _dev(running, "running"), _stream()))
    return running


def q8_quantize_rows(x, q_rows, out_type):
    """Eq. (Q) with the device vector q_rows holding one factor per row (first dimension) of x."""
    rows = int(x.shape[0])
    z = torch.empty(x.shape, dtype=TORCH_DTYPES[out_type], device=x.device)
    _check(lib.q8_quantize_rows(_dev(x, "x"), rows, x.numel() // max(rows, 1), _dev(q_rows, "q_rows"), out_type, _dev(z, "z"),
                                _stream()))
    return z


def q8_concat_branch(x, in_factor, out_factor, out, c_offset):
    """Writes x (re-expressed at out_factor) into channels c_offset.. of the wider tensor `out`."""
    t = {torch.uint8: Q8_U8, torch.int8: Q8_S8}[x.dtype]
    ch = int(x.shape[-1])
    _check(lib.q8_concat_branch(_dev(x, "x"), ch, in_factor, out_factor, t, x.numel() // ch, _dev(out, "out"),
                                int(out.shape[-1]), c_offset, _stream()))
    return out


def q8_pool_out_extent(H, k, stride, pad, ceil_mode=False):
    o = C.c_int()
    _check(lib.q8_pool_out_extent(H, k, stride, pad, int(ceil_mode), C.byref(o)))
    return o.value


def _pool(fn, x, k, stride, pad, ceil_mode, out):
    t = {torch.uint8: Q8_U8, torch.int8: Q8_S8}[x.dtype]
    N, H, W, Cc = x.shape
    P = q8_pool_out_extent(H, k[0], stride[0], pad[0], ceil_mode)
    Q = q8_pool_out_extent(W, k[1], stride[1], pad[1], ceil_mode)
    if out is None:
        out = torch.empty((N, P, Q, Cc), dtype=x.dtype, device=x.device)
    _check(fn(_dev(x, "x"), t, N, H, W, Cc, k[0], k[1], stride[0], stride[1], pad[0], pad[1], int(ceil_mode),
              _dev(out, "out"), _stream()))
    return out


def q8_maxpool2d(x, k, stride, pad=(0, 0), ceil_mode=False, out=None):
    return _pool(lib.q8_maxpool2d, x, k, stride, pad, ceil_mode, out)


def q8_avgpool2d(x, k, stride, pad=(0, 0), ceil_mode=False, out=None):
    return _pool(lib.q8_avgpool2d, x, k, stride, pad, ceil_mode, out)


def q8_l2norm(x, qx, eps, mult, out=None):
    """L2 normalisation across the last dimension of a u8 tensor; mult: CUDA fp32 [C] = gamma qx / qy."""
    Cc = int(x.shape[-1])
    if out is None:
        out = torch.empty_like(x)
    _check(lib.q8_l2norm(_dev(x, "x"), x.numel() // Cc, Cc, qx, eps, _dev(mult, "mult"), _dev(out, "out"), _stream()))
    return out


def q8_add_relu_quantize(a, b, q, out=None):
    """Q_8(max(a + b, 0), q) of two fp32 tensors as u8 (the FP32 route of a residual sum)."""
    if out is None:
        out = torch.empty(a.shape, dtype=torch.uint8, device=a.device)
    _check(lib.q8_add_relu_quantize(_dev(a, "a"), _dev(b, "b"), a.numel(), q, _dev(out, "out"), _stream()))
    return out


def q8_detection_output_workspace_bytes(N, P, classes, background, nms_top_k, keep_top_k):
    n = C.c_size_t()
    _check(lib.q8_detection_output_workspace_bytes(N, P, classes, background, nms_top_k, keep_top_k, C.byref(n)))
    return n.value


def _cell_view(t, what):
    """(pointer, cell stride in floats, cells per image) of a CUDA fp32 tensor [N, cells..., values] whose cells lie a
    fixed stride apart (a contiguous tensor, or a slice of the last dimension of one)."""
    if not (isinstance(t, torch.Tensor) and t.is_cuda and t.dtype == torch.float32 and t.dim() >= 2 and t.stride(-1) == 1):
        raise TypeError(f"{what}: expected a CUDA fp32 tensor with unit stride in its last dimension")
    if t.dim() == 2:
        return t.data_ptr(), int(t.stride(0)), 1
    stride = int(t.stride(-2))
    for i in range(t.dim() - 2):
        if t.shape[i] > 1 and t.stride(i) != t.stride(i + 1) * t.shape[i + 1]:
            raise TypeError(f"{what}: cells are not a fixed stride apart")
    cells = 1
    for v in t.shape[1:-1]:
        cells *= int(v)
    return t.data_ptr(), stride, cells


def q8_detection_output(sources, priors, variances, classes, background=0, conf_thresh=0.01, nms_thresh=0.45,
                        nms_top_k=400, keep_top_k=200, workspace=None, out=None, counts=None):
    """sources: list of (loc, conf, boxes_per_cell) with loc [N, cells..., boxes * 4] and conf [N, cells...,
    boxes * classes] CUDA fp32 tensors, contiguous or slices of the last dimension of a wider tensor (a merged
    head).  priors: CUDA fp32 [P, 4].  Returns (rows [N, keep_top_k, 6], counts [N])."""
    N = int(sources[0][0].shape[0])
    n = len(sources)
    locp, confp = (C.c_void_p * n)(), (C.c_void_p * n)()
    lstr, cstr, cells, boxes = (C.c_int * n)(), (C.c_int * n)(), (C.c_int * n)(), (C.c_int * n)()
    P = 0
    for i, (loc, conf, b) in enumerate(sources):
        locp[i], lstr[i], cells[i] = _cell_view(loc, "loc")
        confp[i], cstr[i], ccells = _cell_view(conf, "conf")
        if ccells != cells[i] or int(conf.shape[0]) != N or int(loc.shape[0]) != N:
            raise ValueError("loc and conf of a source must cover the same cells of the same images")
        boxes[i] = int(b)
        P += cells[i] * int(b)
    dev = sources[0][0].device
    nbytes = q8_detection_output_workspace_bytes(N, P, classes, background, nms_top_k, keep_top_k)
    if workspace is None:
        workspace = torch.empty(nbytes, dtype=torch.uint8, device=dev)
    if out is None:
        out = torch.empty((N, keep_top_k, 6), dtype=torch.float32, device=dev)
    if counts is None:
        counts = torch.empty(N, dtype=torch.int32, device=dev)
    var = (C.c_float * 4)(*[float(v) for v in variances])
    _check(lib.q8_detection_output(n, locp, lstr, confp, cstr, cells, boxes, _dev(priors, "priors"), var, N, classes, background,
                                   conf_thresh, nms_thresh, nms_top_k, keep_top_k, _dev(workspace, "workspace"), workspace.numel(),
                                   _dev(out, "out"), _dev(counts, "counts"), _stream()))
    return out, counts

"""numpy/ctypes face of the C++ oracle (oracle/q8_oracle.cpp).

Each function marshals arrays and calls the C++ routine of the same name; no
arithmetic of the method is done in Python.  Storage-type bounds used with
Eq. (Q): u8 [0, 255], s8 [-128, 127], s32 [-2^31, 2^31 - 1]; ``bounds_p``
gives the literal [-2^p, 2^p - 1].
"""
import ctypes as C

import numpy as np

from . import build as _build

_lib = C.CDLL(_build.build())

_f32p = C.POINTER(C.c_float)
_i32p = C.POINTER(C.c_int32)
_u8p = C.POINTER(C.c_uint8)
_i8p = C.POINTER(C.c_int8)

U8, S8, S32, F32 = 0, 1, 2, 3
BOUNDS = {U8: (0.0, 255.0), S8: (-128.0, 127.0), S32: (-2147483648.0, 2147483647.0)}
NP_TYPES = {U8: np.uint8, S8: np.int8, S32: np.int32, F32: np.float32}


def bounds_p(p):
    """Literal clamp bounds of Eq. (Q)."""
    return (-float(2 ** p), float(2 ** p - 1))


def _ptr(a, t):
    return a.ctypes.data_as(t)


def _f32(a):
    return np.ascontiguousarray(a, dtype=np.float32)


_lib.q8o_maxabs.restype = C.c_float
_lib.q8o_maxabs.argtypes = [_f32p, C.c_size_t, C.c_float]
_lib.q8o_factor.restype = C.c_float
_lib.q8o_factor.argtypes = [C.c_float, C.c_int]
_lib.q8o_quantize.restype = None
_lib.q8o_quantize.argtypes = [_f32p, C.c_size_t, C.c_float, C.c_double, C.c_double, _i32p]
_lib.q8o_dequantize.restype = None
_lib.q8o_dequantize.argtypes = [_i32p, C.c_size_t, C.c_float, _f32p]
_lib.q8o_eltwise_add.restype = C.c_float
_lib.q8o_eltwise_add.argtypes = [_i32p, C.c_float, _i32p, C.c_float, C.c_size_t, C.c_double, C.c_double, _i32p]
_lib.q8o_fold_bn.restype = None
_lib.q8o_fold_bn.argtypes = [_f32p] * 6 + [C.c_double, C.c_int, C.c_size_t, _f32p, _f32p]
_lib.q8o_fold_bn_f64.restype = None
_lib.q8o_fold_bn_f64.argtypes = [_f32p] * 6 + [C.c_double, C.c_int, C.c_size_t, C.POINTER(C.c_double),
                                 C.POINTER(C.c_double)]
_lib.q8o_requant_scale.restype = C.c_float
_lib.q8o_requant_scale.argtypes = [C.c_float] * 3
_lib.q8o_bias_factor.restype = C.c_float
_lib.q8o_bias_factor.argtypes = [C.c_float] * 2
_lib.q8o_conv_acc.restype = None
_lib.q8o_conv_acc.argtypes = [_u8p, C.c_int, _i8p, _i32p] + [C.c_int] * 13 + [_i32p, C.c_int]
_lib.q8o_epilogue.restype = None
_lib.q8o_epilogue.argtypes = [_i32p, C.c_size_t, C.c_int, _f32p, C.c_int, _u8p, C.c_int, C.c_float,
                              C.c_int, C.c_int, C.c_void_p, C.c_size_t, C.c_size_t]
_lib.q8o_concat.restype = None
_lib.q8o_concat.argtypes = [C.c_int, C.POINTER(_u8p), C.POINTER(C.c_int), _f32p, C.c_float, C.c_int,
                            C.c_size_t, _u8p]
_lib.q8o_pool_out.restype = C.c_int
_lib.q8o_pool_out.argtypes = [C.c_int] * 5
_lib.q8o_pool.restype = None
_lib.q8o_pool.argtypes = [_u8p, C.c_int, C.c_int] + [C.c_int] * 11 + [_u8p]
_lib.q8o_hw_threads.restype = C.c_int


def hw_threads():
    return int(_lib.q8o_hw_threads())


def maxabs(r, init=0.0):
    r = _f32(r).ravel()
    return float(np.float32(_lib.q8o_maxabs(_ptr(r, _f32p), r.size, np.float32(init))))


def factor(m, p):
    return float(np.float32(_lib.q8o_factor(np.float32(m), int(p))))


def quantize(r, q, dtype=None, lo=None, hi=None):
    """Eq. (Q).  ``dtype`` in {U8, S8, S32} picks storage bounds and type; or pass lo/hi (int32 result)."""
    r = _f32(r)
    if dtype is not None:
        lo, hi = BOUNDS[dtype]
    z = np.empty(r.shape, dtype=np.int32)
    _lib.q8o_quantize(_ptr(r.ravel(), _f32p), r.size, np.float32(q), lo, hi, _ptr(z, _i32p))
    return z.astype(NP_TYPES[dtype]) if dtype is not None else z


def dequantize(z, q):
    z32 = np.ascontiguousarray(z, dtype=np.int32)
    r = np.empty(z32.shape, dtype=np.float32)
    _lib.q8o_dequantize(_ptr(z32, _i32p), z32.size, np.float32(q), _ptr(r, _f32p))
    return r


def eltwise_add(z1, q1, z2, q2, lo, hi):
    a = np.ascontiguousarray(z1, dtype=np.int32)
    b = np.ascontiguousarray(z2, dtype=np.int32)
    z = np.empty(a.shape, dtype=np.int32)
    qo = _lib.q8o_eltwise_add(_ptr(a, _i32p), np.float32(q1), _ptr(b, _i32p), np.float32(q2), a.size,
                              lo, hi, _ptr(z, _i32p))
    return z, float(np.float32(qo))


def fold_bn(w, b, gamma, beta, mean, var, eps=1e-5, f64=False):
    """Folded (w', b').  ``f64=True`` returns the unrounded fp64 values."""
    w = _f32(w)
    K = w.shape[0]
    epk = w.size // K
    g, be, mu, va = _f32(gamma), _f32(beta), _f32(mean), _f32(var)
    bb = _f32(b) if b is not None else None
    if f64:
        dp = C.POINTER(C.c_double)
        w_out = np.empty(w.shape, dtype=np.float64)
        b_out = np.empty(K, dtype=np.float64)
        _lib.q8o_fold_bn_f64(_ptr(w, _f32p), _ptr(bb, _f32p) if bb is not None else None, _ptr(g, _f32p),
                             _ptr(be, _f32p), _ptr(mu, _f32p), _ptr(va, _f32p), float(eps), K, epk,
                             _ptr(w_out, dp), _ptr(b_out, dp))
        return w_out, b_out
    w_out = np.empty_like(w)
    b_out = np.empty(K, dtype=np.float32)
    _lib.q8o_fold_bn(_ptr(w, _f32p), _ptr(bb, _f32p) if bb is not None else None, _ptr(g, _f32p),
                     _ptr(be, _f32p), _ptr(mu, _f32p), _ptr(va, _f32p), float(eps), K, epk,
                     _ptr(w_out, _f32p), _ptr(b_out, _f32p))
    return w_out, b_out


def requant_scale(qx, qw, qy):
    return float(np.float32(_lib.q8o_requant_scale(np.float32(qx), np.float32(qw), np.float32(qy))))


def bias_factor(qx, qw):
    return float(np.float32(_lib.q8o_bias_factor(np.float32(qx), np.float32(qw))))


def out_hw(H, W, R, S, stride, pad, dil):
    P = (H + 2 * pad[0] - dil[0] * (R - 1) - 1) // stride[0] + 1
    Q = (W + 2 * pad[1] - dil[1] * (S - 1) - 1) // stride[1] + 1
    return P, Q


def conv_acc(x, w, bias=None, stride=(1, 1), pad=(0, 0), dil=(1, 1), threads=1):
    """x: NHWC uint8 or int8; w: KRSC int8; bias: int32[K] or None -> int32 [N,P,Q,K]."""
    assert x.dtype in (np.uint8, np.int8) and w.dtype == np.int8
    x = np.ascontiguousarray(x)
    w = np.ascontiguousarray(w)
    N, H, W, Cc = x.shape
    K, R, S, C2 = w.shape
    assert Cc == C2
    P, Q = out_hw(H, W, R, S, stride, pad, dil)
    acc = np.empty((N, P, Q, K), dtype=np.int32)
    bp = None
    if bias is not None:
        bias = np.ascontiguousarray(bias, dtype=np.int32)
        bp = _ptr(bias, _i32p)
    _lib.q8o_conv_acc(_ptr(x.view(np.uint8), _u8p), int(x.dtype == np.int8), _ptr(w, _i8p), bp,
                      N, H, W, Cc, K, R, S, stride[0], stride[1], pad[0], pad[1], dil[0], dil[1],
                      _ptr(acc, _i32p), int(threads))
    return acc


def epilogue(acc, scale, residual=None, res_scale=0.0, relu=False, y_type=U8, out=None, c_off=0):
    """acc: int32 [..., K].  Returns the output tensor (or writes a channel slice of ``out``)."""
    acc = np.ascontiguousarray(acc, dtype=np.int32)
    K = acc.shape[-1]
    M = acc.size // K
    scale = np.atleast_1d(_f32(scale))
    assert scale.size in (1, K)
    rp, rs = None, 0
    if residual is not None:
        assert residual.dtype in (np.uint8, np.int8) and residual.size == acc.size
        residual = np.ascontiguousarray(residual)
        rp, rs = _ptr(residual.view(np.uint8), _u8p), int(residual.dtype == np.int8)
    if out is None:
        y = np.empty(acc.shape, dtype=NP_TYPES[y_type])
        ldc = K
    else:
        y = out
        assert y.flags.c_contiguous and y.dtype == NP_TYPES[y_type]
        ldc = y.shape[-1]
    _lib.q8o_epilogue(_ptr(acc, _i32p), M, K, _ptr(scale, _f32p), scale.size, rp, rs,
                      np.float32(res_scale), int(relu), int(y_type), y.ctypes.data, ldc, int(c_off))
    return y


def conv2d(x, w, bias, scale, stride=(1, 1), pad=(0, 0), dil=(1, 1), residual=None, res_scale=0.0,
           relu=False, y_type=U8, threads=1, out=None, c_off=0):
    """Quantized affine layer: integer accumulator followed by the epilogue."""
    acc = conv_acc(x, w, bias, stride, pad, dil, threads)
    return epilogue(acc, scale, residual, res_scale, relu, y_type, out, c_off)


def concat(xs, in_factors, out_factor):
    """xs: list of [..., C_i] uint8/int8 arrays with equal leading dims."""
    dt = xs[0].dtype
    xs = [np.ascontiguousarray(a) for a in xs]
    chans = np.array([a.shape[-1] for a in xs], dtype=np.int32)
    pixels = xs[0].size // xs[0].shape[-1]
    y = np.empty(xs[0].shape[:-1] + (int(chans.sum()),), dtype=dt)
    ptrs = (_u8p * len(xs))(*[_ptr(a.view(np.uint8), _u8p) for a in xs])
    fac = _f32(in_factors)
    _lib.q8o_concat(len(xs), ptrs, _ptr(chans, C.POINTER(C.c_int)), _ptr(fac, _f32p),
                    np.float32(out_factor), int(dt == np.int8), pixels, _ptr(y.view(np.uint8), _u8p))
    return y


def pool_out(H, k, st, pad, ceil_mode=False):
    return int(_lib.q8o_pool_out(H, k, st, pad, int(ceil_mode)))


def pool(x, kind, k, stride, pad=(0, 0), ceil_mode=False):
    """kind: 'max' or 'avg'; x NHWC uint8/int8."""
    x = np.ascontiguousarray(x)
    N, H, W, Cc = x.shape
    P = pool_out(H, k[0], stride[0], pad[0], ceil_mode)
    Q = pool_out(W, k[1], stride[1], pad[1], ceil_mode)
    y = np.empty((N, P, Q, Cc), dtype=x.dtype)
    _lib.q8o_pool(_ptr(x.view(np.uint8), _u8p), int(x.dtype == np.int8), int(kind == "avg"), N, H, W, Cc,
                  k[0], k[1], stride[0], stride[1], pad[0], pad[1], int(ceil_mode),
                  _ptr(y.view(np.uint8), _u8p))
    return y


# ------------------------------------------------------------------ SSD tail (oracle/q8_oracle_detect.cpp)
_lib.q8o_l2norm_mult.restype = C.c_float
_lib.q8o_l2norm_mult.argtypes = [C.c_float] * 3
_lib.q8o_l2norm.restype = None
_lib.q8o_l2norm.argtypes = [_u8p, C.c_size_t, C.c_int, C.c_float, C.c_float, _f32p, _u8p]
_lib.q8o_exp.restype = C.c_float
_lib.q8o_exp.argtypes = [C.c_float]
_lib.q8o_softmax.restype = None
_lib.q8o_softmax.argtypes = [_f32p, C.c_size_t, C.c_int, _f32p]
_lib.q8o_decode_boxes.restype = None
_lib.q8o_decode_boxes.argtypes = [_f32p, _f32p, _f32p, C.c_int, C.c_int, _f32p]
_lib.q8o_iou.restype = C.c_float
_lib.q8o_iou.argtypes = [_f32p, _f32p]
_lib.q8o_detection_output.restype = None
_lib.q8o_detection_output.argtypes = [_f32p, _f32p, _f32p, _f32p, C.c_int, C.c_int, C.c_int, C.c_int, C.c_float,
                                      C.c_float, C.c_int, C.c_int, _f32p, _i32p]
_lib.q8o_add_relu_quantize.restype = None
_lib.q8o_add_relu_quantize.argtypes = [_f32p, _f32p, C.c_size_t, C.c_float, _u8p]


def l2norm_mult(gamma, qx, qy):
    """Per-channel multipliers gamma_c q_x / q_y of the L2 normalisation layer."""
    return np.array([_lib.q8o_l2norm_mult(np.float32(g), np.float32(qx), np.float32(qy)) for g in np.ravel(gamma)],
                    dtype=np.float32)


def l2norm(x, qx, eps, mult):
    """x: [..., C] uint8 codes with factor qx; mult: [C] from l2norm_mult.  Returns uint8 codes with factor qy."""
    x = np.ascontiguousarray(x, dtype=np.uint8)
    m = _f32(mult)
    y = np.empty_like(x)
    _lib.q8o_l2norm(_ptr(x, _u8p), x.size // x.shape[-1], x.shape[-1], np.float32(qx), np.float32(eps), _ptr(m, _f32p),
                    _ptr(y, _u8p))
    return y


def exp(x):
    x = _f32(x)
    return np.array([_lib.q8o_exp(v) for v in x.ravel()], dtype=np.float32).reshape(x.shape)


def softmax(conf):
    """conf: [..., classes] fp32 logits."""
    conf = _f32(conf)
    p = np.empty_like(conf)
    _lib.q8o_softmax(_ptr(conf, _f32p), conf.size // conf.shape[-1], conf.shape[-1], _ptr(p, _f32p))
    return p


def decode_boxes(loc, priors, var):
    """loc [N, P, 4], priors [P, 4] (cx, cy, w, h), var [4] -> corner boxes [N, P, 4]."""
    loc, priors, var = _f32(loc), _f32(priors), _f32(var)
    b = np.empty_like(loc)
    _lib.q8o_decode_boxes(_ptr(loc, _f32p), _ptr(priors, _f32p), _ptr(var, _f32p), loc.shape[0], loc.shape[1], _ptr(b, _f32p))
    return b


def iou(a, b):
    a, b = _f32(a), _f32(b)
    return float(_lib.q8o_iou(_ptr(a, _f32p), _ptr(b, _f32p)))


def detection_output(loc, conf, priors, var, background=0, conf_thresh=0.01, nms_thresh=0.45, nms_top_k=400,
                     keep_top_k=200):
    """loc [N, P, 4], conf [N, P, classes] logits.  Returns (rows [N, keep_top_k, 6], counts [N])."""
    loc, conf, priors, var = _f32(loc), _f32(conf), _f32(priors), _f32(var)
    N, P, classes = conf.shape
    out = np.empty((N, keep_top_k, 6), dtype=np.float32)
    counts = np.empty(N, dtype=np.int32)
    _lib.q8o_detection_output(_ptr(loc, _f32p), _ptr(conf, _f32p), _ptr(priors, _f32p), _ptr(var, _f32p), N, P, classes,
                              background, np.float32(conf_thresh), np.float32(nms_thresh), nms_top_k, keep_top_k,
                              _ptr(out, _f32p), _ptr(counts, _i32p))
    return out, counts


def add_relu_quantize(a, b, qy):
    """The FP32 route for a residual sum with a signed summand: Q_8(max(a + b, 0), q_y) as uint8."""
    a, b = _f32(a), _f32(b)
    y = np.empty(a.shape, dtype=np.uint8)
    _lib.q8o_add_relu_quantize(_ptr(a, _f32p), _ptr(b, _f32p), a.size, np.float32(qy), _ptr(y, _u8p))
    return y

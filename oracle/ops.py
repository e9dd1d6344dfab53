"""numpy front-end to the C oracle routines (see lop_oracle.c for the definitions)."""
import ctypes

import numpy as np

from . import build as _build

_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(_build.build())
        _lib.lop_oracle_bf16_rne.restype = ctypes.c_float
        _lib.lop_oracle_bf16_rne.argtypes = [ctypes.c_float]
        _lib.lop_oracle_num_threads.restype = ctypes.c_int
        _lib.lop_oracle_conv2d.restype = None
        _lib.lop_oracle_maxpool2d.restype = None
        _lib.lop_oracle_linear.restype = None
        _lib.lop_oracle_dwconv2d.restype = None
        _lib.lop_oracle_layernorm.restype = None
        _lib.lop_oracle_concat.restype = None
    return _lib


def _fp(a):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_float)) if a is not None else None


def _f32(a):
    return None if a is None else np.ascontiguousarray(a, dtype=np.float32)


def out_size(n, k, s, p, d):
    """Floor-mode output extent of a strided, padded, dilated window (Sec. IV-A block-wise operators)."""
    return (n + 2 * p - d * (k - 1) - 1) // s + 1


def bf16_rne(v):
    return float(lib().lop_oracle_bf16_rne(ctypes.c_float(v)))


def num_threads():
    return int(lib().lop_oracle_num_threads())


def conv2d(x, w, stride=(1, 1), pad=(0, 0), dil=(1, 1), scale=None, shift=None, res=None, res_pos=0,
           act=0, round_bf16=False, rows=None, out=None):
    """Rows ``rows=(lo,hi)`` (default all) of the NHWC convolution with fused epilogue, into ``out``."""
    x, w = _f32(x), _f32(w)
    N, H, W, Cin = x.shape
    Cout, kh, kw, cin2 = w.shape
    assert cin2 == Cin
    Ho, Wo = out_size(H, kh, stride[0], pad[0], dil[0]), out_size(W, kw, stride[1], pad[1], dil[1])
    assert Ho > 0 and Wo > 0
    if out is None:
        out = np.zeros((N, Ho, Wo, Cout), dtype=np.float32)
    assert out.shape == (N, Ho, Wo, Cout) and out.dtype == np.float32 and out.flags.c_contiguous
    scale, shift, res = _f32(scale), _f32(shift), _f32(res)
    if res is not None:
        assert res.shape == out.shape
    lo, hi = (0, Ho) if rows is None else rows
    lib().lop_oracle_conv2d(_fp(x), N, H, W, Cin, _fp(w), Cout, kh, kw, stride[0], stride[1], pad[0], pad[1],
                            dil[0], dil[1], _fp(scale), _fp(shift), _fp(res), int(res_pos), int(act),
                            int(bool(round_bf16)), int(lo), int(hi), _fp(out))
    return out


def maxpool2d(x, k, stride, pad=(0, 0), dil=(1, 1), rows=None, out=None):
    x = _f32(x)
    N, H, W, C = x.shape
    Ho, Wo = out_size(H, k[0], stride[0], pad[0], dil[0]), out_size(W, k[1], stride[1], pad[1], dil[1])
    assert Ho > 0 and Wo > 0
    if out is None:
        out = np.zeros((N, Ho, Wo, C), dtype=np.float32)
    assert out.shape == (N, Ho, Wo, C) and out.dtype == np.float32 and out.flags.c_contiguous
    lo, hi = (0, Ho) if rows is None else rows
    lib().lop_oracle_maxpool2d(_fp(x), N, H, W, C, k[0], k[1], stride[0], stride[1], pad[0], pad[1],
                               dil[0], dil[1], int(lo), int(hi), _fp(out))
    return out


def linear(x, w, scale=None, shift=None, res=None, res_pos=0, act=0, round_bf16=False, rows=None, out=None):
    """The row-wise operator Y = X W^T (Sec. IV-A, Eq. 1) on an NHWC tensor: every pixel's channel vector is a row of X.

    ``w``: [Cout, K] (or [Cout, 1, 1, K]).  ``rows=(lo, hi)``: image rows of every image to compute (default all); the
    matrix rows they stand for are  (n*H + h)*W .. for h in [lo, hi)."""
    x, w = _f32(x), _f32(w)
    N, H, W, K = x.shape
    w2 = w.reshape(w.shape[0], -1)
    Cout = w2.shape[0]
    assert w2.shape[1] == K
    if out is None:
        out = np.zeros((N, H, W, Cout), dtype=np.float32)
    assert out.shape == (N, H, W, Cout) and out.dtype == np.float32 and out.flags.c_contiguous
    scale, shift, res = _f32(scale), _f32(shift), _f32(res)
    if res is not None:
        assert res.shape == out.shape
    lo, hi = (0, H) if rows is None else rows
    M = N * H * W
    for n in range(N):
        lib().lop_oracle_linear(_fp(x), ctypes.c_longlong(M), K, _fp(w2), Cout, _fp(scale), _fp(shift), _fp(res), int(res_pos),
                                int(act), int(bool(round_bf16)), ctypes.c_longlong((n * H + lo) * W),
                                ctypes.c_longlong((n * H + hi) * W), _fp(out))
    return out


LAYERNORM_EPS = 1e-6


def dwconv2d(x, w, stride=(1, 1), pad=(0, 0), dil=(1, 1), scale=None, shift=None, res=None, res_pos=0, act=0,
             round_bf16=False, rows=None, out=None):
    """Rows ``rows`` of the depth-wise convolution (every channel its own kernel); ``w``: [C, kh, kw] (or [C, kh, kw, 1])."""
    x, w = _f32(x), _f32(w)
    N, H, W, C = x.shape
    w3 = w.reshape(w.shape[0], w.shape[1], w.shape[2])
    assert w3.shape[0] == C
    kh, kw = w3.shape[1], w3.shape[2]
    Ho, Wo = out_size(H, kh, stride[0], pad[0], dil[0]), out_size(W, kw, stride[1], pad[1], dil[1])
    assert Ho > 0 and Wo > 0
    if out is None:
        out = np.zeros((N, Ho, Wo, C), dtype=np.float32)
    assert out.shape == (N, Ho, Wo, C) and out.dtype == np.float32 and out.flags.c_contiguous
    scale, shift, res = _f32(scale), _f32(shift), _f32(res)
    lo, hi = (0, Ho) if rows is None else rows
    lib().lop_oracle_dwconv2d(_fp(x), N, H, W, C, _fp(np.ascontiguousarray(w3)), kh, kw, stride[0], stride[1], pad[0], pad[1],
                              dil[0], dil[1], _fp(scale), _fp(shift), _fp(res), int(res_pos), int(act), int(bool(round_bf16)),
                              int(lo), int(hi), _fp(out))
    return out


def layernorm(x, gamma=None, beta=None, eps=LAYERNORM_EPS, round_bf16=False, rows=None, out=None):
    """Layer normalisation over the channels of every pixel; ``rows``: image rows of every image (default all)."""
    x = _f32(x)
    N, H, W, C = x.shape
    if out is None:
        out = np.zeros((N, H, W, C), dtype=np.float32)
    assert out.shape == x.shape and out.dtype == np.float32 and out.flags.c_contiguous
    gamma, beta = _f32(gamma), _f32(beta)
    lo, hi = (0, H) if rows is None else rows
    for n in range(N):
        lib().lop_oracle_layernorm(_fp(x), ctypes.c_longlong(N * H * W), C, _fp(gamma), _fp(beta), ctypes.c_float(eps),
                                   int(bool(round_bf16)), ctypes.c_longlong((n * H + lo) * W), ctypes.c_longlong((n * H + hi) * W), _fp(out))
    return out


def concat(a, b, rows=None, out=None):
    """Channel concatenation of two NHWC tensors of equal N, H, W."""
    a, b = _f32(a), _f32(b)
    N, H, W, Ca = a.shape
    Cb = b.shape[3]
    assert b.shape[:3] == (N, H, W)
    if out is None:
        out = np.zeros((N, H, W, Ca + Cb), dtype=np.float32)
    assert out.shape == (N, H, W, Ca + Cb) and out.dtype == np.float32 and out.flags.c_contiguous
    lo, hi = (0, H) if rows is None else rows
    for n in range(N):
        lib().lop_oracle_concat(_fp(a), Ca, _fp(b), Cb, ctypes.c_longlong(N * H * W), ctypes.c_longlong((n * H + lo) * W),
                                ctypes.c_longlong((n * H + hi) * W), _fp(out))
    return out

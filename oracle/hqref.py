"""ctypes access to the oracle's C++ functions, on numpy (host) arrays.

Each wrapper only marshals arguments; the arithmetic is in hqref.cpp.  Tensors are NHWC; 4-bit
tensors are passed packed (two per byte along the channel axis) with the logical channel count.
"""
from __future__ import annotations

import ctypes as C

import numpy as np

from .build import build

_lib = None

HQREF_OK, HQREF_ERR_INVALID_ARG, HQREF_ERR_RANGE = 0, 1, 4


class OracleError(RuntimeError):
    def __init__(self, code: int):
        super().__init__(f"oracle returned status {code}")
        self.code = code


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        L.hqref_rshift_round.restype = C.c_int64
        L.hqref_rshift_round.argtypes = [C.c_int64, C.c_int32]
        L.hqref_dn.restype = C.c_int64
        L.hqref_dn.argtypes = [C.c_int32, C.c_int32, C.c_int32]
        vp, i32, i64 = C.c_void_p, C.c_int32, C.c_int64
        L.hqref_conv2d.restype = i32
        L.hqref_conv2d.argtypes = [vp, i32, i32, i32, i32, i32, i32, vp, i32, i32, i32, i32, i32, i32,
                                   vp, vp, vp, vp, i32, i32, vp, vp, i32, i32, i32, vp, i32, i32]
        L.hqref_linear.restype = i32
        L.hqref_linear.argtypes = [vp, i32, i32, i32, i32, vp, i32, i32, vp, vp, vp, i32, i32, i32, vp, i32, i32]
        L.hqref_residual_add.restype = i32
        L.hqref_residual_add.argtypes = [vp, i32, i32, vp, vp, vp, i32, i32, vp, vp, i64, i32,
                                         i32, i32, i32, vp, i32, i32]
        L.hqref_avgpool_requant.restype = i32
        L.hqref_avgpool_requant.argtypes = [vp, i32, i32, i32, i32, i32, i32, vp, vp, i32, i32, vp, i32, i32]
        L.hqref_maxpool.restype = i32
        L.hqref_maxpool.argtypes = [vp, i32, i32, i32, i32, i32, i32, i32, i32, i32, vp]
        L.hqref_concat_branch.restype = i32
        L.hqref_concat_branch.argtypes = [vp, i32, i32, vp, vp, i64, i32, i32, i32, i32, vp, i32, i32, i32, i32]
        L.hqref_sumpool.restype = i32
        L.hqref_sumpool.argtypes = [vp, i32, i32, i32, i32, i32, i32, i32, i32, i32, vp]
        L.hqref_num_threads.restype = i32
        _lib = L
    return _lib


def _p(a):
    if a is None:
        return None
    assert a.flags["C_CONTIGUOUS"]
    return a.ctypes.data_as(C.c_void_p)


def _i32(a):
    return None if a is None else np.ascontiguousarray(a, dtype=np.int32)


def _out_array(shape_nhwc, bits, signed):
    n, h, w, c = shape_nhwc
    if bits == 32:
        return np.zeros((n, h, w, c), np.int32)
    if bits == 8:
        return np.zeros((n, h, w, c), np.int8 if signed else np.uint8)
    return np.zeros((n, h, w, c // 2), np.uint8)


def _check(code):
    if code != HQREF_OK:
        raise OracleError(code)


def rshift_round(x: int, c: int) -> int:
    return int(lib().hqref_rshift_round(x, c))


def dn(q: int, b: int, c: int) -> int:
    return int(lib().hqref_dn(q, b, c))


def num_threads() -> int:
    return int(lib().hqref_num_threads())


def conv2d(x, cin, in_bits, in_signed, wgt, cout, kh, kw, stride, pad, bias, b, c,
           res=None, res_bits=0, res_signed=0, rb=None, rc=None,
           relu=1, qmin=0, qmax=255, out_bits=8, out_signed=0):
    """x: (n,h,w,cin or cin/2) array.  Returns the output array (packed if out_bits == 4)."""
    x = np.ascontiguousarray(x)
    wgt = np.ascontiguousarray(wgt)
    n, h, w = x.shape[:3]
    ho = (h + 2 * pad - kh) // stride + 1
    wo = (w + 2 * pad - kw) // stride + 1
    out = _out_array((n, ho, wo, cout), out_bits, out_signed)
    bias, b, c, rb, rc = _i32(bias), _i32(b), _i32(c), _i32(rb), _i32(rc)
    res = None if res is None else np.ascontiguousarray(res)
    _check(lib().hqref_conv2d(_p(x), n, h, w, cin, in_bits, in_signed, _p(wgt), cout, kh, kw, stride, pad,
                              in_bits, _p(bias), _p(b), _p(c), _p(res), res_bits, res_signed, _p(rb), _p(rc),
                              relu, qmin, qmax, _p(out), out_bits, out_signed))
    return out


def conv_case(case: dict):
    """Run a dict produced by the workload generator's conv_case()."""
    return conv2d(case["x"], case["cin"], case["bits"], case["in_signed"], case["wgt"], case["cout"],
                  case["kh"], case["kw"], case["stride"], case["pad"], case["bias"], case["b"], case["c"],
                  case["res"], case["res_bits"], case["res_signed"], case["rb"], case["rc"],
                  case["relu"], case["qmin"], case["qmax"], case["out_bits"], case["out_signed"])


def linear(x, cin, in_bits, in_signed, wgt, cout, bias, b, c, relu, qmin, qmax, out_bits, out_signed):
    x = np.ascontiguousarray(x)
    n = x.shape[0]
    out = _out_array((n, 1, 1, cout), out_bits, out_signed)
    bias, b, c = _i32(bias), _i32(b), _i32(c)
    wgt = np.ascontiguousarray(wgt)
    _check(lib().hqref_linear(_p(x), n, cin, in_bits, in_signed, _p(wgt), cout, in_bits, _p(bias), _p(b), _p(c),
                              relu, qmin, qmax, _p(out), out_bits, out_signed))
    return out


def residual_add(main, main_bits, main_signed, mb, mc, res, res_bits, res_signed, rb, rc, ch,
                 relu, qmin, qmax, out_bits, out_signed):
    main = np.ascontiguousarray(main)
    shape = main.shape[:-1] + (ch,)
    pixels = int(np.prod(shape[:-1]))
    n, h, w = (shape[0], shape[1], shape[2]) if len(shape) == 4 else (pixels, 1, 1)
    out = _out_array((n, h, w, ch), out_bits, out_signed)
    mb, mc, rb, rc = _i32(mb), _i32(mc), _i32(rb), _i32(rc)
    res = None if res is None else np.ascontiguousarray(res)
    _check(lib().hqref_residual_add(_p(main), main_bits, main_signed, _p(mb), _p(mc), _p(res), res_bits,
                                    res_signed, _p(rb), _p(rc), pixels, ch, relu, qmin, qmax,
                                    _p(out), out_bits, out_signed))
    return out


def avgpool_requant(x, ch, in_bits, in_signed, b, c, qmin, qmax, out_bits=8, out_signed=0):
    x = np.ascontiguousarray(x)
    n, h, w = x.shape[:3]
    out = _out_array((n, 1, 1, ch), out_bits, out_signed)
    b, c = _i32(b), _i32(c)
    _check(lib().hqref_avgpool_requant(_p(x), n, h, w, ch, in_bits, in_signed, _p(b), _p(c), qmin, qmax,
                                       _p(out), out_bits, out_signed))
    return out


def concat_requant(branches, relu, qmin, qmax, out_bits=8, out_signed=0):
    """Inception concatenation (Appendix E): `branches` is a list of dicts {x, bits, signed, ch, b, c};
    every branch is rescaled by its own dyadic pairs and written at its channel offset."""
    first = np.ascontiguousarray(branches[0]["x"])
    n, h, w = first.shape[:3]
    pixels = n * h * w
    out_ch = sum(int(br["ch"]) for br in branches)
    out = _out_array((n, h, w, out_ch), out_bits, out_signed)
    off = 0
    for br in branches:
        x = np.ascontiguousarray(br["x"])
        b, c = _i32(br["b"]), _i32(br["c"])
        _check(lib().hqref_concat_branch(_p(x), br["bits"], br["signed"], _p(b), _p(c), pixels, br["ch"],
                                         relu, qmin, qmax, _p(out), out_bits, out_signed, out_ch, off))
        off += int(br["ch"])
    return out


def sumpool(x, ch, bits, signed, k, stride, pad):
    """k x k window sums in INT32 (taps outside the image count as 0): the Inception pooling branch, Appendix E."""
    x = np.ascontiguousarray(x)
    n, h, w = x.shape[:3]
    ho = (h + 2 * pad - k) // stride + 1
    wo = (w + 2 * pad - k) // stride + 1
    out = np.zeros((n, ho, wo, ch), np.int32)
    _check(lib().hqref_sumpool(_p(x), n, h, w, ch, bits, signed, k, stride, pad, _p(out)))
    return out


def maxpool(x, k, stride, pad, signed=0):
    x = np.ascontiguousarray(x)
    n, h, w, ch = x.shape
    ho = (h + 2 * pad - k) // stride + 1
    wo = (w + 2 * pad - k) // stride + 1
    out = np.zeros((n, ho, wo, ch), x.dtype)
    bits = 32 if x.dtype == np.int32 else 8
    _check(lib().hqref_maxpool(_p(x), n, h, w, ch, bits, 1 if bits == 32 else signed, k, stride, pad, _p(out)))
    return out

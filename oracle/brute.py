"""ctypes front end of brute.c (test infrastructure, see that file's header).

`build()` compiles brute.c with gcc into oracle/_build/; the wrappers marshal
numpy arrays and add nothing to the arithmetic except the optional `pad`
step in front of the paper's un-padded equations.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "brute.c")
_OUT_DIR = os.path.join(_HERE, "_build")
_LIB_PATH = os.path.join(_OUT_DIR, "libo2.so")
_lib = None

_I64 = ctypes.c_int64
_FP = ctypes.POINTER(ctypes.c_float)
_DP = ctypes.POINTER(ctypes.c_double)
_LP = ctypes.POINTER(ctypes.c_int64)


def build(force: bool = False) -> str:
    os.makedirs(_OUT_DIR, exist_ok=True)
    if force or not os.path.exists(_LIB_PATH) or os.path.getmtime(_LIB_PATH) < os.path.getmtime(_SRC):
        tmp = _LIB_PATH + ".%d.tmp" % os.getpid()
        subprocess.check_call(
            ["gcc", "-O2", "-march=native", "-fopenmp", "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"]
        )
        os.replace(tmp, _LIB_PATH)
    return _LIB_PATH


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.o2_num_threads.restype = ctypes.c_int
    return _lib


def num_threads() -> int:
    return int(lib().o2_num_threads())


def _f32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float32)


def _fp(a):
    return a.ctypes.data_as(_FP)


def _dp(a):
    return a.ctypes.data_as(_DP)


def pad_hw(x, pads, fill: float) -> np.ndarray:
    """Constant border on the last two dimensions; pads = ((h_lo,h_hi),(w_lo,w_hi))."""
    x = _f32(x)
    (a, b), (c, d) = pads
    if not (a or b or c or d):
        return x
    h, w = x.shape[-2:]
    outer = int(np.prod(x.shape[:-2], dtype=np.int64))
    out = np.empty(x.shape[:-2] + (h + a + b, w + c + d), dtype=np.float32)
    lib().o2_pad_hw(_fp(x), _fp(out), _I64(outer), _I64(h), _I64(w), _I64(a), _I64(b), _I64(c), _I64(d),
                    ctypes.c_float(fill))
    return out


def _conv_dims(x, wt, strides):
    n, c, h, w = x.shape
    o, c2, kh, kw = wt.shape
    if c != c2 or kh > h or kw > w:
        raise ValueError("conv2d shape mismatch")
    ho, wo = (h - kh) // strides[0] + 1, (w - kw) // strides[1] + 1
    return n, c, h, w, o, kh, kw, ho, wo


def conv2d(x, wt, strides=(1, 1), pads=((0, 0), (0, 0))) -> np.ndarray:
    """(N,C,H,W) x (O,C,Kh,Kw) -> float64 (N,O,Ho,Wo), the paper's conv2d equation."""
    x, wt = pad_hw(x, pads, 0.0), _f32(wt)
    n, c, h, w, o, kh, kw, ho, wo = _conv_dims(x, wt, strides)
    out = np.empty((n, o, ho, wo), dtype=np.float64)
    lib().o2_conv2d(_fp(x), _fp(wt), _dp(out), *map(_I64, (n, c, h, w, o, kh, kw, strides[0], strides[1])))
    return out


def conv2d_f32acc(x, wt, strides=(1, 1), pads=((0, 0), (0, 0))) -> np.ndarray:
    x, wt = pad_hw(x, pads, 0.0), _f32(wt)
    n, c, h, w, o, kh, kw, ho, wo = _conv_dims(x, wt, strides)
    out = np.empty((n, o, ho, wo), dtype=np.float32)
    lib().o2_conv2d_f32acc(_fp(x), _fp(wt), _fp(out), *map(_I64, (n, c, h, w, o, kh, kw, strides[0], strides[1])))
    return out


def conv2d_sampled(x, wt, flat_nchw_index, strides=(1, 1), pads=((0, 0), (0, 0))) -> np.ndarray:
    """The conv2d equation at the listed flat offsets into the (N,O,Ho,Wo) result."""
    x, wt = pad_hw(x, pads, 0.0), _f32(wt)
    n, c, h, w, o, kh, kw, ho, wo = _conv_dims(x, wt, strides)
    idx = np.ascontiguousarray(flat_nchw_index, dtype=np.int64)
    vals = np.empty(idx.shape[0], dtype=np.float64)
    lib().o2_conv2d_sampled(_fp(x), _fp(wt), idx.ctypes.data_as(_LP), _I64(idx.shape[0]), _dp(vals),
                            *map(_I64, (n, c, h, w, o, kh, kw, strides[0], strides[1])))
    return vals


def conv_out_shape(x_shape, w_shape, strides, pads):
    n, c, h, w = x_shape
    o, _, kh, kw = w_shape
    hp, wp = h + sum(pads[0]), w + sum(pads[1])
    return n, o, (hp - kh) // strides[0] + 1, (wp - kw) // strides[1] + 1


def matmul(p, q) -> np.ndarray:
    """R_ij = sum_k P_ik Q_kj."""
    p, q = _f32(p), _f32(q)
    i, k = p.shape
    k2, j = q.shape
    if k != k2:
        raise ValueError("matmul shape mismatch")
    r = np.empty((i, j), dtype=np.float64)
    lib().o2_matmul(_fp(p), _fp(q), _dp(r), _I64(i), _I64(k), _I64(j))
    return r


def rowdot(a, b, rows=None) -> np.ndarray:
    """R[m,o] = A[m,:] . B[o,:] for all rows of A, or only for `rows`."""
    a, b = _f32(a), _f32(b)
    m, k = a.shape
    o, k2 = b.shape
    if k != k2:
        raise ValueError("rowdot shape mismatch")
    if rows is None:
        r = np.empty((m, o), dtype=np.float64)
        lib().o2_rowdot(_fp(a), _fp(b), _dp(r), _I64(m), _I64(o), _I64(k), None, _I64(m))
    else:
        rows = np.ascontiguousarray(rows, dtype=np.int64)
        r = np.empty((rows.shape[0], o), dtype=np.float64)
        lib().o2_rowdot(_fp(a), _fp(b), _dp(r), _I64(m), _I64(o), _I64(k), rows.ctypes.data_as(_LP),
                        _I64(rows.shape[0]))
    return r


def maxpool(x, wshape, strides, pads=((0, 0), (0, 0))) -> np.ndarray:
    """(N,C,H,W) -> float32 (N,C,Ho,Wo); padded cells hold -inf."""
    x = pad_hw(x, pads, -np.inf)
    n, c, h, w = x.shape
    kh, kw = wshape
    ho, wo = (h - kh) // strides[0] + 1, (w - kw) // strides[1] + 1
    out = np.empty((n, c, ho, wo), dtype=np.float32)
    lib().o2_maxpool(_fp(x), _fp(out), *map(_I64, (n * c, h, w, kh, kw, strides[0], strides[1])))
    return out


def im2col(x, kh, kw, strides=(1, 1), pads=((0, 0), (0, 0))) -> np.ndarray:
    """flatten(windows((N),(C,H,W)), (C,Kh,Kw), (1,S0,S1)) -> float32 (N*Ho*Wo, C*Kh*Kw)."""
    x = pad_hw(x, pads, 0.0)
    n, c, h, w = x.shape
    ho, wo = (h - kh) // strides[0] + 1, (w - kw) // strides[1] + 1
    out = np.empty((n * ho * wo, c * kh * kw), dtype=np.float32)
    lib().o2_im2col(_fp(x), _fp(out), *map(_I64, (n, c, h, w, kh, kw, strides[0], strides[1])))
    return out


def transpose_021(x) -> np.ndarray:
    """(B,R,C) -> (B,C,R)."""
    x = _f32(x)
    b, r, c = x.shape
    out = np.empty((b, c, r), dtype=np.float32)
    lib().o2_transpose_021(_fp(x), _fp(out), _I64(b), _I64(r), _I64(c))
    return out

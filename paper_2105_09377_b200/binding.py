"""ctypes binding of the C-ABI library (include/gl.h): argument marshalling only.

Every function has the name of the C entry point it calls.  torch supplies
device memory and the current stream; nothing is computed in Python.  If the
shared library is missing, importing this module raises: there is no CPU path.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass
from typing import Optional, Sequence

import torch

GL_MAX_DIMS = 8
GL_BF16, GL_F32 = 1, 2
GL_PAD_ZERO, GL_PAD_NEG_INF = 0, 1
GL_EPILOGUE_RELU = 0x2
GL_DOT_GENERAL_KERNEL = 0x100
GL_OUT_NCHW = 0x4
GL_OUT_BF16 = 0x8
GL_OK = 0

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libglenside.so")


class GlAp(ctypes.Structure):
    _fields_ = [
        ("data", ctypes.c_void_p),
        ("dtype", ctypes.c_int32),
        ("ndim", ctypes.c_int32),
        ("access_ndim", ctypes.c_int32),
        ("reserved_", ctypes.c_int32),
        ("shape", ctypes.c_int64 * GL_MAX_DIMS),
    ]


class GlWindows(ctypes.Structure):
    _fields_ = [
        ("n", ctypes.c_int32),
        ("pad_kind", ctypes.c_int32),
        ("wshape", ctypes.c_int64 * GL_MAX_DIMS),
        ("stride", ctypes.c_int64 * GL_MAX_DIMS),
        ("pad_lo", ctypes.c_int64 * GL_MAX_DIMS),
        ("pad_hi", ctypes.c_int64 * GL_MAX_DIMS),
    ]


EXPORTS = [
    "gl_shape_access", "gl_shape_windows", "gl_shape_flatten", "gl_shape_transpose", "gl_shape_pad",
    "gl_shape_cartesian_dot", "gl_shape_reduce_max", "gl_access_windows", "gl_access_flatten",
    "gl_access_transpose", "gl_access_pad", "gl_cartesian_dot", "gl_cartesian_dot_workspace",
    "gl_compute_reduce_max", "gl_compute_relu", "gl_poll_device_status", "gl_strerror", "gl_version",
    "gl_cartesian_dot_static", "gl_shape_cartesian_dot_nchw",
    "gl_shape_slice", "gl_shape_concat", "gl_shape_pair", "gl_shape_squeeze", "gl_shape_reshape",
    "gl_shape_reduce_sum", "gl_access_slice", "gl_access_concat", "gl_access_pair", "gl_compute_reduce_sum",
    "gl_selftest_bounded_wait",
]


def _load() -> ctypes.CDLL:
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(
            "libglenside.so is not built (run `python -m paper_2105_09377_b200.build`); "
            "there is no fallback path")
    lib = ctypes.CDLL(LIB_PATH)
    ap, win, vp = ctypes.POINTER(GlAp), ctypes.POINTER(GlWindows), ctypes.c_void_p
    i32p = ctypes.POINTER(ctypes.c_int32)
    sig = {
        "gl_shape_access": [ap, ctypes.c_int32, ap],
        "gl_shape_windows": [ap, win, ap],
        "gl_shape_flatten": [ap, ap],
        "gl_shape_transpose": [ap, i32p, ap],
        "gl_shape_pad": [ap, ctypes.c_int32, ctypes.c_int64, ctypes.c_int64, ap],
        "gl_shape_cartesian_dot": [ap, win, ap, ap],
        "gl_shape_cartesian_dot_nchw": [ap, win, ap, ap],
        "gl_shape_reduce_max": [ap, win, ap],
        "gl_shape_slice": [ap, ctypes.c_int32, ctypes.c_int64, ctypes.c_int64, ap],
        "gl_shape_concat": [ap, ap, ctypes.c_int32, ap],
        "gl_shape_pair": [ap, ap, ap],
        "gl_shape_squeeze": [ap, ctypes.c_int32, ap],
        "gl_shape_reshape": [ap, ctypes.POINTER(ctypes.c_int64), ctypes.c_int32, ctypes.c_int32, ap],
        "gl_shape_reduce_sum": [ap, ap],
        "gl_access_slice": [ap, ctypes.c_int32, ctypes.c_int64, ctypes.c_int64, ap, vp],
        "gl_access_concat": [ap, ap, ctypes.c_int32, ap, vp],
        "gl_access_pair": [ap, ap, ap, vp],
        "gl_compute_reduce_sum": [ap, ap, vp],
        "gl_access_windows": [ap, win, ap, vp],
        "gl_access_flatten": [ap, ap],
        "gl_access_transpose": [ap, i32p, ap, vp],
        "gl_access_pad": [ap, ctypes.c_int32, ctypes.c_int64, ctypes.c_int64, ctypes.c_int32, ap, vp],
        "gl_cartesian_dot": [ap, win, ap, ap, ctypes.c_uint32, vp, ctypes.c_size_t, vp],
        "gl_cartesian_dot_static": [ap, win, ap, ap, ctypes.c_uint32, vp],
        "gl_compute_reduce_max": [ap, win, ap, vp],
        "gl_compute_relu": [ap, ap, vp],
        "gl_poll_device_status": [vp],
        "gl_selftest_bounded_wait": [ctypes.c_uint32, vp],
    }
    for name, args in sig.items():
        fn = getattr(lib, name)
        fn.argtypes = args
        fn.restype = ctypes.c_int
    lib.gl_cartesian_dot_workspace.argtypes = [ap, win, ap, ctypes.c_uint32]
    lib.gl_cartesian_dot_workspace.restype = ctypes.c_size_t
    lib.gl_strerror.argtypes = [ctypes.c_int]
    lib.gl_strerror.restype = ctypes.c_char_p
    lib.gl_version.restype = ctypes.c_int
    return lib


LIB = _load()


class GlError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__("%s: %s (code %d)" % (where, LIB.gl_strerror(code).decode(), code))


def _check(code: int, where: str):
    if code != GL_OK:
        raise GlError(code, where)


_DTYPES = {torch.bfloat16: GL_BF16, torch.float32: GL_F32}
_TORCH = {GL_BF16: torch.bfloat16, GL_F32: torch.float32}


@dataclass
class AccessPattern:
    """A dense device tensor viewed as (access dims, compute dims)."""

    tensor: torch.Tensor
    access_ndim: int

    @property
    def access_shape(self):
        return tuple(self.tensor.shape[: self.access_ndim])

    @property
    def compute_shape(self):
        return tuple(self.tensor.shape[self.access_ndim:])

    @property
    def shape(self):
        return (self.access_shape, self.compute_shape)


def _meta(shape: Sequence[int], access_ndim: int, dtype: int, data: int = 0) -> GlAp:
    if len(shape) > GL_MAX_DIMS:
        raise GlError(3, "too many dimensions")
    m = GlAp()
    m.data = data
    m.dtype = dtype
    m.ndim = len(shape)
    m.access_ndim = access_ndim
    for i, s in enumerate(shape):
        m.shape[i] = int(s)
    return m


def _struct(a: AccessPattern) -> GlAp:
    t = a.tensor
    if not t.is_contiguous():
        raise ValueError("access patterns are dense row-major tensors")
    return _meta(tuple(t.shape), a.access_ndim, _DTYPES[t.dtype], t.data_ptr())


def _alloc(meta: GlAp, device) -> AccessPattern:
    shape = tuple(meta.shape[i] for i in range(meta.ndim))
    return AccessPattern(torch.empty(shape, dtype=_TORCH[meta.dtype], device=device), meta.access_ndim)


def _stream(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def windows_spec(wshape, stride, pad_lo=None, pad_hi=None, pad_kind=GL_PAD_ZERO) -> GlWindows:
    n = len(wshape)
    w = GlWindows()
    w.n = n
    w.pad_kind = pad_kind
    pad_lo = pad_lo or [0] * n
    pad_hi = pad_hi or [0] * n
    for i in range(n):
        w.wshape[i], w.stride[i], w.pad_lo[i], w.pad_hi[i] = int(wshape[i]), int(stride[i]), int(pad_lo[i]), int(pad_hi[i])
    return w


def _wptr(w: Optional[GlWindows]):
    return ctypes.byref(w) if w is not None else None


# ---- host-only shape inference: (shape, access_ndim, dtype) in, the same out ----

def _shape_result(m: GlAp):
    return tuple(m.shape[i] for i in range(m.ndim)), m.access_ndim, m.dtype


def gl_shape_access(shape, access_ndim, i, dtype=GL_F32):
    out = GlAp()
    _check(LIB.gl_shape_access(ctypes.byref(_meta(shape, access_ndim, dtype)), i, ctypes.byref(out)), "gl_shape_access")
    return _shape_result(out)


def gl_shape_windows(shape, access_ndim, w: GlWindows, dtype=GL_F32):
    out = GlAp()
    _check(LIB.gl_shape_windows(ctypes.byref(_meta(shape, access_ndim, dtype)), ctypes.byref(w), ctypes.byref(out)),
           "gl_shape_windows")
    return _shape_result(out)


def gl_shape_flatten(shape, access_ndim, dtype=GL_F32):
    out = GlAp()
    _check(LIB.gl_shape_flatten(ctypes.byref(_meta(shape, access_ndim, dtype)), ctypes.byref(out)), "gl_shape_flatten")
    return _shape_result(out)


def gl_shape_transpose(shape, access_ndim, perm, dtype=GL_F32):
    out = GlAp()
    arr = (ctypes.c_int32 * len(perm))(*perm)
    _check(LIB.gl_shape_transpose(ctypes.byref(_meta(shape, access_ndim, dtype)), arr, ctypes.byref(out)),
           "gl_shape_transpose")
    return _shape_result(out)


def gl_shape_pad(shape, access_ndim, dim, lo, hi, dtype=GL_F32):
    out = GlAp()
    _check(LIB.gl_shape_pad(ctypes.byref(_meta(shape, access_ndim, dtype)), dim, lo, hi, ctypes.byref(out)), "gl_shape_pad")
    return _shape_result(out)


def gl_shape_cartesian_dot(shape0, access0, w: Optional[GlWindows], shape1, access1):
    out = GlAp()
    _check(LIB.gl_shape_cartesian_dot(ctypes.byref(_meta(shape0, access0, GL_BF16)), _wptr(w),
                                      ctypes.byref(_meta(shape1, access1, GL_BF16)), ctypes.byref(out)),
           "gl_shape_cartesian_dot")
    return _shape_result(out)


def gl_shape_cartesian_dot_nchw(shape0, access0, w: GlWindows, shape1, access1):
    out = GlAp()
    _check(LIB.gl_shape_cartesian_dot_nchw(ctypes.byref(_meta(shape0, access0, GL_BF16)), ctypes.byref(w),
                                           ctypes.byref(_meta(shape1, access1, GL_BF16)), ctypes.byref(out)),
           "gl_shape_cartesian_dot_nchw")
    return _shape_result(out)


def gl_shape_reduce_max(shape, access_ndim, w: Optional[GlWindows]):
    out = GlAp()
    _check(LIB.gl_shape_reduce_max(ctypes.byref(_meta(shape, access_ndim, GL_F32)), _wptr(w), ctypes.byref(out)),
           "gl_shape_reduce_max")
    return _shape_result(out)


# ---- device operations ----

def gl_access_windows(a: AccessPattern, w: GlWindows, out: Optional[AccessPattern] = None, stream=None) -> AccessPattern:
    sa = _struct(a)
    if out is None:
        m = GlAp()
        _check(LIB.gl_shape_windows(ctypes.byref(sa), ctypes.byref(w), ctypes.byref(m)), "gl_shape_windows")
        out = _alloc(m, a.tensor.device)
    so = _struct(out)
    _check(LIB.gl_access_windows(ctypes.byref(sa), ctypes.byref(w), ctypes.byref(so), _stream(stream)), "gl_access_windows")
    return out


def gl_access_flatten(a: AccessPattern) -> AccessPattern:
    sa, so = _struct(a), GlAp()
    _check(LIB.gl_access_flatten(ctypes.byref(sa), ctypes.byref(so)), "gl_access_flatten")
    assert so.data == sa.data
    shape = tuple(so.shape[i] for i in range(so.ndim))
    return AccessPattern(a.tensor.view(shape), so.access_ndim)


def gl_access_transpose(a: AccessPattern, perm, out: Optional[AccessPattern] = None, stream=None) -> AccessPattern:
    sa = _struct(a)
    arr = (ctypes.c_int32 * len(perm))(*perm)
    if out is None:
        m = GlAp()
        _check(LIB.gl_shape_transpose(ctypes.byref(sa), arr, ctypes.byref(m)), "gl_shape_transpose")
        out = _alloc(m, a.tensor.device)
    so = _struct(out)
    _check(LIB.gl_access_transpose(ctypes.byref(sa), arr, ctypes.byref(so), _stream(stream)), "gl_access_transpose")
    return out


def gl_access_pad(a: AccessPattern, dim: int, lo: int, hi: int, pad_kind=GL_PAD_ZERO,
                  out: Optional[AccessPattern] = None, stream=None) -> AccessPattern:
    sa = _struct(a)
    if out is None:
        m = GlAp()
        _check(LIB.gl_shape_pad(ctypes.byref(sa), dim, lo, hi, ctypes.byref(m)), "gl_shape_pad")
        out = _alloc(m, a.tensor.device)
    so = _struct(out)
    _check(LIB.gl_access_pad(ctypes.byref(sa), dim, lo, hi, pad_kind, ctypes.byref(so), _stream(stream)), "gl_access_pad")
    return out


def gl_cartesian_dot_workspace(a0: AccessPattern, w: Optional[GlWindows], a1: AccessPattern, flags: int = 0) -> int:
    return int(LIB.gl_cartesian_dot_workspace(ctypes.byref(_struct(a0)), _wptr(w), ctypes.byref(_struct(a1)), flags))


def gl_cartesian_dot(a0: AccessPattern, w: Optional[GlWindows], a1: AccessPattern, out: Optional[AccessPattern] = None,
                     flags: int = 0, workspace: Optional[torch.Tensor] = None, stream=None) -> AccessPattern:
    s0, s1 = _struct(a0), _struct(a1)
    if out is None:
        m = GlAp()
        if flags & GL_OUT_NCHW:
            _check(LIB.gl_shape_cartesian_dot_nchw(ctypes.byref(s0), _wptr(w), ctypes.byref(s1), ctypes.byref(m)),
                   "gl_shape_cartesian_dot_nchw")
        else:
            _check(LIB.gl_shape_cartesian_dot(ctypes.byref(s0), _wptr(w), ctypes.byref(s1), ctypes.byref(m)),
                   "gl_shape_cartesian_dot")
        if flags & GL_OUT_BF16:
            m.dtype = GL_BF16
        out = _alloc(m, a0.tensor.device)
    if workspace is None:
        need = int(LIB.gl_cartesian_dot_workspace(ctypes.byref(s0), _wptr(w), ctypes.byref(s1), flags))
        if need:
            workspace = torch.empty(need + 1024, dtype=torch.uint8, device=a0.tensor.device)
    ws_ptr, ws_bytes = 0, 0
    if workspace is not None:
        ws_ptr = (workspace.data_ptr() + 1023) // 1024 * 1024
        ws_bytes = workspace.numel() * workspace.element_size() - (ws_ptr - workspace.data_ptr())
    so = _struct(out)
    _check(LIB.gl_cartesian_dot(ctypes.byref(s0), _wptr(w), ctypes.byref(s1), ctypes.byref(so), flags, ws_ptr, ws_bytes,
                                _stream(stream)), "gl_cartesian_dot")
    return out


GL_STATIC_SCRATCH_BYTES = 32 << 20


def gl_cartesian_dot_static(a0: AccessPattern, w: Optional[GlWindows], a1: AccessPattern, out: AccessPattern,
                            flags: int = 0, stream=None) -> AccessPattern:
    """gl_cartesian_dot without a workspace argument, for callers that may not allocate device
    memory: the scratch is a fixed 32 MiB array inside the library.  `out` must be supplied (this
    wrapper allocates nothing either).  Calls that may overlap on the GPU must be ordered by the
    caller, and the first call on a device should precede any stream capture."""
    s0, s1, so = _struct(a0), _struct(a1), _struct(out)
    _check(LIB.gl_cartesian_dot_static(ctypes.byref(s0), _wptr(w), ctypes.byref(s1), ctypes.byref(so), flags,
                                       _stream(stream)), "gl_cartesian_dot_static")
    return out


def gl_compute_reduce_max(a: AccessPattern, w: Optional[GlWindows], out: Optional[AccessPattern] = None,
                          stream=None) -> AccessPattern:
    sa = _struct(a)
    if out is None:
        m = GlAp()
        _check(LIB.gl_shape_reduce_max(ctypes.byref(sa), _wptr(w), ctypes.byref(m)), "gl_shape_reduce_max")
        out = _alloc(m, a.tensor.device)
    so = _struct(out)
    _check(LIB.gl_compute_reduce_max(ctypes.byref(sa), _wptr(w), ctypes.byref(so), _stream(stream)), "gl_compute_reduce_max")
    return out


def gl_access_slice(a: AccessPattern, dim: int, lo: int, hi: int, out: Optional[AccessPattern] = None,
                    stream=None) -> AccessPattern:
    sa = _struct(a)
    if out is None:
        m = GlAp()
        _check(LIB.gl_shape_slice(ctypes.byref(sa), dim, lo, hi, ctypes.byref(m)), "gl_shape_slice")
        out = _alloc(m, a.tensor.device)
    so = _struct(out)
    _check(LIB.gl_access_slice(ctypes.byref(sa), dim, lo, hi, ctypes.byref(so), _stream(stream)), "gl_access_slice")
    return out


def gl_access_concat(a: AccessPattern, b: AccessPattern, dim: int, out: Optional[AccessPattern] = None,
                     stream=None) -> AccessPattern:
    sa, sb = _struct(a), _struct(b)
    if out is None:
        m = GlAp()
        _check(LIB.gl_shape_concat(ctypes.byref(sa), ctypes.byref(sb), dim, ctypes.byref(m)), "gl_shape_concat")
        out = _alloc(m, a.tensor.device)
    so = _struct(out)
    _check(LIB.gl_access_concat(ctypes.byref(sa), ctypes.byref(sb), dim, ctypes.byref(so), _stream(stream)),
           "gl_access_concat")
    return out


def gl_access_pair(a: AccessPattern, b: AccessPattern, out: Optional[AccessPattern] = None, stream=None) -> AccessPattern:
    sa, sb = _struct(a), _struct(b)
    if out is None:
        m = GlAp()
        _check(LIB.gl_shape_pair(ctypes.byref(sa), ctypes.byref(sb), ctypes.byref(m)), "gl_shape_pair")
        out = _alloc(m, a.tensor.device)
    so = _struct(out)
    _check(LIB.gl_access_pair(ctypes.byref(sa), ctypes.byref(sb), ctypes.byref(so), _stream(stream)), "gl_access_pair")
    return out


def gl_access_squeeze(a: AccessPattern, dim: int) -> AccessPattern:
    """`squeeze` is metadata: the result views the same storage."""
    m = GlAp()
    _check(LIB.gl_shape_squeeze(ctypes.byref(_struct(a)), dim, ctypes.byref(m)), "gl_shape_squeeze")
    return AccessPattern(a.tensor.view(tuple(m.shape[i] for i in range(m.ndim))), m.access_ndim)


def gl_access_reshape(a: AccessPattern, access_shape, compute_shape) -> AccessPattern:
    """`reshape` is metadata: the result views the same storage."""
    shape = tuple(access_shape) + tuple(compute_shape)
    arr = (ctypes.c_int64 * max(1, len(shape)))(*shape)
    m = GlAp()
    _check(LIB.gl_shape_reshape(ctypes.byref(_struct(a)), arr, len(shape), len(access_shape), ctypes.byref(m)),
           "gl_shape_reshape")
    return AccessPattern(a.tensor.view(shape), len(access_shape))


def gl_compute_reduce_sum(a: AccessPattern, out: Optional[AccessPattern] = None, stream=None) -> AccessPattern:
    sa = _struct(a)
    if out is None:
        m = GlAp()
        _check(LIB.gl_shape_reduce_sum(ctypes.byref(sa), ctypes.byref(m)), "gl_shape_reduce_sum")
        out = _alloc(m, a.tensor.device)
    so = _struct(out)
    _check(LIB.gl_compute_reduce_sum(ctypes.byref(sa), ctypes.byref(so), _stream(stream)), "gl_compute_reduce_sum")
    return out


def gl_compute_relu(a: AccessPattern, out: Optional[AccessPattern] = None, stream=None) -> AccessPattern:
    sa = _struct(a)
    if out is None:
        out = AccessPattern(torch.empty_like(a.tensor), a.access_ndim)
    so = _struct(out)
    _check(LIB.gl_compute_relu(ctypes.byref(sa), ctypes.byref(so), _stream(stream)), "gl_compute_relu")
    return out


def gl_poll_device_status(stream=None) -> int:
    return int(LIB.gl_poll_device_status(_stream(stream)))


def gl_selftest_bounded_wait(limit_ms: int, stream=None) -> None:
    _check(LIB.gl_selftest_bounded_wait(limit_ms, _stream(stream)), "gl_selftest_bounded_wait")


def gl_strerror(code: int) -> str:
    return LIB.gl_strerror(code).decode()


def gl_version() -> int:
    return int(LIB.gl_version())


class Prepared:
    """A device call with its argument structures built once, for launch loops
    where Python marshalling would otherwise outweigh a microsecond-scale kernel.
    The stream is looked up at call time, so a prepared call can be captured
    into a CUDA graph."""

    def __init__(self, fn, args, keep):
        self._fn, self._args, self._keep = fn, args, keep

    def __call__(self, stream=None):
        rc = self._fn(*self._args, _stream(stream))
        if rc != GL_OK:
            raise GlError(rc, self._fn.__name__)


def _ws(workspace):
    if workspace is None:
        return 0, 0
    ptr = (workspace.data_ptr() + 1023) // 1024 * 1024
    return ptr, workspace.numel() * workspace.element_size() - (ptr - workspace.data_ptr())


def prepare_cartesian_dot(a0: AccessPattern, w: Optional[GlWindows], a1: AccessPattern, out: AccessPattern,
                          flags: int = 0, workspace: Optional[torch.Tensor] = None) -> Prepared:
    s0, s1, so = _struct(a0), _struct(a1), _struct(out)
    ws_ptr, ws_bytes = _ws(workspace)
    args = (ctypes.byref(s0), _wptr(w), ctypes.byref(s1), ctypes.byref(so), flags, ws_ptr, ws_bytes)
    return Prepared(LIB.gl_cartesian_dot, args, (s0, s1, so, w, a0, a1, out, workspace))


def prepare_access_windows(a: AccessPattern, w: GlWindows, out: AccessPattern) -> Prepared:
    sa, so = _struct(a), _struct(out)
    return Prepared(LIB.gl_access_windows, (ctypes.byref(sa), ctypes.byref(w), ctypes.byref(so)), (sa, so, w, a, out))


def prepare_access_transpose(a: AccessPattern, perm, out: AccessPattern) -> Prepared:
    sa, so = _struct(a), _struct(out)
    arr = (ctypes.c_int32 * len(perm))(*perm)
    return Prepared(LIB.gl_access_transpose, (ctypes.byref(sa), arr, ctypes.byref(so)), (sa, so, arr, a, out))


def prepare_compute_reduce_max(a: AccessPattern, w: Optional[GlWindows], out: AccessPattern) -> Prepared:
    sa, so = _struct(a), _struct(out)
    return Prepared(LIB.gl_compute_reduce_max, (ctypes.byref(sa), _wptr(w), ctypes.byref(so)), (sa, so, w, a, out))


def prepare_access_pad(a: AccessPattern, dim: int, lo: int, hi: int, pad_kind: int, out: AccessPattern) -> Prepared:
    sa, so = _struct(a), _struct(out)
    return Prepared(LIB.gl_access_pad, (ctypes.byref(sa), dim, lo, hi, pad_kind, ctypes.byref(so)), (sa, so, a, out))


def prepare_compute_relu(a: AccessPattern, out: AccessPattern) -> Prepared:
    sa, so = _struct(a), _struct(out)
    return Prepared(LIB.gl_compute_relu, (ctypes.byref(sa), ctypes.byref(so)), (sa, so, a, out))


def output_like(shape_fn_result, device) -> AccessPattern:
    """Allocate the output described by a gl_shape_* result (shape, access_ndim, dtype)."""
    shape, na, dt = shape_fn_result
    return AccessPattern(torch.empty(shape, dtype=_TORCH[dt], device=device), na)

"""Host-only checks of the C-ABI library: it loads without a GPU, exports every
symbol the header declares, infers the shapes of the paper's transformer table
(checked against the interpreter and the printed shape traces) and rejects
malformed arguments before touching the device."""
import ctypes
import os
import re

import numpy as np
import pytest

from oracle import interp as gi

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def gl():
    from paper_2105_09377_b200 import build
    build.build()
    from paper_2105_09377_b200 import binding
    return binding


def test_exports_match_header(gl):
    header = open(os.path.join(ROOT, "include", "gl.h")).read()
    declared = set(re.findall(r"GL_API[^;(]*?\b(gl_[a-z_0-9]+)\s*\(", header))
    assert len(declared) >= 18
    assert declared == set(gl.EXPORTS)
    lib = ctypes.CDLL(gl.LIB_PATH)
    for name in declared:
        assert hasattr(lib, name), name
    assert gl.gl_version() >= 100
    assert gl.gl_strerror(0) == "ok" and "NULL" in gl.gl_strerror(1)


def test_struct_layout_matches_header(gl):
    assert ctypes.sizeof(gl.GlAp) == 8 + 4 * 4 + 8 * 8
    assert ctypes.sizeof(gl.GlWindows) == 8 + 4 * 8 * 8


def test_shape_rules_against_interpreter(gl):
    n, c, h, w, o, kh, kw, sh, sw = 2, 3, 9, 8, 4, 3, 2, 2, 1
    act = gi.access(np.zeros((n, c, h, w)), 1)
    wts = gi.access(np.zeros((o, c, kh, kw)), 1)
    win = gi.windows(act, (c, kh, kw), (1, sh, sw))
    spec = gl.windows_spec((c, kh, kw), (1, sh, sw))
    shp, na, _ = gl.gl_shape_windows((n, c, h, w), 1, spec)
    assert (shp[:na], shp[na:]) == win.shape
    shp, na, dt = gl.gl_shape_cartesian_dot((n, c, h, w), 1, spec, (o, c, kh, kw), 1)
    dot = gi.compute("dotProd", gi.cart_prod(win, wts))
    assert (shp[:na], shp[na:]) == dot.shape and dt == gl.GL_F32
    # flatten of both sides gives the im2col matrices of Section 5.3
    fl, fna, _ = gl.gl_shape_flatten(win.data.shape, win.access_ndim)
    assert (fl[:fna], fl[fna:]) == gi.flatten(win).shape
    shp, na, _ = gl.gl_shape_cartesian_dot(fl, fna, None, (o, c * kh * kw), 1)
    assert shp == (win.data.shape[0] * win.data.shape[1] * win.data.shape[2] * win.data.shape[3], o) and na == 2
    # transpose keeps the split: ((N),(O)) -> ((O),(N))
    assert gl.gl_shape_transpose((6, 9), 1, (1, 0))[:2] == ((9, 6), 1)
    tr = gi.transpose(gi.access(np.zeros((2, 3, 4, 5)), 2), (0, 3, 1, 2))
    shp, na, _ = gl.gl_shape_transpose((2, 3, 4, 5), 2, (0, 3, 1, 2))
    assert (shp[:na], shp[na:]) == tr.shape
    # max pooling
    pool = gi.compute("reduceMax", gi.windows(gi.access(np.zeros((n, c, h, w)), 2), (kh, kw), (sh, sw)))
    shp, na, _ = gl.gl_shape_reduce_max((n, c, h, w), 2, gl.windows_spec((kh, kw), (sh, sw)))
    assert (shp[:na], shp[na:]) == pool.shape
    assert gl.gl_shape_reduce_max((4, 5, 6), 1, None)[:2] == ((4,), 1)
    # Fig. 2a in full: transpose(squeeze(dotProd ...)) -> ((N,O,H',W'),())
    full = gi.transpose(gi.squeeze(dot, 1), (0, 3, 1, 2))
    shp, na, dt = gl.gl_shape_cartesian_dot_nchw((n, c, h, w), 1, spec, (o, c, kh, kw), 1)
    assert (shp[:na], shp[na:]) == full.shape and dt == gl.GL_F32
    cl = gl.windows_spec((kh, kw, c), (sh, sw, 1))
    assert gl.gl_shape_cartesian_dot_nchw((n, h, w, c), 1, cl, (o, kh, kw, c), 1)[0] == full.data.shape
    # access, flatten edge cases, pad
    assert gl.gl_shape_access((2, 3, 4), 1, 3)[:2] == ((2, 3, 4), 3)
    assert gl.gl_shape_flatten((2, 3, 4), 3)[:2] == ((24,), 1)
    assert gl.gl_shape_flatten((2, 3, 4), 0)[:2] == ((24,), 0)
    assert gl.gl_shape_pad((2, 3, 4), 1, 2, 1, 3)[:2] == ((2, 3, 8), 1)


@pytest.mark.parametrize("b,w,s,lo,hi", [(8, 3, 1, 0, 0), (56, 3, 1, 1, 1), (224, 7, 2, 3, 3), (112, 3, 2, 1, 1),
                                         (56, 1, 2, 0, 0), (10, 3, 2, 0, 0), (9, 3, 2, 0, 1)])
def test_windows_extent_with_padding(gl, b, w, s, lo, hi):
    spec = gl.windows_spec((w,), (s,), (lo,), (hi,))
    shp, na, _ = gl.gl_shape_windows((5, b), 1, spec)
    assert shp == (5, gi.windows_out_extent(b + lo + hi, w, s), w) and na == 2


def test_argument_errors(gl):
    E = gl.GlError
    with pytest.raises(E) as e:
        gl.gl_shape_transpose((2, 3), 1, (0, 0))
    assert e.value.code == 5                                   # GL_ERR_PERM
    with pytest.raises(E) as e:
        gl.gl_shape_windows((2, 3), 1, gl.windows_spec((4,), (1,)))      # window > extent
    assert e.value.code == 4
    with pytest.raises(E) as e:
        gl.gl_shape_windows((2, 3), 1, gl.windows_spec((2, 2), (1, 1)))  # wrong count
    assert e.value.code == 4
    with pytest.raises(E) as e:
        gl.gl_shape_windows((2, 5), 1, gl.windows_spec((2,), (1,), (2,), (0,)))   # pad >= window
    assert e.value.code == 4
    with pytest.raises(E) as e:
        gl.gl_shape_cartesian_dot((4, 6), 1, None, (3, 5), 1)   # compute shapes differ
    assert e.value.code == 4
    with pytest.raises(E) as e:
        gl.gl_shape_access((2, 3), 1, 5)
    assert e.value.code == 3
    with pytest.raises(E) as e:
        gl.gl_shape_access((2, 0), 1, 1)                        # extents are positive
    assert e.value.code == 4
    with pytest.raises(E) as e:
        gl.gl_shape_reduce_max((2, 3), 2, None)                 # no compute dims to reduce
    assert e.value.code == 4
    # device calls validate before launching: NULL data is refused on a machine without a GPU too
    a = gl._meta((4, 8), 1, gl.GL_BF16, 0)
    out = gl._meta((4, 4), 2, gl.GL_F32, 0)
    rc = gl.LIB.gl_cartesian_dot(ctypes.byref(a), None, ctypes.byref(a), ctypes.byref(out), 0, None, 0, None)
    assert rc == 1                                              # GL_ERR_NULL
    a.data = 0x1008                                             # misaligned
    rc = gl.LIB.gl_compute_relu(ctypes.byref(a), ctypes.byref(a), None)
    assert rc == 6                                              # GL_ERR_ALIGN
    assert gl.LIB.gl_cartesian_dot_workspace(ctypes.byref(a), None, ctypes.byref(out), 0) == 0


def test_blocking_transformer_shapes(gl, golden_dir):
    """slice / transpose / cartProd / dotProd / pair / reduceSum / concat: the library's shape rules
    reproduce the annotations of the blocked 32x32 matMul (Fig. 8) and agree with the interpreter."""
    import ctypes as ct

    def shape_of(fn, *args):
        out = gl.GlAp()
        rc = fn(*args, ct.byref(out))
        assert rc == 0, rc
        shp = tuple(out.shape[i] for i in range(out.ndim))
        return (shp[:out.access_ndim], shp[out.access_ndim:])

    m = gl._meta
    act = m((32, 32), 1, gl.GL_BF16)
    s1 = gl.GlAp()
    assert gl.LIB.gl_shape_slice(ct.byref(act), 0, 0, 16, ct.byref(s1)) == 0
    assert shape_of(gl.LIB.gl_shape_slice, ct.byref(s1), 1, 0, 16) == ((16,), (16,))
    dot = m((16, 16), 2, gl.GL_F32)
    assert shape_of(gl.LIB.gl_shape_pair, ct.byref(dot), ct.byref(dot)) == ((16, 16), (2,))
    pr = m((16, 16, 2), 2, gl.GL_F32)
    assert shape_of(gl.LIB.gl_shape_reduce_sum, ct.byref(pr)) == ((16, 16), ())
    assert shape_of(gl.LIB.gl_shape_concat, ct.byref(dot), ct.byref(dot), 1) == ((16, 32), ())
    row = m((16, 32), 2, gl.GL_F32)
    assert shape_of(gl.LIB.gl_shape_concat, ct.byref(row), ct.byref(row), 0) == ((32, 32), ())
    # against the interpreter on lopsided shapes
    a = gi.access(np.zeros((2, 3, 4, 5)), 2)
    am = m((2, 3, 4, 5), 2, gl.GL_F32)
    assert shape_of(gl.LIB.gl_shape_slice, ct.byref(am), 2, 1, 3) == gi.slice_(a, 2, 1, 3).shape
    assert shape_of(gl.LIB.gl_shape_pair, ct.byref(am), ct.byref(am)) == gi.pair(a, a).shape
    b = m((2, 3, 6, 5), 2, gl.GL_F32)
    assert shape_of(gl.LIB.gl_shape_concat, ct.byref(am), ct.byref(b), 2) == gi.concat(a, gi.access(np.zeros((2, 3, 6, 5)), 2), 2).shape
    assert shape_of(gl.LIB.gl_shape_squeeze, ct.byref(m((2, 1, 3), 2, gl.GL_F32)), 1) == gi.squeeze(gi.access(np.zeros((2, 1, 3)), 2), 1).shape
    assert shape_of(gl.LIB.gl_shape_squeeze, ct.byref(m((2, 3, 1), 2, gl.GL_F32)), 2) == ((2, 3), ())
    arr = (ct.c_int64 * 3)(6, 2, 10)
    assert shape_of(gl.LIB.gl_shape_reshape, ct.byref(am), arr, 3, 1) == gi.reshape(a, (6,), (2, 10)).shape
    out = gl.GlAp()
    bad = (ct.c_int64 * 2)(3, 40)
    assert gl.LIB.gl_shape_reshape(ct.byref(am), bad, 2, 1, ct.byref(out)) == 4
    assert gl.LIB.gl_shape_slice(ct.byref(am), 2, 3, 3, ct.byref(out)) == 4          # empty range
    assert gl.LIB.gl_shape_concat(ct.byref(am), ct.byref(m((2, 4, 4, 5), 2, gl.GL_F32)), 2, ct.byref(out)) == 4
    assert gl.LIB.gl_shape_squeeze(ct.byref(am), 0, ct.byref(out)) == 4


def test_scratch_sizes_follow_the_layout_rules(gl):
    """gl_cartesian_dot_workspace is pure host arithmetic: the bytes it asks for are those of the layout
    copies each kind of convolution makes (checked against the sizes written out by hand)."""
    def need(x_shape, w_shape, spec, flags=0):
        a = gl._meta(x_shape, 1, gl.GL_BF16)
        b = gl._meta(w_shape, 1, gl.GL_BF16)
        return int(gl.LIB.gl_cartesian_dot_workspace(ctypes.byref(a), ctypes.byref(spec), ctypes.byref(b), flags))

    def up(v, a=1024):
        return (v + a - 1) // a * a

    # channels-last items with a channel count that is a multiple of 8: nothing to copy
    assert need((32, 56, 56, 64), (64, 3, 3, 64), gl.windows_spec((3, 3, 64), (1, 1, 1), (1, 1, 0), (1, 1, 0))) == 0
    # (C,H,W) items, 3x3: channels-last copies of the activations and of the weights
    spec = gl.windows_spec((128, 3, 3), (1, 1, 1), (0, 1, 1), (0, 1, 1))
    assert need((32, 128, 28, 28), (128, 128, 3, 3), spec) == up(32 * 28 * 28 * 128 * 2) + up(128 * 9 * 128 * 2)
    # (C,H,W) items, 1x1 stride 2, no pad: only the pixels the windows touch, weights [O, C]
    spec = gl.windows_spec((256, 1, 1), (1, 2, 2))
    assert need((8, 256, 30, 30), (128, 256, 1, 1), spec) == up(8 * 15 * 15 * 256 * 2) + up(128 * 256 * 2)
    # ... unless the rows are ones the TMA unit can fetch (W a multiple of 8, at most 64): read in place, no copy
    assert need((32, 256, 56, 56), (128, 256, 1, 1), spec) == 0
    # RGB stem, stride 2, either item layout: both operands are read where they are, nothing is copied
    for shape, wshape, spec in (((32, 3, 224, 224), (64, 3, 7, 7), gl.windows_spec((3, 7, 7), (1, 2, 2), (0, 3, 3), (0, 3, 3))),
                                ((32, 224, 224, 3), (64, 7, 7, 3), gl.windows_spec((7, 7, 3), (2, 2, 1), (3, 3, 0), (3, 3, 0)))):
        assert need(shape, wshape, spec) == 0
    # small M, long K: partial planes of the split contraction (26 tiles of 128x256 -> 5 slices of 15 K blocks)
    spec = gl.windows_spec((3, 3, 512), (1, 1, 1), (1, 1, 0), (1, 1, 0))
    assert need((32, 7, 7, 512), (512, 3, 3, 512), spec) == up(5 * 1568 * 512 * 4)

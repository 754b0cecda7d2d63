"""GPU parity of the memory-bound access operators against the CPU checker.
They move or compare values, so every comparison is bit-exact."""
import numpy as np
import pytest
import torch

from oracle import brute
from oracle import interp as gi
from paper_2105_09377_b200 import synth
from tests.gpu_util import to_bf16_device, to_f32_device

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def gl():
    from paper_2105_09377_b200 import binding
    return binding


def _same_bits(got: torch.Tensor, ref: np.ndarray):
    g = got.float().cpu().numpy()
    assert g.shape == ref.shape
    np.testing.assert_array_equal(g.view(np.uint32), np.ascontiguousarray(ref, dtype=np.float32).view(np.uint32))


TRANSPOSE_CASES = [
    ((2, 8, 4, 12), 1, (0, 2, 3, 1)),       # NCHW -> NHWC, vector path
    ((3, 5, 7, 9), 1, (0, 2, 3, 1)),        # odd extents: scalar tiles
    ((2, 6, 5, 16), 2, (0, 3, 1, 2)),       # (N,H',W',O) -> (N,O,H',W') of Fig. 2a
    ((70, 130), 1, (1, 0)),                 # plain matrix, several ragged tiles
    ((4, 3, 200), 1, (1, 0, 2)),            # innermost kept: row gather
    ((4, 3, 37), 1, (1, 0, 2)),
    ((3, 4, 5, 6, 7), 2, (4, 1, 3, 0, 2)),  # rank 5, general permutation
    ((5, 1, 6), 1, (2, 1, 0)),              # size-1 dim in the middle
    ((24,), 1, (0,)),                       # identity
    ((2, 3, 4), 1, (0, 1, 2)),
    ((1, 64, 3, 3, 8, 2, 2, 5), 3, (7, 6, 5, 4, 3, 2, 1, 0)),  # rank 8 reversal
]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("shape,na,perm", TRANSPOSE_CASES)
def test_transpose(gl, shape, na, perm, dtype):
    x = synth.uniform(7, 1, shape, -1.0, 1.0)
    if dtype == "bf16":
        x = synth.bf16_round(x)
    ref = gi.transpose(gi.access(x, na), perm)
    dev = to_f32_device(x) if dtype == "f32" else to_bf16_device(x)
    out = gl.gl_access_transpose(gl.AccessPattern(dev, na), perm)
    assert out.shape == ref.shape
    _same_bits(out.tensor, ref.data.astype(np.float32))


def test_transpose_full_size_nchw_to_nhwc(gl):
    cfg = synth.MEM_TRANSPOSE
    x = cfg.inputs(synth.config_seed(4))
    out = gl.gl_access_transpose(gl.AccessPattern(to_f32_device(x), 1), cfg.perm).tensor
    n, c, h, w = cfg.shape
    ref = brute.transpose_021(x.reshape(n, c, h * w)).reshape(n, h, w, c)
    assert torch.equal(out.cpu(), torch.from_numpy(ref))


WINDOW_CASES = [
    # shape, access_ndim, window, stride, pad_lo, pad_hi, kind
    ((1, 3, 8, 8), 1, (3, 3, 3), (1, 1, 1), (0, 0, 0), (0, 0, 0), 0),       # the tiny conv configuration
    ((2, 4, 9, 10), 1, (4, 3, 3), (1, 1, 1), (0, 1, 1), (0, 1, 1), 0),      # 3x3 pad 1, K multiple of 4
    ((2, 3, 11, 9), 1, (3, 7, 7), (1, 2, 2), (0, 3, 3), (0, 3, 3), 0),      # 7x7 s2 p3, K = 147 (scalar stores)
    ((2, 8, 6, 6), 1, (8, 1, 1), (1, 2, 2), (0, 0, 0), (0, 0, 0), 0),       # 1x1 stride 2
    ((2, 3, 9, 8), 2, (3, 2), (2, 1), (0, 0), (0, 0), 0),                   # pooling-style 2D windows
    ((2, 3, 9, 8), 2, (3, 3), (2, 2), (1, 1), (1, 1), 1),                   # -inf border
    ((3, 10), 1, (4,), (3,), (1,), (2,), 0),                                # 1D windows, uneven pads
    ((2, 5, 6, 7), 1, (2, 3, 2), (2, 1, 3), (1, 0, 1), (0, 2, 0), 0),       # windows over channels too
    ((2, 6, 4), 1, (6, 4), (1, 1), (0, 0), (0, 0), 0),                      # window == whole item
    # rows of whole 16-byte pieces (aligned staging), stride 1, Kw >= 3 (sliding gather)
    ((2, 4, 9, 12), 1, (4, 3, 3), (1, 1, 1), (0, 1, 1), (0, 1, 1), 0),      # K = 36
    ((2, 64, 5, 8), 1, (64, 3, 3), (1, 1, 1), (0, 1, 1), (0, 1, 1), 0),     # K = 576: two channel halves per slab
    ((2, 64, 5, 8), 1, (64, 3, 3), (1, 1, 1), (0, 1, 1), (0, 1, 1), 1),     # the same with a -inf border
    ((1, 4, 8, 16), 1, (4, 5, 5), (1, 1, 1), (0, 2, 2), (0, 2, 2), 0),      # Kw = 5: pieces inside one staged row
    ((1, 8, 6, 8), 1, (8, 2, 4), (1, 1, 1), (0, 0, 1), (0, 1, 2), 1),       # Kw = 4, uneven pads, two halves
    ((1, 4, 3, 136), 1, (4, 3, 3), (1, 1, 1), (0, 1, 1), (0, 1, 1), 0),     # rows longer than 32 pieces
    ((2, 4, 9, 16), 1, (4, 3, 3), (1, 2, 2), (0, 1, 1), (0, 1, 1), 0),      # stride 2: aligned staging, table gather
    ((1, 4, 6, 8), 1, (4, 3, 7), (1, 1, 1), (0, 1, 5), (0, 1, 1), 0),       # left border wider than one piece
    ((1, 4, 4, 4), 1, (4, 3, 3), (1, 1, 1), (0, 0, 0), (0, 0, 0), 0),       # two output columns
    ((3, 16, 4, 60), 1, (16, 3, 3), (1, 1, 1), (0, 1, 1), (0, 1, 1), 0),    # segments with a ragged tail (W' = 60)
    ((1, 128, 4, 8), 1, (128, 3, 3), (1, 1, 1), (0, 1, 1), (0, 1, 1), 0),   # K = 1152: two halves for 2-byte elements too
    ((1, 128, 5, 6), 1, (128, 3, 3), (1, 2, 1), (0, 1, 1), (0, 1, 1), 0),   # two halves, rows that are no whole pieces
]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("shape,na,wshape,stride,lo,hi,kind", WINDOW_CASES)
def test_windows(gl, shape, na, wshape, stride, lo, hi, kind, dtype):
    x = synth.uniform(8, 1, shape, -1.0, 1.0)
    if dtype == "bf16":
        x = synth.bf16_round(x)
    a = gi.access(x, na)
    for i, (l, h) in enumerate(zip(lo, hi)):
        if l or h:
            a = gi.pad(a, na + i, l, h, "neg_inf" if kind else "zero")
    ref = gi.windows(a, wshape, stride)
    dev = to_f32_device(x) if dtype == "f32" else to_bf16_device(x)
    out = gl.gl_access_windows(gl.AccessPattern(dev, na), gl.windows_spec(wshape, stride, lo, hi, kind))
    assert out.shape == ref.shape
    _same_bits(out.tensor, ref.data.astype(np.float32))
    # flatten is metadata: same storage, the im2col matrix view
    flat = gl.gl_access_flatten(out)
    assert flat.tensor.data_ptr() == out.tensor.data_ptr()
    assert flat.shape == gi.flatten(ref).shape


def test_im2col_full_size(gl):
    cfg = synth.MEM_IM2COL
    x = cfg.inputs(synth.config_seed(4))
    n, c, h, w = cfg.shape
    spec = gl.windows_spec((c, 3, 3), (1, 1, 1), (0, 1, 1), (0, 1, 1))
    out = gl.gl_access_windows(gl.AccessPattern(to_f32_device(x), 1), spec)
    assert out.shape == ((n, 1, h, w), (c, 3, 3))
    ref = brute.im2col(x, 3, 3, (1, 1), ((1, 1), (1, 1)))
    got = gl.gl_access_flatten(out).tensor
    assert got.shape == ref.shape
    assert torch.equal(got.cpu(), torch.from_numpy(ref))


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("shape,na,dim,lo,hi,kind", [
    ((2, 3, 5, 8), 1, 2, 1, 1, 0), ((2, 3, 5, 8), 1, 3, 2, 0, 0), ((2, 3, 5, 7), 2, 3, 1, 3, 1),
    ((4, 6), 1, 0, 0, 2, 1), ((9,), 0, 0, 3, 3, 0), ((2, 3, 4), 1, 1, 0, 0, 0),
    ((5, 1), 1, 1, 0, 0, 0), ((7, 3), 1, 1, 0, 2, 1), ((33, 61), 1, 1, 5, 1, 0), ((3, 700), 1, 1, 1, 1, 0),
])
def test_pad(gl, shape, na, dim, lo, hi, kind, dtype):
    x = synth.uniform(9, 1, shape, -1.0, 1.0)
    if dtype == "bf16":
        x = synth.bf16_round(x)
    ref = gi.pad(gi.access(x, na), dim, lo, hi, "neg_inf" if kind else "zero")
    dev = to_f32_device(x) if dtype == "f32" else to_bf16_device(x)
    out = gl.gl_access_pad(gl.AccessPattern(dev, na), dim, lo, hi, kind)
    assert out.shape == ref.shape
    _same_bits(out.tensor, ref.data.astype(np.float32))


POOL_CASES = [
    ((2, 3, 9, 8), 2, (3, 3), (2, 2), (1, 1), (1, 1)),
    ((2, 3, 9, 8), 2, (2, 3), (1, 2), (0, 0), (0, 0)),
    ((1, 2, 12, 12), 2, (3, 3), (2, 2), (1, 1), (1, 1)),
    ((3, 17), 1, (5,), (2,), (2,), (1,)),                   # 1D windows: general kernel
    ((2, 4, 5, 6), 1, (2, 3, 2), (2, 1, 2), (0, 1, 0), (0, 1, 0)),   # 3D windows: general kernel
]


@pytest.mark.parametrize("shape,na,wshape,stride,lo,hi", POOL_CASES)
def test_windows_reduce_max(gl, shape, na, wshape, stride, lo, hi):
    x = synth.uniform(10, 1, shape, -1.0, 1.0) - 2.0          # all negative: a zero border would win
    a = gi.access(x, na)
    for i, (l, h) in enumerate(zip(lo, hi)):
        if l or h:
            a = gi.pad(a, na + i, l, h, "neg_inf")
    ref = gi.compute("reduceMax", gi.windows(a, wshape, stride))
    out = gl.gl_compute_reduce_max(gl.AccessPattern(to_f32_device(x), na),
                                   gl.windows_spec(wshape, stride, lo, hi, gl.GL_PAD_NEG_INF))
    assert out.shape == ref.shape
    _same_bits(out.tensor, ref.data.astype(np.float32))


POOL_HWC_CASES = [
    # n, h, w, c, (kh, kw), (sh, sw), (ph, pw)
    (2, 9, 8, 8, (3, 3), (2, 2), (1, 1)),
    (3, 12, 10, 16, (2, 3), (1, 2), (0, 1)),
    (1, 16, 16, 64, (8, 8), (8, 8), (0, 0)),
    (2, 7, 5, 24, (3, 3), (1, 1), (1, 1)),
]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("n,h,w,c,k,s,pd", POOL_HWC_CASES)
def test_channels_last_max_pool(gl, n, h, w, c, k, s, pd, dtype):
    # ((N),(H,W,C)) items, window (Kh,Kw,1): the pooling of Fig. 2c with channels innermost, against the
    # brute-force pooling of the (C,H,W) view
    x = synth.uniform(12, 1, (n, h, w, c), -1.0, 1.0) - 2.0
    if dtype == "bf16":
        x = synth.bf16_round(x)
    ref = brute.maxpool(np.ascontiguousarray(x.transpose(0, 3, 1, 2)), k, s, ((pd[0], pd[0]), (pd[1], pd[1]))).transpose(0, 2, 3, 1)
    dev = to_bf16_device(x) if dtype == "bf16" else to_f32_device(x)
    spec = gl.windows_spec((k[0], k[1], 1), (s[0], s[1], 1), (pd[0], pd[1], 0), (pd[0], pd[1], 0), gl.GL_PAD_NEG_INF)
    out = gl.gl_compute_reduce_max(gl.AccessPattern(dev, 1), spec)
    assert out.shape == ((n,) + ref.shape[1:], ())
    assert np.array_equal(out.tensor.float().cpu().numpy(), ref)
    # the interpreter's windows + reduceMax on the same items
    a = gi.access(x, 1)
    for i, l in enumerate(pd):
        if l:
            a = gi.pad(a, 1 + i, l, l, "neg_inf")
    prog = gi.compute("reduceMax", gi.windows(a, (k[0], k[1], 1), (s[0], s[1], 1)))
    assert np.array_equal(prog.data.astype(np.float32), ref)


@pytest.mark.parametrize("shape,k,s,pd", [((2, 3, 9, 8), (3, 3), (2, 2), (1, 1)), ((1, 5, 16, 24), (8, 8), (8, 8), (0, 0)),
                                          ((3, 2, 7, 11), (2, 3), (1, 2), (0, 1)), ((2, 2, 14, 16), (3, 3), (2, 2), (1, 1)),
                                          ((1, 3, 33, 40), (3, 3), (2, 2), (1, 1)), ((2, 5, 112, 112), (3, 3), (2, 2), (1, 1)),
                                          ((2, 3, 13, 32), (4, 8), (3, 8), (1, 0)), ((3, 4, 56, 56), (8, 8), (8, 8), (0, 0)),
                                          ((1, 2, 40, 16), (20, 8), (20, 8), (0, 0))])
def test_bf16_plane_max_pool(gl, shape, k, s, pd):
    x = synth.bf16_round(synth.uniform(13, 1, shape, -1.0, 1.0) - 2.0)
    ref = brute.maxpool(x, k, s, ((pd[0], pd[0]), (pd[1], pd[1])))
    out = gl.gl_compute_reduce_max(gl.AccessPattern(to_bf16_device(x), 2), gl.windows_spec(k, s, pd, pd, gl.GL_PAD_NEG_INF))
    assert tuple(out.tensor.shape) == ref.shape and out.tensor.dtype == torch.bfloat16
    assert np.array_equal(out.tensor.float().cpu().numpy(), ref)


def test_reduce_max_whole_items(gl):
    x = synth.uniform(11, 1, (7, 5, 33), -1.0, 1.0)
    ref = gi.compute("reduceMax", gi.access(x, 1))
    out = gl.gl_compute_reduce_max(gl.AccessPattern(to_f32_device(x), 1), None)
    _same_bits(out.tensor, ref.data.astype(np.float32))


def test_maxpool_full_size(gl):
    cfg = synth.MEM_MAXPOOL
    x = cfg.inputs(synth.config_seed(4))
    spec = gl.windows_spec(cfg.window, (cfg.stride,) * 2, (cfg.pad,) * 2, (cfg.pad,) * 2, gl.GL_PAD_NEG_INF)
    out = gl.gl_compute_reduce_max(gl.AccessPattern(to_f32_device(x), 2), spec).tensor
    ref = brute.maxpool(x, cfg.window, (cfg.stride,) * 2, ((cfg.pad,) * 2, (cfg.pad,) * 2))
    assert torch.equal(out.cpu(), torch.from_numpy(ref))


@pytest.mark.parametrize("n", [1, 3, 4, 1000, 4099])
def test_relu(gl, n):
    x = synth.uniform(12, 1, (n,), -1.0, 1.0)
    x[::7] = -0.0
    ref = gi.compute("relu", gi.access(x, 1)).data.astype(np.float32)
    dev = to_f32_device(x)
    out = gl.gl_compute_relu(gl.AccessPattern(dev, 1))
    _same_bits(out.tensor, ref)
    gl.gl_compute_relu(gl.AccessPattern(dev, 1), gl.AccessPattern(dev, 1))    # in place
    _same_bits(dev, ref)


def test_output_metadata_is_checked(gl):
    x = to_f32_device(synth.uniform(13, 1, (4, 6), -1.0, 1.0))
    bad = gl.AccessPattern(torch.empty((6, 5), device="cuda"), 1)
    with pytest.raises(gl.GlError) as e:
        gl.gl_access_transpose(gl.AccessPattern(x, 1), (1, 0), out=bad)
    assert e.value.code == 4
    with pytest.raises(gl.GlError) as e:
        gl.gl_compute_relu(gl.AccessPattern(x.to(torch.bfloat16), 1))
    assert e.value.code == 2


def _guarded(shape, dtype, band=2048):
    """A result tensor of `shape` inside a larger buffer whose guard bands hold -7."""
    count = int(np.prod(shape))
    buf = torch.full((count + 2 * band,), -7.0, device="cuda", dtype=dtype)
    return buf, buf[band:band + count].view(shape), band, count


def _bands_intact(buf, band, count):
    return bool((buf[:band] == -7.0).all()) and bool((buf[band + count:] == -7.0).all())


def test_memory_bound_operators_write_only_their_results(gl):
    # every operator writes into the middle of a buffer whose guard bands must keep their fill; ragged shapes
    x = synth.uniform(14, 1, (3, 5, 13, 18), -1.0, 1.0) - 2.0
    xa = gl.AccessPattern(to_f32_device(x), 1)
    # im2col
    spec = gl.windows_spec((5, 3, 3), (1, 1, 1), (0, 1, 1), (0, 1, 1))
    first = gl.gl_access_windows(xa, spec)
    buf, view, band, count = _guarded(tuple(first.tensor.shape), torch.float32)
    gl.gl_access_windows(xa, spec, out=gl.AccessPattern(view, first.access_ndim))
    assert gl.gl_poll_device_status() == 0 and torch.equal(view, first.tensor) and _bands_intact(buf, band, count)
    # transpose
    first = gl.gl_access_transpose(xa, (0, 2, 3, 1))
    buf, view, band, count = _guarded(tuple(first.tensor.shape), torch.float32)
    gl.gl_access_transpose(xa, (0, 2, 3, 1), out=gl.AccessPattern(view, first.access_ndim))
    assert gl.gl_poll_device_status() == 0 and torch.equal(view, first.tensor) and _bands_intact(buf, band, count)
    assert np.array_equal(view.cpu().numpy(), x.transpose(0, 2, 3, 1).astype(np.float32))
    # pad of the innermost dimension
    first = gl.gl_access_pad(xa, 3, 1, 1)
    buf, view, band, count = _guarded(tuple(first.tensor.shape), torch.float32)
    gl.gl_access_pad(xa, 3, 1, 1, out=gl.AccessPattern(view, first.access_ndim))
    assert gl.gl_poll_device_status() == 0 and torch.equal(view, first.tensor) and _bands_intact(buf, band, count)
    assert np.array_equal(view.cpu().numpy(), np.pad(x, ((0, 0), (0, 0), (0, 0), (1, 1))).astype(np.float32))
    # max pooling, fp32 planes (3x3 stride 2: rows of four column groups and a half) and bf16 planes
    xp = synth.uniform(14, 2, (3, 5, 14, 24), -1.0, 1.0) - 2.0
    pool = gl.windows_spec((3, 3), (2, 2), (1, 1), (1, 1), gl.GL_PAD_NEG_INF)
    ref = brute.maxpool(xp.astype(np.float32), (3, 3), (2, 2), ((1, 1), (1, 1)))
    buf, view, band, count = _guarded(ref.shape, torch.float32)
    nd = gl.gl_compute_reduce_max(gl.AccessPattern(to_f32_device(xp), 2), pool).access_ndim
    gl.gl_compute_reduce_max(gl.AccessPattern(to_f32_device(xp), 2), pool, out=gl.AccessPattern(view, nd))
    assert gl.gl_poll_device_status() == 0 and np.array_equal(view.cpu().numpy(), ref) and _bands_intact(buf, band, count)
    xb = synth.bf16_round(xp)
    refb = brute.maxpool(xb, (3, 3), (2, 2), ((1, 1), (1, 1)))
    buf, view, band, count = _guarded(refb.shape, torch.bfloat16)
    gl.gl_compute_reduce_max(gl.AccessPattern(to_bf16_device(xb), 2), pool, out=gl.AccessPattern(view, nd))
    assert gl.gl_poll_device_status() == 0 and np.array_equal(view.float().cpu().numpy(), refb) and _bands_intact(buf, band, count)
    # relu
    buf, view, band, count = _guarded(x.shape, torch.float32)
    gl.gl_compute_relu(xa, out=gl.AccessPattern(view, 1))
    assert gl.gl_poll_device_status() == 0 and _bands_intact(buf, band, count)
    assert np.array_equal(view.cpu().numpy(), np.maximum(x, 0.0).astype(np.float32))

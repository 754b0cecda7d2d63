"""GPU parity of gl_cartesian_dot (compute dotProd over cartProd, Fig. 2a/2b and
the im2col-rewritten form of Section 5.3) against the CPU checker.

Integer-valued inputs in [-3,3]: every partial sum is an integer below 2^24, so
fp32 accumulation in any order is exact and the comparison is bit for bit.
N(0,1) inputs: max |g-r| / max(|r|, rms(r)) <= 2e-3 against the float64 result.
"""
import numpy as np
import pytest
import torch

from oracle import brute
from oracle import interp as gi
from paper_2105_09377_b200 import synth
from tests.gpu_util import REL_TOL, rel_err, to_bf16_device

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def gl():
    from paper_2105_09377_b200 import binding
    return binding


def _ok(gl):
    assert gl.gl_poll_device_status() == 0


def _conv_gpu(gl, x, wt, stride, pad, channels_last=False, flags=0):
    """conv2d through the C ABI; returns the ((N,1,H',W',O),()) result as (N,H',W',O) numpy."""
    n, c, h, w = x.shape
    o, _, kh, kw = wt.shape
    if channels_last:
        xa = gl.AccessPattern(to_bf16_device(np.ascontiguousarray(x.transpose(0, 2, 3, 1))), 1)
        wa = gl.AccessPattern(to_bf16_device(np.ascontiguousarray(wt.transpose(0, 2, 3, 1))), 1)
        spec = gl.windows_spec((kh, kw, c), (stride[0], stride[1], 1), (pad[0], pad[1], 0), (pad[0], pad[1], 0))
    else:
        xa = gl.AccessPattern(to_bf16_device(x), 1)
        wa = gl.AccessPattern(to_bf16_device(wt), 1)
        spec = gl.windows_spec((c, kh, kw), (1, stride[0], stride[1]), (0, pad[0], pad[1]), (0, pad[0], pad[1]))
    out = gl.gl_cartesian_dot(xa, spec, wa, flags=flags)
    _ok(gl)
    t = out.tensor.float() if out.tensor.dtype == torch.bfloat16 else out.tensor
    if channels_last:
        assert t.shape[3] == 1
        return t.squeeze(3).cpu().numpy()
    assert t.shape[1] == 1
    return t.squeeze(1).cpu().numpy()


def _conv_ref(x, wt, stride, pad):
    """float64 (N,H',W',O) from the brute-force conv2d equation."""
    return brute.conv2d(x, wt, stride, ((pad[0], pad[0]), (pad[1], pad[1]))).transpose(0, 2, 3, 1)


# ---- the tiny configuration: direct form, im2col-rewritten form, interpreter ----

@pytest.mark.parametrize("flags", [0, 0x100])
def test_tiny_conv_direct_and_rewritten(gl, flags):
    cfg = synth.CONV_TINY
    x, wt = cfg.inputs(synth.config_seed(0))
    ref = gi.conv2d_program(x, wt, upto="dotProd")              # ((1,1,6,6,4),())
    xa, wa = gl.AccessPattern(to_bf16_device(x), 1), gl.AccessPattern(to_bf16_device(wt), 1)
    spec = gl.windows_spec((3, 3, 3), (1, 1, 1))
    direct = gl.gl_cartesian_dot(xa, spec, wa, flags=flags)
    _ok(gl)
    assert direct.shape == ref.shape
    assert np.array_equal(direct.tensor.cpu().numpy().astype(np.float64), ref.data)
    # Section 5.3: windows materialised and flattened, weights flattened, plain matmul, reshape
    cols = gl.gl_access_flatten(gl.gl_access_windows(xa, spec))
    wflat = gl.gl_access_flatten(wa)
    assert cols.shape == ((36,), (27,)) and wflat.shape == ((4,), (27,))
    mm = gl.gl_cartesian_dot(cols, None, wflat, flags=flags)
    _ok(gl)
    assert mm.shape == ((36, 4), ())
    assert torch.equal(mm.tensor.view(direct.tensor.shape), direct.tensor)
    # squeeze + transpose (0 3 1 2) of Fig. 2a gives the NCHW result
    nhwo = gl.AccessPattern(direct.tensor.view(1, 6, 6, 4), 4)
    nchw = gl.gl_access_transpose(nhwo, (0, 3, 1, 2))
    full = gi.conv2d_program(x, wt)
    assert np.array_equal(nchw.tensor.cpu().numpy().astype(np.float64), full.data)


CONV_SMALL = [
    # n, c, h, w, o, kh, kw, sh, sw, ph, pw
    (2, 8, 9, 10, 16, 3, 3, 1, 1, 1, 1),      # C = 8: granule path, one M tile
    (3, 16, 12, 11, 24, 3, 2, 2, 1, 1, 0),    # lopsided window, strides and pads
    (2, 64, 14, 14, 64, 3, 3, 1, 1, 1, 1),    # C = 64: swizzled path, 4 ragged M tiles
    (1, 128, 9, 9, 72, 3, 3, 1, 1, 1, 1),     # two channel chunks per tap, O not a tile multiple
    (2, 96, 8, 8, 40, 1, 1, 1, 1, 0, 0),      # C = 96: last chunk half empty
    (2, 3, 20, 20, 8, 7, 7, 2, 2, 3, 3),      # stem-like: C = 3 padded to 8, 49 taps
    (2, 32, 10, 10, 130, 1, 1, 2, 2, 0, 0),   # 1x1 stride 2, O spans two column tiles
    (5, 24, 7, 7, 10, 5, 5, 1, 1, 2, 2),      # several images per tile, window 5x5
    (1, 5, 6, 6, 3, 2, 2, 1, 1, 0, 0),        # odd everything
]


@pytest.mark.parametrize("layout", ["nchw", "nhwc"])
@pytest.mark.parametrize("case", CONV_SMALL)
def test_conv_integer_bit_exact(gl, case, layout):
    n, c, h, w, o, kh, kw, sh, sw, ph, pw = case
    x = synth.uniform_int(21, 1, (n, c, h, w), -3, 3)
    wt = synth.uniform_int(21, 2, (o, c, kh, kw), -3, 3)
    ref = _conv_ref(x, wt, (sh, sw), (ph, pw))
    got = _conv_gpu(gl, x, wt, (sh, sw), (ph, pw), channels_last=(layout == "nhwc"))
    assert got.shape == ref.shape
    assert np.array_equal(got.astype(np.float64), ref)
    again = _conv_gpu(gl, x, wt, (sh, sw), (ph, pw), channels_last=(layout == "nhwc"))
    assert np.array_equal(got, again)                         # same bits on a second run


@pytest.mark.parametrize("case", CONV_SMALL[:4])
def test_conv_general_kernel_bit_exact(gl, case):
    n, c, h, w, o, kh, kw, sh, sw, ph, pw = case
    x = synth.uniform_int(22, 1, (n, c, h, w), -3, 3)
    wt = synth.uniform_int(22, 2, (o, c, kh, kw), -3, 3)
    ref = _conv_ref(x, wt, (sh, sw), (ph, pw))
    for cl in (False, True):
        got = _conv_gpu(gl, x, wt, (sh, sw), (ph, pw), channels_last=cl, flags=gl.GL_DOT_GENERAL_KERNEL)
        assert np.array_equal(got.astype(np.float64), ref)


@pytest.mark.parametrize("case", CONV_SMALL)
def test_conv_gaussian_within_tolerance(gl, case):
    n, c, h, w, o, kh, kw, sh, sw, ph, pw = case
    cc = synth.ConvCase("t", n, c, h, w, o, kh, kw, sh, ph)
    x = synth.bf16_round(synth.normal(23, 1, (n, c, h, w)))
    wt = synth.bf16_round(synth.normal(23, 2, (o, c, kh, kw), np.sqrt(2.0 / cc.kd)))
    ref = _conv_ref(x, wt, (sh, sw), (ph, pw))
    got = _conv_gpu(gl, x, wt, (sh, sw), (ph, pw), channels_last=True)
    assert rel_err(got, ref) <= REL_TOL


@pytest.mark.parametrize("layout", ["nchw", "nhwc"])
@pytest.mark.parametrize("case", [CONV_SMALL[0], CONV_SMALL[2], CONV_SMALL[3], CONV_SMALL[5], CONV_SMALL[7]])
def test_conv_fused_squeeze_transpose_is_fig2a(gl, case, layout):
    # GL_OUT_NCHW: the whole program of Fig. 2a in one call, result ((N,O,H',W'),())
    n, c, h, w, o, kh, kw, sh, sw, ph, pw = case
    x = synth.uniform_int(25, 1, (n, c, h, w), -3, 3)
    wt = synth.uniform_int(25, 2, (o, c, kh, kw), -3, 3)
    ref = brute.conv2d(x, wt, (sh, sw), ((ph, ph), (pw, pw)))                 # (N,O,H',W')
    if layout == "nhwc":
        xa = gl.AccessPattern(to_bf16_device(np.ascontiguousarray(x.transpose(0, 2, 3, 1))), 1)
        wa = gl.AccessPattern(to_bf16_device(np.ascontiguousarray(wt.transpose(0, 2, 3, 1))), 1)
        spec = gl.windows_spec((kh, kw, c), (sh, sw, 1), (ph, pw, 0), (ph, pw, 0))
    else:
        xa, wa = gl.AccessPattern(to_bf16_device(x), 1), gl.AccessPattern(to_bf16_device(wt), 1)
        spec = gl.windows_spec((c, kh, kw), (1, sh, sw), (0, ph, pw), (0, ph, pw))
    for flags in (gl.GL_OUT_NCHW, gl.GL_OUT_NCHW | gl.GL_DOT_GENERAL_KERNEL, gl.GL_OUT_NCHW | gl.GL_EPILOGUE_RELU):
        out = gl.gl_cartesian_dot(xa, spec, wa, flags=flags)
        _ok(gl)
        assert out.shape == ((n, o) + ref.shape[2:], ())
        want = np.maximum(ref, 0.0) if flags & gl.GL_EPILOGUE_RELU else ref
        assert np.array_equal(out.tensor.cpu().numpy().astype(np.float64), want)
    # the same thing in two steps: [M,O] result, then the library's transpose (0 3 1 2)
    two = gl.gl_cartesian_dot(xa, spec, wa)
    t = two.tensor.squeeze(3 if layout == "nhwc" else 1).contiguous()
    nchw = gl.gl_access_transpose(gl.AccessPattern(t, 4), (0, 3, 1, 2))
    assert np.array_equal(nchw.tensor.cpu().numpy().astype(np.float64), ref)
    # the interpreter's full program on a small case
    if n * o * ref.shape[2] * ref.shape[3] * c * kh * kw <= 600000:
        full = gi.conv2d_program(x, wt, (sh, sw), ((ph, ph), (pw, pw)))
        assert full.shape == ((n, o) + ref.shape[2:], ()) and np.array_equal(full.data, ref)


def _random_conv_cases(count, seed):
    rng = np.random.default_rng(seed)
    cases = []
    while len(cases) < count:
        c = int(rng.choice([1, 3, 4, 8, 12, 16, 24, 32, 40, 64, 72, 128, 136]))
        kh, kw = int(rng.integers(1, 5)), int(rng.integers(1, 5))
        sh, sw = int(rng.integers(1, 4)), int(rng.integers(1, 4))
        ph, pw = int(rng.integers(0, kh)), int(rng.integers(0, kw))
        h, w = int(rng.integers(kh, 20)), int(rng.integers(kw, 20))
        n, o = int(rng.integers(1, 5)), int(rng.choice([1, 3, 8, 20, 64, 70, 130, 260]))
        if n * c * h * w * o * kh * kw > 6e7:
            continue
        cases.append((n, c, h, w, o, kh, kw, sh, sw, ph, pw))
    return cases


@pytest.mark.parametrize("case", _random_conv_cases(40, 2105), ids=lambda c: "x".join(map(str, c)))
def test_conv_random_shapes_bit_exact(gl, case):
    # seeded shape fuzzing across all tensor-core modes (dense shortcut, im2col, row-window, granule, K split)
    n, c, h, w, o, kh, kw, sh, sw, ph, pw = case
    x = synth.uniform_int(sum(case), 1, (n, c, h, w), -3, 3)
    wt = synth.uniform_int(sum(case), 2, (o, c, kh, kw), -3, 3)
    ref = _conv_ref(x, wt, (sh, sw), (ph, pw))
    for cl in (False, True):
        got = _conv_gpu(gl, x, wt, (sh, sw), (ph, pw), channels_last=cl)
        assert got.shape == ref.shape
        assert np.array_equal(got.astype(np.float64), ref), "layout channels_last=%s" % cl


@pytest.mark.parametrize("m,o,k", [(int(a), int(b), int(c) * 8) for a, b, c in
                                   np.random.default_rng(99).integers(1, 400, (16, 3))])
def test_dense_random_shapes_bit_exact(gl, m, o, k):
    a = synth.uniform_int(m + o, 1, (m, k), -3, 3)
    b = synth.uniform_int(m + o, 2, (o, k), -3, 3)
    out = gl.gl_cartesian_dot(gl.AccessPattern(to_bf16_device(a), 1), None, gl.AccessPattern(to_bf16_device(b), 1))
    _ok(gl)
    assert np.array_equal(out.tensor.cpu().numpy().astype(np.float64), brute.rowdot(a, b))


def _random_window_kernel_cases(count, seed):
    """Seeded shapes aimed at the kernels that keep windows in shared memory: stride-1 convolutions with 64, 128 or
    192 channels (input block resident across the taps), at most 8 / Sw channels (windows read in place from row
    runs), and 1x1 windows (the layout copy is the matrix).  Both item layouts are run for each."""
    rng = np.random.default_rng(seed)
    cases = []
    while len(cases) < count:
        kind = len(cases) % 3
        if kind == 0:
            c = int(rng.choice([64, 128, 192]))
            kh, kw = int(rng.integers(1, 6)), int(rng.integers(2, 6))
            sh = sw = 1
            h, w = int(rng.integers(kh, 24)), int(rng.integers(kw, 61))
            o = int(rng.choice([4, 60, 64, 68, 128, 200]))
        elif kind == 1:
            sw = int(rng.choice([1, 2, 4]))
            c = int(rng.integers(1, 8 // sw + 1))
            sh = int(rng.integers(1, 4))
            kh, kw = int(rng.integers(1, 8)), int(rng.integers(1, 9))
            h, w = int(rng.integers(kh, 40)), int(rng.integers(kw, 180))
            o = int(rng.choice([4, 8, 36, 64, 128]))
        else:
            c = int(rng.choice([64, 72, 128, 320]))
            kh = kw = 1
            sh, sw = int(rng.integers(1, 4)), int(rng.integers(1, 4))
            h, w = int(rng.integers(1, 30)), int(rng.integers(1, 30))
            o = int(rng.choice([8, 64, 100, 260]))
        ph, pw = (0, 0) if kind == 2 else (int(rng.integers(0, kh)), int(rng.integers(0, kw)))
        n = int(rng.integers(1, 4))
        if n * c * h * w * o * kh * kw > 1.5e8:
            continue
        cases.append((n, c, h, w, o, kh, kw, sh, sw, ph, pw))
    return cases


@pytest.mark.parametrize("case", _random_window_kernel_cases(30, 5309), ids=lambda c: "x".join(map(str, c)))
def test_conv_random_shapes_window_kernels_bit_exact(gl, case):
    n, c, h, w, o, kh, kw, sh, sw, ph, pw = case
    x = synth.uniform_int(sum(case) + 7, 1, (n, c, h, w), -3, 3)
    wt = synth.uniform_int(sum(case) + 7, 2, (o, c, kh, kw), -3, 3)
    ref = _conv_ref(x, wt, (sh, sw), (ph, pw))
    for cl in (False, True):
        got = _conv_gpu(gl, x, wt, (sh, sw), (ph, pw), channels_last=cl)
        assert got.shape == ref.shape
        assert np.array_equal(got.astype(np.float64), ref), "layout channels_last=%s" % cl


# ---- GL_OUT_BF16: results rounded to bf16 as the last step ----

def _bf16(v):
    """float64 array -> the bf16 value nearest to each element (ties to even), as float64."""
    return synth.bf16_round(np.asarray(v, dtype=np.float32)).astype(np.float64)


@pytest.mark.parametrize("m,o,k", [(36, 8, 32), (130, 72, 72), (300, 520, 200), (257, 100, 1000), (2600, 1928, 200), (64, 64, 4096)])
def test_dense_bf16_output_bit_exact(gl, m, o, k):
    # integer sums are exact in fp32, so rounding them to bf16 gives the same bits on both sides
    a = synth.uniform_int(43, 1, (m, k), -3, 3)
    b = synth.uniform_int(43, 2, (o, k), -3, 3)
    ref = brute.rowdot(a, b)
    aa, bb = gl.AccessPattern(to_bf16_device(a), 1), gl.AccessPattern(to_bf16_device(b), 1)
    for flags in (gl.GL_OUT_BF16, gl.GL_OUT_BF16 | gl.GL_EPILOGUE_RELU, gl.GL_OUT_BF16 | gl.GL_DOT_GENERAL_KERNEL):
        out = gl.gl_cartesian_dot(aa, None, bb, flags=flags)
        _ok(gl)
        assert out.tensor.dtype == torch.bfloat16 and out.shape == ((m, o), ())
        want = _bf16(np.maximum(ref, 0.0) if flags & gl.GL_EPILOGUE_RELU else ref)
        assert np.array_equal(out.tensor.float().cpu().numpy().astype(np.float64), want)


CONV_BF16_OUT = [
    # n, c, h, w, o, kh, kw, sh, sw, ph, pw
    (2, 64, 12, 20, 128, 3, 3, 1, 1, 1, 1),    # input block resident, 128-wide tiles
    (2, 64, 14, 14, 64, 3, 3, 1, 1, 1, 1),     # ... 64-wide tiles, two blocks per SM
    (2, 3, 30, 40, 64, 7, 7, 2, 2, 3, 3),      # windows read in place from row runs
    (1, 4, 17, 33, 24, 5, 5, 3, 2, 2, 2),      # ... narrow accumulator (N = 32)
    (2, 64, 13, 13, 72, 3, 3, 2, 2, 1, 1),     # im2col-mode loads (stride 2)
    (2, 128, 10, 10, 64, 1, 1, 2, 2, 0, 0),    # 1x1: the copy is the matrix
    (2, 16, 9, 9, 20, 3, 3, 1, 1, 1, 1),       # granule path, O not a multiple of 8
    (1, 512, 7, 7, 64, 3, 3, 1, 1, 1, 1),      # split contraction, rounded by the summing kernel
]


@pytest.mark.parametrize("case", CONV_BF16_OUT, ids=lambda c: "x".join(map(str, c)))
def test_conv_bf16_output_bit_exact(gl, case):
    n, c, h, w, o, kh, kw, sh, sw, ph, pw = case
    x = synth.uniform_int(44, 1, (n, c, h, w), -3, 3)
    wt = synth.uniform_int(44, 2, (o, c, kh, kw), -3, 3)
    ref = _conv_ref(x, wt, (sh, sw), (ph, pw))
    for cl in (False, True):
        for relu in (0, gl.GL_EPILOGUE_RELU):
            got = _conv_gpu(gl, x, wt, (sh, sw), (ph, pw), channels_last=cl, flags=gl.GL_OUT_BF16 | relu)
            want = _bf16(np.maximum(ref, 0.0) if relu else ref)
            assert np.array_equal(np.asarray(got, dtype=np.float64), want), "channels_last=%s relu=%s" % (cl, bool(relu))
    # fused squeeze + transpose with bf16 results
    out = gl.gl_cartesian_dot(gl.AccessPattern(to_bf16_device(x), 1),
                              gl.windows_spec((c, kh, kw), (1, sh, sw), (0, ph, pw), (0, ph, pw)),
                              gl.AccessPattern(to_bf16_device(wt), 1), flags=gl.GL_OUT_BF16 | gl.GL_OUT_NCHW)
    _ok(gl)
    assert np.array_equal(out.tensor.float().cpu().numpy().astype(np.float64), _bf16(ref.transpose(0, 3, 1, 2)))


def test_bf16_output_gaussian_within_one_rounding(gl):
    # N(0,1) inputs: the fp32 sum differs from the float64 one by ~1e-6 relative, so after rounding to bf16 the two
    # agree or sit on neighbouring bf16 values (2^-8 relative apart)
    case = synth.DenseCase("d512", 512, 768, 1024)
    a, b = case.inputs(45)
    out = gl.gl_cartesian_dot(gl.AccessPattern(to_bf16_device(a), 1), None, gl.AccessPattern(to_bf16_device(b), 1),
                              flags=gl.GL_OUT_BF16)
    _ok(gl)
    got = out.tensor.float().cpu().numpy().astype(np.float64)
    ref = brute.rowdot(a, b)
    assert np.max(np.abs(got - ref) / np.maximum(np.abs(ref), np.sqrt(np.mean(ref * ref)))) <= 2.0 ** -8
    assert np.mean(got == _bf16(ref)) > 0.99


def test_bf16_output_wants_a_bf16_tensor(gl):
    a = gl.AccessPattern(to_bf16_device(synth.uniform_int(46, 1, (16, 32), -3, 3)), 1)
    with pytest.raises(gl.GlError):
        gl.gl_cartesian_dot(a, None, a, out=gl.AccessPattern(torch.empty((16, 16), device="cuda"), 2), flags=gl.GL_OUT_BF16)
    with pytest.raises(gl.GlError):
        gl.gl_cartesian_dot(a, None, a, out=gl.AccessPattern(torch.empty((16, 16), device="cuda", dtype=torch.bfloat16), 2))


def test_out_nchw_needs_a_conv(gl):
    a = gl.AccessPattern(to_bf16_device(synth.uniform_int(26, 1, (8, 16), -3, 3)), 1)
    out = gl.AccessPattern(torch.empty((8, 8), device="cuda"), 2)
    with pytest.raises(gl.GlError):
        gl.gl_cartesian_dot(a, None, a, out=out, flags=gl.GL_OUT_NCHW)


def test_windows_over_other_dims_uses_general_kernel(gl):
    # windows that also slide over the channel dim: not a conv2d, still a valid program
    x = synth.uniform_int(24, 1, (2, 5, 6, 7), -3, 3)
    wt = synth.uniform_int(24, 2, (4, 2, 3, 2), -3, 3)
    a = gi.windows(gi.access(x, 1), (2, 3, 2), (2, 1, 3))
    ref = gi.compute("dotProd", gi.cart_prod(a, gi.access(wt, 1)))
    out = gl.gl_cartesian_dot(gl.AccessPattern(to_bf16_device(x), 1), gl.windows_spec((2, 3, 2), (2, 1, 3)),
                              gl.AccessPattern(to_bf16_device(wt), 1))
    _ok(gl)
    assert out.shape == ref.shape
    assert np.array_equal(out.tensor.cpu().numpy().astype(np.float64), ref.data)


# ---- dense: compute dotProd (cartProd A B), both operands as row vectors ----

DENSE_SMALL = [(36, 4, 27), (1, 1, 8), (128, 256, 64), (130, 70, 72), (300, 520, 200), (257, 129, 1000), (64, 48, 7)]


@pytest.mark.parametrize("m,o,k", DENSE_SMALL)
def test_dense_integer_bit_exact(gl, m, o, k):
    a = synth.uniform_int(31, 1, (m, k), -3, 3)
    b = synth.uniform_int(31, 2, (o, k), -3, 3)
    ref = brute.rowdot(a, b)
    for flags in (0, gl.GL_DOT_GENERAL_KERNEL):
        out = gl.gl_cartesian_dot(gl.AccessPattern(to_bf16_device(a), 1), None, gl.AccessPattern(to_bf16_device(b), 1),
                                  flags=flags)
        _ok(gl)
        assert out.shape == ((m, o), ())
        assert np.array_equal(out.tensor.cpu().numpy().astype(np.float64), ref)


# Problems large enough for 256-wide tiles, which run on pairs of blocks sharing a 256x256 tile:
# an odd number of 128-row tiles (the last pair has an empty half), ragged edges in both directions.  The tile
# counts are not multiples of the resident pairs, so part of each result is computed as half-width tiles.
DENSE_PAIRED = [(2600, 1930, 200), (4001, 1100, 136), (2305, 2309, 72), (2560, 3900, 72)]


@pytest.mark.parametrize("m,o,k", DENSE_PAIRED)
def test_dense_paired_tiles_bit_exact(gl, m, o, k):
    a = synth.uniform_int(37, 1, (m, k), -3, 3)
    b = synth.uniform_int(37, 2, (o, k), -3, 3)
    ref = brute.rowdot(a, b)
    aa, bb = gl.AccessPattern(to_bf16_device(a), 1), gl.AccessPattern(to_bf16_device(b), 1)
    sentinel = torch.full((m + 8, o), -7.0, device="cuda")     # rows around the result must stay untouched
    out = gl.AccessPattern(sentinel[4:m + 4], 2)
    for flags in (0, gl.GL_EPILOGUE_RELU):
        sentinel.fill_(-7.0)
        gl.gl_cartesian_dot(aa, None, bb, out=out, flags=flags)
        _ok(gl)
        want = np.maximum(ref, 0.0) if flags else ref
        assert np.array_equal(sentinel[4:m + 4].cpu().numpy().astype(np.float64), want)
        assert bool((sentinel[:4] == -7.0).all()) and bool((sentinel[m + 4:] == -7.0).all())


GUARDED_CONVS = [
    # n, c, h, w, o, k, stride, pad, channels_last, flags: one case per kernel family
    (2, 128, 28, 28, 128, 3, 1, 1, True, 0),       # resident windows on block pairs
    (2, 64, 20, 20, 64, 3, 1, 1, True, 0),         # resident windows, two blocks per SM
    (2, 3, 40, 40, 64, 7, 2, 3, True, 0),          # few channels read in place, channels-last
    (2, 3, 40, 40, 64, 7, 2, 3, False, 1),         # ... (C,H,W) items, fused squeeze + transpose
    (2, 64, 12, 16, 40, 1, 2, 0, False, 0),        # pixel-major 1x1 windows
    (2, 72, 9, 9, 40, 3, 1, 1, False, 0),          # layout copies + im2col-mode tiles
    (1, 512, 7, 7, 64, 3, 1, 1, True, 0),          # K split: partial planes in the workspace
    (2, 12, 10, 12, 8, 3, 1, 1, False, 0),         # row-window copies
]


@pytest.mark.parametrize("case", GUARDED_CONVS, ids=lambda c: "x".join(map(str, c)))
def test_conv_writes_only_its_result_and_its_workspace(gl, case):
    # guard bands around the result and behind the workspace must keep their fill; the result must be right
    n, c, h, w, o, k, s_, pad, cl, nchw = case
    flags = gl.GL_OUT_NCHW if nchw else 0
    x = synth.uniform_int(48, 1, (n, c, h, w), -3, 3)
    wt = synth.uniform_int(48, 2, (o, c, k, k), -3, 3)
    ref = _conv_ref(x, wt, (s_, s_), (pad, pad))
    if cl:
        xa = gl.AccessPattern(to_bf16_device(np.ascontiguousarray(x.transpose(0, 2, 3, 1))), 1)
        wa = gl.AccessPattern(to_bf16_device(np.ascontiguousarray(wt.transpose(0, 2, 3, 1))), 1)
        spec = gl.windows_spec((k, k, c), (s_, s_, 1), (pad, pad, 0), (pad, pad, 0))
    else:
        xa, wa = gl.AccessPattern(to_bf16_device(x), 1), gl.AccessPattern(to_bf16_device(wt), 1)
        spec = gl.windows_spec((c, k, k), (1, s_, s_), (0, pad, pad), (0, pad, pad))
    ho, wo = ref.shape[1], ref.shape[2]
    count, band = n * ho * wo * o, 4096
    buf = torch.full((count + 2 * band,), -7.0, device="cuda")
    shape = (n, o, ho, wo) if nchw else ((n, ho, wo, 1, o) if cl else (n, 1, ho, wo, o))
    out = gl.AccessPattern(buf[band:band + count].view(shape), 4 if nchw else 5)
    need = gl.gl_cartesian_dot_workspace(xa, spec, wa, flags)
    ws = torch.full((need + 1024 + band,), 0xAB, dtype=torch.uint8, device="cuda")
    first = (ws.data_ptr() + 1023) // 1024 * 1024 - ws.data_ptr()
    gl.gl_cartesian_dot(xa, spec, wa, out=out, flags=flags, workspace=ws[:first + need] if need else None)
    _ok(gl)
    got = buf[band:band + count].view(shape).cpu().numpy().astype(np.float64)
    want = ref.transpose(0, 3, 1, 2) if nchw else (ref[:, :, :, None] if cl else ref[:, None])
    assert np.array_equal(got, want)
    assert bool((buf[:band] == -7.0).all()) and bool((buf[band + count:] == -7.0).all())
    assert bool((ws[first + need:] == 0xAB).all()) and bool((ws[:first] == 0xAB).all())


def test_conv_paired_tiles_bit_exact(gl):
    # 161 row tiles x one 256-wide column tile: the im2col loads of both blocks of a pair
    n, c, h, w, o = 5, 64, 64, 64, 200
    x = synth.uniform_int(38, 1, (n, c, h, w), -3, 3)
    wt = synth.uniform_int(38, 2, (o, c, 3, 3), -3, 3)
    ref = _conv_ref(x, wt, (1, 1), (1, 1))
    got = _conv_gpu(gl, x, wt, (1, 1), (1, 1), channels_last=True)
    assert np.array_equal(got.astype(np.float64), ref)
    got = _conv_gpu(gl, x, wt, (1, 1), (1, 1), channels_last=True, flags=gl.GL_EPILOGUE_RELU)
    assert np.array_equal(got.astype(np.float64), np.maximum(ref, 0.0))


# Stride-1 convolutions whose input block stays in shared memory across the filter taps: weights that
# stay resident (one chunk), weights streamed per filter row, per tap (5x5), two channel chunks, no padding.
CONV_RESIDENT_WINDOWS = [
    (2, 64, 12, 20, 128, 3, 3, 1, 1),
    (1, 128, 12, 20, 96, 5, 5, 2, 2),
    (3, 64, 16, 30, 160, 3, 3, 0, 0),
    (2, 192, 14, 14, 260, 3, 3, 1, 1),
    (2, 64, 9, 40, 68, 2, 4, 1, 2),
]


@pytest.mark.parametrize("case", CONV_RESIDENT_WINDOWS, ids=lambda c: "x".join(map(str, c)))
def test_conv_resident_window_tiles_bit_exact(gl, case):
    n, c, h, w, o, kh, kw, ph, pw = case
    x = synth.uniform_int(39, 1, (n, c, h, w), -3, 3)
    wt = synth.uniform_int(39, 2, (o, c, kh, kw), -3, 3)
    ref = _conv_ref(x, wt, (1, 1), (ph, pw))
    for flags in (0, gl.GL_EPILOGUE_RELU):
        got = _conv_gpu(gl, x, wt, (1, 1), (ph, pw), channels_last=True, flags=flags)
        assert got.shape == ref.shape
        assert np.array_equal(got.astype(np.float64), np.maximum(ref, 0.0) if flags else ref)
    got = _conv_gpu(gl, x, wt, (1, 1), (ph, pw), channels_last=False)
    assert np.array_equal(got.astype(np.float64), ref)


# Few input channels (C <= 8 / Sw): windows read in place from runs of the padded rows.
# n, c, h, w, o, kh, kw, sh, sw, ph, pw
CONV_ROW_RUNS = [
    (2, 3, 30, 300, 64, 7, 7, 2, 2, 3, 3),     # RGB stem, three 128-column segments per output row
    (1, 8, 12, 40, 128, 3, 3, 1, 1, 1, 1),     # stride 1: 8-channel pixels, widest tile
    (2, 4, 17, 33, 20, 5, 5, 3, 2, 2, 2),      # odd sizes, O = 20 (MMA N = 32)
    (2, 2, 16, 64, 12, 3, 6, 1, 4, 1, 0),      # stride 4: 2-channel pixels
    (1, 1, 20, 80, 8, 2, 20, 2, 8, 0, 4),      # stride 8: 1-channel pixels, two MMAs per filter row
    (3, 1, 9, 9, 4, 3, 3, 1, 1, 1, 1),         # one channel, stride 1
]


@pytest.mark.parametrize("case", CONV_ROW_RUNS, ids=lambda c: "x".join(map(str, c)))
def test_conv_row_runs_bit_exact(gl, case):
    n, c, h, w, o, kh, kw, sh, sw, ph, pw = case
    x = synth.uniform_int(40, 1, (n, c, h, w), -3, 3)
    wt = synth.uniform_int(40, 2, (o, c, kh, kw), -3, 3)
    ref = _conv_ref(x, wt, (sh, sw), (ph, pw))
    for cl in (False, True):
        got = _conv_gpu(gl, x, wt, (sh, sw), (ph, pw), channels_last=cl, flags=gl.GL_EPILOGUE_RELU if cl else 0)
        assert got.shape == ref.shape
        assert np.array_equal(got.astype(np.float64), np.maximum(ref, 0.0) if cl else ref), "channels_last=%s" % cl
    again = _conv_gpu(gl, x, wt, (sh, sw), (ph, pw), channels_last=False)
    assert np.array_equal(again.astype(np.float64), ref)           # the scratch copies are rebuilt on every call


# 1x1 unpadded windows over (C,H,W) items: the layout copy keeps only the pixels the windows touch.
CONV_1X1_CHW = [
    (2, 64, 9, 11, 72, 2, 3),      # n, c, h, w, o, sh, sw
    (3, 96, 8, 8, 40, 1, 1),       # C = 96: second chunk half empty
    (1, 200, 7, 7, 260, 1, 1),     # C not a multiple of 64, O spans tiles
    (2, 128, 10, 10, 64, 2, 2),
    (1, 2048, 7, 7, 64, 1, 1),     # one tile, 32 K blocks: the contraction is split and summed by the second kernel
    # rows the TMA unit can fetch (W a multiple of 8, at most 64): read in place as a pixel-major operand, no copy
    (2, 64, 6, 8, 16, 1, 1),
    (3, 72, 9, 16, 40, 2, 2),      # C = 72: second K block mostly zero fill; odd H'
    (1, 128, 5, 64, 130, 1, 1),    # full 64-pixel rows, two column tiles, O not a multiple of 4
    (2, 64, 7, 24, 8, 3, 2),       # row stride 3
    (2, 256, 12, 56, 128, 2, 2),
    (2, 64, 9, 16, 24, 2, 1),      # rows skipped, every pixel of a row used
    # unit strides and H*W a multiple of 8: the image as one run of pixels
    (2, 64, 10, 12, 16, 1, 1),     # H*W = 120: one ragged tile per image
    (1, 128, 28, 28, 64, 1, 1),    # 784 pixels: 6 tiles + 16 pixels
    # H*W a multiple of 4 only: planes the TMA unit cannot address, back to the layout copy
    (2, 64, 6, 6, 24, 1, 1),
    (3, 128, 14, 14, 72, 1, 1),    # 196 pixels: 128 + 68
    (1, 192, 10, 18, 136, 1, 1),   # three K blocks, two column tiles
]


@pytest.mark.parametrize("case", CONV_1X1_CHW, ids=lambda c: "x".join(map(str, c)))
def test_conv_1x1_chw_items_bit_exact(gl, case):
    n, c, h, w, o, sh, sw = case
    x = synth.uniform_int(41, 1, (n, c, h, w), -3, 3)
    wt = synth.uniform_int(41, 2, (o, c, 1, 1), -3, 3)
    ref = _conv_ref(x, wt, (sh, sw), (0, 0))
    got = _conv_gpu(gl, x, wt, (sh, sw), (0, 0), channels_last=False)
    assert got.shape == ref.shape
    assert np.array_equal(got.astype(np.float64), ref)
    got = _conv_gpu(gl, x, wt, (sh, sw), (0, 0), channels_last=False, flags=gl.GL_EPILOGUE_RELU)
    assert np.array_equal(got.astype(np.float64), np.maximum(ref, 0.0))
    if o % 8 == 0:
        got = _conv_gpu(gl, x, wt, (sh, sw), (0, 0), channels_last=False, flags=gl.GL_OUT_BF16)
        assert np.array_equal(np.asarray(got, dtype=np.float64), _bf16(ref))
    # with the fused squeeze + transpose the same items take the general window path
    out = gl.gl_cartesian_dot(gl.AccessPattern(to_bf16_device(x), 1), gl.windows_spec((c, 1, 1), (1, sh, sw)),
                              gl.AccessPattern(to_bf16_device(wt), 1), flags=gl.GL_OUT_NCHW)
    _ok(gl)
    assert np.array_equal(out.tensor.cpu().numpy().astype(np.float64), ref.transpose(0, 3, 1, 2))


def test_dense_interpreter_program_with_relu(gl):
    a = synth.uniform_int(32, 1, (20, 16), -3, 3)
    b = synth.uniform_int(32, 2, (12, 16), -3, 3)
    ref = gi.dense_rows_program(a, b, relu=True)
    aa, bb = gl.AccessPattern(to_bf16_device(a), 1), gl.AccessPattern(to_bf16_device(b), 1)
    fused = gl.gl_cartesian_dot(aa, None, bb, flags=gl.GL_EPILOGUE_RELU)
    two_step = gl.gl_compute_relu(gl.gl_cartesian_dot(aa, None, bb))
    _ok(gl)
    assert np.array_equal(fused.tensor.cpu().numpy().astype(np.float64), ref.data)
    assert torch.equal(fused.tensor, two_step.tensor)


def test_dense_gaussian_1024_full_check(gl):
    case = synth.DenseCase("d1024", 1024, 1024, 1024)
    a, b = case.inputs(41)
    ref = brute.rowdot(a, b)
    out = gl.gl_cartesian_dot(gl.AccessPattern(to_bf16_device(a), 1), None, gl.AccessPattern(to_bf16_device(b), 1))
    _ok(gl)
    assert rel_err(out.tensor.cpu().numpy(), ref) <= REL_TOL


@pytest.mark.parametrize("kind", ["integer", "gaussian"])
def test_dense_4096_whole_result_and_relu(gl, kind):
    # the whole 4096 x 4096 result against the row-vector form of the matMul equation (Section 3.1)
    case = synth.DENSE_4096
    if kind == "integer":
        a = synth.uniform_int(synth.config_seed(1), 1, (case.m, case.k), -3, 3)
        b = synth.uniform_int(synth.config_seed(1), 2, (case.o, case.k), -3, 3)
    else:
        a, b = case.inputs(synth.config_seed(1))
    aa, bb = gl.AccessPattern(to_bf16_device(a), 1), gl.AccessPattern(to_bf16_device(b), 1)
    out = gl.gl_cartesian_dot(aa, None, bb, flags=gl.GL_EPILOGUE_RELU)
    _ok(gl)
    got = out.tensor.cpu().numpy()
    ref = np.maximum(brute.rowdot(a, b), 0.0)
    if kind == "integer":
        assert np.array_equal(got.astype(np.float64), ref)      # |sums| <= 9 * 4096 < 2^24: exact in any order
    else:
        assert rel_err(got, ref) <= REL_TOL
    plain = gl.gl_cartesian_dot(aa, None, bb)
    _ok(gl)
    assert torch.equal(torch.clamp_min(plain.tensor, 0.0), out.tensor)


# ---- the convolution sweeps at full size: the whole result, both layouts, both kinds of input ----

FULL_CONVS = list(synth.CONV_SWEEP_3X3) + list(synth.CONV_STRIDED_1X1)
_FULL = {}


def _full_case(cfg, kind):
    """Inputs and the brute-force (N,H',W',O) result of a full-size workload, computed once per module."""
    key = (cfg.name, kind)
    if key not in _FULL:
        if kind == "integer":
            x = synth.uniform_int(synth.config_seed(2), 1, (cfg.n, cfg.c, cfg.h, cfg.w), -3, 3)
            wt = synth.uniform_int(synth.config_seed(2), 2, (cfg.o, cfg.c, cfg.kh, cfg.kw), -3, 3)
        else:
            x, wt = cfg.inputs(synth.config_seed(2))
        ref = _conv_ref(x, wt, (cfg.stride,) * 2, (cfg.pad,) * 2)
        if kind == "integer":
            assert np.abs(ref).max() < 2 ** 24
            ref = ref.astype(np.float32)                       # integers below 2^24: exact
        _FULL[key] = (x, wt, np.ascontiguousarray(ref))
    return _FULL[key]


@pytest.mark.parametrize("cfg", FULL_CONVS, ids=[c.name for c in FULL_CONVS])
@pytest.mark.parametrize("kind", ["integer", "gaussian"])
@pytest.mark.parametrize("layout", ["nhwc", "nchw"])
def test_full_size_conv_whole_result(gl, cfg, kind, layout):
    x, wt, ref = _full_case(cfg, kind)
    got = _conv_gpu(gl, x, wt, (cfg.stride,) * 2, (cfg.pad,) * 2, channels_last=(layout == "nhwc"))
    assert got.shape == ref.shape == (cfg.n, cfg.ho, cfg.wo, cfg.o)
    if kind == "integer":
        assert np.array_equal(got, ref)
    else:
        assert rel_err(got, ref) <= REL_TOL


@pytest.mark.parametrize("cfg", FULL_CONVS, ids=[c.name for c in FULL_CONVS])
@pytest.mark.parametrize("layout", ["nhwc", "nchw"])
def test_full_size_conv_fused_squeeze_transpose(gl, cfg, layout):
    # GL_OUT_NCHW at full size: the whole program of Fig. 2a, result ((N,O,H',W'),())
    x, wt, ref = _full_case(cfg, "integer")
    if layout == "nhwc":
        xa = gl.AccessPattern(to_bf16_device(np.ascontiguousarray(x.transpose(0, 2, 3, 1))), 1)
        wa = gl.AccessPattern(to_bf16_device(np.ascontiguousarray(wt.transpose(0, 2, 3, 1))), 1)
        spec = gl.windows_spec((cfg.kh, cfg.kw, cfg.c), (cfg.stride, cfg.stride, 1), (cfg.pad, cfg.pad, 0), (cfg.pad, cfg.pad, 0))
    else:
        xa, wa = gl.AccessPattern(to_bf16_device(x), 1), gl.AccessPattern(to_bf16_device(wt), 1)
        spec = gl.windows_spec((cfg.c, cfg.kh, cfg.kw), (1, cfg.stride, cfg.stride), (0, cfg.pad, cfg.pad), (0, cfg.pad, cfg.pad))
    out = gl.gl_cartesian_dot(xa, spec, wa, flags=gl.GL_OUT_NCHW)
    _ok(gl)
    assert tuple(out.tensor.shape) == (cfg.n, cfg.o, cfg.ho, cfg.wo)
    assert np.array_equal(out.tensor.cpu().numpy(), ref.transpose(0, 3, 1, 2))


FEW_CHANNEL_NCHW = [
    # n, c, h, w, o, k, stride, pad: few input channels, so the row-strip kernel takes them
    (2, 3, 38, 40, 24, 7, 2, 3),      # W' = 20: fp32 rows are whole 16-byte pieces, bf16 rows are not (other kernel)
    (2, 3, 30, 64, 40, 7, 2, 3),      # W' = 32, 40 filters: second channel box clipped at O
    (1, 4, 20, 288, 16, 3, 2, 1),     # W' = 144: two pixel segments per row, the second ragged
    (3, 8, 9, 16, 128, 3, 1, 1),      # stride 1, 8 channels, all 128 accumulator columns
    (2, 1, 17, 48, 8, 5, 1, 2),       # one channel, 5x5
]


@pytest.mark.parametrize("layout", ["nchw", "nhwc"])
@pytest.mark.parametrize("case", FEW_CHANNEL_NCHW)
def test_few_channel_conv_fused_squeeze_transpose(gl, case, layout):
    # Fig. 2a's whole program, (N,C,H,W) in and (N,O,H',W') out, on stem-like shapes, fp32 and bf16 results
    n, c, h, w, o, k, s, pad = case
    x = synth.uniform_int(47, 1, (n, c, h, w), -3, 3)
    wt = synth.uniform_int(47, 2, (o, c, k, k), -3, 3)
    ref = _conv_ref(x, wt, (s, s), (pad, pad)).transpose(0, 3, 1, 2)
    if layout == "nhwc":
        xa = gl.AccessPattern(to_bf16_device(np.ascontiguousarray(x.transpose(0, 2, 3, 1))), 1)
        wa = gl.AccessPattern(to_bf16_device(np.ascontiguousarray(wt.transpose(0, 2, 3, 1))), 1)
        spec = gl.windows_spec((k, k, c), (s, s, 1), (pad, pad, 0), (pad, pad, 0))
    else:
        xa, wa = gl.AccessPattern(to_bf16_device(x), 1), gl.AccessPattern(to_bf16_device(wt), 1)
        spec = gl.windows_spec((c, k, k), (1, s, s), (0, pad, pad), (0, pad, pad))
    for flags in (0, gl.GL_EPILOGUE_RELU, gl.GL_OUT_BF16, gl.GL_OUT_BF16 | gl.GL_EPILOGUE_RELU):
        out = gl.gl_cartesian_dot(xa, spec, wa, flags=flags | gl.GL_OUT_NCHW)
        _ok(gl)
        assert tuple(out.tensor.shape) == ref.shape
        want = np.maximum(ref, 0.0) if flags & gl.GL_EPILOGUE_RELU else ref
        if flags & gl.GL_OUT_BF16:
            want = _bf16(want)
        assert np.array_equal(out.tensor.float().cpu().numpy().astype(np.float64), want), "flags=%d" % flags


@pytest.mark.parametrize("cfg", FULL_CONVS, ids=[c.name for c in FULL_CONVS])
def test_full_size_conv_bf16_results(gl, cfg):
    # GL_OUT_BF16 at full size: the exact integer sums rounded once to the nearest-even bf16
    x, wt, ref = _full_case(cfg, "integer")
    got = _conv_gpu(gl, x, wt, (cfg.stride,) * 2, (cfg.pad,) * 2, channels_last=True, flags=gl.GL_OUT_BF16 | gl.GL_EPILOGUE_RELU)
    assert np.array_equal(got, synth.bf16_round(np.maximum(ref, 0.0)))


@pytest.mark.parametrize("kind", ["integer", "gaussian"])
def test_full_size_rewritten_form_equals_direct(gl, kind):
    # Section 5.3 at full size: windows materialised (bf16), flattened, plain matrix product, reshape
    cfg = synth.CONV_SWEEP_3X3[0]
    x, wt, ref = _full_case(cfg, kind)
    xa, wa = gl.AccessPattern(to_bf16_device(x), 1), gl.AccessPattern(to_bf16_device(wt), 1)
    spec = gl.windows_spec((cfg.c, cfg.kh, cfg.kw), (1, 1, 1), (0, cfg.pad, cfg.pad), (0, cfg.pad, cfg.pad))
    cols = gl.gl_access_flatten(gl.gl_access_windows(xa, spec))
    mm = gl.gl_cartesian_dot(cols, None, gl.gl_access_flatten(wa))
    _ok(gl)
    assert mm.shape == ((cfg.m, cfg.o), ())
    got = mm.tensor.view(cfg.n, cfg.ho, cfg.wo, cfg.o).cpu().numpy()
    if kind == "integer":
        assert np.array_equal(got, ref)
    else:
        assert rel_err(got, ref) <= REL_TOL


def test_bounded_wait_reports_timeout_and_context_survives(gl):
    # a wait that nothing completes gives up after its limit, the status word says so, and the
    # context keeps working: no trap, no fault, no hang
    assert gl.gl_poll_device_status() == 0
    gl.gl_selftest_bounded_wait(20)
    assert gl.gl_poll_device_status() == 10          # GL_ERR_TIMEOUT
    assert gl.gl_poll_device_status() == 0           # cleared by the poll
    a = synth.uniform_int(71, 1, (64, 64), -3, 3)
    out = gl.gl_cartesian_dot(gl.AccessPattern(to_bf16_device(a), 1), None, gl.AccessPattern(to_bf16_device(a), 1))
    _ok(gl)
    assert np.array_equal(out.tensor.cpu().numpy().astype(np.float64), brute.rowdot(a, a))
    with pytest.raises(gl.GlError):
        gl.gl_selftest_bounded_wait(5000)


def test_workspace_and_flag_errors_launch_nothing(gl):
    x = to_bf16_device(synth.uniform_int(72, 1, (2, 16, 10, 10), -3, 3))
    wt = to_bf16_device(synth.uniform_int(72, 2, (8, 16, 3, 3), -3, 3))
    spec = gl.windows_spec((16, 3, 3), (1, 1, 1), (0, 1, 1), (0, 1, 1))
    xa, wa = gl.AccessPattern(x, 1), gl.AccessPattern(wt, 1)
    need = gl.gl_cartesian_dot_workspace(xa, spec, wa)
    assert need > 0
    out = gl.output_like(gl.gl_shape_cartesian_dot(tuple(x.shape), 1, spec, tuple(wt.shape), 1), "cuda")
    out.tensor.fill_(5.0)
    small = torch.empty(need // 2 + 1024, dtype=torch.uint8, device="cuda")
    with pytest.raises(gl.GlError) as e:
        gl.gl_cartesian_dot(xa, spec, wa, out=out, workspace=small)
    assert e.value.code == 8
    with pytest.raises(gl.GlError) as e:
        gl.gl_cartesian_dot(xa, spec, wa, out=out, flags=0x40)
    assert e.value.code == 7
    torch.cuda.synchronize()
    assert bool((out.tensor == 5.0).all())

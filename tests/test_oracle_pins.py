"""Pins of the CPU checker to things other than itself: library routines it
does not call (torch.nn.functional on CPU, scipy.signal), closed forms,
special cases that reduce to a textbook routine, the paper's program
equalities (Section 5.3 and 5.4), and agreement of the interpreter with the
independent brute-force C loops.  Shapes are deliberately lopsided
(H != W, Kh != Kw, Sh != Sw, C != O) so a transposed index fails."""
import numpy as np
import pytest
import scipy.signal
import torch
import torch.nn.functional as F

from oracle import brute
from oracle import interp as gi
from paper_2105_09377_b200 import synth


def _ints(seed, tid, shape):
    return synth.uniform_int(seed, tid, shape, -3, 3).astype(np.float64)


def _rand(seed, tid, shape):
    return synth.normal(seed, tid, shape).astype(np.float64)


CONV_CASES = [
    # n, c, h, w, o, kh, kw, sh, sw, ph, pw
    (1, 3, 8, 8, 4, 3, 3, 1, 1, 0, 0),       # the tiny configuration
    (2, 3, 9, 7, 5, 3, 2, 2, 1, 0, 0),
    (2, 2, 7, 10, 3, 2, 3, 1, 2, 1, 2),
    (1, 4, 6, 5, 2, 1, 1, 2, 2, 0, 0),       # 1x1 strided
    (1, 1, 11, 9, 2, 7, 7, 2, 2, 3, 3),      # stem-like 7x7 s2 p3
]


@pytest.mark.parametrize("case", CONV_CASES)
def test_conv2d_against_torch_and_brute(case):
    n, c, h, w, o, kh, kw, sh, sw, ph, pw = case
    x = _rand(11, 1, (n, c, h, w))
    wt = _rand(11, 2, (o, c, kh, kw))
    pads = ((ph, ph), (pw, pw))
    ref = F.conv2d(torch.from_numpy(x), torch.from_numpy(wt), stride=(sh, sw), padding=(ph, pw)).numpy()
    o1 = gi.conv2d_program(x, wt, (sh, sw), pads).data
    o2 = brute.conv2d(x.astype(np.float32), wt.astype(np.float32), (sh, sw), pads)
    assert o1.shape == ref.shape == o2.shape
    np.testing.assert_allclose(o1, ref, rtol=1e-12, atol=1e-12)
    # brute takes float32 inputs: compare on float32-rounded inputs
    x32, w32 = x.astype(np.float32).astype(np.float64), wt.astype(np.float32).astype(np.float64)
    np.testing.assert_allclose(o2, gi.conv2d_program(x32, w32, (sh, sw), pads).data, rtol=1e-12, atol=1e-12)


def test_conv2d_against_scipy_correlate():
    x = _rand(12, 1, (1, 2, 7, 6))
    wt = _rand(12, 2, (3, 2, 3, 2))
    got = gi.conv2d_program(x, wt).data
    for o in range(3):
        acc = sum(scipy.signal.correlate2d(x[0, c], wt[o, c], mode="valid") for c in range(2))
        np.testing.assert_allclose(got[0, o], acc, rtol=1e-12, atol=1e-12)


def test_conv2d_is_cross_correlation_not_flipped():
    # a flipped kernel (true convolution) must NOT match: guards the sign of dx, dy
    x = _rand(13, 1, (1, 1, 6, 6))
    wt = _rand(13, 2, (1, 1, 3, 3))
    good = gi.conv2d_program(x, wt).data
    flipped = gi.conv2d_program(x, wt[:, :, ::-1, ::-1].copy()).data
    ref = F.conv2d(torch.from_numpy(x), torch.from_numpy(wt)).numpy()
    assert np.allclose(good, ref) and not np.allclose(flipped, ref)


@pytest.mark.parametrize("case", CONV_CASES)
def test_direct_and_im2col_programs_agree_exactly(case):
    # Section 5.3: the rewritten program equals the original, cell for cell.
    n, c, h, w, o, kh, kw, sh, sw, ph, pw = case
    x, wt = _ints(14, 1, (n, c, h, w)), _ints(14, 2, (o, c, kh, kw))
    pads = ((ph, ph), (pw, pw))
    a = gi.conv2d_program(x, wt, (sh, sw), pads)
    b = gi.conv2d_im2col_program(x, wt, (sh, sw), pads)
    assert a.shape == b.shape
    assert np.array_equal(a.data, b.data)
    # integers in [-3,3]: float32 accumulation is exact, so all three agree bit for bit
    c32 = brute.conv2d_f32acc(x, wt, (sh, sw), pads)
    assert np.array_equal(a.data, c32.astype(np.float64))


def test_tiny_config_shapes_and_exactness():
    cfg = synth.CONV_TINY
    x, wt = cfg.inputs(synth.config_seed(0))
    assert set(np.unique(x)).issubset(set(range(-3, 4)))
    d = gi.conv2d_program(x, wt, upto="dotProd")
    assert d.shape == ((1, 1, 6, 6, 4), ())
    full = gi.conv2d_program(x, wt)
    assert full.shape == ((1, 4, 6, 6), ())
    assert np.array_equal(full.data, brute.conv2d(x, wt))
    assert np.abs(full.data).max() <= 9 * 27


def test_all_ones_closed_form_with_padding():
    # all-ones input and weights: out = C * (number of in-range taps)
    n, c, h, w, o, k, p = 1, 3, 5, 6, 2, 3, 1
    got = gi.conv2d_program(np.ones((n, c, h, w)), np.ones((o, c, k, k)), (1, 1), ((p, p), (p, p))).data
    for x in range(h):
        for y in range(w):
            taps = sum(1 for dx in range(k) for dy in range(k)
                       if 0 <= x + dx - p < h and 0 <= y + dy - p < w)
            assert got[0, 0, x, y] == c * taps == got[0, 1, x, y]
    assert brute.conv2d(np.ones((n, c, h, w)), np.ones((o, c, k, k)), (1, 1), ((p, p), (p, p)))[0, 0, 0, 0] == c * 4


def test_delta_kernel_shifts_input():
    x = _rand(15, 1, (1, 1, 6, 7))
    wt = np.zeros((1, 1, 3, 2))
    wt[0, 0, 2, 1] = 1.0                      # picks A[x+2, y+1]
    got = gi.conv2d_program(x, wt).data
    np.testing.assert_array_equal(got[0, 0], x[0, 0, 2:, 1:])
    np.testing.assert_array_equal(brute.conv2d(x, wt)[0, 0], x.astype(np.float32)[0, 0, 2:, 1:])


def test_one_by_one_conv_is_matmul():
    n, c, h, w, o = 2, 5, 3, 4, 6
    x, wt = _rand(16, 1, (n, c, h, w)), _rand(16, 2, (o, c, 1, 1))
    got = gi.conv2d_program(x, wt, upto="dotProd").data.reshape(n * h * w, o)
    ref = x.transpose(0, 2, 3, 1).reshape(-1, c) @ wt.reshape(o, c).T
    np.testing.assert_allclose(got, ref, rtol=1e-12, atol=1e-12)


def test_matmul_forms():
    p, q = _rand(17, 1, (5, 7)), _rand(17, 2, (7, 3))
    ref = p @ q
    np.testing.assert_allclose(gi.matmul_program(p, q).data, ref, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(gi.dense_rows_program(p, q.T.copy()).data, ref, rtol=1e-12, atol=1e-12)
    p32, q32 = p.astype(np.float32), q.astype(np.float32)
    ref32 = p32.astype(np.float64) @ q32.astype(np.float64)
    np.testing.assert_allclose(brute.matmul(p32, q32), ref32, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(brute.rowdot(p32, q32.T.copy()), ref32, rtol=1e-12, atol=1e-12)
    rows = np.array([4, 0, 2])
    np.testing.assert_allclose(brute.rowdot(p32, q32.T.copy(), rows), ref32[rows], rtol=1e-12, atol=1e-12)


def test_dense_identity_and_relu():
    a = _rand(18, 1, (6, 4))
    out = gi.dense_rows_program(a, np.eye(4)).data
    np.testing.assert_array_equal(out, a)
    r = gi.dense_rows_program(a, np.eye(4), relu=True).data
    np.testing.assert_array_equal(r, np.maximum(a, 0.0))
    assert not np.signbit(r).any()            # relu yields +0, never -0


def test_dotprod_commutes_and_transpose_inverts():
    a, b = _rand(19, 1, (3, 5)), _rand(19, 2, (4, 5))
    ab = gi.compute("dotProd", gi.cart_prod(gi.access(a, 1), gi.access(b, 1)))
    ba = gi.compute("dotProd", gi.cart_prod(gi.access(b, 1), gi.access(a, 1)))
    np.testing.assert_array_equal(ab.data, ba.data.T)
    t = gi.access(_rand(19, 3, (2, 3, 4, 5)), 2)
    perm = (2, 0, 3, 1)
    inv = tuple(np.argsort(perm))
    np.testing.assert_array_equal(gi.transpose(gi.transpose(t, perm), inv).data, t.data)
    np.testing.assert_array_equal(gi.transpose(t, perm).data, np.transpose(t.data, perm))


def test_transpose_large_path_matches_small_path():
    t = gi.access(_rand(20, 1, (5, 9, 10, 11)), 1)            # > 4096 cells: library path
    perm = (0, 2, 3, 1)
    big = gi.transpose(t, perm).data
    for idx in [(0, 0, 0, 0), (4, 9, 10, 8), (2, 3, 7, 5)]:
        n, h, w, c = idx
        assert big[idx] == t.data[n, c, h, w]
    np.testing.assert_array_equal(brute.transpose_021(t.data.reshape(5, 9, 110)).reshape(5, 10, 11, 9),
                                  big.astype(np.float32))


@pytest.mark.parametrize("k,s,p", [((3, 3), (2, 2), 1), ((2, 3), (1, 2), 0), ((3, 2), (3, 1), 1)])
def test_maxpool_against_torch(k, s, p):
    x = _rand(21, 1, (2, 3, 9, 8))
    ref = F.max_pool2d(torch.from_numpy(x), k, s, padding=p).numpy()
    pads = ((p, p), (p, p))
    got = gi.maxpool_program(x, k, s, pads).data
    np.testing.assert_array_equal(got, ref)
    x32 = x.astype(np.float32)
    ref32 = F.max_pool2d(torch.from_numpy(x32), k, s, padding=p).numpy()
    np.testing.assert_array_equal(brute.maxpool(x32, k, s, pads), ref32)


def test_maxpool_negative_input_with_padding():
    # -inf padding: a zero border would win over an all-negative window
    x = -np.abs(_rand(22, 1, (1, 1, 4, 4))) - 1.0
    got = gi.maxpool_program(x, (3, 3), (2, 2), ((1, 1), (1, 1))).data
    assert (got < 0).all() and np.isfinite(got).all()


def test_windows_against_unfold():
    n, c, h, w, kh, kw, sh, sw, p = 2, 3, 7, 6, 3, 2, 2, 1, 1
    x = _rand(23, 1, (n, c, h, w))
    ref = F.unfold(torch.from_numpy(x), (kh, kw), padding=p, stride=(sh, sw)).numpy()   # (n, c*kh*kw, L)
    act = gi._pad_hw(gi.access(x, 1), ((p, p), (p, p)), "zero")
    col = gi.flatten(gi.windows(act, (c, kh, kw), (1, sh, sw))).data
    np.testing.assert_array_equal(col.reshape(n, -1, c * kh * kw), ref.transpose(0, 2, 1))
    got2 = brute.im2col(x.astype(np.float32), kh, kw, (sh, sw), ((p, p), (p, p)))
    np.testing.assert_array_equal(got2, col.astype(np.float32))


def test_windows_special_cases():
    a = gi.access(_rand(24, 1, (2, 4, 6)), 1)
    # window == whole extent: a single window that is the item itself
    whole = gi.windows(a, (4, 6), (1, 1))
    assert whole.shape == ((2, 1, 1), (4, 6))
    np.testing.assert_array_equal(whole.data.reshape(2, 4, 6), a.data)
    # window 1 stride 1: every cell becomes a (1,1) item
    one = gi.windows(a, (1, 1), (1, 1))
    assert one.shape == ((2, 4, 6), (1, 1))
    np.testing.assert_array_equal(one.data.reshape(2, 4, 6), a.data)
    # stride == window (no overlap): reshape + transpose
    tiles = gi.windows(a, (2, 3), (2, 3))
    ref = a.data.reshape(2, 2, 2, 2, 3).transpose(0, 1, 3, 2, 4)
    np.testing.assert_array_equal(tiles.data, ref)
    # single-cell definition agrees with the whole result
    w = gi.windows(a, (2, 3), (1, 2))
    for idx in [(0, 0, 0, 0, 0), (1, 2, 1, 1, 2), (1, 1, 0, 0, 1)]:
        assert gi.windows_element(a, (2, 3), (1, 2), idx) == w.data[idx]


def test_cartprod_members():
    a, b = gi.access(_rand(25, 1, (2, 3)), 1), gi.access(_rand(25, 2, (4, 3)), 1)
    cp = gi.cart_prod(a, b)
    assert cp.shape == ((2, 4), (2, 3))
    for i in range(2):
        for j in range(4):
            np.testing.assert_array_equal(cp.data[i, j, 0], a.data[i])
            np.testing.assert_array_equal(cp.data[i, j, 1], b.data[j])
    with pytest.raises(ValueError):
        gi.cart_prod(a, gi.access(np.zeros((4, 2)), 1))


def test_operators():
    item = gi.access(np.array([[1.0, -2.0, 3.0], [4.0, 5.0, -6.0]]), 0)
    assert gi.compute("reduceSum", item).data == 5.0
    assert gi.compute("reduceMax", item).data == 5.0
    assert gi.compute("dotProd", item).data == 1 * 4 - 2 * 5 - 3 * 6
    three = gi.access(np.array([[1.0, 2.0], [3.0, 4.0], [5.0, 6.0]]), 0)
    assert gi.compute("dotProd", three).data == 1 * 3 * 5 + 2 * 4 * 6
    assert gi.compute("relu", gi.access(np.array([-1.0, 0.0, 2.0]), 1)).data.tolist() == [0.0, 0.0, 2.0]


# ---- Section 5.3: the three im2col rewrites as equalities -----------------

def test_rewrite_flatten_reshape_is_identity():
    a = gi.access(_rand(26, 1, (2, 3, 4, 5)), 2)
    back = gi.reshape(gi.flatten(a), a.access_shape, a.compute_shape)
    assert back.shape == a.shape
    np.testing.assert_array_equal(back.data, a.data)


def test_rewrite_cartprod_commutes_with_reshape():
    a0, a1 = gi.access(_rand(27, 1, (6, 8)), 1), gi.access(_rand(27, 2, (4, 8)), 1)
    lhs = gi.cart_prod(gi.reshape(a0, (2, 3), (2, 4)), gi.reshape(a1, (4,), (2, 4)))
    rhs = gi.reshape(gi.cart_prod(a0, a1), (2, 3, 4), (2, 2, 4))
    assert lhs.shape == rhs.shape
    np.testing.assert_array_equal(lhs.data, rhs.data)


def test_rewrite_dotprod_commutes_with_reshape():
    a = gi.access(_rand(28, 1, (6, 2, 8)), 1)
    lhs = gi.compute("dotProd", gi.reshape(a, (2, 3), (2, 2, 4)))
    rhs = gi.reshape(gi.compute("dotProd", a), (2, 3), ())
    np.testing.assert_allclose(lhs.data, rhs.data, rtol=1e-13, atol=1e-13)


# ---- Section 5.4: the blocking rewrites as equalities ---------------------

def test_rewrite_slice_concat_is_identity():
    a = gi.access(_rand(29, 1, (4, 6)), 1)
    for d, n in ((0, 4), (1, 6)):
        back = gi.concat(gi.slice_(a, d, 0, n // 2), gi.slice_(a, d, n // 2, n), d)
        np.testing.assert_array_equal(back.data, a.data)


def test_rewrite_concat_bubbles_through_cartprod_and_dotprod():
    a = gi.access(_ints(30, 1, (4, 6)), 1)
    b0, b1 = gi.access(_ints(30, 2, (2, 6)), 1), gi.access(_ints(30, 3, (3, 6)), 1)
    # access-dimension concat of the second argument
    lhs = gi.cart_prod(a, gi.concat(b0, b1, 0))
    rhs = gi.concat(gi.cart_prod(a, b0), gi.cart_prod(a, b1), 1)
    np.testing.assert_array_equal(lhs.data, rhs.data)
    # compute (shape) dimension concat on both arguments
    a0, a1 = gi.slice_(a, 1, 0, 2), gi.slice_(a, 1, 2, 6)
    c0, c1 = gi.slice_(b0, 1, 0, 2), gi.slice_(b0, 1, 2, 6)
    lhs2 = gi.cart_prod(gi.concat(a0, a1, 1), gi.concat(c0, c1, 1))
    rhs2 = gi.concat(gi.cart_prod(a0, c0), gi.cart_prod(a1, c1), 3)
    np.testing.assert_array_equal(lhs2.data, rhs2.data)
    # dotProd over an access-dimension concat
    p, q = gi.cart_prod(a, b0), gi.cart_prod(a, b1)
    np.testing.assert_array_equal(gi.compute("dotProd", gi.concat(p, q, 1)).data,
                                  gi.concat(gi.compute("dotProd", p), gi.compute("dotProd", q), 1).data)
    # dotProd over a shape-dimension concat = reduceSum of the pair
    x0, x1 = gi.cart_prod(a0, c0), gi.cart_prod(a1, c1)
    whole = gi.compute("dotProd", gi.concat(x0, x1, 3))
    parts = gi.compute("reduceSum", gi.pair(gi.compute("dotProd", x0), gi.compute("dotProd", x1)))
    np.testing.assert_array_equal(whole.data, parts.data)


def test_blocked_32x32_is_eight_16x16_matmuls():
    p, q = _ints(31, 1, (32, 32)), _ints(31, 2, (32, 32))
    act, wts = gi.access(p, 1), gi.access(q, 1)
    count = 0
    rows = []
    for i in (0, 16):
        cols = []
        for j in (0, 16):
            parts = []
            for k in (0, 16):
                a_blk = gi.slice_(gi.slice_(act, 0, i, i + 16), 1, k, k + 16)
                w_blk = gi.transpose(gi.slice_(gi.slice_(wts, 0, k, k + 16), 1, j, j + 16), (1, 0))
                parts.append(gi.compute("dotProd", gi.cart_prod(a_blk, w_blk)))
                count += 1
            cols.append(gi.compute("reduceSum", gi.pair(parts[0], parts[1])))
        rows.append(gi.concat(cols[0], cols[1], 1))
    blocked = gi.concat(rows[0], rows[1], 0)
    assert count == 8
    np.testing.assert_array_equal(blocked.data, p @ q)
    np.testing.assert_array_equal(blocked.data, gi.matmul_program(p, q).data)


# ---- the sampled form of the conv2d equation (used on full-size results) ----

SAMPLED_CASES = [
    # n, c, h, w, o, kh, kw, sh, sw, ph, pw: strides and pads unequal, N and O above 1
    (2, 3, 13, 10, 5, 7, 7, 2, 1, 3, 2),     # stem-like 7x7, stride 2 only along H, pads 3 and 2
    (3, 4, 9, 8, 6, 1, 1, 2, 3, 0, 0),       # 1x1 with strides 2 and 3
    (2, 2, 7, 11, 3, 3, 2, 1, 2, 1, 0),      # lopsided window, one padded dimension
]


@pytest.mark.parametrize("case", SAMPLED_CASES)
def test_conv2d_sampled_against_full_brute_torch_and_interpreter(case):
    # every flat (n,o,x,y) offset, then a shuffled subset with repeats: the values must be the cells of
    # the full brute-force result, of the interpreter's Fig. 2a program and of torch's conv2d
    n, c, h, w, o, kh, kw, sh, sw, ph, pw = case
    x = synth.bf16_round(synth.normal(61, 1, (n, c, h, w)))
    wt = synth.bf16_round(synth.normal(61, 2, (o, c, kh, kw)))
    pads = ((ph, ph), (pw, pw))
    full = brute.conv2d(x, wt, (sh, sw), pads)
    assert full.shape == brute.conv_out_shape(x.shape, wt.shape, (sh, sw), pads)
    every = np.arange(full.size, dtype=np.int64)
    got = brute.conv2d_sampled(x, wt, every, (sh, sw), pads)
    np.testing.assert_array_equal(got, full.ravel())
    prog = gi.conv2d_program(x.astype(np.float64), wt.astype(np.float64), (sh, sw), pads).data
    np.testing.assert_allclose(got, prog.ravel(), rtol=1e-12, atol=1e-12)
    ref = F.conv2d(torch.from_numpy(x.astype(np.float64)), torch.from_numpy(wt.astype(np.float64)), stride=(sh, sw),
                   padding=(ph, pw)).numpy()
    np.testing.assert_allclose(got, ref.ravel(), rtol=1e-12, atol=1e-12)
    rng = np.random.default_rng(3)
    pick = rng.integers(0, full.size, 257)
    np.testing.assert_array_equal(brute.conv2d_sampled(x, wt, pick, (sh, sw), pads), full.ravel()[pick])


def test_conv2d_sampled_pin_catches_a_wrong_offset_order():
    # the pin must tell (n,o,x,y) offsets from (n,x,y,o) offsets: feeding offsets of the other order
    # (a plausible slip in a caller or in the decode) gives different values
    n, c, h, w, o, kh, kw = 2, 3, 6, 7, 4, 3, 2
    x = synth.bf16_round(synth.normal(62, 1, (n, c, h, w)))
    wt = synth.bf16_round(synth.normal(62, 2, (o, c, kh, kw)))
    full = brute.conv2d(x, wt)
    _, _, ho, wo = full.shape
    nn, oo, xx, yy = np.meshgrid(np.arange(n), np.arange(o), np.arange(ho), np.arange(wo), indexing="ij")
    right = ((nn * o + oo) * ho + xx) * wo + yy
    wrong = ((nn * ho + xx) * wo + yy) * o + oo
    np.testing.assert_array_equal(brute.conv2d_sampled(x, wt, right.ravel()), full.ravel())
    assert not np.array_equal(brute.conv2d_sampled(x, wt, wrong.ravel()), full.ravel())


# ---- sensitivity: a planted mistake in the checker is caught --------------

def test_pins_catch_a_planted_mistake(monkeypatch):
    x, wt = _rand(32, 1, (1, 2, 6, 5)), _rand(32, 2, (3, 2, 3, 2))
    ref = F.conv2d(torch.from_numpy(x), torch.from_numpy(wt), stride=(2, 1)).numpy()
    assert np.allclose(gi.conv2d_program(x, wt, (2, 1)).data, ref)
    real = gi.windows

    def swapped(a, wshape, strides):          # H and W strides exchanged
        s = list(strides)
        s[-1], s[-2] = s[-2], s[-1]
        return real(a, wshape, s)

    monkeypatch.setattr(gi, "windows", swapped)
    wrong = gi.conv2d_program(x, wt, (2, 1)).data
    assert wrong.shape != ref.shape or not np.allclose(wrong, ref)


def test_synth_is_seeded_and_bf16_exact():
    a = synth.normal(5, 1, (1000,))
    b = synth.normal(5, 1, (1000,))
    np.testing.assert_array_equal(a, b)
    assert abs(float(a.mean())) < 0.15 and 0.85 < float(a.std()) < 1.15
    assert not np.array_equal(a, synth.normal(6, 1, (1000,)))
    r = synth.bf16_round(a)
    t = torch.from_numpy(a).to(torch.bfloat16).to(torch.float32).numpy()
    np.testing.assert_array_equal(r, t)       # RNE agrees with torch's conversion
    u = synth.uniform(5, 2, (1000,), -1.0, 1.0)
    assert u.min() >= -1.0 and u.max() < 1.0
    i = synth.uniform_int(5, 3, (7000,), -3, 3)
    assert sorted(set(i.tolist())) == [-3, -2, -1, 0, 1, 2, 3]

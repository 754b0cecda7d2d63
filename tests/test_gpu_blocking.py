"""The remaining transformers and reduceSum on the GPU (slice, concat, pair, squeeze, reshape),
each against the interpreter, and the worked example of Section 5.4: a 32x32 matMul evaluated as
eight 16x16 matMuls that are summed in pairs (reduceSum (pair ..)) and concatenated (Fig. 8)."""
import numpy as np
import pytest
import torch

from oracle import interp as gi
from paper_2105_09377_b200 import synth
from tests.gpu_util import REL_TOL, rel_err, to_bf16_device, to_f32_device

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def gl():
    from paper_2105_09377_b200 import binding
    return binding


def _bits(t):
    return t.float().cpu().numpy().view(np.uint32)


def _dev(x, dtype):
    return to_f32_device(x) if dtype == "f32" else to_bf16_device(x)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("shape,na,dim,lo,hi", [((4, 6, 8), 1, 0, 1, 3), ((4, 6, 8), 1, 1, 2, 6), ((4, 6, 8), 2, 2, 0, 8),
                                                ((5, 7), 1, 1, 3, 4), ((3, 5, 2, 9), 2, 1, 1, 5), ((32, 32), 1, 0, 16, 32)])
def test_slice(gl, shape, na, dim, lo, hi, dtype):
    x = synth.bf16_round(synth.uniform(41, 1, shape, -1.0, 1.0))
    ref = gi.slice_(gi.access(x, na), dim, lo, hi)
    out = gl.gl_access_slice(gl.AccessPattern(_dev(x, dtype), na), dim, lo, hi)
    assert out.shape == ref.shape
    np.testing.assert_array_equal(_bits(out.tensor), ref.data.astype(np.float32).view(np.uint32))


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("sa,sb,na,dim", [((4, 6), (3, 6), 1, 0), ((4, 6), (4, 2), 1, 1), ((2, 3, 8), (2, 5, 8), 2, 1),
                                          ((2, 3, 5), (2, 3, 7), 1, 2), ((16, 16), (16, 16), 2, 1)])
def test_concat(gl, sa, sb, na, dim, dtype):
    a = synth.bf16_round(synth.uniform(42, 1, sa, -1.0, 1.0))
    b = synth.bf16_round(synth.uniform(42, 2, sb, -1.0, 1.0))
    ref = gi.concat(gi.access(a, na), gi.access(b, na), dim)
    out = gl.gl_access_concat(gl.AccessPattern(_dev(a, dtype), na), gl.AccessPattern(_dev(b, dtype), na), dim)
    assert out.shape == ref.shape
    np.testing.assert_array_equal(_bits(out.tensor), ref.data.astype(np.float32).view(np.uint32))
    # slice undoes concat (first blocking rewrite of Fig. 7, read right to left)
    back = gl.gl_access_slice(out, dim, 0, sa[dim])
    np.testing.assert_array_equal(_bits(back.tensor), a.view(np.uint32))


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("shape,na", [((4, 6), 1), ((4, 6), 2), ((3, 5, 8), 1), ((7,), 0), ((16, 16), 2)])
def test_pair(gl, shape, na, dtype):
    a = synth.bf16_round(synth.uniform(43, 1, shape, -1.0, 1.0))
    b = synth.bf16_round(synth.uniform(43, 2, shape, -1.0, 1.0))
    ref = gi.pair(gi.access(a, na), gi.access(b, na))
    out = gl.gl_access_pair(gl.AccessPattern(_dev(a, dtype), na), gl.AccessPattern(_dev(b, dtype), na))
    assert out.shape == ref.shape
    np.testing.assert_array_equal(_bits(out.tensor), ref.data.astype(np.float32).view(np.uint32))


def test_squeeze_and_reshape_are_views(gl):
    x = synth.uniform(44, 1, (2, 1, 6, 4), -1.0, 1.0)
    a = gl.AccessPattern(to_f32_device(x), 2)
    sq = gl.gl_access_squeeze(a, 1)
    assert sq.shape == gi.squeeze(gi.access(x, 2), 1).shape and sq.tensor.data_ptr() == a.tensor.data_ptr()
    rs = gl.gl_access_reshape(sq, (2,), (3, 8))
    assert rs.shape == gi.reshape(gi.squeeze(gi.access(x, 2), 1), (2,), (3, 8)).shape
    assert rs.tensor.data_ptr() == a.tensor.data_ptr()
    with pytest.raises(gl.GlError):
        gl.gl_access_reshape(sq, (3,), (16,))          # access side would change its element count
    with pytest.raises(gl.GlError):
        gl.gl_access_squeeze(a, 2)                     # extent 6, not 1


@pytest.mark.parametrize("shape,na", [((5, 7), 1), ((3, 4, 100), 2), ((6, 2), 1), ((2, 3, 4, 5), 1), ((1000,), 0)])
def test_reduce_sum(gl, shape, na):
    xi = synth.uniform_int(45, 1, shape, -3, 3)
    ref = gi.compute("reduceSum", gi.access(xi, na))
    out = gl.gl_compute_reduce_sum(gl.AccessPattern(to_f32_device(xi), na))
    assert out.shape == ref.shape
    assert np.array_equal(out.tensor.cpu().numpy().astype(np.float64), ref.data)      # integer sums: exact
    xf = synth.normal(45, 2, shape)
    reff = gi.compute("reduceSum", gi.access(xf, na)).data
    dev = to_f32_device(xf)
    one = gl.gl_compute_reduce_sum(gl.AccessPattern(dev, na)).tensor
    two = gl.gl_compute_reduce_sum(gl.AccessPattern(dev, na)).tensor
    assert torch.equal(one, two)                                                        # fixed order
    assert rel_err(np.atleast_1d(one.cpu().numpy()), np.atleast_1d(reff)) <= REL_TOL


def test_fig8_blocked_matmul_on_device(gl):
    """Section 5.4 / Fig. 8: matMul(32x32) = concat over row blocks and column blocks of
    reduceSum(pair(dotProd(block k=0), dotProd(block k=1))), eight 16x16 products in all."""
    p = synth.uniform_int(46, 1, (32, 32), -3, 3)
    q = synth.uniform_int(46, 2, (32, 32), -3, 3)
    act = gl.AccessPattern(to_bf16_device(p), 1)          # (access activations 1)
    wts = gl.AccessPattern(to_bf16_device(q), 1)          # (access weights 1)
    products = 0
    rows = []
    for i in (0, 16):
        cols = []
        for j in (0, 16):
            parts = []
            for k in (0, 16):
                a_blk = gl.gl_access_slice(gl.gl_access_slice(act, 0, i, i + 16), 1, k, k + 16)
                w_blk = gl.gl_access_transpose(gl.gl_access_slice(gl.gl_access_slice(wts, 0, k, k + 16), 1, j, j + 16), (1, 0))
                parts.append(gl.gl_cartesian_dot(a_blk, None, w_blk))            # ((16,16),())
                products += 1
            cols.append(gl.gl_compute_reduce_sum(gl.gl_access_pair(parts[0], parts[1])))   # ((16,16),(2)) -> ((16,16),())
        rows.append(gl.gl_access_concat(cols[0], cols[1], 1))                     # ((16,32),())
    blocked = gl.gl_access_concat(rows[0], rows[1], 0)                            # ((32,32),())
    assert products == 8 and gl.gl_poll_device_status() == 0
    assert blocked.shape == ((32, 32), ())
    whole = gl.gl_cartesian_dot(act, None, gl.gl_access_transpose(wts, (1, 0)))    # Fig. 2b in one call
    ref = gi.matmul_program(p, q).data
    assert np.array_equal(blocked.tensor.cpu().numpy().astype(np.float64), ref)
    assert torch.equal(blocked.tensor, whole.tensor)

"""Operators composed into one program on the device: the conv2d of Fig. 2a (squeeze and transpose
fused, relu in the epilogue) followed by the max pooling of Fig. 2c, against the same chain run by
the CPU checker.  Integer inputs: every intermediate is exact, so the comparison is bit for bit."""
import numpy as np
import pytest

from oracle import brute
from oracle import interp as gi
from paper_2105_09377_b200 import synth
from tests.gpu_util import to_bf16_device

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def gl():
    from paper_2105_09377_b200 import binding
    return binding


@pytest.mark.parametrize("n,c,h,w,o", [(2, 3, 23, 21, 8), (1, 16, 18, 18, 24), (2, 64, 12, 12, 64)])
def test_conv_relu_maxpool_chain(gl, n, c, h, w, o):
    x = synth.uniform_int(61, 1, (n, c, h, w), -3, 3)
    wt = synth.uniform_int(61, 2, (o, c, 3, 3), -3, 3)
    # device: conv 3x3 pad 1 -> relu -> (N,O,H,W) -> max pool 3x3 stride 2 pad 1
    spec = gl.windows_spec((c, 3, 3), (1, 1, 1), (0, 1, 1), (0, 1, 1))
    act = gl.gl_cartesian_dot(gl.AccessPattern(to_bf16_device(x), 1), spec, gl.AccessPattern(to_bf16_device(wt), 1),
                              flags=gl.GL_OUT_NCHW | gl.GL_EPILOGUE_RELU)
    assert act.shape == ((n, o, h, w), ())
    pooled = gl.gl_compute_reduce_max(gl.AccessPattern(act.tensor, 2),
                                      gl.windows_spec((3, 3), (2, 2), (1, 1), (1, 1), gl.GL_PAD_NEG_INF))
    assert gl.gl_poll_device_status() == 0
    # checker: the same chain from the brute-force equations
    conv = np.maximum(brute.conv2d(x, wt, (1, 1), ((1, 1), (1, 1))), 0.0)
    ref = brute.maxpool(conv.astype(np.float32), (3, 3), (2, 2), ((1, 1), (1, 1)))
    assert pooled.tensor.shape == ref.shape
    assert np.array_equal(pooled.tensor.cpu().numpy(), ref)
    if n * c * h * w * o < 40000:          # and from the interpreter's programs on the smallest case
        prog = gi.maxpool_program(gi.compute("relu", gi.conv2d_program(x, wt, (1, 1), ((1, 1), (1, 1)))).data,
                                  (3, 3), (2, 2), ((1, 1), (1, 1)))
        assert np.array_equal(prog.data, ref.astype(np.float64))


def test_conv_relu_maxpool_dense_chain(gl):
    """The chain continued by the dense layer of Fig. 2b: flatten the pooled activations per image and take
    dot products with the rows of a weight matrix.  All values stay small integers (three input channels),
    so the bf16 operands of the dense layer and every sum are exact."""
    import torch
    n, c, h, w, o, units = 2, 3, 23, 21, 8, 10
    x = synth.uniform_int(62, 1, (n, c, h, w), -3, 3)
    wt = synth.uniform_int(62, 2, (o, c, 3, 3), -3, 3)
    spec = gl.windows_spec((c, 3, 3), (1, 1, 1), (0, 1, 1), (0, 1, 1))
    act = gl.gl_cartesian_dot(gl.AccessPattern(to_bf16_device(x), 1), spec, gl.AccessPattern(to_bf16_device(wt), 1),
                              flags=gl.GL_OUT_NCHW | gl.GL_EPILOGUE_RELU)
    pooled = gl.gl_compute_reduce_max(gl.AccessPattern(act.tensor, 2),
                                      gl.windows_spec((3, 3), (2, 2), (1, 1), (1, 1), gl.GL_PAD_NEG_INF))
    feat = gl.gl_access_flatten(gl.AccessPattern(pooled.tensor, 1))            # ((N), (O*H'*W'))
    k = feat.tensor.shape[1]
    assert float(pooled.tensor.abs().max()) <= 256.0                            # exact in bf16
    dense_w = synth.uniform_int(62, 3, (units, k), -3, 3)
    feat_bf16 = gl.AccessPattern(feat.tensor.to(torch.bfloat16), 1)             # storage type of the next layer's operand
    logits = gl.gl_cartesian_dot(feat_bf16, None, gl.AccessPattern(to_bf16_device(dense_w), 1), flags=gl.GL_EPILOGUE_RELU)
    assert gl.gl_poll_device_status() == 0
    conv = np.maximum(brute.conv2d(x, wt, (1, 1), ((1, 1), (1, 1))), 0.0)
    ref_pool = brute.maxpool(conv.astype(np.float32), (3, 3), (2, 2), ((1, 1), (1, 1)))
    ref = np.maximum(brute.rowdot(ref_pool.reshape(n, -1).astype(np.float32), dense_w), 0.0)
    assert logits.shape == ((n, units), ())
    assert np.array_equal(logits.tensor.cpu().numpy().astype(np.float64), ref)


def test_two_convolutions_chained_through_bf16_results(gl):
    """conv -> relu -> conv with channels-last items: the first layer stores its results as bf16 (GL_OUT_BF16), which
    is exactly the operand the second layer reads.  Three input channels keep the first layer's results below 256,
    so they are exact in bf16 and the whole chain is bit for bit the checker's."""
    n, c, h, w, o1, o2 = 2, 3, 17, 19, 8, 16
    x = synth.uniform_int(63, 1, (n, c, h, w), -3, 3)
    w1 = synth.uniform_int(63, 2, (o1, c, 3, 3), -3, 3)
    w2 = synth.uniform_int(63, 3, (o2, o1, 3, 3), -3, 3)
    nhwc = lambda t: np.ascontiguousarray(t.transpose(0, 2, 3, 1))
    spec1 = gl.windows_spec((3, 3, c), (1, 1, 1), (1, 1, 0), (1, 1, 0))
    y1 = gl.gl_cartesian_dot(gl.AccessPattern(to_bf16_device(nhwc(x)), 1), spec1, gl.AccessPattern(to_bf16_device(nhwc(w1)), 1),
                             flags=gl.GL_OUT_BF16 | gl.GL_EPILOGUE_RELU)          # ((N,H,W,1,O1),()) in bf16
    act = gl.AccessPattern(y1.tensor.view(n, h, w, o1), 1)                        # squeeze: items (H,W,O1)
    spec2 = gl.windows_spec((3, 3, o1), (2, 2, 1), (1, 1, 0), (1, 1, 0))
    y2 = gl.gl_cartesian_dot(act, spec2, gl.AccessPattern(to_bf16_device(nhwc(w2)), 1))
    assert gl.gl_poll_device_status() == 0
    r1 = np.maximum(brute.conv2d(x, w1, (1, 1), ((1, 1), (1, 1))), 0.0)
    assert r1.max() <= 256.0
    r2 = brute.conv2d(r1.astype(np.float32), w2, (2, 2), ((1, 1), (1, 1))).transpose(0, 2, 3, 1)
    assert np.array_equal(y2.tensor.squeeze(3).cpu().numpy().astype(np.float64), r2)

"""gl_cartesian_dot_static: the convolution entry point for hosts that cannot allocate.

Some users of this library run where device memory cannot be requested: inside another
framework's operator, in a plug-in that only receives its input and output buffers, or in a
process whose memory all belongs to a pool.  They cannot hand gl_cartesian_dot a workspace,
so this variant keeps its scratch in a fixed array inside the library.  The test calls it
through the C ABI on a convolution that needs scratch (the (C,H,W) layout) and compares with
the ordinary entry point, twice in a row with different data, because the array is shared
by all calls and keeps the previous call's contents."""
import numpy as np
import pytest
import torch

from paper_2105_09377_b200 import synth
from tests.gpu_util import REL_TOL, rel_err, to_bf16_device

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def gl():
    from paper_2105_09377_b200 import binding
    return binding


def _conv_operands(gl, seed, n, c, h, w, o, k, integer):
    if integer:
        x = synth.uniform_int(seed, 1, (n, c, h, w), -3, 3)
        wt = synth.uniform_int(seed, 2, (o, c, k, k), -3, 3)
    else:
        x = synth.bf16_round(synth.normal(seed, 1, (n, c, h, w)))
        wt = synth.bf16_round(synth.normal(seed, 2, (o, c, k, k), np.sqrt(2.0 / (c * k * k))))
    spec = gl.windows_spec((c, k, k), (1, 1, 1), (0, k // 2, k // 2), (0, k // 2, k // 2))
    return gl.AccessPattern(to_bf16_device(x), 1), spec, gl.AccessPattern(to_bf16_device(wt), 1)


def test_static_scratch_matches_workspace_entry_point_twice(gl):
    for seed, shape, integer in ((51, (3, 20, 13, 11, 24, 3), True), (52, (2, 64, 14, 14, 48, 3), False)):
        xa, spec, wa = _conv_operands(gl, seed, *shape, integer)
        assert gl.gl_cartesian_dot_workspace(xa, spec, wa) > 0          # this case does use scratch
        want = gl.gl_cartesian_dot(xa, spec, wa)
        got = gl.AccessPattern(torch.full_like(want.tensor, float("nan")), want.access_ndim)
        gl.gl_cartesian_dot_static(xa, spec, wa, got)
        assert gl.gl_poll_device_status() == 0
        g, r = got.tensor.cpu().numpy(), want.tensor.cpu().numpy()
        if integer:
            assert np.array_equal(g, r)                                  # exact sums: same bits
        assert rel_err(g, r) <= REL_TOL
        # a second call on the now-dirty array, same answer
        again = gl.AccessPattern(torch.empty_like(want.tensor), want.access_ndim)
        gl.gl_cartesian_dot_static(xa, spec, wa, again, flags=gl.GL_EPILOGUE_RELU)
        assert torch.equal(again.tensor, torch.clamp_min(got.tensor, 0.0))


def test_static_scratch_rejects_oversized_requests(gl):
    n, c, h, w = 40, 64, 112, 112                                        # 40x112x112x64 bf16 = 61 MiB of scratch
    x = torch.zeros((n, c, h, w), dtype=torch.bfloat16, device="cuda")
    wt = torch.zeros((8, c, 3, 3), dtype=torch.bfloat16, device="cuda")
    spec = gl.windows_spec((c, 3, 3), (1, 1, 1), (0, 1, 1), (0, 1, 1))
    xa, wa = gl.AccessPattern(x, 1), gl.AccessPattern(wt, 1)
    assert gl.gl_cartesian_dot_workspace(xa, spec, wa) > gl.GL_STATIC_SCRATCH_BYTES
    out = gl.output_like(gl.gl_shape_cartesian_dot(tuple(x.shape), 1, spec, tuple(wt.shape), 1), "cuda")
    out.tensor.fill_(7.0)
    with pytest.raises(gl.GlError) as e:
        gl.gl_cartesian_dot_static(xa, spec, wa, out)
    assert e.value.code == 8 and "workspace" in str(e.value)             # GL_ERR_WORKSPACE
    torch.cuda.synchronize()
    assert bool((out.tensor == 7.0).all())                               # nothing was launched

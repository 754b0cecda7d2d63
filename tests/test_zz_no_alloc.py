"""gl_cartesian_dot_static: the convolution entry point for hosts that cannot allocate.

Some users of this library run where device memory cannot be requested: inside another
framework's operator, in a plug-in that only receives its input and output buffers, or in a
process whose memory all belongs to a pool.  They cannot hand gl_cartesian_dot a workspace,
so this variant keeps its scratch in a fixed array inside the library.  The tests call it
through the C ABI on problems that need scratch (the (C,H,W) layout, few-channel windows, a
split contraction) and compare with the ordinary entry point and with the CPU checker, twice
in a row, because the array is shared by all calls and keeps the previous call's contents;
they also check that the device's free memory does not move across a call."""
import gc

import numpy as np
import pytest
import torch

from oracle import brute
from paper_2105_09377_b200 import synth
from tests.gpu_util import REL_TOL, rel_err, to_bf16_device

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def gl():
    from paper_2105_09377_b200 import binding
    return binding


def _conv_operands(gl, seed, n, c, h, w, o, k, integer, stride=1):
    if integer:
        x = synth.uniform_int(seed, 1, (n, c, h, w), -3, 3)
        wt = synth.uniform_int(seed, 2, (o, c, k, k), -3, 3)
    else:
        x = synth.bf16_round(synth.normal(seed, 1, (n, c, h, w)))
        wt = synth.bf16_round(synth.normal(seed, 2, (o, c, k, k), np.sqrt(2.0 / (c * k * k))))
    spec = gl.windows_spec((c, k, k), (1, stride, stride), (0, k // 2, k // 2), (0, k // 2, k // 2))
    ref = brute.conv2d(x, wt, (stride, stride), ((k // 2, k // 2), (k // 2, k // 2))).transpose(0, 2, 3, 1)
    return gl.AccessPattern(to_bf16_device(x), 1), spec, gl.AccessPattern(to_bf16_device(wt), 1), ref


def _dirty_the_scratch(gl):
    """A call whose scratch footprint covers every later case, with operands that are all NaN: any cell a
    later call reads without having written it first shows up in that call's result."""
    n, c, h, w, o = 4, 72, 56, 56, 8
    x = torch.full((n, c, h, w), float("nan"), dtype=torch.bfloat16, device="cuda")
    wt = torch.full((o, c, 3, 3), float("nan"), dtype=torch.bfloat16, device="cuda")
    spec = gl.windows_spec((c, 3, 3), (1, 1, 1), (0, 1, 1), (0, 1, 1))
    xa, wa = gl.AccessPattern(x, 1), gl.AccessPattern(wt, 1)
    out = gl.output_like(gl.gl_shape_cartesian_dot(tuple(x.shape), 1, spec, tuple(wt.shape), 1), "cuda")
    gl.gl_cartesian_dot_static(xa, spec, wa, out)
    assert gl.gl_poll_device_status() == 0
    assert bool(torch.isnan(out.tensor).all())
    return gl.gl_cartesian_dot_workspace(xa, spec, wa)


CASES = [
    # seed, (n, c, h, w, o, k), integer inputs, stride
    (51, (3, 20, 13, 11, 24, 3), True, 1),       # channels padded 20 -> 24: zero-filled cells in the copies
    (52, (2, 64, 14, 14, 48, 3), False, 1),      # N(0,1) inputs, resident-window kernel behind the layout copy
    (53, (2, 3, 30, 30, 136, 7), True, 2),       # RGB stem 7x7 stride 2 pad 3 with 136 filters: row-window copies
    (54, (2, 12, 10, 12, 8, 3), True, 1),        # row-window copies with zero borders and zero weight tails
    (55, (1, 2048, 7, 7, 64, 1), True, 1),       # one tile, 32 K blocks: split contraction, partial planes in the scratch
]


def test_static_scratch_matches_workspace_entry_point_and_checker_twice(gl):
    covered = _dirty_the_scratch(gl)
    for seed, shape, integer, stride in CASES:
        xa, spec, wa, ref = _conv_operands(gl, seed, *shape, integer, stride)
        need = gl.gl_cartesian_dot_workspace(xa, spec, wa)
        assert 0 < need <= covered                                       # this case does use scratch, all of it dirtied
        want = gl.gl_cartesian_dot(xa, spec, wa)
        got = gl.AccessPattern(torch.full_like(want.tensor, float("nan")), want.access_ndim)
        gl.gl_cartesian_dot_static(xa, spec, wa, got)
        assert gl.gl_poll_device_status() == 0
        g, r = got.tensor.cpu().numpy(), want.tensor.cpu().numpy()
        if integer:
            assert np.array_equal(g, r)                                  # exact sums: same bits
            assert np.array_equal(g.squeeze(1).astype(np.float64), ref)  # and the conv2d equation itself
        assert rel_err(g, r) <= REL_TOL
        assert rel_err(g.squeeze(1), ref) <= REL_TOL
        # a second call on the now-dirty array: same answer, and no device memory changes hands
        again = gl.AccessPattern(torch.empty_like(want.tensor), want.access_ndim)
        gc.collect()                  # tensors of earlier tests that are still waiting for the collector go now,
        gc.disable()                  # not between the two readings
        try:
            torch.cuda.synchronize()
            held, free = torch.cuda.memory_allocated(), torch.cuda.mem_get_info()[0]
            gl.gl_cartesian_dot_static(xa, spec, wa, again, flags=gl.GL_EPILOGUE_RELU)
            torch.cuda.synchronize()
            held_after, free_after = torch.cuda.memory_allocated(), torch.cuda.mem_get_info()[0]
        finally:
            gc.enable()
        assert (held_after, free_after) == (held, free)
        assert torch.equal(again.tensor, torch.clamp_min(got.tensor, 0.0))


def test_static_scratch_dense_split_contraction(gl):
    # a plain product whose contraction is split: the partial planes are the only scratch
    _dirty_the_scratch(gl)
    a = synth.uniform_int(56, 1, (100, 4096), -3, 3)
    b = synth.uniform_int(56, 2, (60, 4096), -3, 3)
    aa, bb = gl.AccessPattern(to_bf16_device(a), 1), gl.AccessPattern(to_bf16_device(b), 1)
    assert gl.gl_cartesian_dot_workspace(aa, None, bb) > 0
    got = gl.output_like(gl.gl_shape_cartesian_dot(a.shape, 1, None, b.shape, 1), "cuda")
    for _ in range(2):
        got.tensor.fill_(float("nan"))
        gl.gl_cartesian_dot_static(aa, None, bb, got)
        assert gl.gl_poll_device_status() == 0
        assert np.array_equal(got.tensor.cpu().numpy().astype(np.float64), brute.rowdot(a, b))


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

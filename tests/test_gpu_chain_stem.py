"""The kernels of Fig. 2 composed into one program at the scale of a network stem (conv 7x7 stride 2 + relu,
max pool, conv 3x3 + relu, max pool, flatten, dense), run in both item layouts, against the same chain of
brute-force equations.  Layer results are stored as bf16; the checker rounds its float64 layer results the same
way.  With inputs from {-1, 0, 1} every sum is an integer below 2^24 and exact in fp32, so the device's rounded
layer results are the checker's bit for bit and so is the final result."""
import numpy as np
import pytest

from oracle import brute
from paper_2105_09377_b200 import synth

pytestmark = pytest.mark.gpu

CASES = {
    "small": synth.ChainCase("chain_small", 3, 45, 37, 16, 24, 2, 10, integer=True),
    "stem_integer": synth.ChainCase("chain_stem_int", 32, 224, 224, 64, 64, 8, 1000, integer=True),
    "stem_gaussian": synth.CHAIN_STEM,
}


def _checker_chain(cfg, x, w1, w2, wd):
    """(N, units) float64 from the brute-force equations, layer results rounded to bf16 as the device stores them."""
    y1 = synth.bf16_round(np.maximum(brute.conv2d(x, w1, (2, 2), ((3, 3), (3, 3))), 0.0).astype(np.float32))
    p1 = brute.maxpool(y1, (3, 3), (2, 2), ((1, 1), (1, 1)))
    y2 = synth.bf16_round(np.maximum(brute.conv2d(p1, w2, (1, 1), ((1, 1), (1, 1))), 0.0).astype(np.float32))
    p2 = brute.maxpool(y2, (cfg.pool2,) * 2, (cfg.pool2,) * 2)
    feat = p2.reshape(cfg.n, -1)
    return brute.rowdot(feat, wd.reshape(cfg.units, -1)), feat


@pytest.fixture(scope="module")
def refs():
    return {}


@pytest.mark.parametrize("layout", ["nhwc", "nchw"])
@pytest.mark.parametrize("name", list(CASES))
def test_chain_both_layouts(name, layout, refs):
    import torch
    from paper_2105_09377_b200 import binding as gl
    from paper_2105_09377_b200 import run_workload as rw
    from tests.gpu_util import REL_TOL, rel_err
    cfg = CASES[name]
    seed = 77
    if name not in refs:
        refs[name] = _checker_chain(cfg, *cfg.inputs(seed))
    ref, feat = refs[name]
    run, logits, nsteps = rw.build_chain(cfg, layout, torch.device("cuda", 0), seed)
    assert nsteps == 5
    logits.tensor.fill_(float("nan"))
    run()
    assert gl.gl_poll_device_status() == 0
    got = logits.tensor.cpu().numpy()
    assert got.shape == ref.shape == (cfg.n, cfg.units)
    if cfg.integer:
        assert np.abs(feat).sum(axis=1).max() < 2 ** 24          # every partial sum of the dense layer is exact
        assert np.array_equal(got.astype(np.float64), ref)
    else:
        assert rel_err(got, ref) <= REL_TOL

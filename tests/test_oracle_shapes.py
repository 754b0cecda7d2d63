"""The interpreter's shapes against the shape annotations printed in the paper
(Fig. 2a-c, Fig. 6, Fig. 8) and the closed forms of the transformer table."""
import math
import os

import numpy as np
import pytest

from oracle import interp as gi


def _parse(golden_dir):
    traces = {}
    with open(os.path.join(golden_dir, "shape_traces.txt")) as fh:
        for line in fh:
            line = line.split("#")[0].strip()
            if not line:
                continue
            name, rest = line.split(":")
            acc, comp = rest.split("|")
            traces[name.strip()] = (acc.strip(), comp.strip())
    return traces


def _inst(side: str, env):
    if not side:
        return ()
    out = []
    for term in side.split(","):
        v = 1
        for f in term.strip().split("*"):
            f = f.strip()
            v *= int(f) if f.isdigit() else env[f]
        out.append(v)
    return tuple(out)


def _expect(traces, key, env):
    acc, comp = traces[key]
    return (_inst(acc, env), _inst(comp, env))


ENV = {"N": 2, "C": 3, "H": 9, "W": 8, "O": 4, "Kh": 3, "Kw": 2, "Sh": 2, "Sw": 1}
ENV["H'"] = (ENV["H"] - ENV["Kh"]) // ENV["Sh"] + 1
ENV["W'"] = (ENV["W"] - ENV["Kw"]) // ENV["Sw"] + 1


def test_conv2d_trace(golden_dir):
    t = _parse(golden_dir)
    e = ENV
    act = gi.access(np.zeros((e["N"], e["C"], e["H"], e["W"])), 1)
    wts = gi.access(np.zeros((e["O"], e["C"], e["Kh"], e["Kw"])), 1)
    assert act.shape == _expect(t, "conv2d.activations", e)
    assert wts.shape == _expect(t, "conv2d.weights", e)
    win = gi.windows(act, (e["C"], e["Kh"], e["Kw"]), (1, e["Sh"], e["Sw"]))
    assert win.shape == _expect(t, "conv2d.windows", e)
    cp = gi.cart_prod(win, wts)
    assert cp.shape == _expect(t, "conv2d.cartProd", e)
    dp = gi.compute("dotProd", cp)
    assert dp.shape == _expect(t, "conv2d.dotProd", e)
    sq = gi.squeeze(dp, 1)
    assert sq.shape == _expect(t, "conv2d.squeeze", e)
    tr = gi.transpose(sq, (0, 3, 1, 2))
    assert tr.shape == _expect(t, "conv2d.transpose", e)


def test_matmul_trace(golden_dir):
    t = _parse(golden_dir)
    e = {"M": 5, "K": 7, "O": 3}
    act = gi.access(np.zeros((5, 7)), 1)
    wts = gi.access(np.zeros((7, 3)), 1)
    assert act.shape == _expect(t, "matmul.activations", e)
    assert wts.shape == _expect(t, "matmul.weights", e)
    wt = gi.transpose(wts, (1, 0))
    assert wt.shape == _expect(t, "matmul.transpose", e)
    cp = gi.cart_prod(act, wt)
    assert cp.shape == _expect(t, "matmul.cartProd", e)
    assert gi.compute("dotProd", cp).shape == _expect(t, "matmul.dotProd", e)


def test_maxpool_trace(golden_dir):
    t = _parse(golden_dir)
    e = ENV
    act = gi.access(np.zeros((e["N"], e["C"], e["H"], e["W"])), 2)
    assert act.shape == _expect(t, "maxpool.activations", e)
    win = gi.windows(act, (e["Kh"], e["Kw"]), (e["Sh"], e["Sw"]))
    assert win.shape == _expect(t, "maxpool.windows", e)
    assert gi.compute("reduceMax", win).shape == _expect(t, "maxpool.reduceMax", e)


def test_im2col_trace(golden_dir):
    t = _parse(golden_dir)
    e = ENV
    act = gi.access(np.zeros((e["N"], e["C"], e["H"], e["W"])), 1)
    wts = gi.access(np.zeros((e["O"], e["C"], e["Kh"], e["Kw"])), 1)
    win = gi.windows(act, (e["C"], e["Kh"], e["Kw"]), (1, e["Sh"], e["Sw"]))
    fa, fw = gi.flatten(win), gi.flatten(wts)
    assert fa.shape == _expect(t, "im2col.flatten_act", e)
    assert fw.shape == _expect(t, "im2col.flatten_wts", e)
    dp = gi.compute("dotProd", gi.cart_prod(fa, fw))
    assert dp.shape == _expect(t, "im2col.dotProd", e)
    rs = gi.reshape(dp, win.access_shape + wts.access_shape, ())
    assert rs.shape == _expect(t, "im2col.reshape", e)


def test_blocked_trace(golden_dir):
    t = _parse(golden_dir)
    act = gi.access(np.zeros((32, 32)), 1)
    wts = gi.access(np.zeros((32, 32)), 1)
    sa = gi.slice_(gi.slice_(act, 0, 0, 16), 1, 0, 16)
    assert sa.shape == _expect(t, "blocked.slice_act", {})
    tw = gi.transpose(gi.slice_(gi.slice_(wts, 0, 0, 16), 1, 0, 16), (1, 0))
    assert tw.shape == _expect(t, "blocked.transpose", {})
    cp = gi.cart_prod(sa, tw)
    assert cp.shape == _expect(t, "blocked.cartProd", {})
    dp = gi.compute("dotProd", cp)
    assert dp.shape == _expect(t, "blocked.dotProd", {})
    pr = gi.pair(dp, dp)
    assert pr.shape == _expect(t, "blocked.pair", {})
    rs = gi.compute("reduceSum", pr)
    assert rs.shape == _expect(t, "blocked.reduceSum", {})
    ci = gi.concat(rs, rs, 1)
    assert ci.shape == _expect(t, "blocked.concat_inner", {})
    assert gi.concat(ci, ci, 0).shape == _expect(t, "blocked.concat_outer", {})


@pytest.mark.parametrize("b,w,s", [(8, 3, 1), (9, 3, 2), (10, 3, 2), (7, 7, 1), (230, 7, 2), (114, 3, 2), (5, 1, 3)])
def test_windows_extent_closed_form(b, w, s):
    # ceil((b-(w-1))/s) of the table equals the usual floor((b-w)/s)+1
    assert gi.windows_out_extent(b, w, s) == (b - w) // s + 1 == math.ceil((b - (w - 1)) / s)


def test_windows_rejects_oversized_window():
    with pytest.raises(ValueError):
        gi.windows_out_extent(2, 3, 1)


def test_table_rows_misc():
    a = gi.access(np.zeros((2, 3, 4, 5)), 2)
    assert gi.access(a, 3).shape == ((2, 3, 4), (5,))
    assert gi.access(a, 0).shape == ((), (2, 3, 4, 5))
    assert gi.flatten(a).shape == ((6,), (20,))
    assert gi.flatten(gi.access(a, 4)).shape == ((120,), ())
    assert gi.flatten(gi.access(a, 0)).shape == ((), (120,))
    assert gi.slice_(a, 2, 1, 3).shape == ((2, 3), (2, 5))
    assert gi.reshape(a, (6,), (2, 10)).shape == ((6,), (2, 10))
    with pytest.raises(ValueError):
        gi.reshape(a, (3,), (40,))
    assert gi.pair(a, a).shape == ((2, 3), (2, 4, 5))
    assert gi.squeeze(gi.access(np.zeros((2, 1, 3)), 2), 1).shape == ((2,), (3,))
    assert gi.squeeze(gi.access(np.zeros((2, 3, 1)), 2), 2).shape == ((2, 3), ())
    assert gi.pad(a, 3, 1, 2).shape == ((2, 3), (4, 8))
    assert gi.transpose(gi.access(np.zeros((6, 9)), 1), (1, 0)).shape == ((9,), (6,))

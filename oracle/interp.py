"""Reference interpreter of Glenside access-pattern programs (test infrastructure).

This file is a checker, not a product: only the tests, the smoke check and the
benchmark's CPU-baseline leg may import it.  It shares no code with the CUDA
library and never calls it.  Everything is dense row-major numpy in float64.

An access pattern (paper Section 4.1) is a tensor together with a split of its
dimensions into *access* dimensions S_A (iterated over) and *compute*
dimensions S_C (computed on); the tensor's shape is S_A ++ S_C.

Each function below states one row of the paper's Table of access-pattern
transformers (Section 4, first table) or of the operator table (Section 4.3)
as the definition written out, with no blocking or fusion.

Readings taken where the paper is silent or inconsistent
  * windows: the table writes k_i in the formula and w_i in the argument list;
    both mean the window extent.  ceil((b-(w-1))/s) equals floor((b-w)/s)+1 for
    b >= w; a window larger than its dimension is an error.
  * transpose: the permutation ranges over all dimensions (access and compute);
    the split position is kept (Section 4.2: ((N),(O)) becomes ((O),(N))).
  * cartProd: the first argument supplies tuple member 0 and the leading
    access dimensions (Fig. 2a passes windows first, weights second, and
    annotates ((N,1,H',W',O),(2,C,Kh,Kw))).
  * dotProd on an item (t, s...) multiplies the t members elementwise and sums.
  * flatten: a side with no dimensions stays empty.
  * pair: the new axis of size 2 is the first compute dimension.
  * concat (used in the blocking figure, absent from the table): ordinary
    concatenation along one dimension.
  * pad and relu are not in the paper (parity unpinned by the paper): pad
    grows one dimension by lo+hi cells holding 0 or -inf; relu(x) is x if
    x > 0 else +0, itemwise, shape kept.
"""
from __future__ import annotations

import itertools
import math
from dataclasses import dataclass

import numpy as np


@dataclass
class AP:
    """Access pattern: `data` has shape S_A ++ S_C, `access_ndim` = |S_A|."""

    data: np.ndarray
    access_ndim: int

    def __post_init__(self):
        self.data = np.asarray(self.data, dtype=np.float64)
        if not 0 <= self.access_ndim <= self.data.ndim:
            raise ValueError("access_ndim out of range")

    @property
    def access_shape(self):
        return tuple(self.data.shape[: self.access_ndim])

    @property
    def compute_shape(self):
        return tuple(self.data.shape[self.access_ndim:])

    @property
    def shape(self):
        """The pair (S_A, S_C)."""
        return (self.access_shape, self.compute_shape)


# --------------------------------------------------------------------------
# Transformers (Section 4.2, transformer table)
# --------------------------------------------------------------------------

def access(t, i: int) -> AP:
    """`access`: (re)split the dimensions at index i.  Data untouched."""
    data = t.data if isinstance(t, AP) else np.asarray(t, dtype=np.float64)
    if not 0 <= i <= data.ndim:
        raise ValueError("access index out of range")
    return AP(data, i)


def transpose(a: AP, perm) -> AP:
    """`transpose`: output dimension j is input dimension perm[j]."""
    perm = tuple(int(p) for p in perm)
    if sorted(perm) != list(range(a.data.ndim)):
        raise ValueError("not a permutation of all dimensions")
    out_shape = tuple(a.data.shape[p] for p in perm)
    if a.data.size > 4096:
        # numpy's axis permutation as a library step (same index rule)
        return AP(np.ascontiguousarray(np.transpose(a.data, perm)), a.access_ndim)
    out = np.empty(out_shape, dtype=np.float64)
    for idx in np.ndindex(*out_shape):
        src = [0] * len(perm)
        for j, p in enumerate(perm):
            src[p] = idx[j]
        out[idx] = a.data[tuple(src)]
    return AP(out, a.access_ndim)


def cart_prod(a: AP, b: AP) -> AP:
    """`cartProd`: pair every item of `a` with every item of `b`.

    ((a...),(c...)) x ((b...),(c...)) -> ((a..., b...),(2, c...)).
    """
    if a.compute_shape != b.compute_shape:
        raise ValueError("cartProd needs equal compute shapes")
    sa, sb, sc = a.access_shape, b.access_shape, a.compute_shape
    out = np.empty(sa + sb + (2,) + sc, dtype=np.float64)
    for ia in np.ndindex(*sa):
        for ib in np.ndindex(*sb):
            out[ia + ib + (0,)] = a.data[ia]
            out[ia + ib + (1,)] = b.data[ib]
    return AP(out, len(sa) + len(sb))


def windows_out_extent(b: int, w: int, s: int) -> int:
    """b' = ceil((b - (w - 1)) / s), the table's formula."""
    if w < 1 or s < 1:
        raise ValueError("window extent and stride must be positive")
    if w > b:
        raise ValueError("window larger than the dimension")
    return -((-(b - (w - 1))) // s)


def windows(a: AP, wshape, strides) -> AP:
    """`windows`: out[a..., p_0..p_n, q_0..q_n] = in[a..., p_i*s_i + q_i].

    ((a...),(b_0..b_n)) -> ((a..., b'_0..b'_n),(w_0..w_n)).
    """
    wshape = tuple(int(w) for w in wshape)
    strides = tuple(int(s) for s in strides)
    cs = a.compute_shape
    if len(wshape) != len(cs) or len(strides) != len(cs):
        raise ValueError("one window extent and stride per compute dimension")
    bp = tuple(windows_out_extent(b, w, s) for b, w, s in zip(cs, wshape, strides))
    sa = a.access_shape
    out = np.empty(sa + bp + wshape, dtype=np.float64)
    for p in np.ndindex(*bp):
        sel = tuple(slice(pi * si, pi * si + wi) for pi, si, wi in zip(p, strides, wshape))
        # every access index at once; the window itself is copied cell by cell
        out[(Ellipsis,) + p + (slice(None),) * len(wshape)] = a.data[(Ellipsis,) + sel]
    return AP(out, len(sa) + len(bp))


def windows_element(a: AP, wshape, strides, index) -> float:
    """One cell of `windows` by its definition (for sampled checks at sizes
    where the whole result is too large to build)."""
    na = a.access_ndim
    n = len(wshape)
    acc = tuple(index[:na])
    p = index[na:na + n]
    q = index[na + n:]
    src = tuple(pi * si + qi for pi, si, qi in zip(p, strides, q))
    return float(a.data[acc + src])


def slice_(a: AP, d: int, lo: int, hi: int) -> AP:
    """`slice`: keep [lo, hi) of dimension d."""
    if not 0 <= d < a.data.ndim or not 0 <= lo <= hi <= a.data.shape[d]:
        raise ValueError("bad slice")
    sel = [slice(None)] * a.data.ndim
    sel[d] = slice(lo, hi)
    return AP(a.data[tuple(sel)].copy(), a.access_ndim)


def squeeze(a: AP, d: int) -> AP:
    """`squeeze`: drop dimension d, which must have size 1."""
    if a.data.shape[d] != 1:
        raise ValueError("squeeze needs a size-1 dimension")
    na = a.access_ndim - 1 if d < a.access_ndim else a.access_ndim
    return AP(a.data.reshape(a.data.shape[:d] + a.data.shape[d + 1:]).copy(), na)


def flatten(a: AP) -> AP:
    """`flatten`: ((a...),(b...)) -> ((prod a),(prod b)); an empty side stays empty."""
    sa, sc = a.access_shape, a.compute_shape
    new = (() if not sa else (math.prod(sa),)) + (() if not sc else (math.prod(sc),))
    return AP(a.data.reshape(new).copy(), 0 if not sa else 1)


def reshape(a: AP, access_shape, compute_shape) -> AP:
    """`reshape`: row-major re-view; each side's element count must be kept."""
    access_shape = tuple(access_shape)
    compute_shape = tuple(compute_shape)
    if math.prod(access_shape) != math.prod(a.access_shape):
        raise ValueError("access sizes differ")
    if math.prod(compute_shape) != math.prod(a.compute_shape):
        raise ValueError("compute sizes differ")
    return AP(a.data.reshape(access_shape + compute_shape).copy(), len(access_shape))


def pair(a: AP, b: AP) -> AP:
    """`pair`: stack two equal-shape patterns; the 2 is the first compute dimension."""
    if a.shape != b.shape:
        raise ValueError("pair needs equal shapes")
    return AP(np.stack([a.data, b.data], axis=a.access_ndim), a.access_ndim)


def concat(a: AP, b: AP, d: int) -> AP:
    """`concat` (blocking figure): join along dimension d."""
    if a.access_ndim != b.access_ndim:
        raise ValueError("concat needs the same split")
    return AP(np.concatenate([a.data, b.data], axis=d), a.access_ndim)


def pad(a: AP, d: int, lo: int, hi: int, kind: str = "zero") -> AP:
    """`pad` (not in the paper): dimension d grows by lo + hi cells of 0 or -inf."""
    fill = {"zero": 0.0, "neg_inf": -np.inf}[kind]
    if lo < 0 or hi < 0 or not 0 <= d < a.data.ndim:
        raise ValueError("bad pad")
    shp = list(a.data.shape)
    shp[d] += lo + hi
    out = np.full(shp, fill, dtype=np.float64)
    sel = [slice(None)] * a.data.ndim
    sel[d] = slice(lo, lo + a.data.shape[d])
    out[tuple(sel)] = a.data
    return AP(out, a.access_ndim)


# --------------------------------------------------------------------------
# Operators (Section 4.3, operator table) applied by `compute`
# --------------------------------------------------------------------------

def _reduce_sum(item: np.ndarray) -> np.ndarray:
    return np.asarray(math.fsum(item.ravel().tolist()))


def _reduce_max(item: np.ndarray) -> np.ndarray:
    return np.asarray(item.max())


def _dot_prod(item: np.ndarray) -> np.ndarray:
    # item has shape (t, s...): multiply the t members cell by cell, sum all
    prod = np.ones(item.shape[1:], dtype=np.float64)
    for j in range(item.shape[0]):
        prod = prod * item[j]
    return np.asarray(prod.sum())


def _relu(item: np.ndarray) -> np.ndarray:
    return np.where(item > 0.0, item, 0.0)


OPERATORS = {
    "reduceSum": _reduce_sum,
    "reduceMax": _reduce_max,
    "dotProd": _dot_prod,
    "relu": _relu,
}


def compute(op: str, a: AP) -> AP:
    """`compute f A`: apply f to every item; the access dimensions never change."""
    f = OPERATORS[op]
    sa = a.access_shape
    first = f(a.data[(0,) * len(sa)]) if a.data.size else None
    if op == "dotProd" and a.data.shape[a.access_ndim] < 1:
        raise ValueError("dotProd needs a tuple axis")
    item_shape = () if first is None else first.shape
    out = np.empty(sa + item_shape, dtype=np.float64)
    for ia in np.ndindex(*sa):
        out[ia] = f(a.data[ia])
    return AP(out, len(sa))


# --------------------------------------------------------------------------
# The kernel specifications of Fig. 2 and the rewritten form of Section 5.3
# --------------------------------------------------------------------------

def _pad_hw(act: AP, pads, kind: str) -> AP:
    """Optional `pad` of the last two dimensions (H and W) before `windows`."""
    (ph_lo, ph_hi), (pw_lo, pw_hi) = pads
    nd = act.data.ndim
    if ph_lo or ph_hi:
        act = pad(act, nd - 2, ph_lo, ph_hi, kind)
    if pw_lo or pw_hi:
        act = pad(act, nd - 1, pw_lo, pw_hi, kind)
    return act


def conv2d_program(activations, weights, strides=(1, 1), pads=((0, 0), (0, 0)), upto="transpose"):
    """Fig. 2a: transpose(squeeze(compute dotProd(cartProd(windows(access act 1)
    (C,Kh,Kw) (1,Sh,Sw)) (access weights 1))) 1) (0 3 1 2)).

    `upto` = "dotProd" stops at the ((N,1,H',W',O),()) pattern.
    """
    act = _pad_hw(access(activations, 1), pads, "zero")
    wts = access(weights, 1)
    c, kh, kw = wts.compute_shape
    win = windows(act, (c, kh, kw), (1, strides[0], strides[1]))
    dot = compute("dotProd", cart_prod(win, wts))
    if upto == "dotProd":
        return dot
    return transpose(squeeze(dot, 1), (0, 3, 1, 2))


def conv2d_im2col_program(activations, weights, strides=(1, 1), pads=((0, 0), (0, 0)), upto="transpose"):
    """Fig. 6 (Section 5.3): the same conv2d after the three im2col rewrites:
    reshape(compute dotProd(cartProd(flatten(windows ...)) (flatten(access weights 1)))) ?shape),
    with ?shape = ((N,1,H',W',O),()), then squeeze and transpose as before."""
    act = _pad_hw(access(activations, 1), pads, "zero")
    wts = access(weights, 1)
    c, kh, kw = wts.compute_shape
    win = windows(act, (c, kh, kw), (1, strides[0], strides[1]))
    lhs = flatten(win)            # ((N*1*H'*W'),(C*Kh*Kw)): the im2col matrix
    rhs = flatten(wts)            # ((O),(C*Kh*Kw))
    dot = compute("dotProd", cart_prod(lhs, rhs))      # ((N*1*H'*W', O),())
    dot = reshape(dot, win.access_shape + wts.access_shape, ())
    if upto == "dotProd":
        return dot
    return transpose(squeeze(dot, 1), (0, 3, 1, 2))


def matmul_program(activations, weights):
    """Fig. 2b: compute dotProd (cartProd (access act 1) (transpose (access weights 1) (1 0)))."""
    return compute("dotProd", cart_prod(access(activations, 1), transpose(access(weights, 1), (1, 0))))


def dense_rows_program(a_rows, b_rows, relu=False):
    """Dense layer with both operands already accessed as row vectors
    ((M),(K)) and ((O),(K)): compute dotProd (cartProd A B), optionally
    followed by compute relu."""
    out = compute("dotProd", cart_prod(access(a_rows, 1), access(b_rows, 1)))
    return compute("relu", out) if relu else out


def maxpool_program(activations, wshape, strides, pads=((0, 0), (0, 0))):
    """Fig. 2c: compute reduceMax (windows (access act 2) (Kh,Kw) (Sh,Sw)),
    optionally preceded by a -inf pad of H and W."""
    act = _pad_hw(access(activations, 2), pads, "neg_inf")
    return compute("reduceMax", windows(act, wshape, strides))

"""Run one workload of the table in `synth` a few times on cuda:0.

    python -m paper_2105_09377_b200.run_workload --workload conv3x3_56x56x64 --layout nhwc --iters 3

Prints the mean time per call (CUDA events).  Meant for profilers and quick
checks; the benchmark proper is bench.py.
"""
from __future__ import annotations

import argparse
import functools

import numpy as np
import torch

from . import binding as gl
from . import synth


def _bf16(x, device):
    return torch.from_numpy(synth.bf16_bits(x).view(np.int16)).to(device).view(torch.bfloat16).reshape(x.shape)


@functools.lru_cache(maxsize=2)
def _inputs(cfg, seed):
    """Host inputs of a workload, kept so that several buffer sets can be filled from one draw."""
    return cfg.inputs(seed)


def workloads():
    table = {c.name: c for c in (synth.CONV_TINY,) + synth.CONV_SWEEP_3X3 + synth.CONV_STRIDED_1X1}
    table.update({c.name: c for c in (synth.MEM_IM2COL, synth.MEM_TRANSPOSE, synth.MEM_MAXPOOL, synth.MEM_RELU,
                                      synth.MEM_PAD)})
    table[synth.DENSE_4096.name] = synth.DENSE_4096
    return table


def build_call(cfg, layout: str, device, batch=None, flags=0):
    """Returns (prepared call, flops, algorithmic bytes)."""
    if isinstance(cfg, synth.DenseCase):
        a, b = _inputs(cfg, synth.config_seed(1))
        aa, bb = gl.AccessPattern(_bf16(a, device), 1), gl.AccessPattern(_bf16(b, device), 1)
        out = gl.output_like(gl.gl_shape_cartesian_dot(a.shape, 1, None, b.shape, 1), device)
        if flags & gl.GL_OUT_BF16:
            out = gl.AccessPattern(out.tensor.to(torch.bfloat16), out.access_ndim)
        return gl.prepare_cartesian_dot(aa, None, bb, out, flags | gl.GL_EPILOGUE_RELU), cfg.flops, cfg.algorithmic_bytes
    if isinstance(cfg, synth.ConvCase):
        if batch:
            cfg = synth.ConvCase(cfg.name, batch, cfg.c, cfg.h, cfg.w, cfg.o, cfg.kh, cfg.kw, cfg.stride, cfg.pad, cfg.integer)
        x, wt = _inputs(cfg, synth.config_seed(2))
        if layout == "rewritten":
            # Section 5.3: flatten(windows(act)) materialised as the im2col matrix, flatten(weights), plain matmul
            spec = gl.windows_spec((cfg.c, cfg.kh, cfg.kw), (1, cfg.stride, cfg.stride), (0, cfg.pad, cfg.pad), (0, cfg.pad, cfg.pad))
            xa, wa = gl.AccessPattern(_bf16(x, device), 1), gl.AccessPattern(_bf16(wt, device), 1)
            cols = gl.output_like(gl.gl_shape_windows(x.shape, 1, spec, gl.GL_BF16), device)
            flat, wflat = gl.gl_access_flatten(cols), gl.gl_access_flatten(wa)
            out = gl.output_like(gl.gl_shape_cartesian_dot(tuple(flat.tensor.shape), 1, None, tuple(wflat.tensor.shape), 1), device)
            need = gl.gl_cartesian_dot_workspace(flat, None, wflat, flags)
            ws = torch.empty(need + 1024, dtype=torch.uint8, device=device) if need else None
            steps = (gl.prepare_access_windows(xa, spec, cols), gl.prepare_cartesian_dot(flat, None, wflat, out, flags, ws))

            def both(stream=None):
                for step in steps:
                    step(stream)
            return both, cfg.flops, cfg.algorithmic_bytes
        if layout == "nhwc":
            x, wt = x.transpose(0, 2, 3, 1).copy(), wt.transpose(0, 2, 3, 1).copy()
            spec = gl.windows_spec((cfg.kh, cfg.kw, cfg.c), (cfg.stride, cfg.stride, 1), (cfg.pad, cfg.pad, 0), (cfg.pad, cfg.pad, 0))
        else:
            spec = gl.windows_spec((cfg.c, cfg.kh, cfg.kw), (1, cfg.stride, cfg.stride), (0, cfg.pad, cfg.pad), (0, cfg.pad, cfg.pad))
        xa, wa = gl.AccessPattern(_bf16(x, device), 1), gl.AccessPattern(_bf16(wt, device), 1)
        out = gl.output_like(gl.gl_shape_cartesian_dot(x.shape, 1, spec, wt.shape, 1), device)
        if flags & gl.GL_OUT_NCHW:      # Fig. 2a's whole program: squeeze + transpose (0 3 1 2) fused, ((N,O,H',W'),())
            out = gl.AccessPattern(torch.empty((cfg.n, cfg.o, cfg.ho, cfg.wo), dtype=torch.float32, device=device), 4)
        if flags & gl.GL_OUT_BF16:      # results stored as bf16: half the bytes written
            out = gl.AccessPattern(out.tensor.to(torch.bfloat16), out.access_ndim)
        need = gl.gl_cartesian_dot_workspace(xa, spec, wa, flags)
        ws = torch.empty(need + 1024, dtype=torch.uint8, device=device) if need else None
        return gl.prepare_cartesian_dot(xa, spec, wa, out, flags, ws), cfg.flops, cfg.algorithmic_bytes
    if batch:
        cfg = synth.MemCase(cfg.name, cfg.kind, (batch,) + tuple(cfg.shape[1:]), cfg.window, cfg.stride, cfg.pad, cfg.perm)
    x = torch.from_numpy(_inputs(cfg, synth.config_seed(4))).to(device)
    if cfg.kind == "transpose":
        out = gl.output_like(gl.gl_shape_transpose(cfg.shape, 1, cfg.perm), device)
        return gl.prepare_access_transpose(gl.AccessPattern(x, 1), cfg.perm, out), 0.0, cfg.algorithmic_bytes
    if cfg.kind == "relu":
        a = gl.AccessPattern(x, 4)
        return gl.prepare_compute_relu(a, gl.AccessPattern(torch.empty_like(x), 4)), 0.0, cfg.algorithmic_bytes
    if cfg.kind == "pad":
        out = gl.output_like(gl.gl_shape_pad(cfg.shape, 1, 3, cfg.pad, cfg.pad), device)
        return gl.prepare_access_pad(gl.AccessPattern(x, 1), 3, cfg.pad, cfg.pad, gl.GL_PAD_ZERO, out), 0.0, cfg.algorithmic_bytes
    if cfg.kind == "im2col":
        c = cfg.shape[1]
        spec = gl.windows_spec((c,) + cfg.window, (1, cfg.stride, cfg.stride), (0, cfg.pad, cfg.pad), (0, cfg.pad, cfg.pad))
        out = gl.output_like(gl.gl_shape_windows(cfg.shape, 1, spec), device)
        return gl.prepare_access_windows(gl.AccessPattern(x, 1), spec, out), 0.0, cfg.algorithmic_bytes
    spec = gl.windows_spec(cfg.window, (cfg.stride,) * 2, (cfg.pad,) * 2, (cfg.pad,) * 2, gl.GL_PAD_NEG_INF)
    out = gl.output_like(gl.gl_shape_reduce_max(cfg.shape, 2, spec), device)
    return gl.prepare_compute_reduce_max(gl.AccessPattern(x, 2), spec, out), 0.0, cfg.algorithmic_bytes


def build_chain(cfg, layout: str, device, seed=None):
    """The program of `synth.ChainCase` as a list of prepared calls plus the access pattern of its result.

    layout "nhwc": items (H,W,C), layer results stored as bf16 rows [pixels, channels] (GL_OUT_BF16) which are the
    next layer's items as they stand.  layout "nchw": the paper's (C,H,W) items, every convolution followed by the
    squeeze + transpose of Fig. 2a (GL_OUT_NCHW).  The dense weights are laid out to match the flatten order of the
    layout, so both layouts compute the same numbers."""
    x, w1, w2, wd = cfg.inputs(synth.config_seed(5) if seed is None else seed)
    (h1, wd1), (h2, wd2), (h3, wd3) = cfg.dims()
    n, c1, c2, k2 = cfg.n, cfg.c1, cfg.c2, cfg.pool2
    relu_bf16 = gl.GL_EPILOGUE_RELU | gl.GL_OUT_BF16
    steps = []

    def conv(xa, spec, wa, out_shape, flags):
        out = gl.AccessPattern(torch.empty(out_shape, dtype=torch.bfloat16, device=device), len(out_shape))
        need = gl.gl_cartesian_dot_workspace(xa, spec, wa, flags)
        ws = torch.empty(need + 1024, dtype=torch.uint8, device=device) if need else None
        steps.append(gl.prepare_cartesian_dot(xa, spec, wa, out, flags, ws))
        return out

    def pool(a, spec, out_shape, na):
        out = gl.AccessPattern(torch.empty(out_shape, dtype=torch.bfloat16, device=device), na)
        steps.append(gl.prepare_compute_reduce_max(a, spec, out))
        return out

    if layout == "nhwc":
        t = lambda a: np.ascontiguousarray(a.transpose(0, 2, 3, 1))
        xa = gl.AccessPattern(_bf16(t(x), device), 1)
        y1 = conv(xa, gl.windows_spec((7, 7, 3), (2, 2, 1), (3, 3, 0), (3, 3, 0)), gl.AccessPattern(_bf16(t(w1), device), 1),
                  (n, h1, wd1, 1, c1), relu_bf16)
        p1 = pool(gl.AccessPattern(y1.tensor.view(n, h1, wd1, c1), 1),
                  gl.windows_spec((3, 3, 1), (2, 2, 1), (1, 1, 0), (1, 1, 0), gl.GL_PAD_NEG_INF), (n, h2, wd2, c1), 4)
        y2 = conv(gl.AccessPattern(p1.tensor, 1), gl.windows_spec((3, 3, c1), (1, 1, 1), (1, 1, 0), (1, 1, 0)),
                  gl.AccessPattern(_bf16(t(w2), device), 1), (n, h2, wd2, 1, c2), relu_bf16)
        p2 = pool(gl.AccessPattern(y2.tensor.view(n, h2, wd2, c2), 1), gl.windows_spec((k2, k2, 1), (k2, k2, 1)),
                  (n, h3, wd3, c2), 4)
        feat = gl.AccessPattern(p2.tensor.view(n, h3 * wd3 * c2), 1)                 # flatten: metadata
        wdense = gl.AccessPattern(_bf16(t(wd).reshape(cfg.units, -1), device), 1)
    else:
        xa = gl.AccessPattern(_bf16(x, device), 1)
        nchw = relu_bf16 | gl.GL_OUT_NCHW
        y1 = conv(xa, gl.windows_spec((3, 7, 7), (1, 2, 2), (0, 3, 3), (0, 3, 3)), gl.AccessPattern(_bf16(w1, device), 1),
                  (n, c1, h1, wd1), nchw)
        p1 = pool(gl.AccessPattern(y1.tensor, 2), gl.windows_spec((3, 3), (2, 2), (1, 1), (1, 1), gl.GL_PAD_NEG_INF),
                  (n, c1, h2, wd2), 4)
        y2 = conv(gl.AccessPattern(p1.tensor, 1), gl.windows_spec((c1, 3, 3), (1, 1, 1), (0, 1, 1), (0, 1, 1)),
                  gl.AccessPattern(_bf16(w2, device), 1), (n, c2, h2, wd2), nchw)
        p2 = pool(gl.AccessPattern(y2.tensor, 2), gl.windows_spec((k2, k2), (k2, k2)), (n, c2, h3, wd3), 4)
        feat = gl.AccessPattern(p2.tensor.view(n, c2 * h3 * wd3), 1)
        wdense = gl.AccessPattern(_bf16(wd.reshape(cfg.units, -1), device), 1)
    logits = gl.AccessPattern(torch.empty((n, cfg.units), dtype=torch.float32, device=device), 2)
    need = gl.gl_cartesian_dot_workspace(feat, None, wdense, 0)
    ws = torch.empty(need + 1024, dtype=torch.uint8, device=device) if need else None
    steps.append(gl.prepare_cartesian_dot(feat, None, wdense, logits, 0, ws))

    def run(stream=None):
        for step in steps:
            step(stream)
    return run, logits, len(steps)


def main():
    table = workloads()
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", required=True, choices=sorted(table))
    ap.add_argument("--layout", default="nhwc", choices=["nhwc", "nchw", "rewritten"])
    ap.add_argument("--iters", type=int, default=3)
    ap.add_argument("--batch", type=int, default=0, help="override the leading (batch) extent")
    ap.add_argument("--graph", action="store_true", help="time one CUDA graph holding all iterations")
    ap.add_argument("--general", action="store_true", help="use the general SIMT kernel for dot products")
    ap.add_argument("--bf16-out", action="store_true", help="store dot-product results as bf16 (GL_OUT_BF16)")
    args = ap.parse_args()
    device = torch.device("cuda", 0)
    torch.cuda.set_device(device)
    call, flops, nbytes = build_call(table[args.workload], args.layout, device, args.batch or None,
                                     (gl.GL_DOT_GENERAL_KERNEL if args.general else 0) | (gl.GL_OUT_BF16 if args.bf16_out else 0))
    call()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if args.graph:
        # replay the calls from one CUDA graph: host launch cost no longer paces short kernels
        side = torch.cuda.Stream()
        with torch.cuda.stream(side):
            call()
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            for _ in range(args.iters):
                call()
        graph.replay()
        torch.cuda.synchronize()
        e0.record()
        graph.replay()
        e1.record()
    else:
        e0.record()
        for _ in range(args.iters):
            call()
        e1.record()
    torch.cuda.synchronize()
    status = gl.gl_poll_device_status()
    us = e0.elapsed_time(e1) * 1e3 / args.iters
    print("%s %s: %.2f us/call, %.1f TFLOP/s, %.0f GB/s (algorithmic), status %d"
          % (args.workload, args.layout, us, flops / us / 1e6, nbytes / us / 1e3, status))
    return 0 if status == 0 else 1


if __name__ == "__main__":
    raise SystemExit(main())

"""Whole-tensor and band-wise execution of a layer list on the CPU.  TEST INFRASTRUCTURE ONLY.

Whole-tensor execution is the plain definition: every layer computed over its full
output, one after the other.  Band-wise execution follows Sec. IV-B of the paper: each
band's operations run as soon as their inputs exist, using only the rows the plan says
they depend on; the stitched result must equal whole-tensor execution exactly
("without sacrificing accuracy").  To make a missing dependency visible, every row a
band was not given is filled with +inf before the band runs.
"""
import numpy as np

from . import ops, planner

NO_RESIDUAL = -2
POISON = np.float32(np.inf)


def run_layer(l, src, res, rows, round_bf16, out):
    """Rows ``rows`` of layer ``l`` applied to the full-size tensor ``src`` (residual ``res``) into ``out``."""
    if l.op == 3:                       # depth-wise convolution: a block-wise operator, every channel its own filter
        return ops.dwconv2d(src, l.weight, (l.sh, l.sw), (l.ph, l.pw), (l.dh, l.dw), l.scale, l.shift, res,
                            l.residual_pos if res is not None else 0, l.act, round_bf16, rows, out)
    if l.op == 4:                       # layer normalisation over the channels of a pixel: rows map one to one
        return ops.layernorm(src, l.scale, l.shift, ops.LAYERNORM_EPS, round_bf16, rows, out)
    if l.op == 5:                       # channel concatenation of the main input and the second input
        return ops.concat(src, res, rows, out)
    if l.op == 2:                       # row-wise operator (Sec. IV-A, Eq. 1): rows map one to one
        return ops.linear(src, l.weight, l.scale, l.shift, res, l.residual_pos if res is not None else 0, l.act, round_bf16, rows, out)
    if l.op == 0:
        return ops.conv2d(src, l.weight, (l.sh, l.sw), (l.ph, l.pw), (l.dh, l.dw), l.scale, l.shift,
                          res, l.residual_pos if res is not None else 0, l.act, round_bf16, rows, out)
    return ops.maxpool2d(src, (l.kh, l.kw), (l.sh, l.sw), (l.ph, l.pw), (l.dh, l.dw), rows, out)


def run_whole(layers, x, round_bf16, keep_all=False):
    """Unpartitioned execution.  Returns the last layer's output (or every layer's if keep_all)."""
    outs = []

    def tensor(idx):
        return x if idx == -1 else outs[idx]

    for l in layers:
        res = tensor(l.residual_from) if l.residual_from != NO_RESIDUAL else None
        outs.append(run_layer(l, tensor(l.input_from), res, None, round_bf16, None))
    return outs if keep_all else outs[-1]


def run_banded(layers, x, plan, round_bf16, reuse=False, band_order=None):
    """Band-wise execution according to ``plan``; returns the stitched last-layer output.

    independent mode: each band starts from poisoned tensors, receives only its planned input
    rows and recomputes every intermediate row it needs (the paper's operation replication).
    reuse mode: tensors persist across bands; each band receives and computes only rows no
    earlier band produced (the paper's "only what is missing is transmitted").
    """
    N = x.shape[0]
    L = len(layers)

    def fresh():
        t = {-1: np.full(x.shape, POISON, dtype=np.float32)}
        for i, (h, w, c) in enumerate(plan.shapes):
            t[i] = np.full((N, h, w, c), POISON, dtype=np.float32)
        return t

    stitched = np.full((N,) + tuple(plan.shapes[-1]), POISON, dtype=np.float32)
    order = range(plan.n_bands) if band_order is None else band_order
    if reuse:
        assert band_order is None, "reuse mode needs bands in ascending order"
        t = fresh()
    for b in order:
        if not reuse:
            t = fresh()
        lo, hi, new_lo = plan.input_need[b]
        c0 = new_lo if reuse else lo
        t[-1][:, c0:hi] = x[:, c0:hi]
        for i, l in enumerate(layers):
            r = plan.ranges[b][i]
            r0 = r.new_lo if reuse else r.out_lo
            if r0 >= r.out_hi:
                continue
            res = t[l.residual_from] if l.residual_from != NO_RESIDUAL else None
            run_layer(l, t[l.input_from], res, (r0, r.out_hi), round_bf16, t[i])
        r = plan.ranges[b][L - 1]
        r0 = r.new_lo if reuse else r.out_lo
        stitched[:, r0:r.out_hi] = t[L - 1][:, r0:r.out_hi]
    return stitched


def run_band_block(layers, x, plan, round_bf16, b0, b1, reuse=False):
    """Bands [b0, b1) on a device that runs no other band (the paper's operation replication across devices,
    Sec. IV-C): tensors start poisoned, only the chain-input rows those bands need are present, and -- in reuse mode -- a band computes only the rows the
    block itself has not yet produced (so the block's first band computes every row it needs).  Returns the last layer's output with the block's rows filled in and poison elsewhere."""
    N = x.shape[0]
    L = len(layers)
    t = {-1: np.full(x.shape, POISON, dtype=np.float32)}
    for i, (h, w, c) in enumerate(plan.shapes):
        t[i] = np.full((N, h, w, c), POISON, dtype=np.float32)
    stitched = np.full((N,) + tuple(plan.shapes[-1]), POISON, dtype=np.float32)
    done = [0] * L                                     # rows [.., done) of layer i this block has produced so far
    for b in range(b0, b1):
        lo, hi, _ = plan.input_need[b]
        t[-1][:, lo:hi] = x[:, lo:hi]
        if not reuse and b != b0:                      # independent bands never read another band's rows
            for i in range(L):
                t[i][...] = POISON
        for i, l in enumerate(layers):
            r = plan.ranges[b][i]
            if r.out_lo >= r.out_hi:
                continue
            r0 = min(max(r.out_lo, done[i]), r.out_hi) if reuse else r.out_lo
            done[i] = max(done[i], r.out_hi)
            if r0 >= r.out_hi:
                continue
            res = t[l.residual_from] if l.residual_from != NO_RESIDUAL else None
            run_layer(l, t[l.input_from], res, (r0, r.out_hi), round_bf16, t[i])
        r = plan.ranges[b][L - 1]
        stitched[:, r.out_lo:r.out_hi] = t[L - 1][:, r.out_lo:r.out_hi]
    return stitched


def run_workload(wl, banded=False, reuse=False, keep_segments=False):
    """Run every segment of a workload in order; each segment's output feeds the next."""
    rb = wl.dtype == "bf16"
    x = wl.x
    outs = []
    for seg in wl.segments:
        if banded:
            _, H, W, C = x.shape
            plan = planner.make_plan(seg.layers, H, W, C, seg.n_bands, reuse)
            x = run_banded(seg.layers, x, plan, rb, reuse)
        else:
            x = run_whole(seg.layers, x, rb)
        outs.append(x)
    return outs if keep_segments else x


def flops(wl):
    """2 * multiply-accumulates of the unpartitioned convolutions of a workload."""
    total = 0
    H, W, C = wl.H, wl.W, wl.C
    for seg in wl.segments:
        shapes = planner.infer_shapes(seg.layers, H, W, C)
        for l, (h, w, c) in zip(seg.layers, shapes):
            if l.op in (0, 2):
                total += 2 * wl.N * h * w * c * l.kh * l.kw * l.cin
            elif l.op == 3:
                total += 2 * wl.N * h * w * c * l.kh * l.kw
        H, W, C = shapes[-1]
    return total

"""Integer band planner of the CPU oracle.  TEST INFRASTRUCTURE ONLY.

A segment is a list of local operators (Sec. IV-A) in topological order.  The rows of
its LAST layer's output are cut into ``n_bands`` contiguous intervals (the paper's
contiguous-interval constraint on the operations of one device, Sec. IV-C
"Computational Efficiency", and its rule that every operation is executed, Sec. IV-C
"Data Partitioning").  For each band the planner walks the layers from last to first and
derives which rows of every earlier tensor the band depends on -- the inverse of the
paper's ``child(.)`` relation (Sec. IV-C "Data Dependency"): a dependency exists if any
part of an output is used (Sec. IV-B).

Where the paper is silent the following readings are taken:
  * bands are the floor partition  [i*H/B, (i+1)*H/B)  and may be empty when B > H;
  * output extents use floor rounding only;
  * stride belongs to the block-size parameters although Sec. IV-A lists only kernel
    size, padding and dilation;
  * a range holds only rows that exist and are read (rows in the padding create no
    dependency), and it is narrowed this way at EVERY layer before it is propagated further;
  * only H is split; W and the batch are never split.

All ranges are half-open row intervals (lo, hi); the empty interval is written (0, 0).
"""
from collections import namedtuple

Range = namedtuple("Range", "out_lo out_hi in_lo in_hi pad_top pad_bot new_lo")
EMPTY = (0, 0)
NO_RESIDUAL = -2


class PlanError(ValueError):
    pass


def out_extent(n_in, k, s, p, d):
    """Floor-mode output extent of a window operator."""
    return (n_in + 2 * p - d * (k - 1) - 1) // s + 1


def infer_shapes(layers, H, W, C):
    """(H, W, C) of every layer's output; raises PlanError on an invalid layer list."""
    shapes = []

    def shape_of(idx):
        return (H, W, C) if idx == -1 else shapes[idx]

    for i, l in enumerate(layers):
        if min(l.kh, l.kw, l.sh, l.sw, l.dh, l.dw) < 1 or min(l.ph, l.pw) < 0:
            raise PlanError("layer %d: bad kernel/stride/padding/dilation" % i)
        if not (-1 <= l.input_from < i):
            raise PlanError("layer %d: input_from must name the segment input or an earlier layer" % i)
        hin, win, cin = shape_of(l.input_from)
        if cin != l.cin:
            raise PlanError("layer %d: cin %d but its input has %d channels" % (i, l.cin, cin))
        if l.op == 2 and (l.kh, l.kw, l.sh, l.sw, l.ph, l.pw, l.dh, l.dw) != (1, 1, 1, 1, 0, 0, 1, 1):
            raise PlanError("layer %d: a row-wise operator has no window" % i)
        if l.op in (1, 3, 4) and l.cout != l.cin:
            raise PlanError("layer %d: pooling, depth-wise convolution and layer normalisation keep the channel count" % i)
        if l.op in (4, 5) and (l.kh, l.kw, l.sh, l.sw, l.ph, l.pw, l.dh, l.dw) != (1, 1, 1, 1, 0, 0, 1, 1):
            raise PlanError("layer %d: a per-pixel operator has no window" % i)
        if l.op == 5 and l.residual_from == NO_RESIDUAL:
            raise PlanError("layer %d: a concatenation needs its second input (residual_from)" % i)
        ho = out_extent(hin, l.kh, l.sh, l.ph, l.dh)
        wo = out_extent(win, l.kw, l.sw, l.pw, l.dw)
        if ho <= 0 or wo <= 0:
            raise PlanError("layer %d: empty output" % i)
        if l.residual_from != NO_RESIDUAL:
            if not (-1 <= l.residual_from < i):
                raise PlanError("layer %d: residual_from must name the segment input or an earlier layer" % i)
            if l.op == 5:
                if shape_of(l.residual_from) != (ho, wo, l.cout - l.cin):
                    raise PlanError("layer %d: the second input of a concatenation must bring cout - cin channels" % i)
            else:
                if l.op not in (0, 2, 3) or l.residual_pos not in (1, 2):
                    raise PlanError("layer %d: a residual needs a convolution and a position" % i)
                if shape_of(l.residual_from) != (ho, wo, l.cout):
                    raise PlanError("layer %d: residual shape mismatch" % i)
        shapes.append((ho, wo, l.cout))
    return shapes


def band_partition(h_out, n_bands):
    """Band i covers rows [floor(i*H/B), floor((i+1)*H/B))."""
    return [((i * h_out) // n_bands, ((i + 1) * h_out) // n_bands) for i in range(n_bands)]


def hull(a, b):
    if a[0] >= a[1]:
        return b
    if b[0] >= b[1]:
        return a
    return (min(a[0], b[0]), max(a[1], b[1]))


def input_rows(o0, o1, k, s, p, d, h_in):
    """Rows of the input that output rows [o0, o1) actually read, by enumeration.

    Output row o reads, through tap t = 0..k-1, the row  o*s - p + t*d.  Every (output row, tap)
    pair is visited; a row inside [0, h_in) is a dependency (Sec. IV-B: a dependency exists as
    soon as any part of the producer's output is used), a row outside it lies in the padding,
    is nobody's output and creates none.  The range returned is the smallest interval that
    holds every dependency; pad_top / pad_bot are how far above / below the tensor the taps
    reach.  With d == 1 and p <= k-1 the result is the analytic receptive range
    [o0*s - p, (o1-1)*s - p + (k-1)*d] cut to the tensor.

    Returns (in_lo, in_hi, pad_top, pad_bot).
    """
    read = []
    pad_top = pad_bot = 0
    for o in range(o0, o1):
        for t in range(k):
            r = o * s - p + t * d
            if r < 0:
                pad_top = max(pad_top, -r)
            elif r >= h_in:
                pad_bot = max(pad_bot, r - (h_in - 1))
            else:
                read.append(r)
    if not read:
        return 0, 0, pad_top, pad_bot
    return min(read), max(read) + 1, pad_top, pad_bot


class Plan:
    """ranges[band][layer] -> Range; input_need[band] -> (lo, hi, new_lo) rows of the segment input."""

    def __init__(self, shapes, in_shape, ranges, input_need, n_bands, reuse):
        self.shapes, self.in_shape = shapes, in_shape
        self.ranges, self.input_need = ranges, input_need
        self.n_bands, self.reuse = n_bands, reuse


def make_plan(layers, H, W, C, n_bands, reuse=False):
    if n_bands < 1 or not layers:
        raise PlanError("need at least one band and one layer")
    shapes = infer_shapes(layers, H, W, C)
    L = len(layers)
    bands = band_partition(shapes[-1][0], n_bands)
    ranges, input_need = [], []
    done = {idx: 0 for idx in range(-1, L)}       # rows [.., done) already produced by earlier bands
    for band in bands:
        need = {idx: EMPTY for idx in range(-1, L)}
        need[L - 1] = band if band[0] < band[1] else EMPTY
        rec = [None] * L
        for i in range(L - 1, -1, -1):
            l = layers[i]
            o0, o1 = need[i]
            if o0 >= o1:
                rec[i] = (0, 0, 0, 0, 0, 0)
                continue
            h_in = H if l.input_from == -1 else shapes[l.input_from][0]
            lo, hi, pt, pb = input_rows(o0, o1, l.kh, l.sh, l.ph, l.dh, h_in)
            need[l.input_from] = hull(need[l.input_from], (lo, hi))
            if l.residual_from != NO_RESIDUAL:
                need[l.residual_from] = hull(need[l.residual_from], (o0, o1))
            rec[i] = (o0, o1, lo, hi, pt, pb)
        row = []
        for i in range(L):
            o0, o1 = rec[i][0], rec[i][1]
            new_lo = 0 if o0 >= o1 else min(max(o0, done[i]), o1)
            if o0 < o1:
                done[i] = max(done[i], o1)
            row.append(Range(*rec[i], new_lo))
        ranges.append(row)
        lo, hi = need[-1]
        new_lo = 0 if lo >= hi else min(max(lo, done[-1]), hi)
        if lo < hi:
            done[-1] = max(done[-1], hi)
        input_need.append((lo, hi, new_lo))
    return Plan(shapes, (H, W, C), ranges, input_need, n_bands, reuse)

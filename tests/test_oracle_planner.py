"""Pins for the oracle's band planner: closed form, brute-force touch marking, hand-derived
ranges, invariants, and stitched == whole on the oracle itself."""
import random

import numpy as np
import pytest

import lop_inputs as li
from lop_inputs.workloads import Layer, NO_RESIDUAL
from oracle import chain, planner


def rows_of(r):
    return (r.in_lo, r.in_hi)


# ----------------------------------------------------------------------------- closed form, one layer
def test_single_layer_closed_form():
    rnd = random.Random(5)
    for _ in range(3000):
        k, s, p, d = rnd.randint(1, 7), rnd.randint(1, 3), rnd.randint(0, 3), rnd.randint(1, 3)
        H = rnd.randint(1, 64)
        Ho = (H + 2 * p - d * (k - 1) - 1) // s + 1
        if Ho <= 0:
            continue
        B = rnd.randint(1, Ho + 1)
        l = Layer(0, 1, 1, k, 1, s, 1, p, 0, d, 1, input_from=-1)
        plan = planner.make_plan([l], H, 8, 1, B)
        for i in range(B):
            o0, o1 = (i * Ho) // B, ((i + 1) * Ho) // B
            r = plan.ranges[i][0]
            if o0 == o1:
                assert tuple(r) == (0, 0, 0, 0, 0, 0, 0)
                continue
            a, b = o0 * s - p, (o1 - 1) * s - p + (k - 1) * d           # analytic receptive rows, inclusive
            assert (r.out_lo, r.out_hi) == (o0, o1)
            assert r.pad_top == max(0, -a) and r.pad_bot == max(0, b - (H - 1))
            lo, hi = max(a, 0), min(b, H - 1)
            clamped = (lo, hi + 1) if lo <= hi else (0, 0)
            if d == 1 and p <= k - 1:
                assert rows_of(r) == clamped                 # regular case: the clamped analytic range
            else:                                            # taps skip rows: never wider, at most d-1 / p rows tighter
                assert clamped[0] <= r.in_lo and r.in_hi <= clamped[1]


def per_tap_interval(o0, o1, k, s, p, d, h_in):
    """The same interval from index arithmetic instead of enumeration: for tap t the first output row whose tap is
    not above the tensor is ceil((p - t*d)/s), the last whose tap is not below it is floor((h_in-1 + p - t*d)/s)."""
    lo = hi = None
    for t in range(k):
        first = max(o0, -((t * d - p) // s))
        if first < o1 and first * s - p + t * d < h_in:
            r = first * s - p + t * d
            lo = r if lo is None else min(lo, r)
        last = min(o1 - 1, (h_in - 1 + p - t * d) // s)
        if last >= o0 and last * s - p + t * d >= 0:
            r = last * s - p + t * d
            hi = r if hi is None else max(hi, r)
    return (0, 0) if lo is None or hi is None else (lo, hi + 1)


def test_enumerated_input_rows_equal_the_per_tap_closed_form():
    rnd = random.Random(77)
    for _ in range(20000):
        k, s, p, d = rnd.randint(1, 7), rnd.randint(1, 4), rnd.randint(0, 9), rnd.randint(1, 4)
        h_in = rnd.randint(1, 40)
        ho = (h_in + 2 * p - d * (k - 1) - 1) // s + 1
        if ho <= 0:
            continue
        o0 = rnd.randint(0, ho - 1)
        o1 = rnd.randint(o0 + 1, ho)
        lo, hi, pt, pb = planner.input_rows(o0, o1, k, s, p, d, h_in)
        assert (lo, hi) == per_tap_interval(o0, o1, k, s, p, d, h_in)
        assert pt == max(0, p - o0 * s) and pb == max(0, (o1 - 1) * s - p + (k - 1) * d - (h_in - 1))


# ----------------------------------------------------------------------------- brute-force touch marking
def random_stack(rnd):
    """A random layer list with optional residual edges; all H extents stay positive."""
    while True:
        H = rnd.randint(1, 64)
        L = rnd.randint(1, 5)
        layers, heights = [], [H]
        ok = True
        for i in range(L):
            src = i - 1 if rnd.random() < 0.8 else rnd.randint(-1, i - 1)
            k, s, p, d = rnd.randint(1, 7), rnd.randint(1, 3), rnd.randint(0, 3), rnd.randint(1, 3)
            hin = heights[src + 1]
            ho = (hin + 2 * p - d * (k - 1) - 1) // s + 1
            if ho <= 0:
                ok = False
                break
            op = 0 if rnd.random() < 0.8 else 1
            l = Layer(op, 1, 1, k, 1, s, 1, p, 0, d, 1, input_from=src)
            if op == 0 and rnd.random() < 0.4:
                cands = [j for j in range(-1, i) if heights[j + 1] == ho]
                if cands:
                    l.residual_from, l.residual_pos = rnd.choice(cands), rnd.choice((1, 2))
            layers.append(l)
            heights.append(ho)
        if ok:
            return layers, H


def touch_marking(layers, H, band):
    """Sets of rows, no interval arithmetic: which rows does computing ``band`` of the last layer read?

    Each layer's operations on one device form one contiguous run (Sec. IV-C), so once some
    rows of a layer are wanted, every row between the smallest and largest wanted one is
    computed, and each computed row marks every in-bounds input row one of its taps reads.
    """
    L = len(layers)
    heights = {-1: H}
    for i, l in enumerate(layers):
        heights[i] = (heights[l.input_from] + 2 * l.ph - l.dh * (l.kh - 1) - 1) // l.sh + 1
    wanted = {i: set() for i in range(-1, L)}
    wanted[L - 1] = set(range(band[0], band[1]))
    reads = {}
    for i in range(L - 1, -1, -1):
        if not wanted[i]:
            reads[i] = (set(), set())
            continue
        l = layers[i]
        computed = range(min(wanted[i]), max(wanted[i]) + 1)
        touched, outside = set(), set()
        for o in computed:
            for t in range(l.kh):
                r = o * l.sh - l.ph + t * l.dh
                (touched if 0 <= r < heights[l.input_from] else outside).add(r)
        wanted[l.input_from] |= touched
        if l.residual_from != NO_RESIDUAL:
            wanted[l.residual_from] |= set(computed)
        reads[i] = (touched, outside)
    return wanted, reads, heights


def test_plan_equals_touch_marking_on_random_stacks():
    rnd = random.Random(2024)
    checked = 0
    for _ in range(10000):
        layers, H = random_stack(rnd)
        HL = None
        B = rnd.randint(1, 6)
        plan = planner.make_plan(layers, H, 4, 1, B)
        HL = plan.shapes[-1][0]
        for b in range(B):
            band = ((b * HL) // B, ((b + 1) * HL) // B)
            wanted, reads, heights = touch_marking(layers, H, band)
            for i in range(len(layers)):
                r = plan.ranges[b][i]
                if not wanted[i]:
                    assert (r.out_lo, r.out_hi) == (0, 0)
                    continue
                assert (r.out_lo, r.out_hi) == (min(wanted[i]), max(wanted[i]) + 1)
                touched, outside = reads[i]
                if touched:
                    assert rows_of(r) == (min(touched), max(touched) + 1)
                else:
                    assert rows_of(r) == (0, 0)
                hin = heights[layers[i].input_from]
                assert r.pad_top == max([0] + [-t for t in outside if t < 0])
                assert r.pad_bot == max([0] + [t - (hin - 1) for t in outside if t >= hin])
            lo, hi, _ = plan.input_need[b]
            if wanted[-1]:
                assert (lo, hi) == (min(wanted[-1]), max(wanted[-1]) + 1)
            else:
                assert (lo, hi) == (0, 0)
            checked += 1
    assert checked > 20000


# ----------------------------------------------------------------------------- hand-derived ranges
def test_single_conv_four_bands():
    # 3x3 s1 p1 on 32 rows, bands of 8: rows [8i-1, 8i+8] clamped
    wl = li.build("single_conv", with_data=False)
    plan = planner.make_plan(wl.segments[0].layers, 32, 32, 16, 4)
    assert [rows_of(plan.ranges[b][0]) for b in range(4)] == [(0, 9), (7, 17), (15, 25), (23, 32)]
    assert [plan.ranges[b][0].pad_top for b in range(4)] == [1, 0, 0, 0]
    assert [plan.ranges[b][0].pad_bot for b in range(4)] == [0, 0, 0, 1]
    assert [plan.input_need[b][:2] for b in range(4)] == [(0, 9), (7, 17), (15, 25), (23, 32)]


def clamp(lo, hi_incl, H):
    return (max(lo, 0), min(hi_incl, H - 1) + 1)


def test_vgg_block_eight_bands():
    # pool 2x2 s2 rows [14i,14i+14) <- conv2 rows [28i, 28i+28) <- conv1 rows [28i-1, 28i+29) <- image [28i-2, 28i+30)
    wl = li.build("vgg_block", with_data=False)
    plan = planner.make_plan(wl.segments[0].layers, 224, 224, 3, 8)
    for i in range(8):
        r = plan.ranges[i]
        assert (r[2].out_lo, r[2].out_hi) == (14 * i, 14 * i + 14)
        assert rows_of(r[2]) == (28 * i, 28 * i + 28)
        assert (r[1].out_lo, r[1].out_hi) == (28 * i, 28 * i + 28)
        assert rows_of(r[1]) == clamp(28 * i - 1, 28 * i + 28, 224)
        assert (r[0].out_lo, r[0].out_hi) == clamp(28 * i - 1, 28 * i + 28, 224)
        assert rows_of(r[0]) == clamp(28 * i - 2, 28 * i + 29, 224)
        assert plan.input_need[i][:2] == clamp(28 * i - 2, 28 * i + 29, 224)


def test_resnet_stem_and_stage1():
    wl = li.build("resnet18", with_data=False)
    stem = planner.make_plan(wl.segments[0].layers, 224, 224, 3, 8)
    assert stem.shapes == [(112, 112, 64), (56, 56, 64)]
    for i in range(8):
        r = stem.ranges[i]
        assert (r[1].out_lo, r[1].out_hi) == (7 * i, 7 * i + 7)
        assert rows_of(r[1]) == clamp(14 * i - 1, 14 * i + 13, 112)           # 3x3 s2 p1 pool
        assert rows_of(r[0]) == clamp(28 * i - 5, 28 * i + 29, 224)           # 7x7 s2 p3 stem
    # stage 1: two BasicBlocks of 3x3 s1 p1 convolutions -> four rows of halo on each side
    st1 = planner.make_plan(wl.segments[1].layers, 56, 56, 64, 8)
    for i in range(8):
        assert st1.input_need[i][:2] == clamp(7 * i - 4, 7 * i + 10, 56)
    # stage 2 opens with a 3x3 s2 and a 1x1 s2 projection reading the same input: the hull wins,
    # and the 1x1 s2 alone never reads the last row of a 56-row input
    st2 = planner.make_plan(wl.segments[2].layers, 56, 56, 64, 1)
    assert rows_of(st2.ranges[0][1]) == (0, 55) and rows_of(st2.ranges[0][0]) == (0, 56)
    assert st2.input_need[0][:2] == (0, 56)


def test_csp_stack_one_row_bands():
    wl = li.build("csp_stack", with_data=False)
    plan = planner.make_plan(wl.segments[0].layers, 1024, 1024, 3, 32)
    assert plan.shapes[-1][0] == 32
    for r in (0, 1, 7, 16, 31):
        assert plan.input_need[r][:2] == clamp(32 * r - 59, 32 * r + 59, 1024)
        rr = plan.ranges[r]
        assert (rr[0].out_lo, rr[0].out_hi) == clamp(16 * r - 29, 16 * r + 29, 512)
        assert (rr[1].out_lo, rr[1].out_hi) == clamp(8 * r - 14, 8 * r + 14, 256)
        assert (rr[2].out_lo, rr[2].out_hi) == clamp(8 * r - 14, 8 * r + 14, 256)     # 1x1: same rows as its input
        assert (rr[3].out_lo, rr[3].out_hi) == clamp(8 * r - 13, 8 * r + 13, 256)
        assert (rr[4].out_lo, rr[4].out_hi) == clamp(4 * r - 6, 4 * r + 6, 128)
        assert (rr[5].out_lo, rr[5].out_hi) == clamp(4 * r - 6, 4 * r + 6, 128)
        assert (rr[6].out_lo, rr[6].out_hi) == clamp(4 * r - 5, 4 * r + 5, 128)
        assert (rr[7].out_lo, rr[7].out_hi) == clamp(2 * r - 2, 2 * r + 2, 64)
        assert (rr[8].out_lo, rr[8].out_hi) == clamp(2 * r - 2, 2 * r + 2, 64)
        assert (rr[9].out_lo, rr[9].out_hi) == clamp(2 * r - 1, 2 * r + 1, 64)
        assert (rr[10].out_lo, rr[10].out_hi) == (r, r + 1) == (rr[11].out_lo, rr[11].out_hi)


# ----------------------------------------------------------------------------- invariants
@pytest.mark.parametrize("name,kw", [("vgg_block", dict(H=40, W=8)), ("resnet18", dict(H=64, W=8, width=8)),
                                     ("resnet50", dict(H=64, W=8, width=8, N=1)), ("csp_stack", dict(H=256, W=32)),
                                     ("convnext_block", dict(H=23, W=8, C=8)), ("dense_layer", dict(H=14, W=6, C=8, growth=4))])
def test_invariants(name, kw):
    wl = li.build(name, with_data=False, **kw)
    H, W, C = wl.H, wl.W, wl.C
    for seg in wl.segments:
        shapes = planner.infer_shapes(seg.layers, H, W, C)
        HL = shapes[-1][0]
        full = planner.make_plan(seg.layers, H, W, C, 1)
        for B in (1, 2, 3, HL, HL + 1):
            plan = planner.make_plan(seg.layers, H, W, C, B)
            last = [plan.ranges[b][-1] for b in range(B)]
            pos = 0
            for r in last:                                   # bands tile [0, HL): no gap, no overlap
                if r.out_lo < r.out_hi:
                    assert r.out_lo == pos
                    pos = r.out_hi
            assert pos == HL
            for i in range(len(seg.layers)):                 # ranges move monotonically with the band
                lo = hi = 0
                for b in range(B):
                    r = plan.ranges[b][i]
                    if r.out_lo < r.out_hi:
                        assert r.out_lo >= lo and r.out_hi >= hi
                        lo, hi = r.out_lo, r.out_hi
                        assert r.out_lo <= r.new_lo <= r.out_hi
            # the union of what the bands read from the segment input is what one band reads
            need = [plan.input_need[b][:2] for b in range(B) if plan.input_need[b][0] < plan.input_need[b][1]]
            assert min(n[0] for n in need) == full.input_need[0][0]
            assert max(n[1] for n in need) == full.input_need[0][1]
            # rows newly fetched by each band are disjoint and add up to that union
            new = sum(hi - nl for (lo, hi, nl) in plan.input_need if lo < hi)
            assert new <= full.input_need[0][1] - full.input_need[0][0]
        for i, r in enumerate(full.ranges[0]):               # one band: every used layer is computed in full
            if r.out_lo < r.out_hi:
                assert (r.out_lo, r.out_hi) == (0, shapes[i][0])
        H, W, C = shapes[-1]


def test_invalid_layer_lists_are_rejected():
    good = Layer(0, 4, 4, 3, 3, 1, 1, 1, 1, 1, 1, input_from=-1)
    for field, val in (("kh", 0), ("sh", 0), ("dh", 0), ("ph", -1), ("cin", 5), ("input_from", 0), ("input_from", 3)):
        bad = Layer(**{**good.__dict__, field: val})
        with pytest.raises(planner.PlanError):
            planner.make_plan([bad], 8, 8, 4, 2)
    with pytest.raises(planner.PlanError):                   # kernel larger than the padded input
        planner.make_plan([Layer(0, 4, 4, 7, 7, 1, 1, 0, 0, 1, 1, input_from=-1)], 5, 5, 4, 1)
    with pytest.raises(planner.PlanError):                   # residual of another shape
        planner.make_plan([Layer(0, 4, 4, 3, 3, 2, 2, 1, 1, 1, 1, input_from=-1, residual_from=-1, residual_pos=1)],
                          8, 8, 4, 1)
    with pytest.raises(planner.PlanError):
        planner.make_plan([good], 8, 8, 4, 0)


# ----------------------------------------------------------------------------- stitched == whole
SMALL = [("single_conv", dict(H=13, W=6, C=4)), ("vgg_block", dict(H=22, W=10, width=8)),
         ("resnet18", dict(H=48, W=16, width=8)), ("resnet50", dict(N=2, H=40, W=16, width=4, depths=(2, 1, 2, 1))),
         ("csp_stack", dict(H=96, W=32, base=4)), ("pointwise_mlp", dict(H=9, W=7, C=8, hidden=24)),
         ("convnext_block", dict(H=17, W=9, C=8)), ("dense_layer", dict(H=11, W=6, C=8, growth=4))]


@pytest.mark.parametrize("name,kw", SMALL)
@pytest.mark.parametrize("reuse", [False, True])
def test_stitched_bands_equal_whole_tensor_execution(name, kw, reuse):
    wl = li.build(name, **kw)
    rb = wl.dtype == "bf16"
    x = wl.x
    for seg in wl.segments:
        whole = chain.run_whole(seg.layers, x, rb)
        HL = whole.shape[1]
        for B in (1, 2, 3, HL, HL + 1):
            plan = planner.make_plan(seg.layers, x.shape[1], x.shape[2], x.shape[3], B, reuse)
            got = chain.run_banded(seg.layers, x, plan, rb, reuse)
            assert np.array_equal(got, whole), (name, B, reuse)
        if not reuse:                                          # independent bands run in any order
            plan = planner.make_plan(seg.layers, x.shape[1], x.shape[2], x.shape[3], 3)
            assert np.array_equal(chain.run_banded(seg.layers, x, plan, rb, False, band_order=[2, 0, 1]), whole)
        x = whole
    assert np.all(np.isfinite(x))


@pytest.mark.parametrize("name,kw", SMALL)
@pytest.mark.parametrize("reuse", [False, True])
def test_band_blocks_on_separate_devices_tile_the_whole_output(name, kw, reuse):
    """A block of bands run alone (poisoned tensors, only its own input rows) gives exactly its rows of the
    whole-tensor result, whichever way the bands are dealt out to 1, 2, 3 or more devices."""
    wl = li.build(name, **kw)
    rb = wl.dtype == "bf16"
    x = wl.x
    for seg in wl.segments:
        whole = chain.run_whole(seg.layers, x, rb)
        for B in (min(6, whole.shape[1] + 1), 2 * whole.shape[1] + 3):       # the second: most bands are empty
            plan = planner.make_plan(seg.layers, x.shape[1], x.shape[2], x.shape[3], B, reuse)
            for world in (1, 2, 3, B + 1):
                seen = np.zeros(whole.shape[1], dtype=bool)
                for rank in range(world):
                    b0, b1 = rank * B // world, (rank + 1) * B // world
                    got = chain.run_band_block(seg.layers, x, plan, rb, b0, b1, reuse)
                    rows = np.isfinite(got).all(axis=(0, 2, 3))
                    assert not (rows & seen).any()
                    assert np.array_equal(got[:, rows], whole[:, rows]), (name, B, world, rank, reuse)
                    seen |= rows
                assert seen.all()
        x = whole


def test_a_plan_one_row_short_is_caught():
    """Planting a mistake in the plan (one halo row dropped) must break stitched == whole."""
    wl = li.build("vgg_block", H=22, W=10, width=8)
    seg = wl.segments[0]
    whole = chain.run_whole(seg.layers, wl.x, True)
    plan = planner.make_plan(seg.layers, 22, 10, 3, 3)
    lo, hi, nl = plan.input_need[1]
    plan.input_need[1] = (lo + 1, hi, nl)
    assert not np.array_equal(chain.run_banded(seg.layers, wl.x, plan, True), whole)
    plan = planner.make_plan(seg.layers, 22, 10, 3, 3)
    r = plan.ranges[0][0]
    plan.ranges[0][0] = r._replace(out_hi=r.out_hi - 1)
    assert not np.array_equal(chain.run_banded(seg.layers, wl.x, plan, True), whole)


def test_flops_of_the_named_workloads():
    assert chain.flops(li.build("single_conv", with_data=False)) == 2 * 32 * 32 * 16 * 144
    v = chain.flops(li.build("vgg_block", with_data=False))
    assert v == 2 * 224 * 224 * 64 * (27 + 576)


def test_row_wise_operators_need_no_halo():
    """Sec. IV-A, Eq. 1: a block of output rows of a row-wise operator depends on the same rows of its input."""
    wl = li.build("pointwise_mlp", with_data=False)
    seg = wl.segments[0]
    plan = planner.make_plan(seg.layers, wl.H, wl.W, wl.C, seg.n_bands)
    for b in range(seg.n_bands):
        band = ((b * wl.H) // seg.n_bands, ((b + 1) * wl.H) // seg.n_bands)
        for i in range(len(seg.layers)):
            r = plan.ranges[b][i]
            assert (r.out_lo, r.out_hi) == band and rows_of(r) == band and r.pad_top == 0 and r.pad_bot == 0
        assert plan.input_need[b][:2] == band
    bad = li.linear(8, 8)
    bad.input_from, bad.kh = -1, 3
    with pytest.raises(planner.PlanError):
        planner.make_plan([bad], 8, 8, 8, 2)


def test_convnext_block_and_dense_layer_ranges():
    """Depth-wise 7x7: three rows of halo at the block's first layer, none behind it; concatenation: both inputs 1:1."""
    wl = li.build("convnext_block", with_data=False)
    seg = wl.segments[0]
    plan = planner.make_plan(seg.layers, wl.H, wl.W, wl.C, seg.n_bands)
    for b in range(seg.n_bands):
        lo, hi = (b * wl.H) // seg.n_bands, ((b + 1) * wl.H) // seg.n_bands
        assert rows_of(plan.ranges[b][0]) == clamp(lo - 3, hi + 2, wl.H)
        for i in (1, 2, 3):
            assert rows_of(plan.ranges[b][i]) == (lo, hi)
        assert plan.input_need[b][:2] == clamp(lo - 3, hi + 2, wl.H)      # hull of the halo and the shortcut's own rows
    wl = li.build("dense_layer", with_data=False)
    seg = wl.segments[0]
    plan = planner.make_plan(seg.layers, wl.H, wl.W, wl.C, seg.n_bands)
    assert plan.shapes[-1] == (wl.H, wl.W, wl.C + 32)
    for b in range(seg.n_bands):
        lo, hi = (b * wl.H) // seg.n_bands, ((b + 1) * wl.H) // seg.n_bands
        assert (plan.ranges[b][2].out_lo, plan.ranges[b][2].out_hi) == (lo, hi)
        assert (plan.ranges[b][1].out_lo, plan.ranges[b][1].out_hi) == (lo, hi)       # the concatenation's second input
        assert plan.input_need[b][:2] == clamp(lo - 1, hi, wl.H)                      # 3x3 halo through the 1x1
    bad = li.concat(8, 4, input_from=-1)
    with pytest.raises(planner.PlanError):
        planner.make_plan([bad], 8, 8, 8, 2)

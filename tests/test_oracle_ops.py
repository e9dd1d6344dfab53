"""Pins for the oracle's operators: closed forms, brute force, library special cases."""
import math

import numpy as np
import pytest
import torch
import torch.nn.functional as F

import lop_inputs as li
from oracle import ops


def rnd(shape, seed, stream=0):
    return li.uniform(seed, stream, shape, -1.0, 1.0)


# ----------------------------------------------------------------------------- bf16 rounding
def test_bf16_rne_fixed_points_all_patterns():
    bits = np.arange(65536, dtype=np.uint16)
    vals = li.from_bf16_bits(bits)
    for v in vals[::37]:                       # every pattern is slow through ctypes; stride + edges below
        if math.isnan(v):
            continue
        assert ops.bf16_rne(float(v)) == v
    for b in (0x0000, 0x8000, 0x0001, 0x7F7F, 0xFF7F, 0x7F80, 0xFF80, 0x3F80):
        v = float(li.from_bf16_bits(np.array([b], dtype=np.uint16))[0])
        r = ops.bf16_rne(v)
        assert r == v and math.copysign(1, r) == math.copysign(1, v)


def test_bf16_rne_ties_to_even():
    u = 2.0 ** -7                                            # bf16 ulp at 1.0
    assert ops.bf16_rne(1.0 + u / 2) == 1.0                   # tie -> even mantissa (0)
    assert ops.bf16_rne(1.0 + 3 * u / 2) == 1.0 + 2 * u       # tie -> even mantissa (2)
    assert ops.bf16_rne(1.0 + u / 2 + 2.0 ** -20) == 1.0 + u  # just above the tie
    assert ops.bf16_rne(1.0 + u / 2 - 2.0 ** -20) == 1.0      # just below
    assert ops.bf16_rne(-(1.0 + u / 2)) == -1.0
    assert ops.bf16_rne(-(1.0 + 3 * u / 2)) == -(1.0 + 2 * u)
    big = float(li.from_bf16_bits(np.array([0x7F7F], dtype=np.uint16))[0])   # largest finite bf16
    f32 = lambda bits: float(np.array([bits], dtype=np.uint32).view(np.float32)[0])
    assert ops.bf16_rne(f32(0x7F7F7FFF)) == big                # below the midpoint to infinity
    assert ops.bf16_rne(f32(0x7F7F8000)) == math.inf           # the midpoint: odd mantissa rounds up
    assert math.isnan(ops.bf16_rne(math.nan))


def test_bf16_rne_matches_library_conversion():
    x = np.concatenate([li.normal(7, 0, (20000,), 0, 1), li.normal(7, 1, (2000,), 0, 1e-30),
                        li.normal(7, 2, (2000,), 0, 1e30)]).astype(np.float32)
    want = torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy()
    got = np.array([ops.bf16_rne(float(v)) for v in x], dtype=np.float32)
    assert np.array_equal(got, want)
    assert np.array_equal(li.round_to_bf16(x), want)          # the generator's own rounding


# ----------------------------------------------------------------------------- convolution closed forms
def test_conv_identity_kernel_returns_input():
    x = rnd((2, 9, 7, 5), 1)
    w = np.zeros((5, 3, 3, 5), np.float32)
    for c in range(5):
        w[c, 1, 1, c] = 1.0
    assert np.array_equal(ops.conv2d(x, w, pad=(1, 1)), x)


@pytest.mark.parametrize("a,b", [(0, 0), (0, 2), (2, 1), (1, 0)])
def test_conv_shifted_delta_shifts_input_with_zero_border(a, b):
    x = rnd((1, 8, 6, 3), 2)
    w = np.zeros((3, 3, 3, 3), np.float32)
    for c in range(3):
        w[c, a, b, c] = 1.0
    y = ops.conv2d(x, w, pad=(1, 1))
    want = np.zeros_like(x)
    for oh in range(8):
        for ow in range(6):
            ih, iw = oh - 1 + a, ow - 1 + b
            if 0 <= ih < 8 and 0 <= iw < 6:
                want[0, oh, ow] = x[0, ih, iw]
    assert np.array_equal(y, want)


def test_conv_all_ones_counts_in_bounds_taps():
    cin = 4
    x = np.ones((1, 6, 5, cin), np.float32)
    w = np.ones((2, 3, 3, cin), np.float32)
    y = ops.conv2d(x, w, pad=(1, 1))
    assert y[0, 2, 2, 0] == 9 * cin and y[0, 0, 2, 1] == 6 * cin and y[0, 0, 0, 0] == 4 * cin
    assert y[0, 5, 4, 1] == 4 * cin and y[0, 3, 4, 0] == 6 * cin
    # dilation 2, pad 2: the corner sees taps (1..2, 1..2) -> 4, the centre of a 6x5 image fewer than 9
    y = ops.conv2d(x, w, pad=(2, 2), dil=(2, 2))
    assert y.shape == (1, 6, 5, 2) and y[0, 0, 0, 0] == 4 * cin and y[0, 2, 2, 0] == 9 * cin
    assert y[0, 1, 2, 0] == 6 * cin      # rows -1(out),1,3 -> 2 rows; cols 0,2,4 -> 3


def test_conv_linearity():
    x1, x2 = rnd((1, 7, 7, 3), 3), rnd((1, 7, 7, 3), 4)
    w1, w2 = rnd((4, 3, 3, 3), 5), rnd((4, 3, 3, 3), 6)
    kw = dict(stride=(2, 1), pad=(1, 2), dil=(1, 2))
    a = ops.conv2d(x1 + x2, w1, **kw)
    b = ops.conv2d(x1, w1, **kw) + ops.conv2d(x2, w1, **kw)
    assert np.allclose(a, b, atol=1e-5)
    a = ops.conv2d(x1, w1 + w2, **kw)
    b = ops.conv2d(x1, w1, **kw) + ops.conv2d(x1, w2, **kw)
    assert np.allclose(a, b, atol=1e-5)
    assert np.allclose(ops.conv2d(2.5 * x1, w1, **kw), 2.5 * ops.conv2d(x1, w1, **kw), atol=1e-5)


def test_conv_1x1_is_a_per_pixel_matrix_product():
    x = rnd((2, 5, 4, 6), 8)
    w = rnd((7, 1, 1, 6), 9)
    y = ops.conv2d(x, w)
    want = (x.reshape(-1, 6).astype(np.float64) @ w.reshape(7, 6).astype(np.float64).T).reshape(2, 5, 4, 7)
    assert np.allclose(y, want.astype(np.float32), rtol=0, atol=1e-6)
    ys = ops.conv2d(x, w, stride=(2, 2))                       # stride 2 just subsamples the pixels
    assert np.array_equal(ys, y[:, ::2, ::2])


def naive_conv_nchw(x, w, s, p, d):
    """A second, separately written definition: NCHW, gather the window, then dot."""
    N, H, W, C = x.shape
    K, kh, kw, _ = w.shape
    xc = np.transpose(x, (0, 3, 1, 2)).astype(np.float64)
    wc = np.transpose(w, (0, 3, 1, 2)).astype(np.float64)
    Ho = (H + 2 * p[0] - d[0] * (kh - 1) - 1) // s[0] + 1
    Wo = (W + 2 * p[1] - d[1] * (kw - 1) - 1) // s[1] + 1
    xp = np.zeros((N, C, H + 2 * p[0], W + 2 * p[1]))
    xp[:, :, p[0]:p[0] + H, p[1]:p[1] + W] = xc
    y = np.zeros((N, K, Ho, Wo))
    for n in range(N):
        for k in range(K):
            for i in range(Ho):
                for j in range(Wo):
                    win = xp[n, :, i * s[0]:i * s[0] + d[0] * (kh - 1) + 1:d[0],
                             j * s[1]:j * s[1] + d[1] * (kw - 1) + 1:d[1]]
                    y[n, k, i, j] = np.sum(win * wc[k])
    return np.transpose(y, (0, 2, 3, 1))


CASES = [  # H, W, cin, cout, k, s, p, d
    (6, 7, 3, 4, (3, 3), (1, 1), (1, 1), (1, 1)),
    (9, 8, 2, 3, (3, 2), (2, 1), (0, 1), (1, 2)),
    (11, 5, 4, 2, (5, 3), (3, 2), (2, 0), (2, 1)),
    (7, 7, 1, 1, (7, 7), (2, 2), (3, 3), (1, 1)),
    (5, 9, 3, 5, (1, 1), (2, 3), (0, 0), (1, 1)),
    (4, 4, 2, 2, (3, 3), (1, 1), (3, 3), (3, 3)),
]


@pytest.mark.parametrize("case", CASES)
def test_conv_matches_naive_nchw_and_library(case):
    H, W, cin, cout, k, s, p, d = case
    x = rnd((2, H, W, cin), 11 + H)
    w = rnd((cout, k[0], k[1], cin), 12 + W)
    y = ops.conv2d(x, w, s, p, d)
    assert np.allclose(y, naive_conv_nchw(x, w, s, p, d), rtol=0, atol=1e-6)
    t = F.conv2d(torch.from_numpy(x).permute(0, 3, 1, 2), torch.from_numpy(w).permute(0, 3, 1, 2),
                 stride=s, padding=p, dilation=d).permute(0, 2, 3, 1).numpy()
    assert np.allclose(y, t, rtol=0, atol=1e-5)


# ----------------------------------------------------------------------------- epilogue
def test_epilogue_order_and_activations():
    x, w = rnd((1, 6, 6, 3), 21), rnd((4, 3, 3, 3), 22)
    scale, shift = li.normal(23, 0, (4,), 1, 0.1), li.normal(23, 1, (4,), 0, 0.1)
    raw = ops.conv2d(x, w, pad=(1, 1))
    res = rnd(raw.shape, 24)
    lin = (scale * raw + shift).astype(np.float32)
    relu = lambda t: np.maximum(t, 0)
    silu = lambda t: (t / (1 + np.exp(-t.astype(np.float64)))).astype(np.float32)
    kw = dict(pad=(1, 1), scale=scale, shift=shift)
    assert np.array_equal(ops.conv2d(x, w, pad=(1, 1), scale=None, shift=None), raw)
    assert np.allclose(ops.conv2d(x, w, **kw), lin, atol=1e-6)
    assert np.allclose(ops.conv2d(x, w, act=1, **kw), relu(lin), atol=1e-6)
    assert np.allclose(ops.conv2d(x, w, act=2, **kw), silu(lin), atol=1e-6)
    assert np.allclose(ops.conv2d(x, w, act=1, res=res, res_pos=1, **kw), relu(lin + res), atol=1e-6)
    assert np.allclose(ops.conv2d(x, w, act=1, res=res, res_pos=2, **kw), relu(lin) + res, atol=1e-6)
    assert np.allclose(ops.conv2d(x, w, act=2, res=res, res_pos=2, **kw), silu(lin) + res, atol=1e-6)
    # pre- and post-activation placement differ wherever lin + res changes sign
    assert not np.allclose(relu(lin + res), relu(lin) + res)
    # scalar identities of SiLU: silu(0)=0, silu(t) - silu(-t) = t
    z = ops.conv2d(np.zeros((1, 1, 1, 1), np.float32), np.ones((1, 1, 1, 1), np.float32), act=2)
    assert z[0, 0, 0, 0] == 0
    one = np.ones((1, 1, 1, 1), np.float32)
    for t in (0.5, 2.0, 7.0):
        a = ops.conv2d(one * t, one, act=2)[0, 0, 0, 0]
        b = ops.conv2d(one * -t, one, act=2)[0, 0, 0, 0]
        assert abs((a - b) - t) < 1e-6


def test_bf16_path_rounds_stored_outputs():
    x, w = li.round_to_bf16(rnd((1, 6, 6, 8), 31)), li.round_to_bf16(rnd((4, 3, 3, 8), 32))
    full = ops.conv2d(x, w, pad=(1, 1))
    r = ops.conv2d(x, w, pad=(1, 1), round_bf16=True)
    assert np.array_equal(r, li.round_to_bf16(full))
    assert not np.array_equal(r, full)


def test_rows_argument_computes_exactly_those_rows():
    x, w = rnd((2, 10, 6, 3), 41), rnd((4, 3, 3, 3), 42)
    whole = ops.conv2d(x, w, stride=(2, 1), pad=(1, 1))
    out = np.full_like(whole, 123.0)
    ops.conv2d(x, w, stride=(2, 1), pad=(1, 1), rows=(1, 3), out=out)
    assert np.array_equal(out[:, 1:3], whole[:, 1:3])
    assert np.all(out[:, :1] == 123.0) and np.all(out[:, 3:] == 123.0)
    pw = ops.maxpool2d(x, (3, 3), (2, 2), (1, 1))
    po = np.full_like(pw, 123.0)
    ops.maxpool2d(x, (3, 3), (2, 2), (1, 1), rows=(2, 5), out=po)
    assert np.array_equal(po[:, 2:5], pw[:, 2:5]) and np.all(po[:, :2] == 123.0)


# ----------------------------------------------------------------------------- max pooling
def test_pool_ramp_closed_form():
    H, W = 9, 8
    x = (np.arange(H)[:, None] * W + np.arange(W)[None, :]).astype(np.float32).reshape(1, H, W, 1)
    for k, s, p in ((2, 2, 0), (3, 2, 1), (3, 1, 1), (2, 3, 1)):
        y = ops.maxpool2d(x, (k, k), (s, s), (p, p))
        Ho, Wo = (H + 2 * p - k) // s + 1, (W + 2 * p - k) // s + 1
        assert y.shape == (1, Ho, Wo, 1)
        for i in range(Ho):
            for j in range(Wo):
                ih, iw = min(i * s - p + k - 1, H - 1), min(j * s - p + k - 1, W - 1)   # last in-bounds tap
                assert y[0, i, j, 0] == ih * W + iw


def test_pool_constant_and_negative_inputs_ignore_padding():
    x = np.full((1, 5, 5, 2), -3.5, np.float32)
    y = ops.maxpool2d(x, (3, 3), (2, 2), (1, 1))
    assert np.all(y == -3.5)                    # zero padding would have produced 0 at the border


@pytest.mark.parametrize("k,s,p,d", [((2, 2), (2, 2), (0, 0), (1, 1)), ((3, 3), (2, 2), (1, 1), (1, 1)),
                                     ((3, 2), (1, 2), (1, 0), (2, 1)), ((5, 5), (3, 3), (2, 2), (1, 1))])
def test_pool_matches_naive_and_library(k, s, p, d):
    x = rnd((2, 11, 9, 3), 51)
    y = ops.maxpool2d(x, k, s, p, d)
    N, H, W, C = x.shape
    want = np.full(y.shape, -np.inf, np.float32)
    for i in range(y.shape[1]):
        for j in range(y.shape[2]):
            for a in range(k[0]):
                for b in range(k[1]):
                    ih, iw = i * s[0] - p[0] + a * d[0], j * s[1] - p[1] + b * d[1]
                    if 0 <= ih < H and 0 <= iw < W:
                        want[:, i, j] = np.maximum(want[:, i, j], x[:, ih, iw])
    assert np.array_equal(y, want)
    t = F.max_pool2d(torch.from_numpy(x).permute(0, 3, 1, 2), k, s, p, d).permute(0, 2, 3, 1).numpy()
    assert np.array_equal(y, t)


# ----------------------------------------------------------------------------- row-wise operator (Sec. IV-A, Eq. 1)
def test_linear_equals_a_float64_matrix_product():
    rnd = np.random.default_rng(21)
    x = rnd.standard_normal((2, 5, 7, 19)).astype(np.float32)
    w = rnd.standard_normal((11, 19)).astype(np.float32)
    y = ops.linear(x, w)
    want = (x.reshape(-1, 19).astype(np.float64) @ w.astype(np.float64).T).reshape(2, 5, 7, 11)
    assert np.max(np.abs(y - want)) <= 1e-6 * np.max(np.abs(want))


def test_linear_with_the_identity_matrix_returns_its_input_and_transposition_matters():
    rnd = np.random.default_rng(22)
    x = rnd.standard_normal((1, 3, 4, 6)).astype(np.float32)
    assert np.array_equal(ops.linear(x, np.eye(6, dtype=np.float32)), x)
    w = np.zeros((6, 6), dtype=np.float32)
    w[2, 5] = 1.0                                    # output channel 2 reads input channel 5 (W is [cout][cin])
    y = ops.linear(x, w)
    assert np.array_equal(y[..., 2], x[..., 5]) and not y[..., [0, 1, 3, 4, 5]].any()


def test_linear_row_blocks_computed_apart_stack_to_the_whole():
    """Eq. 1: the rows of X may be partitioned freely, the parameter matrix is shared, nothing is summed across blocks."""
    rnd = np.random.default_rng(23)
    x = rnd.standard_normal((2, 9, 5, 8)).astype(np.float32)
    w = rnd.standard_normal((4, 8)).astype(np.float32)
    sc, sh = rnd.standard_normal(4).astype(np.float32), rnd.standard_normal(4).astype(np.float32)
    whole = ops.linear(x, w, sc, sh, act=2)
    parts = np.full_like(whole, np.inf)
    for lo, hi in ((0, 2), (2, 3), (3, 9)):
        ops.linear(x, w, sc, sh, act=2, rows=(lo, hi), out=parts)
        assert np.all(np.isinf(parts[:, hi:]))       # rows outside the block are left alone
    assert np.array_equal(parts, whole)


def test_linear_is_the_pointwise_convolution_and_shares_its_epilogue():
    rnd = np.random.default_rng(24)
    x = rnd.standard_normal((2, 4, 6, 10)).astype(np.float32)
    w = rnd.standard_normal((7, 10)).astype(np.float32)
    sc, sh = rnd.standard_normal(7).astype(np.float32), rnd.standard_normal(7).astype(np.float32)
    res = rnd.standard_normal((2, 4, 6, 7)).astype(np.float32)
    for pos in (1, 2):
        a = ops.linear(x, w, sc, sh, res, pos, act=1, round_bf16=True)
        b = ops.conv2d(x, w.reshape(7, 1, 1, 10), scale=sc, shift=sh, res=res, res_pos=pos, act=1, round_bf16=True)
        assert np.array_equal(a, b)
    lin = ops.linear(x, w)                           # linear in x
    assert np.allclose(ops.linear(2.0 * x, w), 2.0 * lin, rtol=1e-6, atol=1e-6)


# ----------------------------------------------------------------------------- depth-wise conv, layer norm, concat, GELU
def test_depthwise_convolution_is_the_convolution_with_block_diagonal_weights():
    rnd = np.random.default_rng(31)
    for k, s_, p, d in ((7, 1, 3, 1), (3, 2, 1, 1), (3, 1, 2, 2)):
        x = rnd.standard_normal((2, 11, 9, 5)).astype(np.float32)
        w = rnd.standard_normal((5, k, k)).astype(np.float32)
        full = np.zeros((5, k, k, 5), dtype=np.float32)
        for c in range(5):
            full[c, :, :, c] = w[c]
        sc, sh = rnd.standard_normal(5).astype(np.float32), rnd.standard_normal(5).astype(np.float32)
        a = ops.dwconv2d(x, w, (s_, s_), (p, p), (d, d), sc, sh, act=1)
        b = ops.conv2d(x, full, (s_, s_), (p, p), (d, d), sc, sh, act=1)
        assert a.shape == b.shape and np.max(np.abs(a - b)) <= 1e-6 * max(1.0, np.max(np.abs(b)))
    delta = np.zeros((5, 3, 3), dtype=np.float32)
    delta[:, 1, 1] = 1.0
    x = rnd.standard_normal((1, 6, 7, 5)).astype(np.float32)
    assert np.array_equal(ops.dwconv2d(x, delta, pad=(1, 1)), x)          # the centre tap alone returns the input


def test_depthwise_convolution_matches_the_grouped_library_convolution():
    import torch
    import torch.nn.functional as F
    rnd = np.random.default_rng(32)
    x = rnd.standard_normal((2, 12, 10, 6)).astype(np.float32)
    w = rnd.standard_normal((6, 7, 7)).astype(np.float32)
    got = ops.dwconv2d(x, w, pad=(3, 3))
    want = F.conv2d(torch.from_numpy(x).permute(0, 3, 1, 2).double(), torch.from_numpy(w).unsqueeze(1).double(), padding=3, groups=6)
    assert np.max(np.abs(got - want.permute(0, 2, 3, 1).numpy())) <= 1e-5


def test_layernorm_rows_have_zero_mean_unit_variance_and_ignore_shift_and_scale_of_their_input():
    import torch
    import torch.nn.functional as F
    rnd = np.random.default_rng(33)
    x = (3.0 * rnd.standard_normal((2, 4, 5, 32)) + 7.0).astype(np.float32)
    y = ops.layernorm(x)
    assert np.max(np.abs(y.mean(axis=-1))) < 1e-5 and np.max(np.abs(y.var(axis=-1) - 1.0)) < 1e-4
    y2 = ops.layernorm((5.0 * x - 2.0).astype(np.float32))             # an affine map of the row changes nothing
    assert np.max(np.abs(y2 - y)) < 1e-4
    g, b = rnd.standard_normal(32).astype(np.float32), rnd.standard_normal(32).astype(np.float32)
    want = F.layer_norm(torch.from_numpy(x).double(), (32,), torch.from_numpy(g).double(), torch.from_numpy(b).double(), eps=1e-6).numpy()
    assert np.max(np.abs(ops.layernorm(x, g, b) - want)) < 1e-5
    const = np.full((1, 2, 2, 8), 3.5, dtype=np.float32)
    assert np.allclose(ops.layernorm(const, None, b[:8]), b[:8], atol=1e-6)    # no spread: only beta is left
    part = np.full_like(y, np.inf)
    ops.layernorm(x, rows=(1, 3), out=part)
    assert np.array_equal(part[:, 1:3], y[:, 1:3]) and np.all(np.isinf(part[:, :1])) and np.all(np.isinf(part[:, 3:]))


def test_concat_puts_the_main_input_first():
    rnd = np.random.default_rng(34)
    a, b = rnd.standard_normal((2, 3, 4, 5)).astype(np.float32), rnd.standard_normal((2, 3, 4, 2)).astype(np.float32)
    y = ops.concat(a, b)
    assert y.shape == (2, 3, 4, 7) and np.array_equal(y[..., :5], a) and np.array_equal(y[..., 5:], b)
    part = np.full_like(y, np.inf)
    ops.concat(a, b, rows=(2, 3), out=part)
    assert np.array_equal(part[:, 2:3], y[:, 2:3]) and np.all(np.isinf(part[:, :2]))


def test_gelu_identities():
    import math
    x = np.linspace(-6, 6, 97, dtype=np.float32).reshape(1, 1, 97, 1)
    w = np.ones((1, 1, 1, 1), dtype=np.float32)
    g = ops.conv2d(x, w, act=3).reshape(-1)
    gm = ops.conv2d(-x, w, act=3).reshape(-1)
    xs = x.reshape(-1)
    assert np.max(np.abs((g - gm) - xs)) < 1e-6                         # x Phi(x) + x Phi(-x) = x
    assert abs(g[48]) == 0.0 and abs(g[-1] - 6.0) < 1e-6 and abs(gm[-1]) < 1e-6
    one = ops.conv2d(np.ones((1, 1, 1, 1), dtype=np.float32), w, act=3)[0, 0, 0, 0]
    assert abs(one - 0.5 * (1.0 + math.erf(1.0 / math.sqrt(2.0)))) < 1e-7     # Phi(1) = 0.8413447...
    assert abs(one - 0.8413447) < 1e-6

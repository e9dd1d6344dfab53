"""Layer lists and seeded tensors for the five workload families.

The paper evaluates torchvision VGGNet / ResNet / ConvNeXt / DenseNet and two robot
applications with trained weights (Sec. V-B "Task").  None of those weights or data
are available, so every workload here takes only the *shapes* of such models and
fills them with seeded random tensors:

  weights  ~ N(0, 2 / (kh*kw*cin))      (He initialisation)
  scale    ~ N(1, 0.1), shift ~ N(0, 0.1)   (a folded batch-norm), fp32
  input    ~ U[-1, 1]  (U[0, 1] for the high-resolution detector stack)

A chain is cut into *segments*; each segment is planned with its own band count on
its own last layer (the segment boundary plays the role of the paper's barrier in
front of a global operator, Sec. IV-B).

Layer indices inside a segment: -1 is the segment input, 0.. are layers in list
(= topological) order.  ``residual_from == -2`` means "no residual".
"""
from dataclasses import dataclass
from typing import List, Optional

import numpy as np

from . import rng

CONV, POOL, LINEAR, DWCONV, LAYERNORM, CONCAT = 0, 1, 2, 3, 4, 5
ACT_NONE, ACT_RELU, ACT_SILU, ACT_GELU = 0, 1, 2, 3
RES_NONE, RES_PRE_ACT, RES_POST_ACT = 0, 1, 2
NO_RESIDUAL = -2


@dataclass
class Layer:
    op: int
    cin: int
    cout: int
    kh: int
    kw: int
    sh: int = 1
    sw: int = 1
    ph: int = 0
    pw: int = 0
    dh: int = 1
    dw: int = 1
    act: int = ACT_NONE
    input_from: Optional[int] = None         # None until the builder resolves it to "previous layer"
    residual_from: int = NO_RESIDUAL
    residual_pos: int = RES_NONE
    weight: Optional[np.ndarray] = None      # [cout, kh, kw, cin] float32 (bf16-representable on the bf16 path)
    scale: Optional[np.ndarray] = None       # [cout] float32 or None (=> 1)
    shift: Optional[np.ndarray] = None       # [cout] float32 or None (=> 0)


@dataclass
class Segment:
    layers: List[Layer]
    n_bands: int


@dataclass
class Workload:
    name: str
    dtype: str                    # "f32" | "bf16"
    N: int
    H: int
    W: int
    C: int
    segments: List[Segment]
    x: Optional[np.ndarray] = None           # [N, H, W, C] float32 (bf16-representable on the bf16 path)
    seed: int = 0
    notes: str = ""
    input_range: tuple = (-1.0, 1.0)
    affine: bool = True


def conv(cin, cout, k, s=1, p=None, d=1, act=ACT_RELU, input_from=None, residual_from=NO_RESIDUAL,
         residual_pos=RES_NONE):
    if p is None:
        p = d * (k - 1) // 2
    return Layer(CONV, cin, cout, k, k, s, s, p, p, d, d, act, input_from, residual_from, residual_pos)


def linear(cin, cout, act=ACT_NONE, input_from=None, residual_from=NO_RESIDUAL, residual_pos=RES_NONE):
    """The row-wise operator of Sec. IV-A (Eq. 1): every pixel's channel vector times a shared [cout, cin] matrix."""
    return Layer(LINEAR, cin, cout, 1, 1, 1, 1, 0, 0, 1, 1, act, input_from, residual_from, residual_pos)


def dwconv(c, k, s=1, p=None, d=1, act=ACT_NONE, input_from=None, residual_from=NO_RESIDUAL, residual_pos=RES_NONE):
    """Depth-wise convolution: every channel filtered by its own k x k kernel (weight [c, k, k, 1])."""
    if p is None:
        p = d * (k - 1) // 2
    return Layer(DWCONV, c, c, k, k, s, s, p, p, d, d, act, input_from, residual_from, residual_pos)


def layernorm(c, input_from=None):
    """Layer normalisation over the channels of every pixel (scale = gamma, shift = beta)."""
    return Layer(LAYERNORM, c, c, 1, 1, 1, 1, 0, 0, 1, 1, ACT_NONE, input_from)


def concat(c_main, c_second, input_from=None, second_from=NO_RESIDUAL):
    """Channel concatenation (main input's channels first); the second input is named like a residual."""
    return Layer(CONCAT, c_main, c_main + c_second, 1, 1, 1, 1, 0, 0, 1, 1, ACT_NONE, input_from, second_from, RES_NONE)


def pool(c, k, s, p=0, input_from=None):
    return Layer(POOL, c, c, k, k, s, s, p, p, 1, 1, ACT_NONE, input_from)


def _chain(layers):
    """A layer built without an explicit ``input_from`` reads the layer before it (-1 for the first)."""
    for i, l in enumerate(layers):
        if l.input_from is None:
            l.input_from = i - 1
    return layers


def fill_parameters(wl: Workload):
    """Draw weights / scale / shift for every conv layer; one sub-stream per tensor."""
    bf16 = wl.dtype == "bf16"
    stream = 16
    for seg in wl.segments:
        for l in seg.layers:
            if l.op in (CONV, LINEAR, DWCONV):
                cin_w = 1 if l.op == DWCONV else l.cin
                fan_in = l.kh * l.kw * cin_w
                w = rng.normal(wl.seed, stream, (l.cout, l.kh, l.kw, cin_w), 0.0, float(np.sqrt(2.0 / fan_in)))
                l.weight = rng.round_to_bf16(w) if bf16 else w
                if wl.affine:
                    l.scale = rng.normal(wl.seed, stream + 1, (l.cout,), 1.0, 0.1)
                    l.shift = rng.normal(wl.seed, stream + 2, (l.cout,), 0.0, 0.1)
            elif l.op == LAYERNORM:
                l.scale = rng.normal(wl.seed, stream + 1, (l.cout,), 1.0, 0.1)       # gamma
                l.shift = rng.normal(wl.seed, stream + 2, (l.cout,), 0.0, 0.1)       # beta
            stream += 4
    return wl


def make_input(wl: Workload):
    x = rng.uniform(wl.seed, 1, (wl.N, wl.H, wl.W, wl.C), wl.input_range[0], wl.input_range[1])
    wl.x = rng.round_to_bf16(x) if wl.dtype == "bf16" else x
    return wl


# ----------------------------------------------------------------------------------------------
# the five families
# ----------------------------------------------------------------------------------------------

def single_conv(N=1, H=32, W=32, C=16, n_bands=4, dtype="f32", seed=101):
    """One 3x3 stride-1 pad-1 convolution, no affine, no activation."""
    layers = _chain([conv(C, C, 3, act=ACT_NONE)])
    return Workload("single_conv3x3", dtype, N, H, W, C, [Segment(layers, n_bands)], seed=seed, affine=False)


def vgg_block(N=1, H=224, W=224, n_bands=8, dtype="bf16", seed=202, width=64):
    layers = _chain([conv(3, width, 3), conv(width, width, 3), pool(width, 2, 2)])
    return Workload("vgg_block", dtype, N, H, W, 3, [Segment(layers, n_bands)], seed=seed)


def _stem(width=64):
    return _chain([conv(3, width, 7, s=2, p=3), pool(width, 3, 2, 1)])


def _basic_block(layers, cin, cout, stride, src):
    """Append a ResNet BasicBlock reading layer index ``src``; return the index of its output."""
    a = len(layers)
    layers.append(conv(cin, cout, 3, s=stride, input_from=src))
    if stride != 1 or cin != cout:
        layers.append(conv(cin, cout, 1, s=stride, p=0, act=ACT_NONE, input_from=src))
        short = len(layers) - 1
    else:
        short = src
    layers.append(conv(cout, cout, 3, input_from=a, residual_from=short, residual_pos=RES_PRE_ACT))
    return len(layers) - 1


def resnet18(N=1, H=224, W=224, n_bands=8, dtype="bf16", seed=303, width=64):
    segs = [Segment(_stem(width), n_bands)]
    cin = width
    for stage, mult in enumerate((1, 2, 4, 8)):
        cout = width * mult
        layers, src = [], -1
        for b in range(2):
            src = _basic_block(layers, cin, cout, 2 if (b == 0 and stage > 0) else 1, src)
            cin = cout
        segs.append(Segment(_chain(layers), n_bands))
    return Workload("resnet18_trunk", dtype, N, H, W, 3, segs, seed=seed)


def _bottleneck(layers, cin, mid, stride, src, project):
    cout = 4 * mid
    layers.append(conv(cin, mid, 1, p=0, input_from=src))
    a = len(layers) - 1
    layers.append(conv(mid, mid, 3, s=stride, input_from=a))
    b = len(layers) - 1
    if project:
        layers.append(conv(cin, cout, 1, s=stride, p=0, act=ACT_NONE, input_from=src))
        short = len(layers) - 1
    else:
        short = src
    layers.append(conv(mid, cout, 1, p=0, input_from=b, residual_from=short, residual_pos=RES_PRE_ACT))
    return len(layers) - 1


def resnet50(N=8, H=224, W=224, n_bands=16, dtype="bf16", seed=404, width=64, depths=(3, 4, 6, 3)):
    segs = [Segment(_stem(width), n_bands)]
    cin = width
    for stage, nblocks in enumerate(depths):
        mid = width * (1 << stage)
        layers, src = [], -1
        for b in range(nblocks):
            src = _bottleneck(layers, cin, mid, 2 if (b == 0 and stage > 0) else 1, src, project=(b == 0))
            cin = 4 * mid
        segs.append(Segment(_chain(layers), n_bands))
    return Workload("resnet50_trunk", dtype, N, H, W, 3, segs, seed=seed)


def csp_stack(N=1, H=1024, W=1024, n_bands=32, dtype="bf16", seed=505, base=32):
    """Twelve 3x3 / 1x1 SiLU convolutions, five stride-2 stages, three post-activation residual joins."""
    c1, c2, c3, c4, c5 = base, 2 * base, 4 * base, 8 * base, 16 * base
    S = ACT_SILU
    layers = [
        conv(3, c1, 3, s=2, act=S),                                                         # 0
        conv(c1, c2, 3, s=2, act=S),                                                        # 1
        conv(c2, c2, 1, p=0, act=S),                                                        # 2
        conv(c2, c2, 3, act=S, residual_from=1, residual_pos=RES_POST_ACT),                 # 3
        conv(c2, c3, 3, s=2, act=S),                                                        # 4
        conv(c3, c3, 1, p=0, act=S),                                                        # 5
        conv(c3, c3, 3, act=S, residual_from=4, residual_pos=RES_POST_ACT),                 # 6
        conv(c3, c4, 3, s=2, act=S),                                                        # 7
        conv(c4, c4, 1, p=0, act=S),                                                        # 8
        conv(c4, c4, 3, act=S, residual_from=7, residual_pos=RES_POST_ACT),                 # 9
        conv(c4, c5, 3, s=2, act=S),                                                        # 10
        conv(c5, c5, 1, p=0, act=S),                                                        # 11
    ]
    wl = Workload("csp_stack", dtype, N, H, W, 3, [Segment(_chain(layers), n_bands)], seed=seed,
                  input_range=(0.0, 1.0))
    return wl


def pointwise_mlp(N=2, H=56, W=56, C=128, hidden=512, n_bands=8, dtype="bf16", seed=606):
    """Row-wise local operators only (Sec. IV-A, Eq. 1), shaped like the point-wise MLP of a ConvNeXt block: every
    pixel's channel vector through  linear(C -> hidden) + SiLU,  linear(hidden -> C) + shortcut.  Rows map one to one
    through both layers, so bands need no halo at all."""
    layers = [linear(C, hidden, act=ACT_SILU), linear(hidden, C, act=ACT_NONE, residual_from=-1, residual_pos=RES_POST_ACT)]
    return Workload("pointwise_mlp", dtype, N, H, W, C, [Segment(_chain(layers), n_bands)], seed=seed)


def convnext_block(N=2, H=56, W=56, C=128, n_bands=8, dtype="bf16", seed=707):
    """One ConvNeXt block (the paper evaluates ConvNeXt, Sec. V-B): depth-wise 7x7, layer normalisation over the
    channels, point-wise MLP C -> 4C (GELU) -> C, shortcut.  A block-wise operator (3-row halo) followed by per-pixel and
    row-wise ones."""
    layers = [dwconv(C, 7), layernorm(C), linear(C, 4 * C, act=ACT_GELU),
              linear(4 * C, C, act=ACT_NONE, residual_from=-1, residual_pos=RES_POST_ACT)]
    return Workload("convnext_block", dtype, N, H, W, C, [Segment(_chain(layers), n_bands)], seed=seed)


def dense_layer(N=2, H=28, W=28, C=64, growth=32, n_bands=4, dtype="bf16", seed=808):
    """One DenseNet layer (Sec. V-B): 1x1 bottleneck to 4*growth, 3x3 to growth channels, concatenated behind the input."""
    layers = [conv(C, 4 * growth, 1, p=0, act=ACT_RELU), conv(4 * growth, growth, 3, act=ACT_RELU),
              concat(C, growth, input_from=-1, second_from=1)]
    layers[0].input_from, layers[1].input_from = -1, 0
    return Workload("dense_layer", dtype, N, H, W, C, [Segment(layers, n_bands)], seed=seed)


WORKLOADS = {
    "single_conv": single_conv,
    "vgg_block": vgg_block,
    "resnet18": resnet18,
    "resnet50": resnet50,
    "csp_stack": csp_stack,
    "pointwise_mlp": pointwise_mlp,
    "convnext_block": convnext_block,
    "dense_layer": dense_layer,
}


def build(name, with_data=True, **overrides):
    """Instantiate a workload family; ``overrides`` shrink it for tests (N, H, W, n_bands, width...)."""
    wl = WORKLOADS[name](**overrides)
    if with_data:
        fill_parameters(wl)
        make_input(wl)
    return wl

"""Parity of the CUDA library (through the C ABI) against the CPU oracle.  Needs a B200."""
import numpy as np
import pytest
import torch

import lop_inputs as li
import paper_2507_05829_b200 as lop
from lop_inputs.workloads import Layer, Segment, Workload, conv, pool
from oracle import chain as ochain
from paper_2507_05829_b200.chain import DeviceChain, to_host_f32

pytestmark = pytest.mark.gpu

TOL = {"f32": 1e-4, "bf16": 2e-2}       # max |gpu - oracle| / max |oracle|


def rel_err(got, want):
    scale = float(np.max(np.abs(want)))
    return float(np.max(np.abs(got.astype(np.float64) - want.astype(np.float64)))) / (scale if scale > 0 else 1.0)


def oracle_layers(wl):
    """Every layer's output of every segment, whole-tensor execution on the CPU: [segment][layer] -> array."""
    x, out = wl.x, []
    for seg in wl.segments:
        out.append(ochain.run_whole(seg.layers, x, wl.dtype == "bf16", keep_all=True))
        x = out[-1][-1]
    return out


def check_layers(dc, want_layers, tol, what, independent_bands=False):
    """Every layer output the GPU run has stored (workspace tensors and segment outputs) against the oracle.

    In reuse-halo and whole-tensor runs every row of every layer has been computed; with independent bands (each band
    recomputing its halo into the same full-size tensors) the rows are complete as well -- the last band to write a
    row wrote the same bits."""
    for s, layers in enumerate(want_layers):
        for i, w in enumerate(layers):
            t = dc.layer_output(s, i)
            if t is None:                    # folded into the next layer's stage: that layer's tensor is checked instead
                continue
            g = to_host_f32(t)
            assert g.shape == w.shape, (what, s, i)
            assert np.all(np.isfinite(g)), (what, "segment", s, "layer", i)
            e = rel_err(g, w)
            assert e <= tol, (what, "segment", s, "layer", i, "rel err", e)


def check_workload(wl, flags=0, modes=("whole", "banded", "pipelined", "pipelined_copy"), n_bands=None, tol=None):
    """Run every segment on the GPU in each mode and compare EVERY LAYER's output with the oracle (the intermediate
    tensors are read out of the workspaces), then the modes with each other bit for bit.

    pipelined: the kernel fetches the bands from the pinned host tensor itself (where the plan runs on the persistent
    kernel); pipelined_copy: the bands come by copy-engine copies on the side stream."""
    want_layers = oracle_layers(wl)
    want = [layers[-1] for layers in want_layers]
    tol = TOL[wl.dtype] if tol is None else tol
    results = {}
    for mode in modes:
        dc = DeviceChain(wl, flags=flags | (lop.LOP_FLAG_COPY_ENGINE if mode == "pipelined_copy" else 0), n_bands=n_bands)
        if mode in ("pipelined", "pipelined_copy"):
            dc.run_pipelined(dc.pinned_input())
        elif mode == "banded":
            dc.run_banded(dc.input_tensor())
        else:
            dc.run_whole(dc.input_tensor())
        torch.cuda.synchronize()
        dc.check_device()
        check_layers(dc, want_layers, tol, (wl.name, mode))
        outs = [to_host_f32(o) for o in dc.outs]
        for s, (g, w) in enumerate(zip(outs, want)):
            assert g.shape == w.shape
        results[mode] = outs
    base = results[modes[0]]
    for mode in modes[1:]:                   # band-wise execution reproduces whole-tensor execution bit for bit
        for a, b in zip(base, results[mode]):
            assert np.array_equal(a, b), (wl.name, mode, "differs from", modes[0])
    return results


def one_layer(l, N, H, W, dtype="bf16", n_bands=3, seed=9, affine=True):
    wl = Workload("one_layer", dtype, N, H, W, l.cin, [Segment([l], n_bands)], seed=seed, affine=affine)
    l.input_from = -1
    li.fill_parameters(wl)
    li.make_input(wl)
    return wl


# ------------------------------------------------------------------------------------ fp32 path
def test_single_conv_fp32_four_bands():
    wl = li.build("single_conv")
    check_workload(wl)


@pytest.mark.parametrize("k,s,p,d,cin,cout,H,W", [
    (3, 1, 1, 1, 5, 7, 11, 13), (5, 2, 2, 1, 3, 8, 17, 9), (3, 1, 2, 2, 4, 4, 12, 12), (1, 2, 0, 1, 9, 3, 10, 7),
    (7, 3, 3, 1, 2, 5, 23, 23), (2, 2, 0, 1, 6, 70, 8, 8),
])
def test_fp32_conv_general_shapes(k, s, p, d, cin, cout, H, W):
    wl = one_layer(conv(cin, cout, k, s=s, p=p, d=d, act=li.ACT_SILU), 2, H, W, dtype="f32")
    check_workload(wl, modes=("whole", "banded"))


def test_fp32_vgg_block_small():
    check_workload(li.build("vgg_block", H=30, W=22, dtype="f32", width=16, n_bands=4))


# ------------------------------------------------------------------------------------ bf16 tensor-core conv, per shape
TC_CASES = [  # k, s, p, d, cin, cout, N, H, W
    (3, 1, 1, 1, 64, 64, 1, 20, 32),
    (3, 1, 1, 1, 64, 64, 2, 9, 56),        # ragged W against the tile width
    (3, 1, 1, 1, 128, 256, 1, 14, 14),
    (3, 2, 1, 1, 64, 128, 2, 28, 28),      # stride 2, even extent
    (3, 2, 1, 1, 32, 64, 1, 31, 45),       # stride 2, odd extents, 32-channel slabs
    (1, 1, 0, 1, 256, 64, 3, 7, 7),        # pointwise, tiny image, batch folded into the tile
    (1, 2, 0, 1, 64, 256, 2, 15, 15),      # strided pointwise projection
    (7, 2, 3, 1, 3, 64, 2, 38, 38),        # stem: 3 input channels, padded to 16
    (3, 1, 1, 1, 3, 32, 1, 24, 40),
    (3, 1, 1, 1, 5, 32, 2, 9, 21),         # 45 patch values -> 48: 16-channel chunks, tiny images
    (3, 2, 1, 1, 7, 64, 3, 13, 13),        # 63 -> 64: one 64-channel chunk, strided stem
    (5, 1, 2, 2, 3, 48, 1, 20, 20),        # dilated stem, 75 -> 80
    (3, 1, 2, 2, 64, 32, 1, 16, 16),       # dilation 2
    (3, 1, 1, 1, 16, 16, 1, 10, 10),       # 16-channel slabs
    (5, 1, 2, 1, 64, 48, 1, 12, 12),       # 48 output channels
    (3, 1, 1, 1, 512, 512, 1, 7, 7),
    (3, 1, 1, 1, 64, 64, 1, 5, 300),       # wider than two 128-pixel tiles
]


@pytest.mark.parametrize("case", TC_CASES)
def test_bf16_tensor_core_conv_shapes(case):
    k, s, p, d, cin, cout, N, H, W = case
    wl = one_layer(conv(cin, cout, k, s=s, p=p, d=d, act=li.ACT_RELU), N, H, W)
    dc = DeviceChain(wl)
    assert dc.plans[0].layer_kernel(0) == 2
    check_workload(wl, modes=("whole", "banded"))                                   # persistent wavefront launch
    check_workload(wl, modes=("whole", "banded"), flags=lop.LOP_FLAG_PER_LAYER)     # one launch per (band, layer)
    check_workload(wl, modes=("whole",), flags=lop.LOP_FLAG_FORCE_SIMT)


@pytest.mark.parametrize("pos,act", [(li.RES_PRE_ACT, li.ACT_RELU), (li.RES_POST_ACT, li.ACT_SILU)])
def test_bf16_residual_and_activation_epilogues(pos, act):
    layers = [conv(64, 64, 3, act=act), conv(64, 64, 3, act=act, residual_from=0, residual_pos=pos),
              conv(64, 64, 1, p=0, act=li.ACT_NONE, residual_from=-1, residual_pos=pos)]
    for i, l in enumerate(layers):
        l.input_from = i - 1
    wl = Workload("res", "bf16", 2, 18, 24, 64, [Segment(layers, 4)], seed=5)
    li.fill_parameters(wl)
    li.make_input(wl)
    check_workload(wl)
    check_workload(wl, flags=lop.LOP_FLAG_PER_LAYER | lop.LOP_FLAG_REUSE_HALO)


# ------------------------------------------------------------------------------------ convolution + 2x2 pooling in one stage
POOL_FUSE_CASES = [  # layers (cin, cout, k) of the convolution in front of the pooling, N, H, W, C
    ((64, 64, 3), 2, 20, 27, 64),          # odd width: the last column has no partner
    ((64, 32, 1), 3, 6, 6, 64),            # pointwise, tiny images folded into one tile
    ((3, 64, 3), 1, 24, 40, 3),            # gathered stem straight into the pooling
    ((64, 128, 5), 1, 16, 16, 64),         # wider halo, two channel tiles
]


@pytest.mark.parametrize("case", POOL_FUSE_CASES)
def test_conv_then_pool2x2_is_pooled_in_the_epilogue(case):
    (cin, cout, k), N, H, W, C = case
    layers = [conv(cin, cout, k, act=li.ACT_RELU), pool(cout, 2, 2, 0)]
    for i, l in enumerate(layers):
        l.input_from = i - 1
    wl = Workload("convpool", "bf16", N, H, W, C, [Segment(layers, 3)], seed=11)
    li.fill_parameters(wl)
    li.make_input(wl)
    a = check_workload(wl, flags=lop.LOP_FLAG_REUSE_HALO)["whole"]
    b = check_workload(wl, flags=lop.LOP_FLAG_REUSE_HALO | lop.LOP_FLAG_PER_LAYER, modes=("whole", "banded"))["whole"]
    for x, y in zip(a, b):
        assert np.array_equal(x, y)
    check_workload(wl)                                           # independent bands


def test_pooling_is_not_folded_when_the_convolution_has_another_reader():
    layers = [conv(64, 64, 3, act=li.ACT_RELU), pool(64, 2, 2, 0),
              conv(64, 64, 3, s=2, act=li.ACT_NONE, residual_from=1, residual_pos=li.RES_POST_ACT)]
    layers[0].input_from, layers[1].input_from, layers[2].input_from = -1, 0, 0     # layer 2 also reads the convolution
    wl = Workload("convpool2", "bf16", 1, 16, 24, 64, [Segment(layers, 2)], seed=12)
    li.fill_parameters(wl)
    li.make_input(wl)
    check_workload(wl, flags=lop.LOP_FLAG_REUSE_HALO)


# ------------------------------------------------------------------------------------ pooling
@pytest.mark.parametrize("dtype,C", [("bf16", 64), ("bf16", 6), ("f32", 8), ("f32", 3)])
@pytest.mark.parametrize("k,s,p", [(2, 2, 0), (3, 2, 1)])
def test_maxpool(dtype, C, k, s, p):
    l = pool(C, k, s, p)
    wl = one_layer(l, 2, 21, 18, dtype=dtype)
    res = check_workload(wl, modes=("whole", "banded"), tol=0.0)   # pooling only selects: exact


# ------------------------------------------------------------------------------------ depth-wise, layer norm, concat, GELU
@pytest.mark.parametrize("dtype,C", [("bf16", 64), ("bf16", 40), ("bf16", 6), ("f32", 8), ("f32", 3)])
@pytest.mark.parametrize("k,s,p,d", [(7, 1, 3, 1), (3, 2, 1, 1), (3, 1, 2, 2), (5, 1, 0, 1)])
def test_depthwise_convolution(dtype, C, k, s, p, d):
    l = li.dwconv(C, k, s=s, p=p, d=d, act=li.ACT_GELU)
    check_workload(one_layer(l, 2, 23, 18, dtype=dtype, n_bands=4), modes=("whole", "banded", "pipelined"))


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("pos,act", [(li.RES_PRE_ACT, li.ACT_RELU), (li.RES_POST_ACT, li.ACT_SILU)])
def test_depthwise_convolution_with_a_shortcut(dtype, pos, act):
    l = li.dwconv(32, 3, act=act, residual_from=-1, residual_pos=pos)
    check_workload(one_layer(l, 2, 14, 11, dtype=dtype), modes=("whole", "banded"))
    check_workload(one_layer(l, 2, 14, 11, dtype=dtype), flags=lop.LOP_FLAG_REUSE_HALO, modes=("whole", "banded"))


@pytest.mark.parametrize("dtype,C", [("bf16", 64), ("bf16", 520), ("bf16", 40), ("bf16", 7), ("f32", 12), ("f32", 5), ("f32", 260)])
def test_layer_normalisation(dtype, C):
    wl = one_layer(li.layernorm(C), 2, 13, 9, dtype=dtype)
    wl.x = (wl.x * 3.0 + 1.5).astype(np.float32)               # a mean and a spread the normalisation has to remove
    if dtype == "bf16":
        wl.x = li.round_to_bf16(wl.x)
    check_workload(wl, modes=("whole", "banded", "pipelined"))


@pytest.mark.parametrize("dtype,ca,cb", [("bf16", 16, 8), ("bf16", 64, 32), ("bf16", 5, 3), ("f32", 8, 4), ("f32", 3, 2)])
def test_concatenation(dtype, ca, cb):
    layers = [conv(ca, cb, 3, act=li.ACT_RELU), li.concat(ca, cb, input_from=-1, second_from=0)]
    layers[0].input_from = -1
    wl = Workload("concat", dtype, 2, 12, 10, ca, [Segment(layers, 3)], seed=21)
    li.fill_parameters(wl)
    li.make_input(wl)
    for flags in (0, lop.LOP_FLAG_REUSE_HALO):
        res = check_workload(wl, flags=flags, modes=("whole", "banded", "pipelined"))
        assert np.array_equal(res["whole"][0][..., :ca], wl.x)                 # the copied half is bit-exact


@pytest.mark.parametrize("dtype,cin,cout,flags", [("bf16", 64, 64, 0), ("bf16", 64, 64, lop.LOP_FLAG_PER_LAYER),
                                                  ("bf16", 64, 64, lop.LOP_FLAG_FORCE_SIMT), ("f32", 5, 9, 0)])
def test_gelu_in_the_convolution_epilogue(dtype, cin, cout, flags):
    """The persistent kernel's, the per-layer tensor-core kernel's and the CUDA-core kernel's epilogues."""
    wl = one_layer(conv(cin, cout, 3, act=li.ACT_GELU), 2, 20, 16, dtype=dtype)
    check_workload(wl, flags=flags, modes=("whole", "banded"))


# ------------------------------------------------------------------------------------ chains, reduced sizes
SMALL = [("vgg_block", dict(H=44, W=36)), ("resnet18", dict(H=64, W=64)),
         ("resnet50", dict(N=2, H=64, W=64, depths=(2, 2, 2, 2))), ("csp_stack", dict(H=256, W=128)),
         ("pointwise_mlp", dict(H=21, W=19, C=64, hidden=192, n_bands=4)),      # row-wise operators (Sec. IV-A, Eq. 1)
         ("convnext_block", dict(H=29, W=17, C=64, n_bands=5)), ("dense_layer", dict(H=19, W=14, n_bands=3)),
         ("convnext_block", dict(H=15, W=9, C=12, n_bands=3, dtype="f32"))]


@pytest.mark.parametrize("name,kw", SMALL)
@pytest.mark.parametrize("flags", [0, lop.LOP_FLAG_REUSE_HALO, lop.LOP_FLAG_PER_LAYER,
                                   lop.LOP_FLAG_PER_LAYER | lop.LOP_FLAG_REUSE_HALO])
def test_chains_small(name, kw, flags):
    check_workload(li.build(name, **kw), flags=flags)


@pytest.mark.parametrize("name,kw", [("single_conv", {}), ("vgg_block", dict(H=30, W=22, dtype="f32", width=16, n_bands=4)),
                                     ("resnet18", dict(H=64, W=64)), ("convnext_block", dict(H=29, W=17, C=64, n_bands=5)),
                                     ("convnext_block", dict(H=15, W=9, C=12, n_bands=3, dtype="f32")), ("dense_layer", dict(H=19, W=14, n_bands=3))])
def test_checked_execution_finds_nothing_and_changes_nothing(name, kw):
    """LOP_FLAG_DEBUG_BOUNDS: the kernels test every address they compute.  On a correct library the status word stays
    clear (check_device inside check_workload raises otherwise) and the results are those of the unchecked per-layer
    kernels, bit for bit."""
    wl = li.build(name, **kw)
    for reuse in (0, lop.LOP_FLAG_REUSE_HALO):
        a = check_workload(wl, flags=reuse | lop.LOP_FLAG_DEBUG_BOUNDS, modes=("whole", "banded", "pipelined_copy"))
        b = check_workload(wl, flags=reuse | lop.LOP_FLAG_PER_LAYER, modes=("banded",))
        for x, y in zip(a["banded"], b["banded"]):
            assert np.array_equal(x, y)


def test_tensor_core_and_cuda_core_paths_agree():
    wl = li.build("resnet18", H=64, W=64)
    a = check_workload(wl, modes=("whole",))["whole"]
    b = check_workload(wl, modes=("whole",), flags=lop.LOP_FLAG_FORCE_SIMT)["whole"]
    for x, y in zip(a, b):
        assert rel_err(x, y) <= 2e-2


# ------------------------------------------------------------------------------------ several plans, one launch
def _chain_args(dc):
    return [o.data_ptr() for o in dc.outs], [w.data_ptr() for w in dc.ws]


@pytest.mark.parametrize("flags", [0, lop.LOP_FLAG_REUSE_HALO])
def test_chain_entry_points_run_all_plans_in_one_launch(flags):
    """lop_run_chain_*: one persistent launch for the whole multi-segment network, same bits as plan after plan."""
    wl = li.build("resnet18", H=64, W=64)
    ref = DeviceChain(wl, flags=flags)
    ref.per_plan = True                                  # the plans one by one
    ref.run_banded(ref.input_tensor())
    torch.cuda.synchronize()
    assert sum(p.last_launches() for p in ref.plans) >= len(ref.plans) > 1
    s = torch.cuda.current_stream().cuda_stream
    for mode in ("banded", "pipelined"):
        dc = DeviceChain(wl, flags=flags)
        outs, wss = _chain_args(dc)
        x_dev, x_host = dc.input_tensor(), dc.pinned_input()
        for call in range(2):                            # the first call also pads the stem's weights, once
            if mode == "banded":
                lop.run_chain_banded(dc.plans, x_dev.data_ptr(), outs, wss, s)
            else:
                lop.run_chain_pipelined(dc.plans, x_host.data_ptr(), dc.staging.data_ptr(), outs, wss, s)
            torch.cuda.synchronize()
        dc.check_device()
        assert dc.plans[0].last_launches() == 1 and all(p.last_launches() == 0 for p in dc.plans[1:])
        for a, b in zip(ref.outs, dc.outs):
            assert torch.equal(a, b), mode


def test_chain_entry_points_refuse_plans_that_do_not_follow_each_other():
    wl = li.build("resnet18", H=64, W=64)
    dc = DeviceChain(wl)
    outs, wss = _chain_args(dc)
    s = torch.cuda.current_stream().cuda_stream
    x = dc.input_tensor()
    with pytest.raises(lop.LopError) as e:                 # plan 3 does not take plan 0's output
        lop.run_chain_banded([dc.plans[0], dc.plans[3]], x.data_ptr(), [outs[0], outs[3]], [wss[0], wss[3]], s)
    assert e.value.status == -2
    simt = DeviceChain(wl, flags=lop.LOP_FLAG_FORCE_SIMT)  # CUDA-core plans are not taken by the persistent kernel
    o2, w2 = _chain_args(simt)
    with pytest.raises(lop.LopError) as e:
        lop.run_chain_banded(simt.plans, simt.input_tensor().data_ptr(), o2, w2, s)
    assert e.value.status == -3
    simt.run_banded(simt.input_tensor())                   # the wrapper falls back to plan after plan
    torch.cuda.synchronize()
    assert simt.per_plan
    assert rel_err(to_host_f32(simt.outs[-1]), ochain.run_workload(wl)) <= TOL["bf16"]


# ------------------------------------------------------------------------------------ band blocks (sharding over devices)
@pytest.mark.parametrize("flags", [0, lop.LOP_FLAG_REUSE_HALO, lop.LOP_FLAG_REUSE_HALO | lop.LOP_FLAG_PER_LAYER])
@pytest.mark.parametrize("name,kw", [("vgg_block", dict(H=44, W=36)), ("resnet18", dict(H=64, W=64))])
def test_band_blocks_run_alone_give_their_rows_of_the_banded_result(name, kw, flags):
    """lop_run_shard for every rank of 1, 2 and 3 devices, one after the other on this GPU, each on a workspace of
    its own and with only its input rows present: the stitched rows equal lop_run_banded bit for bit."""
    wl = li.build(name, **kw)
    ref = DeviceChain(wl, flags=flags)
    ref.per_plan = True
    ref.run_banded(ref.input_tensor())
    torch.cuda.synchronize()
    s = torch.cuda.current_stream().cuda_stream
    for world in (1, 2, 3):
        x = ref.input_tensor()
        for si, plan in enumerate(ref.plans):
            stitched = torch.full_like(ref.outs[si], float("nan"))
            for rank in range(world):
                dc = DeviceChain(wl, flags=flags)                  # this rank's device: its own tensors
                b0, b1, r0, r1, i0, i1 = dc.plans[si].shard(rank, world)
                x_mine = torch.full_like(x, float("nan"))
                x_mine[:, i0:i1] = x[:, i0:i1]
                dc.outs[si].fill_(float("nan"))
                dc.plans[si].run_shard(b0, b1, x_mine.data_ptr(), dc.outs[si].data_ptr(), dc.ws[si].data_ptr(), s)
                torch.cuda.synchronize()
                dc.plans[si].check_device(dc.ws[si].data_ptr())
                got = dc.outs[si]
                assert not torch.isnan(got[:, r0:r1]).any()
                assert torch.isnan(got[:, :r0]).all() and torch.isnan(got[:, r1:]).all()      # nothing but its rows written
                stitched[:, r0:r1] = got[:, r0:r1]
            assert torch.equal(stitched, ref.outs[si]), (name, world, si)
            x = ref.outs[si]
    assert rel_err(to_host_f32(ref.outs[-1]), ochain.run_workload(wl)) <= TOL["bf16"]


def test_sharded_chain_with_one_rank_is_the_banded_run():
    from paper_2507_05829_b200.shard import ShardedChain
    wl = li.build("resnet18", H=64, W=64)
    ref = DeviceChain(wl, flags=lop.LOP_FLAG_REUSE_HALO)
    ref.run_banded(ref.input_tensor())
    dc = DeviceChain(wl, flags=lop.LOP_FLAG_REUSE_HALO)
    out = ShardedChain(dc, 0, 1).run(dc.input_tensor())
    torch.cuda.synchronize()
    dc.check_device()
    assert torch.equal(out, ref.outs[-1])


def test_sharded_chain_on_a_stream_that_is_not_current():
    """The launches and the row exchange are ordered on the stream that was passed, also when torch's current stream is
    another one: the result equals the banded run and the current stream never sees half-written rows."""
    from paper_2507_05829_b200 import shard
    wl = li.build("resnet18", H=64, W=64)
    ref = DeviceChain(wl, flags=lop.LOP_FLAG_REUSE_HALO)
    ref.run_banded(ref.input_tensor())
    torch.cuda.synchronize()
    dc = DeviceChain(wl, flags=lop.LOP_FLAG_REUSE_HALO)
    side = torch.cuda.Stream()
    x = dc.input_tensor()
    torch.cuda.synchronize()
    out = shard.ShardedChain(dc, 0, 1).run(x, stream=side)
    side.synchronize()
    dc.check_device()
    assert torch.equal(out, ref.outs[-1])
    # the copy path of the exchange for two ranks, driven by hand on the side stream: rank 0's rows stay, rank 1's arrive
    table = shard.shard_table(dc.plans[-1], 2)
    full = ref.outs[-1]
    mine = torch.zeros_like(full)
    mine[:, table[0][2]:table[0][3]] = full[:, table[0][2]:table[0][3]]
    torch.cuda.synchronize()

    class FakeGroup:
        pass

    def fake_all_gather(parts, tensor, group=None):
        n_max = tensor.shape[1]
        for r, part in enumerate(parts):
            lo, hi = table[r][2], table[r][3]
            part.zero_()
            part[:, :hi - lo].copy_(full[:, lo:hi])

    import torch.distributed as dist
    keep = dist.all_gather
    dist.all_gather = fake_all_gather
    try:
        with torch.cuda.stream(side):
            got = shard.all_gather_rows(mine, table, 0)
        side.synchronize()
    finally:
        dist.all_gather = keep
    assert torch.equal(got, full)


def test_set_params_on_a_later_plan_of_a_chain_takes_effect():
    """A chain program is cached in the first plan; re-pointing the parameters of a LATER plan must not leave it in use."""
    wl = li.build("resnet18", H=64, W=64)
    dc = DeviceChain(wl, flags=lop.LOP_FLAG_REUSE_HALO)
    x = dc.input_tensor()
    first = dc.run_banded(x).clone()
    torch.cuda.synchronize()
    assert not dc.per_plan                                  # the plans ran as one launch
    seg_i = 2
    seg = wl.segments[seg_i]
    keep = []
    for i, l in enumerate(seg.layers):
        if l.weight is None:
            continue
        l.weight = -l.weight
        w = torch.from_numpy(l.weight).to(torch.bfloat16).cuda().contiguous()
        sc = torch.from_numpy(l.scale).cuda() if l.scale is not None else None
        sh = torch.from_numpy(l.shift).cuda() if l.shift is not None else None
        keep += [w, sc, sh]
        dc.plans[seg_i].set_params(i, w.data_ptr(), sc.data_ptr() if sc is not None else None, sh.data_ptr() if sh is not None else None)
    want = oracle_layers(wl)
    for mode in ("banded", "pipelined"):
        got = dc.run_banded(x) if mode == "banded" else dc.run_pipelined(dc.pinned_input())
        torch.cuda.synchronize()
        dc.check_device()
        assert not dc.per_plan
        check_layers(dc, want, TOL["bf16"], ("resnet18 re-pointed", mode))
    assert not torch.equal(first, dc.outs[-1])


def test_fetch_band_alone_brings_exactly_its_rows():
    """lop_fetch_band: the transfer step of the fetched transport by itself (what a pipelined run has to hide)."""
    wl = li.build("vgg_block", H=44, W=36)
    dc = DeviceChain(wl, flags=lop.LOP_FLAG_REUSE_HALO)
    plan = dc.plans[0]
    x, xd = dc.pinned_input(), dc.input_tensor()
    s = torch.cuda.current_stream().cuda_stream
    dc.staging.fill_(float("nan"))
    plan.fetch_band(-1, x.data_ptr(), dc.staging.data_ptr(), dc.ws[0].data_ptr(), s)
    torch.cuda.synchronize()
    plan.check_device(dc.ws[0].data_ptr())
    assert plan.last_launches() >= 1 and plan.last_copies() == 0
    assert torch.equal(dc.staging.view(-1), xd.view(-1))
    for b in (0, 2):
        r = plan.get_range(b, lop.LOP_INPUT)
        dc.staging.fill_(float("nan"))
        plan.fetch_band(b, x.data_ptr(), dc.staging.data_ptr(), dc.ws[0].data_ptr(), s)
        torch.cuda.synchronize()
        assert torch.equal(dc.staging[:, r.new_lo:r.out_hi], xd[:, r.new_lo:r.out_hi])
        assert torch.isnan(dc.staging[:, :r.new_lo].float()).all() and torch.isnan(dc.staging[:, r.out_hi:].float()).all()
    dc.run_pipelined(x)                                     # and the plan still runs
    torch.cuda.synchronize()
    dc.check_device()
    assert rel_err(to_host_f32(dc.outs[-1]), ochain.run_workload(wl)) <= TOL["bf16"]


def test_a_band_that_never_arrives_ends_the_launch_with_a_status_not_a_hang():
    """The bounded device-side wait, made to run out on purpose: band 1 is never copied and its arrival flag never
    written; with a limit of a few thousand polls the kernel gives up within milliseconds, returns by itself, the status
    word names the loader's dependency wait (0x10), and the plan works again afterwards."""
    wl = li.build("vgg_block", H=44, W=36)
    dc = DeviceChain(wl, flags=lop.LOP_FLAG_REUSE_HALO | lop.LOP_FLAG_COPY_ENGINE)
    plan, ws = dc.plans[0], dc.ws[0]
    x, xd = dc.pinned_input(), dc.input_tensor()
    s = torch.cuda.current_stream().cuda_stream
    dc.run_pipelined(x)
    torch.cuda.synchronize()
    dc.check_device()
    good = dc.outs[-1].clone()
    with pytest.raises(lop.LopError):                       # refuses to run without a short limit
        plan.run_pipelined_withheld(1, x.data_ptr(), dc.staging.data_ptr(), dc.outs[0].data_ptr(), ws.data_ptr(), s)
    plan.set_wait_limit(4000)
    dc.outs[-1].zero_()
    t0 = torch.cuda.Event(enable_timing=True)
    t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    plan.run_pipelined_withheld(1, x.data_ptr(), dc.staging.data_ptr(), dc.outs[0].data_ptr(), ws.data_ptr(), s)
    t1.record()
    torch.cuda.synchronize()                                # returns: the kernel ended by itself
    assert t0.elapsed_time(t1) < 2000.0
    with pytest.raises(lop.LopError) as e:
        plan.check_device(ws.data_ptr())
    assert e.value.status == -7
    word = int(str(e.value).split("0x")[1].split(":")[0].split()[0], 16)
    assert word & 0x10
    plan.check_device(ws.data_ptr())                        # the word was cleared, the device tables dropped
    plan.set_wait_limit(0)
    for mode in ("pipelined", "banded"):
        dc.outs[-1].zero_()
        if mode == "pipelined":
            dc.run_pipelined(x)
        else:
            dc.run_banded(xd)
        torch.cuda.synchronize()
        dc.check_device()
        assert torch.equal(dc.outs[-1], good), mode


@pytest.mark.parametrize("name,kw", [("vgg_block", dict(H=44, W=36)), ("resnet18", dict(H=64, W=64)),
                                     ("convnext_block", dict(H=29, W=17, C=64, n_bands=6)), ("dense_layer", dict(H=19, W=14, n_bands=6))])
def test_halo_exchange_between_emulated_ranks_on_one_gpu(name, kw):
    """The transmission form of band sharding (Sec. IV-C: trade halo rows instead of recomputing them), two and three
    ranks taking turns on this GPU, each with tensors of its own: lop_run_layer computes every row of every layer once,
    a mailbox carries the halo rows, and every rank's rows equal the whole-tensor run bit for bit."""
    from paper_2507_05829_b200 import shard
    wl = li.build(name, **kw)
    flags = lop.LOP_FLAG_REUSE_HALO | lop.LOP_FLAG_PER_LAYER
    ref = DeviceChain(wl, flags=flags)
    ref.run_whole(ref.input_tensor())
    torch.cuda.synchronize()
    s = torch.cuda.current_stream().cuda_stream
    for world in (2, 3):
        x = ref.input_tensor()
        for si, seg in enumerate(wl.segments):
            box = shard.MailboxTransport()
            ranks = []
            for r in range(world):
                dc = DeviceChain(wl, flags=flags)
                plan = dc.plans[si]
                table = shard.shard_table(plan, world)
                xin = torch.full_like(x, float("nan"))
                xin[:, table[r][4]:table[r][5]] = x[:, table[r][4]:table[r][5]]
                dc.ws[si].view(torch.bfloat16).fill_(float("nan"))
                dc.outs[si].fill_(float("nan"))

                def tensor(idx, dc=dc, xin=xin):
                    return xin if idx < 0 else dc.layer_output(si, idx)

                def compute(layer, lo, hi, dc=dc, xin=xin, plan=plan):
                    plan.run_layer(layer, lo, hi, xin.data_ptr(), dc.outs[si].data_ptr(), dc.ws[si].data_ptr(), s)

                ranks.append((shard.HaloExchangeRank(plan, seg.layers, table, r, tensor, compute, box), dc, table))
            for i in range(len(seg.layers)):
                for hx, _, _ in ranks:
                    hx.post_sends(i)
                torch.cuda.synchronize()
                for hx, _, _ in ranks:
                    hx.receive_and_compute(i)
                torch.cuda.synchronize()
            for r, (hx, dc, table) in enumerate(ranks):
                for i in range(len(seg.layers)):
                    lo, hi = shard.owned_rows(dc.plans[si], i, table, r)
                    want = ref.layer_output(si, i)
                    assert torch.equal(dc.layer_output(si, i)[:, lo:hi], want[:, lo:hi]), (name, world, si, r, i)
            assert sum(hx.rows_computed for hx, _, _ in ranks) == sum(ref.plans[si].out_shape(i)[0] for i in range(len(seg.layers)))
            x = ref.outs[si]


# ------------------------------------------------------------------------------------ edge cases
def test_very_wide_image_gathers_patches_without_staging_rows():
    """Three rows of a 4200-pixel image do not fit the shared staging tile: the gather reads the image in place."""
    wl = one_layer(conv(3, 32, 3, act=li.ACT_RELU), 1, 6, 4200, n_bands=2)
    check_workload(wl, flags=lop.LOP_FLAG_REUSE_HALO)


def test_set_params_takes_effect_on_a_plan_that_has_already_run():
    wl = li.build("vgg_block", H=44, W=36)
    dc = DeviceChain(wl, flags=lop.LOP_FLAG_REUSE_HALO)
    x = dc.input_tensor()
    first = dc.run_banded(x).clone()
    torch.cuda.synchronize()
    seg = wl.segments[0]
    for l in seg.layers:                                  # new weights: the old ones negated
        if l.weight is not None:
            l.weight = -l.weight
    want = ochain.run_workload(wl)
    keep = []
    for i, l in enumerate(seg.layers):
        if l.weight is None:
            continue
        w = torch.from_numpy(l.weight).to(torch.bfloat16).cuda().contiguous()
        sc = torch.from_numpy(l.scale).cuda() if l.scale is not None else None
        sh = torch.from_numpy(l.shift).cuda() if l.shift is not None else None
        keep += [w, sc, sh]
        dc.plans[0].set_params(i, w.data_ptr(), sc.data_ptr() if sc is not None else None, sh.data_ptr() if sh is not None else None)
    for mode in ("banded", "whole"):
        got = dc.run_banded(x) if mode == "banded" else dc.run_whole(x)
        torch.cuda.synchronize()
        dc.check_device()
        assert rel_err(to_host_f32(got), want) <= TOL["bf16"], mode
    assert not torch.equal(first, dc.outs[-1])


def test_more_bands_than_rows_and_single_band():
    wl = li.build("vgg_block", H=12, W=20)
    for nb in (1, 6, 7, 13):                                     # 6 output rows: empty bands from 7 on
        check_workload(wl, n_bands=nb)
    for wl in (li.build("convnext_block", H=9, W=12, C=32), li.build("dense_layer", H=9, W=10)):
        for nb in (1, 9, 10, 19):                                # 9 output rows
            check_workload(wl, n_bands=nb)
            check_workload(wl, n_bands=nb, flags=lop.LOP_FLAG_REUSE_HALO, modes=("whole", "banded"))


def test_bands_in_any_order_without_reuse():
    wl = li.build("vgg_block", H=44, W=36)
    want = ochain.run_workload(wl)
    dc = DeviceChain(wl)
    dc.run_bands_one_by_one(dc.input_tensor(), order=lambda n: list(reversed(range(n))))
    torch.cuda.synchronize()
    assert rel_err(to_host_f32(dc.outs[-1]), want) <= TOL["bf16"]
    ref = DeviceChain(wl)
    ref.run_whole(ref.input_tensor())
    torch.cuda.synchronize()
    assert torch.equal(ref.outs[-1], dc.outs[-1])


def test_run_band_writes_only_its_rows():
    wl = li.build("vgg_block", H=44, W=36)
    dc = DeviceChain(wl)
    dc.outs[0].fill_(123.0)
    plan = dc.plans[0]
    plan.run_band(2, dc.input_tensor().data_ptr(), dc.outs[0].data_ptr(), dc.ws[0].data_ptr(),
                  torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    r = plan.get_range(2, plan.num_layers() - 1)
    out = to_host_f32(dc.outs[0])
    want = ochain.run_workload(wl)
    assert np.all(out[:, :r.out_lo] == 123.0) and np.all(out[:, r.out_hi:] == 123.0)
    assert rel_err(out[:, r.out_lo:r.out_hi], want[:, r.out_lo:r.out_hi]) <= TOL["bf16"]


def test_pipelined_timing_and_launch_count():
    wl = li.build("vgg_block")
    dc = DeviceChain(wl, flags=lop.LOP_FLAG_REUSE_HALO | lop.LOP_FLAG_TIME_LAYERS)
    x = dc.pinned_input()
    for _ in range(3):
        dc.run_pipelined(x)
    torch.cuda.synchronize()
    t = dc.plans[0].last_timing()
    assert t.n_copies == 8 and t.total_ms > 0 and 0 < t.first_copy_ms <= t.copy_ms
    assert dc.plans[0].last_launches() == 8 * (1 + 3)            # channel pad + three layers per band
    assert dc.plans[0].last_copies() == 8                        # one 2-D copy per band
    assert dc.plans[0].layer_time(0, 1) > 0 and dc.plans[0].layer_time(3, 2) > 0


@pytest.mark.parametrize("copy_engine", [False, True])
def test_wavefront_launch_counts_and_repeatability(copy_engine):
    wl = li.build("vgg_block")
    dc = DeviceChain(wl, flags=lop.LOP_FLAG_REUSE_HALO | (lop.LOP_FLAG_COPY_ENGINE if copy_engine else 0))
    x, xd = dc.pinned_input(), dc.input_tensor()
    first = None
    for i in range(5):                                           # run counters advance from launch to launch
        dc.staging.zero_()
        dc.run_pipelined(x)
        torch.cuda.synchronize()
        if i == 0:
            assert dc.plans[0].last_launches() == 1 + 1          # one persistent launch (+ weight padding once)
        else:                                                    # fetched: the launch is the only command of the call
            assert dc.plans[0].last_launches() == 1 and dc.plans[0].last_copies() == (8 if copy_engine else 0)
        assert torch.equal(dc.staging.view(-1), xd.view(-1)), "the input was not brought to the device in full"
        out = dc.outs[-1].clone()
        first = out if first is None else first
        assert torch.equal(out, first)
        dc.outs[-1].zero_()
    dc.run_banded(xd)
    torch.cuda.synchronize()
    assert dc.plans[0].last_launches() == 1 and torch.equal(dc.outs[-1], first)
    dc.check_device()


def test_fetched_pipeline_reads_the_host_buffer_afresh_on_every_call():
    """The kernel reads pinned host memory directly: a later call must see what the host wrote in between."""
    wl = li.build("vgg_block", H=44, W=36)
    dc = DeviceChain(wl, flags=lop.LOP_FLAG_REUSE_HALO)
    x = dc.pinned_input()
    dc.run_pipelined(x)
    torch.cuda.synchronize()
    first = dc.outs[-1].clone()
    keep = x.clone()
    x.mul_(-0.5)                                                 # the host changes its buffer in place
    wl.x = -0.5 * wl.x
    want = ochain.run_workload(wl)
    for _ in range(2):
        dc.run_pipelined(x)
        torch.cuda.synchronize()
        dc.check_device()
        assert rel_err(to_host_f32(dc.outs[-1]), want) <= TOL["bf16"]
        assert not torch.equal(dc.outs[-1], first)
    x.copy_(keep)
    dc.run_pipelined(x)
    torch.cuda.synchronize()
    assert torch.equal(dc.outs[-1], first)


@pytest.mark.parametrize("name,kw", [("vgg_block", dict(H=44, W=36)), ("resnet18", dict(H=64, W=64)), ("single_conv", {})])
def test_output_straight_into_pinned_host_memory(name, kw):
    """The last layer may store into host memory the device can address: same bits as the device tensor."""
    wl = li.build(name, **kw)
    dc = DeviceChain(wl, flags=lop.LOP_FLAG_REUSE_HALO)
    x = dc.pinned_input()
    dc.run_pipelined(x)
    torch.cuda.synchronize()
    want = dc.outs[-1].clone()
    dc.outs[-1].zero_()
    host = torch.zeros(want.shape, dtype=want.dtype).pin_memory()
    for _ in range(2):
        host.zero_()
        got = dc.run_pipelined(x, out_pinned=host)
        torch.cuda.synchronize()
        dc.check_device()
        assert got is host and torch.equal(host, want.cpu())
    assert not dc.outs[-1].any()                                 # the device output tensor was not touched
    s = torch.cuda.current_stream().cuda_stream
    host.zero_()
    xd = dc.input_tensor() if len(dc.plans) == 1 else dc.outs[-2]
    dc.plans[-1].run_whole(xd.data_ptr(), host.data_ptr(), dc.ws[-1].data_ptr(), s)
    torch.cuda.synchronize()
    assert torch.equal(host, want.cpu())


@pytest.mark.parametrize("N,H,W,C,cout", [(2, 21, 37, 3, 32), (3, 9, 21, 5, 32), (1, 33, 50, 64, 64), (2, 16, 9, 7, 64)])
def test_fetched_rows_of_any_length_and_alignment(N, H, W, C, cout):
    """Row lengths that are no multiple of 16 bytes: every fetch entry then starts and ends inside a 16-byte vector
    (2-byte head and tail around the vector body); several images, several bands, both band modes."""
    wl = one_layer(conv(C, cout, 3, act=li.ACT_RELU), N, H, W, n_bands=4)
    for flags in (0, lop.LOP_FLAG_REUSE_HALO):
        res = check_workload(wl, flags=flags, modes=("whole", "pipelined", "pipelined_copy"))
    dc = DeviceChain(wl, flags=lop.LOP_FLAG_REUSE_HALO, n_bands=4)
    x = dc.pinned_input()
    dc.staging.fill_(float("nan"))
    dc.run_pipelined(x)
    torch.cuda.synchronize()
    assert dc.plans[0].last_copies() == 0                       # the kernel brought the input itself ...
    assert torch.equal(dc.staging.cpu().view(-1), x.view(-1))   # ... all of it, bit for bit


def test_unaligned_and_unpinned_host_buffers_take_the_copy_path():
    wl = li.build("vgg_block", H=44, W=36)
    dc = DeviceChain(wl, flags=lop.LOP_FLAG_REUSE_HALO)
    x = dc.pinned_input()
    dc.run_pipelined(x)
    torch.cuda.synchronize()
    want = dc.outs[-1].clone()
    assert dc.plans[0].last_copies() == 0
    big = torch.empty(x.numel() + 8, dtype=x.dtype).pin_memory()
    off = big[1:1 + x.numel()].view(x.shape)                     # 2 bytes off the staging tensor's alignment
    off.copy_(x)
    pageable = x.clone()                                         # ordinary host memory
    assert not pageable.is_pinned()
    s = torch.cuda.current_stream().cuda_stream
    for host in (off, pageable):
        dc.outs[-1].zero_()
        dc.plans[0].run_pipelined(host.data_ptr(), dc.staging.data_ptr(), dc.outs[0].data_ptr(), dc.ws[0].data_ptr(), s)
        torch.cuda.synchronize()
        dc.check_device()
        assert dc.plans[0].last_copies() == dc.plans[0].num_bands()
        assert torch.equal(dc.outs[-1], want)


def test_wavefront_and_per_layer_executors_agree_bit_for_bit():
    for name, kw in (("resnet18", dict(H=96, W=96)), ("csp_stack", dict(H=256, W=256)), ("convnext_block", dict(H=40, W=24, C=96)),
                     ("dense_layer", {})):
        wl = li.build(name, **kw)
        a = DeviceChain(wl, flags=lop.LOP_FLAG_REUSE_HALO)
        b = DeviceChain(wl, flags=lop.LOP_FLAG_REUSE_HALO | lop.LOP_FLAG_PER_LAYER)
        a.run_banded(a.input_tensor())
        b.run_banded(b.input_tensor())
        torch.cuda.synchronize()
        for x, y in zip(a.outs, b.outs):
            assert torch.equal(x, y)


# ------------------------------------------------------------------------------------ the named configurations, full size
@pytest.mark.parametrize("name", ["vgg_block", "resnet18", "csp_stack", "pointwise_mlp", "convnext_block", "dense_layer"])
def test_named_configurations_full_size(name):
    check_workload(li.build(name), flags=lop.LOP_FLAG_REUSE_HALO, modes=("whole", "pipelined", "pipelined_copy"))


def test_resnet50_batch8_full_size():
    check_workload(li.build("resnet50"), flags=lop.LOP_FLAG_REUSE_HALO, modes=("pipelined", "pipelined_copy"))

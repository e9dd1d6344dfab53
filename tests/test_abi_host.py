"""Host-only checks of the C-ABI library: it loads, exports what include/lop.h declares, and its
planner agrees bit for bit with the oracle's planner.  No GPU is touched."""
import ctypes
import os
import random
import re

import pytest

import lop_inputs as li
import paper_2507_05829_b200 as lop
from lop_inputs.workloads import Layer
from oracle import planner
from test_oracle_planner import random_stack

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    L = lop.lib()
    header = open(os.path.join(ROOT, "include", "lop.h")).read()
    declared = set(re.findall(r"\b(lop_[a-z_]+)\s*\(", header))
    declared -= {"lop_plan_t"}
    assert declared == set(lop.EXPORTS)
    for name in declared:
        assert hasattr(L, name), name


def compare(layers, H, W, C, B, N=1, dtype=lop.LOP_F32):
    p = lop.Plan(layers, N, H, W, C, dtype, B)
    o = planner.make_plan(layers, H, W, C, B)
    assert p.num_bands() == B and p.num_layers() == len(layers)
    for i in range(len(layers)):
        assert p.out_shape(i) == tuple(o.shapes[i])
    assert p.out_shape(-1) == (H, W, C)
    for b in range(B):
        for i in range(len(layers)):
            assert p.get_range(b, i).astuple() == tuple(o.ranges[b][i]), (b, i)
        r = p.get_range(b, -1)
        assert (r.out_lo, r.out_hi, r.new_lo) == tuple(o.input_need[b])
        assert (r.in_lo, r.in_hi, r.pad_top, r.pad_bot) == (0, 0, 0, 0)
    p.destroy()
    return o


@pytest.mark.parametrize("name", list(li.WORKLOADS))
def test_plans_of_the_five_workloads_match_the_oracle_bit_for_bit(name):
    wl = li.build(name, with_data=False)
    H, W, C = wl.H, wl.W, wl.C
    dt = lop.LOP_BF16 if wl.dtype == "bf16" else lop.LOP_F32
    for seg in wl.segments:
        for B in {seg.n_bands, 1, 3}:
            o = compare(seg.layers, H, W, C, B, wl.N, dt)
        H, W, C = o.shapes[-1]


def test_random_stacks_match_the_oracle_bit_for_bit():
    rnd = random.Random(77)
    for _ in range(10000):
        layers, H = random_stack(rnd)
        compare(layers, H, 5, 1, rnd.randint(1, 7))


def test_flops_and_sizes():
    wl = li.build("vgg_block", with_data=False)
    p = lop.Plan(wl.segments[0].layers, 1, 224, 224, 3, lop.LOP_BF16, 8)
    assert p.flops() == 2.0 * 224 * 224 * 64 * (27 + 576)
    assert p.staging_bytes() == 224 * 224 * 3 * 2
    assert p.workspace_bytes() >= 224 * 224 * 64 * 2 * 2
    assert [p.layer_kernel(i) for i in range(3)] == [2, 2, 0]
    q = lop.Plan(wl.segments[0].layers, 1, 224, 224, 3, lop.LOP_BF16, 8, lop.LOP_FLAG_FORCE_SIMT)
    assert [q.layer_kernel(i) for i in range(3)] == [1, 1, 0]
    f = lop.Plan(li.build("single_conv", with_data=False).segments[0].layers, 1, 32, 32, 16, lop.LOP_F32, 4)
    assert f.layer_kernel(0) == 1 and f.staging_bytes() == 32 * 32 * 16 * 4


def test_errors_are_reported_not_raised_in_c():
    good = Layer(0, 4, 4, 3, 3, 1, 1, 1, 1, 1, 1, input_from=-1)
    for field, val, status in (("kh", 0, -2), ("sh", 0, -2), ("ph", -1, -2), ("cin", 5, -2), ("input_from", 0, -2),
                               ("op", 7, -1), ("act", 9, -1)):
        bad = Layer(**{**good.__dict__, field: val})
        with pytest.raises(lop.LopError) as e:
            lop.Plan([bad], 1, 8, 8, 4, lop.LOP_F32, 2)
        assert e.value.status == status, field
        assert str(e.value)
    for kw, status in ((dict(n_bands=0), -1), (dict(dtype=5), -1), (dict(N=0), -2), (dict(flags=64), -1)):
        args = dict(N=1, H=8, W=8, C=4, dtype=lop.LOP_F32, n_bands=2, flags=0)
        args.update(kw)
        with pytest.raises(lop.LopError) as e:
            lop.Plan([good], **args)
        assert e.value.status == status
    with pytest.raises(lop.LopError):
        lop.Plan([], 1, 8, 8, 4, lop.LOP_F32, 2)
    L = lop.lib()
    assert L.lop_plan_num_bands(None) == -1 and L.lop_plan_get_range(None, 0, 0, None) == -1
    assert L.lop_strerror(-5) == b"CUDA error" and L.lop_strerror(0) == b"success"
    L.lop_plan_destroy(None)
    assert L.lop_run_chain_banded(None, 0, None, None, None, None) == -1
    assert L.lop_run_chain_pipelined(None, 1, None, None, None, None, None) == -1
    p = lop.Plan([good], 1, 8, 8, 4, lop.LOP_F32, 2)
    with pytest.raises(lop.LopError):
        p.get_range(2, 0)
    with pytest.raises(lop.LopError):
        p.get_range(0, 1)
    # execution entry points validate on the host before touching CUDA
    assert L.lop_run_whole(p._h, None, None, None, None) == -1
    assert L.lop_run_band(p._h, 0, ctypes.c_void_p(16), ctypes.c_void_p(16), None, None) == -6
    assert L.lop_copy_band(p._h, 5, ctypes.c_void_p(16), ctypes.c_void_p(16), None) == -1


def test_row_wise_operator_must_not_carry_a_window():
    ok = li.linear(8, 16)
    ok.input_from = -1
    p = lop.Plan([ok], 1, 6, 5, 8, lop.LOP_BF16, 3)
    assert p.out_shape(0) == (6, 5, 16) and p.layer_kernel(0) == 2         # runs on the tensor-core pointwise path
    assert p.flops() == 2.0 * 6 * 5 * 16 * 8
    for field, val in (("kh", 3), ("sw", 2), ("ph", 1), ("dh", 2)):
        bad = li.linear(8, 16)
        bad.input_from = -1
        setattr(bad, field, val)
        with pytest.raises(lop.LopError) as e:
            lop.Plan([bad], 1, 6, 5, 8, lop.LOP_BF16, 3)
        assert e.value.status == -1 and "row-wise" in str(e.value)


def test_the_developer_trace_build_compiles(tmp_path):
    """-DLOP_WF_TRACE adds per-item time stamps of the persistent kernel's roles and the lop_debug_* readers (a developer
    build, never the shipped library): it must keep compiling for sm_100a as the kernel changes."""
    import glob
    import subprocess
    csrc = os.path.join(ROOT, "paper_2507_05829_b200", "csrc")
    out = str(tmp_path / "trace.o")
    cmd = ["/usr/local/cuda/bin/nvcc", "-gencode", "arch=compute_100a,code=sm_100a", "-std=c++17", "-DLOP_WF_TRACE", "-I",
           os.path.join(ROOT, "include"), "-I", csrc, "-c", os.path.join(csrc, "lop_wavefront.cu"), "-o", out]
    r = subprocess.run(cmd, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stderr[-2000:]
    syms = subprocess.run(["nm", "-g", out], capture_output=True, text=True).stdout
    assert "lop_debug_trace_copy" in syms and "lop_debug_last_items" in syms
    assert not any("lop_debug" in e for e in lop.EXPORTS)          # the shipped library exports none of them

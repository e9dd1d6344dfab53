"""lop_run_whole_static: the execution entry point for callers that may not allocate.

A plug-in inside an application that forbids cudaMalloc after start-up, or a loop that must never
wait on the allocator, cannot hand the library a workspace.  This entry point takes its scratch
from a fixed array inside the library instead.  The checks here: it computes exactly what
lop_run_whole computes, it keeps doing so when the shared array is dirty from another plan's
call, it performs no device allocation, and it refuses plans that do not fit.

The file name sorts last on purpose: a run that stops at the first failure has then already run
every other test.
"""
import ctypes

import numpy as np
import pytest
import torch

import lop_inputs as li
import paper_2507_05829_b200 as lop
from oracle import chain as ochain
from paper_2507_05829_b200.chain import DeviceChain


def test_plan_larger_than_the_built_in_scratch_is_refused():
    """Host-only: the size check comes before any CUDA call and names both sizes."""
    wl = li.build("csp_stack", with_data=False)
    p = lop.Plan(wl.segments[0].layers, wl.N, wl.H, wl.W, wl.C, lop.LOP_BF16, 32)
    assert p.workspace_bytes() > lop.LOP_STATIC_SCRATCH_BYTES
    with pytest.raises(lop.LopError) as e:
        p.run_whole_static(ctypes.c_void_p(256), ctypes.c_void_p(256), None, None)
    assert e.value.status == -3
    assert str(lop.LOP_STATIC_SCRATCH_BYTES) in str(e.value) and str(p.workspace_bytes()) in str(e.value)
    assert lop.lib().lop_run_whole_static(None, None, None, None, None) == -1


TOL = {"f32": 1e-4, "bf16": 2e-2}       # max |gpu - oracle| / max |oracle|, the tolerances of the other GPU tests


def _oracle_err(got, want):
    """Distance of a device tensor from the CPU oracle's result, relative to the oracle's output scale."""
    g = got.detach().to("cpu", torch.float32).numpy().astype(np.float64)
    return float(np.max(np.abs(g - want))) / float(np.max(np.abs(want)))


def _reference(wl):
    dc = DeviceChain(wl)
    x = dc.input_tensor()
    want = dc.run_whole(x).clone()
    torch.cuda.synchronize()
    dc.check_device()
    return dc, x, want


@pytest.mark.gpu
def test_static_scratch_entry_point_matches_run_whole_on_two_calls_in_a_row():
    # the benchmark block at full size (tensor-core convolutions, channel-padded input, pooling) and a
    # residual chain that mixes kernels; the second one dirties the shared array between the two calls
    vgg = li.build("vgg_block")
    res = li.build("resnet18", H=64, W=64)
    dcv, xv, want_v = _reference(vgg)
    dcr, xr, _ = _reference(res)
    want_r = dcr.outs[0].clone()
    assert dcv.plans[0].workspace_bytes() <= lop.LOP_STATIC_SCRATCH_BYTES
    stream = torch.cuda.Stream()
    status = torch.full((1,), 77, dtype=torch.int32, device="cuda")
    out_v = torch.empty_like(want_v)
    out_r = torch.empty_like(want_r)
    s = stream.cuda_stream
    stream.wait_stream(torch.cuda.current_stream())

    # first call on this device resolves the array's address; then measure that nothing is allocated
    dcv.plans[0].run_whole_static(xv.data_ptr(), out_v.data_ptr(), status.data_ptr(), s)
    stream.synchronize()
    assert torch.equal(out_v, want_v) and int(status.item()) == 0
    # the oracle's results: the whole VGG block, and the first segment (stem + pooling) of the residual network
    oracle_v = ochain.run_workload(vgg)
    oracle_r = ochain.run_whole(res.segments[0].layers, res.x, True)
    free_before = None
    for call in range(3):
        out_v.fill_(-5.0)
        out_r.fill_(-5.0)
        status.fill_(77)
        dcv.plans[0].run_whole_static(xv.data_ptr(), out_v.data_ptr(), status.data_ptr(), s)
        dcr.plans[0].run_whole_static(xr.data_ptr(), out_r.data_ptr(), None, s)      # segment 0: stem + pool
        stream.synchronize()
        assert torch.equal(out_v, want_v), "call %d differs from lop_run_whole" % call
        assert torch.equal(out_r, want_r), "call %d (second plan) differs from lop_run_whole" % call
        assert _oracle_err(out_v, oracle_v) <= TOL["bf16"], "call %d differs from the oracle" % call
        assert _oracle_err(out_r, oracle_r) <= TOL["bf16"], "call %d (second plan) differs from the oracle" % call
        assert int(status.item()) == 0
        if free_before is None:                 # torch's own caches for fill_/equal/item are warm from here on
            free_before, _ = torch.cuda.mem_get_info()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before, "device memory was allocated during the calls"


@pytest.mark.gpu
def test_static_scratch_entry_point_fp32_and_cuda_core_paths():
    for wl, flags in ((li.build("single_conv"), 0), (li.build("vgg_block", H=44, W=36), lop.LOP_FLAG_FORCE_SIMT)):
        dc = DeviceChain(wl, flags=flags)
        x = dc.input_tensor()
        want = dc.run_whole(x).clone()
        torch.cuda.synchronize()
        got = torch.zeros_like(want)
        for _ in range(2):
            got.zero_()
            dc.plans[0].run_whole_static(x.data_ptr(), got.data_ptr(), None, torch.cuda.current_stream().cuda_stream)
            torch.cuda.synchronize()
            assert torch.equal(got, want)
            assert _oracle_err(got, ochain.run_workload(wl)) <= TOL[wl.dtype]

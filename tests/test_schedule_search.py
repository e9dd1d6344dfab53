"""The band-count search (the paper's scheduling optimisation re-targeted to one GPU behind a host link)."""
import numpy as np
import pytest

import lop_inputs as li
from paper_2507_05829_b200 import schedule_search as ss


def test_differential_evolution_finds_the_minimum_of_a_known_cost():
    target = (8, 2, 32, 1)

    def cost(bands):
        return sum(abs(ss.BAND_CHOICES.index(b) - ss.BAND_CHOICES.index(t)) ** 2 for b, t in zip(bands, target)) + 3.0

    best, value, evals = ss.search(cost, 4, seed=5, generations=40)
    assert best == target and value == 3.0
    assert evals < len(ss.BAND_CHOICES) ** 4          # far fewer evaluations than the grid has points


def test_the_model_charges_the_transfer_and_the_per_band_overhead():
    wl = li.build("vgg_block", with_data=False)
    slow_link = dict(ss.MACHINE, link_gbs=2.0)
    fast_link = dict(ss.MACHINE, link_gbs=200.0)
    # a slow link: one band waits for the whole image before it computes anything, several bands overlap the transfer
    assert ss.cost_model(wl, (8,), slow_link) < ss.cost_model(wl, (1,), slow_link)
    # the faster the link, the less there is to gain from overlapping it
    gain = lambda m: ss.cost_model(wl, (1,), m) - min(ss.cost_model(wl, (b,), m) for b in ss.BAND_CHOICES)
    assert 0.0 <= gain(fast_link) < gain(slow_link)
    # and a faster link never makes the same plan slower
    for b in ss.BAND_CHOICES:
        assert ss.cost_model(wl, (b,), fast_link) <= ss.cost_model(wl, (b,), slow_link)


def test_choose_returns_the_fastest_measured_candidate_with_a_stub_device():
    wl = li.build("resnet18", with_data=False, H=64, W=64)
    calls = []

    def fake_measure(w, bands):
        calls.append(bands)
        return 100.0 + sum(bands)                     # the stub device likes few bands

    best, us, report = ss.choose(wl, measure_top=3, measure=fake_measure)
    assert best in calls and us == 100.0 + sum(best)
    assert tuple(seg.n_bands for seg in wl.segments) in calls          # the workload's own plan is always measured too
    assert us == min(100.0 + sum(b) for b in calls)
    assert report["candidates_modelled"] > len(calls)


@pytest.mark.gpu
def test_search_with_the_measured_objective_on_the_device():
    """On the GPU: the chosen band counts are never slower than the workload's own (both measured the same way), and the
    chain still matches the oracle with them."""
    import numpy as np
    import torch
    import paper_2507_05829_b200 as lop
    from oracle import chain as ochain
    from paper_2507_05829_b200.chain import DeviceChain, to_host_f32
    wl = li.build("csp_stack", H=256, W=256)
    best, us, report = ss.choose(wl, measure_top=3)
    own = str(tuple(seg.n_bands for seg in wl.segments))
    assert us <= report["measured_us"][own] + 1e-9
    dc = DeviceChain(wl, flags=lop.LOP_FLAG_REUSE_HALO, n_bands=list(best))
    dc.run_pipelined(dc.pinned_input())
    torch.cuda.synchronize()
    dc.check_device()
    want = ochain.run_workload(wl)
    got = to_host_f32(dc.outs[-1])
    assert float(np.max(np.abs(got - want))) / float(np.max(np.abs(want))) <= 2e-2


def test_model_covers_every_operator_kind():
    """Depth-wise convolution, layer normalisation and concatenation are costed as row items: the model returns a
    finite latency for the ConvNeXt block and the DenseNet layer, and more bands never cost less than the launch."""
    for name in ("convnext_block", "dense_layer", "pointwise_mlp"):
        wl = li.build(name, with_data=False)
        for nb in (1, 4, 8):
            t = ss.cost_model(wl, [nb])
            assert np.isfinite(t) and t > ss.MACHINE["launch_us"]

"""Runs one named case of the library a few times, for captures under a profiler.

    python -m paper_2507_05829_b200.profile_case <case> [launches]

Cases: a named workload (``vgg_block``, ``resnet18``, ``resnet50``, ``csp_stack``: all bands from a device-resident
input, one persistent launch per run; ``<name>:pipelined`` streams the bands from pinned host memory), ``pool`` (a
3x3 stride-2 max pooling of an 8 x 224 x 224 x 64 bf16 tensor by the stand-alone kernel and, with ``pool:persistent``,
by pooling items of the persistent kernel), ``gather`` (patch gather + 7x7 stride-2 stem convolution of 8 images by
the stand-alone kernels; ``gather:persistent`` inside the persistent kernel), ``convnext_block`` / ``dense_layer``
(depth-wise convolution, layer normalisation, concatenation: items of the persistent kernel; ``<name>:per_layer``
runs the stand-alone kernels, one launch per layer), ``dwconv`` / ``layernorm`` / ``concat`` (one such operator on an
8 x 224 x 224 x 64 tensor, stand-alone kernel or ``:persistent``).  The L2 is flushed before every run.
"""
import sys

import torch

import lop_inputs as li
from lop_inputs.workloads import Segment, Workload, conv, pool

from . import binding as B
from .chain import DeviceChain


def build_case(name):
    base, _, mode = name.partition(":")
    if base in ("vgg_block", "resnet18", "resnet50", "csp_stack", "single_conv", "pointwise_mlp", "convnext_block", "dense_layer"):
        if mode == "per_layer":                                   # one stand-alone kernel per layer, whole tensors
            return li.build(base), "whole", B.LOP_FLAG_PER_LAYER
        return li.build(base), (mode or "banded"), 0
    if base == "pool":
        l = pool(64, 3, 2, 1)
        l.input_from = -1
        wl = Workload("pool_only", "bf16", 8, 224, 224, 64, [Segment([l], 1)], seed=1)
    elif base in ("dwconv", "layernorm", "concat"):
        # the memory-bound operators on a tensor larger than the L2: 8 x 224 x 224 x 64 bf16 (51 MB)
        if base == "dwconv":
            layers = [li.dwconv(64, 7)]
        elif base == "layernorm":
            layers = [li.layernorm(64)]
        else:
            layers = [pool(64, 1, 1, 0), li.concat(64, 64, input_from=-1, second_from=0)]     # a copy, then input ++ copy
        layers[0].input_from = -1
        wl = Workload(base + "_only", "bf16", 8, 224, 224, 64, [Segment(layers, 1)], seed=1)
    elif base == "gather":
        l = conv(3, 64, 7, s=2, p=3, act=li.ACT_RELU)
        l.input_from = -1
        wl = Workload("stem_only", "bf16", 8, 224, 224, 3, [Segment([l], 1)], seed=1)
    else:
        raise SystemExit("unknown case %r" % name)
    li.fill_parameters(wl)
    li.make_input(wl)
    return wl, "whole", (0 if mode == "persistent" else B.LOP_FLAG_PER_LAYER)


def record_traffic(workload, ncu_csv):
    """Reads dram__bytes_read.sum + dram__bytes_write.sum of the persistent kernel's captured launch from an ``ncu --csv``
    log and stores their sum under ``workload`` in profiles/dram_traffic.json, together with the hash of the kernel's
    sources (bench.py reports the figure only while that hash still matches)."""
    import csv
    import json
    import os
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    sys.path.insert(0, root)
    import bench
    total, units = 0.0, {"byte": 1.0, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9}
    rows = [r for r in csv.reader(open(ncu_csv)) if len(r) > 10]
    hdr = rows[0]
    for r in rows[1:]:
        d = dict(zip(hdr, r))
        if "wavefront_kernel" in d.get("Kernel Name", "") and d.get("Metric Name") in ("dram__bytes_read.sum", "dram__bytes_write.sum"):
            total += float(d["Metric Value"].replace(",", "")) * units[d["Metric Unit"]]
    if total <= 0:
        raise SystemExit("no DRAM counters of the persistent kernel in %s" % ncu_csv)
    path = os.path.join(root, "profiles", "dram_traffic.json")
    rec = {"kernel_hash": bench.kernel_hash(), "bytes_per_launch": {}}
    if os.path.exists(path):
        old = json.load(open(path))
        if old.get("kernel_hash") == rec["kernel_hash"]:
            rec = old
    rec["bytes_per_launch"][workload] = total
    rec["what"] = "dram__bytes_read.sum + dram__bytes_write.sum of one wavefront_kernel launch (all bands, device-resident input), ncu, L2 flushed before the launch"
    json.dump(rec, open(path, "w"), indent=1, sort_keys=True)
    print("%s: %.1f MB per launch (kernel %s)" % (workload, total / 1e6, rec["kernel_hash"]))


def main():
    if len(sys.argv) > 1 and sys.argv[1] == "--record-traffic":
        return record_traffic(sys.argv[2], sys.argv[3])
    name = sys.argv[1] if len(sys.argv) > 1 else "resnet50"
    launches = int(sys.argv[2]) if len(sys.argv) > 2 else 3
    wl, mode, flags = build_case(name)
    dc = DeviceChain(wl, flags=B.LOP_FLAG_REUSE_HALO | flags)
    x_dev, x_pin = dc.input_tensor(), dc.pinned_input()
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    for _ in range(launches):
        flush.zero_()
        if mode == "pipelined":
            dc.run_pipelined(x_pin)
        elif mode == "whole":
            dc.run_whole(x_dev)
        else:
            dc.run_banded(x_dev)
        torch.cuda.synchronize()
    dc.check_device()
    print("%s: %d run(s) of mode %s, %d launch(es) of the library's kernels per run" % (name, launches, mode, dc.launches()))


if __name__ == "__main__":
    main()

#!/usr/bin/env python
"""Benchmark of the band-pipelined local-operator chain on B200.

One *step* = one pass of the whole hot path over one batch of synthetic input: plan lookup,
per band the pinned-host -> device transfer, channel padding, every convolution / pooling
layer on the band's rows, and the stitched write of the output.

  value   images/s with the input already resident in HBM (all bands, no transfer)
  e2e     images/s through the C ABI from PINNED HOST input (band copies overlapped with
          compute on a side stream) plus the device -> host read of the output
  roofline   the dominant kernel (tensor-core convolution of the widest layer) against the
             measured bf16 peak, timed with CUDA events around each of its launches
  cpu_baseline  the CPU oracle, as it stands, timed on this machine's host cores

Usage:  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]
Multi-GPU (torchrun): every rank runs the same chain on its own images (independent replicas,
no data-path collective); the time is the maximum over ranks.
"""
import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

# dram__bytes_read.sum + dram__bytes_write.sum of one wavefront_kernel launch (ncu --set full, see
# profiles/wavefront_kernel_vgg_block.md and profiles/wavefront_kernel_resnet18_resnet50_csp_stack.md); None for workloads not captured, or once the kernel has changed since
TRAFFIC = {"vgg_block": 509.2e3, "resnet18": 22.8e6, "resnet50": 236.3e6, "csp_stack": 37.0e6}

METRIC = "band-pipelined conv-chain images/s"
UNIT = "images/s"
DEFAULT_WORKLOAD = "vgg_block"
WORKLOAD_NOTES = {
    "single_conv": "cfg1 single conv3x3 16->16 1x32x32 fp32, 4 bands",
    "vgg_block": "cfg2 VGG block conv3x3(3->64)+ReLU, conv3x3(64->64)+ReLU, maxpool2x2; 1x224x224x3 bf16, 8 row bands",
    "resnet18": "cfg3 ResNet-18 conv trunk 1x224x224x3 bf16, 5 segments x 8 bands",
    "resnet50": "cfg4 ResNet-50 bottleneck trunk 8x224x224x3 bf16, 5 segments x 16 bands, pinned-host input",
    "csp_stack": "cfg5 CSP-style 12-layer stack 1x1024x1024x3 bf16, 32 bands, pinned-host input",
}


def load_peaks():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), "source": "measured"}
    except Exception:
        return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.idx, self.proc, self.lines = gpu_index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.idx), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.12)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                mx.append(float(f[2]))
            except ValueError:
                continue
            for name, v in zip(names, f[5:9]):
                if v == "Active":
                    reasons.add(name)
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def time_oracle(wl, min_seconds):
    """The CPU oracle, as it stands, on whole images of the workload until ``min_seconds`` have passed."""
    from oracle import chain as ochain, ops
    t0 = time.perf_counter()
    runs = 0
    while True:
        ochain.run_workload(wl)
        runs += 1
        dt = time.perf_counter() - t0
        if dt >= min_seconds or runs >= 64:
            break
    return {"value": wl.N * runs / dt, "unit": UNIT, "cores": ops.num_threads(), "kind": "oracle",
            "sample": "%d whole pass(es) of the workload (N=%d), %.1f s" % (runs, wl.N, dt)}, dt / runs


def max_over_ranks(ms, device=None):
    """The slowest rank's time: every rank runs its own replica, the job is as slow as the slowest of them."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(ms)
    t = torch.tensor([float(ms)], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_images_per_s(images_per_rank, world, ms_per_step):
    """Whole-job throughput of `world` independent replicas (weak scaling, no data-path collective)."""
    return images_per_rank * world / (ms_per_step * 1e-3)


def run_reference(args):
    """The reference arm: the CPU oracle timed on the host cores, rank 0 only."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    import lop_inputs as li
    wl = li.build(args.workload)
    for _ in range(min(args.warmup, 1)):
        time_oracle(wl, 0.0)
    per_step = []
    budget = 150.0
    t_all = time.perf_counter()
    for _ in range(args.steps):
        cb, sec = time_oracle(wl, 0.0)
        per_step.append(sec)
        if time.perf_counter() - t_all > budget:
            break
    from oracle import ops
    ms = 1e3 * sum(per_step) / len(per_step)
    val = wl.N / (ms / 1e3)
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
            "steps": len(per_step), "warmup": min(args.warmup, 1), "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64 accumulate, %s storage" % wl.dtype,
            "data": "synthetic", "config": {"workload": WORKLOAD_NOTES[args.workload]},
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": ops.num_threads(), "kind": "oracle",
                             "sample": "each step = one whole pass of the workload on the host cores"},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=list(WORKLOAD_NOTES))
    ap.add_argument("--impl", default="native", choices=["native", "reference"])
    ap.add_argument("--no-graph", action="store_true", help="enqueue every step launch by launch instead of replaying a CUDA graph")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()

    if args.impl == "reference":
        args.steps = 3 if args.steps is None else args.steps
        args.warmup = 1 if args.warmup is None else args.warmup
        run_reference(args)
        return
    args.steps = 1000 if args.steps is None else args.steps
    args.warmup = 20 if args.warmup is None else max(args.warmup, 3)

    import numpy as np
    import torch
    import torch.distributed as dist
    import lop_inputs as li
    import paper_2507_05829_b200 as lop
    from paper_2507_05829_b200.chain import DeviceChain

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU path (use --impl reference for the oracle)")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if world > 1:
            dist.barrier()

    peaks = load_peaks()
    wl = li.build(args.workload)
    flags = lop.LOP_FLAG_REUSE_HALO
    dc = DeviceChain(wl, flags=flags, device=dev)
    x_dev = dc.input_tensor()
    x_pin = dc.pinned_input()
    out_pin = torch.empty(dc.outs[-1].shape, dtype=dc.outs[-1].dtype).pin_memory()
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)      # > 126 MB L2
    stream = torch.cuda.Stream(device=dev)

    def step_resident():
        dc.run_banded(x_dev, stream)

    def step_e2e():
        # input: the kernel fetches the bands from pinned host memory; result: the last layer stores it straight into
        # pinned host memory -- both transfers are inside the timed region, neither is a separate copy command
        dc.run_pipelined(x_pin, stream, out_pinned=out_pin)

    def make_runner(fn, graph=True):
        """Either the function itself or a CUDA graph of one step (captured after an eager warm-up)."""
        with torch.cuda.stream(stream):
            fn()
        stream.synchronize()
        if args.no_graph or not graph:
            return fn, None
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            fn()
        return g.replay, g

    def timed(run, steps, warmup):
        with torch.cuda.stream(stream):
            for _ in range(warmup):
                flush.zero_()
                run()
            stream.synchronize()
            barrier()
            torch.cuda.synchronize()
            evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
            for a, b in evs:
                flush.zero_()                                      # L2 flush between timed iterations
                a.record(stream)
                run()
                b.record(stream)
            stream.synchronize()
            torch.cuda.synchronize()
            barrier()
        total = sum(a.elapsed_time(b) for a, b in evs)
        return max_over_ranks(total, dev) / steps

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    run_res, g1 = make_runner(step_resident)
    ms_res = timed(run_res, args.steps, args.warmup)
    launches_res = dc.launches()
    # the end-to-end arm is plain calls, the way a user makes them: replaying the kernel + copies + arrival writes from a
    # graph was measured slower than enqueueing them
    run_e2e, g2 = make_runner(step_e2e, graph=False)
    ms_e2e = timed(run_e2e, args.steps, args.warmup)
    clocks = sampler.stop() if rank == 0 else None
    dc.check_device()
    if not torch.equal(out_pin, dc.outs[-1].cpu()):                # the resident arm left the same result on the device
        raise SystemExit("bench: the end-to-end arm's host result differs from the resident arm's device result")

    # ---- pipeline accounting: copies alone, compute alone, both overlapped (eager launches, with events)
    def copies_only():
        for b in range(dc.plans[0].num_bands()):
            dc.plans[0].copy_band(b, x_pin.data_ptr(), dc.staging.data_ptr(), stream.cuda_stream)

    def pipe_only():
        dc.run_pipelined(x_pin, stream)

    def first_copy_only():
        dc.plans[0].copy_band(0, x_pin.data_ptr(), dc.staging.data_ptr(), stream.cuda_stream)

    def first_copy_only():
        dc.plans[0].copy_band(0, x_pin.data_ptr(), dc.staging.data_ptr(), stream.cuda_stream)

    n_acc = max(20, min(200, args.steps))
    t_copy = timed(copies_only, n_acc, 3)
    t_first = timed(first_copy_only, n_acc, 3)
    t_comp = timed(step_resident, n_acc, 3)
    t_pipe = timed(pipe_only, n_acc, 3)
    exposed = max(0.0, t_pipe - t_comp)
    hidden = 100.0 * (1.0 - exposed / t_copy) if t_copy > 0 else None
    # no schedule can hide band 0's copy, nor more copy time than there is compute
    bound = 100.0 * min(1.0 - t_first / t_copy if t_copy > 0 else 0.0, t_comp / t_copy if t_copy > 0 else 1.0)

    # ---- dominant kernel: the persistent wavefront kernel; in the `value` arm one step is exactly one launch of
    # it, so the per-step CUDA events of the timed region are its launch durations
    conv_fl = dc.flops()
    achieved = conv_fl / (ms_res * 1e-3) / 1e12
    if wl.dtype == "bf16":
        roofline = {"bound": "tensor", "kernel": "wavefront_kernel (all-bands program: every gather / conv / pool stage of the step in one persistent launch per segment)",
                    "achieved": achieved, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                    "frac": achieved / peaks["bf16_tflops"],
                    "peak_source": "%s TFLOP/s burst bf16 (of %s)" % (peaks["bf16_tflops"], peaks["source"]),
                    "flops_per_launch": conv_fl, "avg_launch_us": ms_res * 1e3, "launches_per_step": launches_res,
                    "traffic": TRAFFIC.get(args.workload)}
    else:
        # fp32 storage runs on the CUDA cores: plain-ALU peak = SMs x 128 FMA lanes x 2 flop x max SM clock
        props = torch.cuda.get_device_properties(dev)
        mhz = (clocks or {}).get("sm_max_mhz") or 1965.0
        alu_peak = props.multi_processor_count * 128 * 2 * mhz * 1e6 / 1e12
        roofline = {"bound": "alu", "kernel": "conv_simt_kernel (one launch per band)", "achieved": achieved, "peak": alu_peak,
                    "unit": "TFLOP/s", "frac": achieved / alu_peak,
                    "peak_source": "derived: %d SMs x 128 fp32 FMA lanes x 2 x %.0f MHz" % (props.multi_processor_count, mhz),
                    "flops_per_launch": conv_fl / max(launches_res, 1), "avg_launch_us": ms_res * 1e3 / max(launches_res, 1),
                    "launches_per_step": launches_res, "traffic": None}

    # ---- per-layer view: whole-tensor launches, one kernel per layer, CUDA events around each (eager)
    dct = DeviceChain(wl, flags=lop.LOP_FLAG_PER_LAYER | lop.LOP_FLAG_TIME_LAYERS, device=dev)
    acc = {}
    reps = 20
    for r in range(reps + 3):
        with torch.cuda.stream(stream):
            flush.zero_()
            dct.run_whole(x_dev, stream)
        stream.synchronize()
        if r < 3:
            continue
        for s_, (seg, plan) in enumerate(zip(wl.segments, dct.plans)):
            for i in range(len(seg.layers)):
                acc[(s_, i)] = acc.get((s_, i), 0.0) + plan.layer_time(-1, i)
    per_layer = []
    es = 2 if wl.dtype == "bf16" else 4
    for s_, (seg, plan) in enumerate(zip(wl.segments, dct.plans)):
        for i, l in enumerate(seg.layers):
            ms = acc[(s_, i)] / reps
            ho, wo, co = plan.out_shape(i)
            hi, wi, ci = plan.out_shape(l.input_from)
            if l.op == 0:
                fl = 2.0 * wl.N * ho * wo * co * l.kh * l.kw * l.cin
                per_layer.append({"segment": s_, "layer": i, "op": "conv%dx%d s%d %d->%d" % (l.kh, l.kw, l.sh, l.cin, l.cout),
                                  "kernel": ["pool", "cuda-core", "tcgen05"][plan.layer_kernel(i)], "us": ms * 1e3,
                                  "tflops": fl / (ms * 1e-3) / 1e12,
                                  "pct_of_burst_peak": 100.0 * fl / (ms * 1e-3) / 1e12 / peaks["bf16_tflops"]})
            else:
                by = wl.N * (hi * wi * ci + ho * wo * co) * es
                per_layer.append({"segment": s_, "layer": i, "op": "maxpool%dx%d s%d" % (l.kh, l.kw, l.sh), "kernel": "pool",
                                  "us": ms * 1e3, "gbs": by / (ms * 1e-3) / 1e9,
                                  "pct_of_hbm_peak": 100.0 * by / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"]})
    if len(per_layer) > 16:                                   # keep the line readable: the slowest layers only
        per_layer = sorted(per_layer, key=lambda d: -d["us"])[:16]

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    line = {
        "metric": METRIC, "value": job_images_per_s(wl.N, world, ms_res), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_res, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16" if wl.dtype == "bf16" else "f32", "data": "synthetic",
        "config": {"workload": WORKLOAD_NOTES[args.workload], "images_per_step_per_gpu": wl.N,
                   "mode": "reuse-halo bands", "launch": "eager" if args.no_graph else "value: cuda-graph replay of one step; e2e: eager calls",
                   "e2e_transport": "input bands fetched from pinned host memory by the persistent kernel's fetch warps; result "
                                    "stored by the last layer straight into pinned host memory; one launch, no copy commands",
                   "l2": "256 MiB buffer written between timed steps", "multi_gpu": "independent replicas"},
        "e2e": {"value": job_images_per_s(wl.N, world, ms_e2e), "unit": UNIT, "ms_per_step": ms_e2e,
                "h2d_bytes_per_step": int(x_pin.numel() * x_pin.element_size()),
                "d2h_bytes_per_step": int(out_pin.numel() * out_pin.element_size())},
        "gpu_launches": int(launches_res * args.steps),
        "clocks": clocks,
        "roofline": roofline,
        "conv_tflops": {"whole_step_useful": achieved, "pct_of_burst_peak": 100.0 * achieved / peaks["bf16_tflops"],
                        "pct_of_sustained_peak": 100.0 * achieved / peaks["bf16_tflops_sustained"],
                        "per_layer_launches": per_layer},
        "pipeline": {"t_copy_ms": t_copy, "t_compute_ms": t_comp, "t_pipelined_ms": t_pipe, "exposed_ms": exposed,
                     "hidden_pct": hidden, "hidden_pct_bound": bound, "first_copy_ms": t_first,
                     "n_bands": dc.plans[0].num_bands(),
                     "note": "t_copy / first_copy: the bands as copy-engine copies alone, back to back on one stream (the "
                             "transmission the pipeline has to hide; the bound is computed from them). t_pipelined: one "
                             "launch whose fetch warps read the bands from pinned host memory while the other warps compute, "
                             "output left on the device; it can beat the bound because the kernel's fetch has no per-copy "
                             "command cost",
                     "launch": "eager calls"},
    }
    if world == 1 and not args.no_cpu_baseline:
        cb, _ = time_oracle(wl, 10.0)
        line["cpu_baseline"] = cb
    else:
        line["cpu_baseline"] = None
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()

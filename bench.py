#!/usr/bin/env python
"""Benchmark of the band-pipelined local-operator chain on B200.

One *step* = one pass of the whole hot path over one batch of synthetic input: the bands' transfer from
pinned host memory, the patch gather of the image, every convolution / pooling layer on every band's rows,
the stitched write of the output -- one call of the library's pipelined entry point.

  value      images/s of the BAND-PIPELINED path: input bands stream from pinned host memory while the
             rows already there are computed (lop_run_chain_pipelined / lop_run_pipelined), output left on
             the device.  The transfer starts inside the timed region; only the buffers are resident.
  e2e        the same call with the result also stored to pinned host memory (host to host)
  resident   extra key: all bands from a device-resident input (no transfer) -- the compute-only time
  steady_state  R requests back to back on one stream, N*R / T
  roofline   the dominant kernel (the persistent wavefront kernel: one launch per step) against the
             measured bf16 peak, from the CUDA-event time of its launches in the timed region
  pipeline   per transport (kernel fetch / copy engine): transfer alone, first band alone, compute alone,
             pipelined; hidden % and its bound
  per_config the other configurations, measured the same way with fewer steps
  cpu_baseline  the CPU oracle, as it stands, timed on this machine's host cores

Usage:  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]
Multi-GPU (torchrun): every rank runs the same chain on its own images (independent replicas,
no data-path collective); the time is the maximum over ranks.
"""
import argparse
import hashlib
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "band-pipelined conv-chain images/s"
UNIT = "images/s"
DEFAULT_WORKLOAD = "resnet50"
WORKLOAD_NOTES = {
    "single_conv": "cfg1 single conv3x3 16->16 1x32x32 fp32, 4 bands",
    "vgg_block": "cfg2 VGG block conv3x3(3->64)+ReLU, conv3x3(64->64)+ReLU, maxpool2x2; 1x224x224x3 bf16, 8 row bands",
    "resnet18": "cfg3 ResNet-18 conv trunk 1x224x224x3 bf16, 5 segments x 8 bands",
    "resnet50": "cfg4 ResNet-50 bottleneck trunk 8x224x224x3 bf16, 5 segments x 16 bands, bands streamed from pinned host memory",
    "csp_stack": "cfg5 CSP-style 12-layer stack 1x1024x1024x3 bf16, 32 bands, bands streamed from pinned host memory",
}
STEADY_REQUESTS = 8
KERNEL_SOURCES = ("lop_wavefront.cu", "lop_wavefront.cuh", "lop_program.cu", "lop_ptx.cuh", "lop_gather.cuh", "lop_rowops.cuh")


def kernel_hash():
    """Identifies the persistent kernel's sources: DRAM counters taken from another version are not reported."""
    h = hashlib.sha256()
    for name in KERNEL_SOURCES:
        with open(os.path.join(ROOT, "paper_2507_05829_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def dram_traffic(workload):
    """dram__bytes_read.sum + dram__bytes_write.sum of one launch of the persistent kernel on this workload, from the
    counters the profiling step left beside its summaries -- or None when there are none for this kernel version."""
    try:
        with open(os.path.join(ROOT, "profiles", "dram_traffic.json")) as f:
            rec = json.load(f)
        if rec.get("kernel_hash") != kernel_hash():
            return None
        return rec["bytes_per_launch"].get(workload)
    except Exception:
        return None


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


class Timer:
    """CUDA-event timing of steps on one stream, L2 flushed between steps, maximum over ranks."""

    def __init__(self, torch, stream, flush, barrier, dev):
        self.torch, self.stream, self.flush, self.barrier, self.dev = torch, stream, flush, barrier, dev

    def __call__(self, run, steps, warmup, per_step=1):
        """Mean milliseconds of one step; a step is `per_step` back-to-back calls of run() behind one L2 flush."""
        torch = self.torch
        with torch.cuda.stream(self.stream):
            for _ in range(warmup):
                self.flush.zero_()
                for _ in range(per_step):
                    run()
            self.stream.synchronize()
            self.barrier()
            torch.cuda.synchronize()
            evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
            for a, b in evs:
                self.flush.zero_()                                 # L2 flush between timed iterations
                a.record(self.stream)
                for _ in range(per_step):
                    run()
                b.record(self.stream)
            self.stream.synchronize()
            torch.cuda.synchronize()
            self.barrier()
        total = sum(a.elapsed_time(b) for a, b in evs)
        return max_over_ranks(total, self.dev) / steps


def transport_account(t_copy, t_first, t_comp, t_pipe, carrier=0.0):
    """Exposed / hidden transfer time of one transport.  No schedule hides band 0's own transfer, nor more transfer
    time than there is compute: bound = min(1 - (T_first - carrier) / T_copy, T_comp / T_copy).  carrier: the part of
    a stand-alone transfer that is not transfer -- the launch of the kernel that carries an in-kernel fetch; in the
    pipelined run that same launch carries the compute, so it is never exposed (0 for copy-engine copies)."""
    exposed = max(0.0, t_pipe - t_comp)
    hidden = 100.0 * (1.0 - exposed / t_copy) if t_copy > 0 else None
    bound = 100.0 * min(1.0 - (t_first - carrier) / t_copy, t_comp / t_copy) if t_copy > 0 else None
    return {"t_copy_ms": t_copy, "t_first_ms": t_first, "t_compute_ms": t_comp, "t_pipelined_ms": t_pipe, "exposed_ms": exposed,
            "carrier_launch_ms": carrier, "hidden_pct": hidden, "hidden_pct_bound": bound,
            "within_bound": (hidden is not None and hidden <= bound + 1.0)}


def measure_workload(name, steps, warmup, timer, lop, li, DeviceChain, torch, dev, stream, peaks, clocks_mhz=None, copy_engine=True):
    """Everything bench.py reports about one workload: pipelined / end-to-end / resident / steady-state throughput, the
    dominant kernel's roofline fraction and the transfer accounting of both transports."""
    wl = li.build(name)
    dc = DeviceChain(wl, flags=lop.LOP_FLAG_REUSE_HALO, device=dev)
    x_dev, x_pin = dc.input_tensor(), dc.pinned_input()
    out_pin = torch.empty(dc.outs[-1].shape, dtype=dc.outs[-1].dtype).pin_memory()
    cs = stream.cuda_stream

    def step_pipe():
        dc.run_pipelined(x_pin, stream)

    def step_e2e():
        # input: bands from pinned host memory; result: stored by the last layer straight into pinned host memory --
        # both transfers are inside the timed region
        dc.run_pipelined(x_pin, stream, out_pinned=out_pin)

    def step_res():
        dc.run_banded(x_dev, stream)

    for fn in (step_pipe, step_e2e, step_res):                     # first calls build the device programs
        with torch.cuda.stream(stream):
            fn()
        stream.synchronize()
    ms_pipe = timer(step_pipe, steps, warmup)
    launches_pipe, copies_pipe = dc.launches(), sum(p.last_copies() for p in dc.plans)
    ms_e2e = timer(step_e2e, steps, warmup)
    ms_res = timer(step_res, steps, warmup)
    launches_res = dc.launches()
    ms_steady = timer(step_pipe, max(5, steps // STEADY_REQUESTS), 3, per_step=STEADY_REQUESTS) / STEADY_REQUESTS
    dc.check_device()
    with torch.cuda.stream(stream):
        step_res()
    stream.synchronize()
    if not torch.equal(out_pin, dc.outs[-1].cpu()):               # same bits from every arm
        raise SystemExit("bench: %s: the end-to-end arm's host result differs from the resident arm's device result" % name)

    # ---- transfer accounting, one transport at a time: the transfer alone, its first band alone, compute alone, both
    n_acc = max(20, min(100, steps))
    plan0 = dc.plans[0]
    transports = {}
    fetched = launches_pipe >= 1 and copies_pipe == 0              # the value arm's bands were fetched by the kernel
    if fetched:
        t_copy = timer(lambda: plan0.fetch_band(-1, x_pin.data_ptr(), dc.staging.data_ptr(), dc.ws[0].data_ptr(), cs), n_acc, 3)
        t_first = timer(lambda: plan0.fetch_band(0, x_pin.data_ptr(), dc.staging.data_ptr(), dc.ws[0].data_ptr(), cs), n_acc, 3)
        h2d = int(x_pin.numel() * x_pin.element_size())
        # the launch that carries a fetch running alone, from the two measurements: T = carrier + bytes / rate
        r0 = plan0.get_range(0, lop.LOP_INPUT)
        b0 = max(0, r0.out_hi - r0.new_lo) * (h2d // wl.H)
        carrier = 0.0
        if t_copy > t_first and h2d > b0:
            carrier = min(t_first, max(0.0, t_first - b0 * (t_copy - t_first) / (h2d - b0)))
        transports["kernel_fetch"] = transport_account(t_copy, t_first, ms_res, ms_pipe, carrier)
        transports["kernel_fetch"]["link_gbs_alone"] = h2d / (t_copy * 1e-3) / 1e9
    if copy_engine or not fetched:
        dcc = DeviceChain(wl, flags=lop.LOP_FLAG_REUSE_HALO | lop.LOP_FLAG_COPY_ENGINE, device=dev)
        with torch.cuda.stream(stream):
            dcc.run_pipelined(x_pin, stream)
        stream.synchronize()

        def copies_only():
            for b in range(dcc.plans[0].num_bands()):
                dcc.plans[0].copy_band(b, x_pin.data_ptr(), dcc.staging.data_ptr(), cs)

        t_copy_c = timer(copies_only, n_acc, 3)
        t_first_c = timer(lambda: dcc.plans[0].copy_band(0, x_pin.data_ptr(), dcc.staging.data_ptr(), cs), n_acc, 3)
        t_pipe_c = timer(lambda: dcc.run_pipelined(x_pin, stream), n_acc, 3)
        dcc.check_device()
        transports["copy_engine"] = transport_account(t_copy_c, t_first_c, ms_res, t_pipe_c)
        transports["copy_engine"]["link_gbs_alone"] = int(x_pin.numel() * x_pin.element_size()) / (t_copy_c * 1e-3) / 1e9
        del dcc

    flops = dc.flops()
    ach_pipe = flops / (ms_pipe * 1e-3) / 1e12
    ach_res = flops / (ms_res * 1e-3) / 1e12
    if wl.dtype == "bf16":
        roofline = {"bound": "tensor",
                    "kernel": "wavefront_kernel (one persistent launch per step: the fetch of the bands, every gather / conv / pool stage of every band)",
                    "achieved": ach_pipe, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s", "frac": ach_pipe / peaks["bf16_tflops"],
                    "peak_source": "%s TFLOP/s burst bf16 (of %s)" % (peaks["bf16_tflops"], peaks["source"]),
                    "flops_per_launch": flops, "avg_launch_us": ms_pipe * 1e3, "launches_per_step": launches_pipe,
                    "frac_resident": ach_res / peaks["bf16_tflops"], "frac_of_sustained": ach_pipe / peaks["bf16_tflops_sustained"],
                    "traffic": dram_traffic(name)}
    else:
        # fp32 storage runs on the CUDA cores: plain-ALU peak = SMs x 128 FMA lanes x 2 flop x max SM clock
        props = torch.cuda.get_device_properties(dev)
        mhz = clocks_mhz or 1965.0
        alu_peak = props.multi_processor_count * 128 * 2 * mhz * 1e6 / 1e12
        roofline = {"bound": "alu", "kernel": "conv_simt_kernel", "achieved": ach_pipe, "peak": alu_peak, "unit": "TFLOP/s",
                    "frac": ach_pipe / alu_peak,
                    "peak_source": "derived: %d SMs x 128 fp32 FMA lanes x 2 x %.0f MHz" % (props.multi_processor_count, mhz),
                    "flops_per_launch": flops / max(launches_pipe, 1), "avg_launch_us": ms_pipe * 1e3 / max(launches_pipe, 1),
                    "launches_per_step": launches_pipe, "frac_resident": ach_res / alu_peak, "traffic": None}
    return {"wl": wl, "dc": dc, "x_dev": x_dev, "ms_pipe": ms_pipe, "ms_e2e": ms_e2e, "ms_res": ms_res, "ms_steady": ms_steady,
            "launches_pipe": launches_pipe, "launches_res": launches_res, "fetched": fetched,
            "h2d": int(x_pin.numel() * x_pin.element_size()), "d2h": int(out_pin.numel() * out_pin.element_size()),
            "roofline": roofline, "transports": transports, "flops": flops}


def per_layer_table(wl, x_dev, lop, DeviceChain, torch, dev, stream, flush, peaks):
    """Whole-tensor launches, one kernel per layer, CUDA events around each (eager): the slowest layers."""
    dct = DeviceChain(wl, flags=lop.LOP_FLAG_PER_LAYER | lop.LOP_FLAG_TIME_LAYERS, device=dev)
    acc = {}
    reps = 10
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
    return sorted(per_layer, key=lambda d: -d["us"])[:12]          # keep the line readable: the slowest layers only


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=list(WORKLOAD_NOTES))
    ap.add_argument("--impl", default="native", choices=["native", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-per-config", action="store_true", help="measure only --workload, not the other configurations")
    ap.add_argument("--skip-copy-engine", action="store_true",
                    help="leave out the copy-engine transport's accounting: its persistent kernel waits for copies on other streams, "
                         "which a profiler that serialises kernels never lets run (the kernel's bounded wait then ends the run with an error)")
    args = ap.parse_args()

    if args.impl == "reference":
        args.steps = 3 if args.steps is None else args.steps
        args.warmup = 1 if args.warmup is None else args.warmup
        run_reference(args)
        return
    args.steps = 300 if args.steps is None else args.steps
    args.warmup = 10 if args.warmup is None else max(args.warmup, 3)

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
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)      # > 126 MB L2
    stream = torch.cuda.Stream(device=dev)
    timer = Timer(torch, stream, flush, barrier, dev)

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    m = measure_workload(args.workload, args.steps, args.warmup, timer, lop, li, DeviceChain, torch, dev, stream, peaks,
                         copy_engine=not args.skip_copy_engine)
    clocks = sampler.stop() if rank == 0 else None
    wl = m["wl"]

    per_layer = per_layer_table(wl, m["x_dev"], lop, DeviceChain, torch, dev, stream, flush, peaks)

    # ---- the other configurations, fewer steps (single-GPU runs only: the scaling runs time the named workload)
    per_config = {}
    if world == 1 and not args.no_per_config:
        for name in WORKLOAD_NOTES:
            if name == args.workload:
                continue
            mm = measure_workload(name, max(20, args.steps // 3), 5, timer, lop, li, DeviceChain, torch, dev, stream, peaks,
                                  clocks_mhz=(clocks or {}).get("sm_max_mhz"), copy_engine=not args.skip_copy_engine)
            n = mm["wl"].N
            best = "kernel_fetch" if "kernel_fetch" in mm["transports"] else "copy_engine"
            per_config[name] = {
                "workload": WORKLOAD_NOTES[name], "value": n / (mm["ms_pipe"] * 1e-3), "ms_per_step": mm["ms_pipe"],
                "e2e": n / (mm["ms_e2e"] * 1e-3), "resident": n / (mm["ms_res"] * 1e-3), "ms_resident": mm["ms_res"],
                "steady_state": n / (mm["ms_steady"] * 1e-3),
                "roofline_bound": mm["roofline"]["bound"], "roofline_frac": mm["roofline"]["frac"],
                "roofline_frac_resident": mm["roofline"]["frac_resident"], "conv_tflops": mm["roofline"]["achieved"],
                "transport": best, "hidden_pct": mm["transports"][best]["hidden_pct"],
                "hidden_pct_bound": mm["transports"][best]["hidden_pct_bound"], "pipeline": mm["transports"],
            }
            del mm

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    n = wl.N
    best = "kernel_fetch" if "kernel_fetch" in m["transports"] else "copy_engine"
    line = {
        "metric": METRIC, "value": job_images_per_s(n, world, m["ms_pipe"]), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": m["ms_pipe"], "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16" if wl.dtype == "bf16" else "f32", "data": "synthetic",
        "config": {"workload": WORKLOAD_NOTES[args.workload], "images_per_step_per_gpu": n, "mode": "reuse-halo bands",
                   "value_path": "lop_run_chain_pipelined: input bands from pinned host memory inside the timed region, output left on the device",
                   "transport": "input bands fetched from pinned host memory by the persistent kernel's fetch warps (one launch, no copy "
                                "commands)" if m["fetched"] else "copy-engine band copies on a side stream",
                   "e2e_path": "the same call with the last layer storing the result straight into pinned host memory",
                   "launch": "eager calls", "l2": "256 MiB buffer written between timed steps", "multi_gpu": "independent replicas"},
        "e2e": {"value": job_images_per_s(n, world, m["ms_e2e"]), "unit": UNIT, "ms_per_step": m["ms_e2e"],
                "h2d_bytes_per_step": m["h2d"], "d2h_bytes_per_step": m["d2h"]},
        "resident": {"value": job_images_per_s(n, world, m["ms_res"]), "unit": UNIT, "ms_per_step": m["ms_res"],
                     "what": "all bands from a device-resident input (lop_run_chain_banded): compute without any transfer"},
        "steady_state": {"value": job_images_per_s(n, world, m["ms_steady"]), "unit": UNIT, "ms_per_request": m["ms_steady"],
                         "requests": STEADY_REQUESTS, "what": "R pipelined requests back to back on one stream behind one L2 flush, N*R / T"},
        "gpu_launches": int(m["launches_pipe"] * args.steps),
        "clocks": clocks,
        "roofline": m["roofline"],
        "conv_tflops": {"whole_step_useful": m["roofline"]["achieved"], "pct_of_burst_peak": 100.0 * m["roofline"]["frac"],
                        "pct_of_sustained_peak": 100.0 * m["roofline"]["achieved"] / peaks["bf16_tflops_sustained"],
                        "resident_pct_of_burst_peak": 100.0 * m["roofline"]["frac_resident"],
                        "per_layer_launches": per_layer},
        "pipeline": dict(m["transports"][best], transport=best, n_bands=m["dc"].plans[0].num_bands(),
                         note="every figure of one transport: T_copy = that transport moving all bands alone, T_first = its "
                              "band 0 alone, T_compute = the resident run, T_pipelined = the pipelined run with that transport; "
                              "bound = min(1 - (T_first - carrier)/T_copy, T_compute/T_copy), carrier = the launch that carries a stand-alone in-kernel fetch (estimated from T_first, T_copy and the two byte counts; 0 for copy-engine copies)"),
        "pipeline_by_transport": m["transports"],
        "per_config": per_config,
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

"""Choosing the band counts of a chain: the paper's scheduling optimisation, re-targeted from a phone and a server over
Wi-Fi to one B200 behind a host link.

The paper's LOSS (Sec. IV-C) takes per-operation times from a profile and the link's bandwidth, describes a plan by
contiguous intervals of operations, and searches the plan that minimises the latency of one inference with differential
evolution, offline.  Here both "devices" are the same GPU, the transmission is the host link, and what is left to
choose is how finely each segment of the chain is cut into bands: more bands start computing sooner behind the
transfer and overlap more of it, fewer bands pay less per-band overhead and recompute or re-stream less.

  cost_model()   a coarse latency model of one pipelined request from the planner's exact row ranges (what each band
                 transfers and computes) and a handful of measured machine constants
  search()       differential evolution over the vector of per-segment band counts (powers of two), for any objective
  measured()     the objective measured on the device: the pipelined entry point timed with CUDA events
  choose()       model-guided search, then the best few candidates are measured and the fastest is returned

Only the search and the model live here; every operator still runs in the C-ABI library.
"""
import math
import random

from . import binding as B

BAND_CHOICES = (1, 2, 4, 8, 16, 32)

# Machine constants, measured on B200 with this library (microseconds unless said otherwise): a kernel launch and its
# completion; one dependency hop between layers (producer's stores visible -> consumer's first operands in shared
# memory -> its tile finished and published); one convolution tile of 128 pixels x 64 channels per 64-channel chunk and
# tap; one pooling / gather row item; the host link as the kernel's fetch warps drive it.
MACHINE = {"launch_us": 6.0, "hop_us": 4.5, "tile_chunk_tap_us": 0.09, "row_item_us": 2.5, "link_gbs": 30.0, "ctas": 148}


def _tiles(rows, width, n):
    return math.ceil(max(rows, 0) * width * n / 128.0)


def cost_model(wl, bands, machine=MACHINE):
    """Estimated latency (us) of one pipelined request of workload ``wl`` with ``bands[s]`` bands in segment ``s``.

    Per segment the library's planner gives every band's rows at every layer (reuse-halo mode: the rows no earlier
    band produced).  Band b of the first segment can start when its input rows have arrived over the link; a band's
    layers form a chain of dependency hops; the layers' tiles share the CTAs.  The model walks the bands in order and
    keeps, per layer, the time the machine is free again (a list-scheduling estimate, in the spirit of the profile-
    driven cost terms of the paper's LOSS: compute time per operation, transmission time per edge)."""
    N, H, W, C = wl.N, wl.H, wl.W, wl.C
    es = 2 if wl.dtype == "bf16" else 4
    t_ready_prev = None                      # per output row of the previous segment: when it exists
    total_end = machine["launch_us"]
    for s, seg in enumerate(wl.segments):
        nb = bands[s]
        plan = B.Plan(seg.layers, N, H, W, C, B.LOP_BF16 if wl.dtype == "bf16" else B.LOP_F32, nb, B.LOP_FLAG_REUSE_HALO)
        L = len(seg.layers)
        shapes = [plan.out_shape(i) for i in range(L)]
        layer_free = [0.0] * L                # when the machine has finished the layer's earlier tiles
        link_free = machine["launch_us"]
        row_bytes = W * C * es * N
        out_ready = [0.0] * shapes[-1][0]
        for b in range(nb):
            need = plan.get_range(b, B.LOP_INPUT)
            if s == 0:
                new_rows = max(0, need.out_hi - need.new_lo)
                link_free += new_rows * row_bytes / (machine["link_gbs"] * 1e3)
                t = link_free
            else:
                t = max(t_ready_prev[need.out_lo:need.out_hi], default=0.0) if need.out_hi > need.out_lo else 0.0
            for i, l in enumerate(seg.layers):
                r = plan.get_range(b, i)
                rows = max(0, r.out_hi - r.new_lo)
                if rows == 0:
                    continue
                ho, wo, co = shapes[i]
                if l.op in (1, 3, 4, 5):      # pooling, depth-wise convolution, layer normalisation, concatenation: row items of the worker warps
                    items = rows * N
                    per_item = machine["row_item_us"] * (2.0 if l.op == 3 else 1.0)
                    work = math.ceil(items / machine["ctas"]) * per_item
                else:
                    chunks = math.ceil(l.cin / 64.0) if l.cin >= 16 else 1
                    taps = l.kh * l.kw if l.cin >= 16 else 1
                    per_item = 1.0 + machine["tile_chunk_tap_us"] * chunks * taps * 4
                    items = _tiles(rows, wo, N) * max(1, co // 64)
                    work = math.ceil(items / machine["ctas"]) * per_item if items > machine["ctas"] else per_item
                start = max(t + machine["hop_us"], layer_free[i])
                t = start + work
                # a stage with fewer items than CTAs leaves the rest of the machine to the next band's stage
                layer_free[i] = start + work * min(1.0, items / machine["ctas"])
            last = plan.get_range(b, L - 1)
            for row in range(last.new_lo, last.out_hi):
                out_ready[row] = t
            total_end = max(total_end, t)
        t_ready_prev = out_ready
        H, W, C = shapes[-1]
        plan.destroy()
    return total_end


def search(objective, n_segments, choices=BAND_CHOICES, population=12, generations=20, seed=0, start=None):
    """Differential evolution (the paper's solver, Sec. IV-C) over per-segment band counts.

    A candidate is a vector of indices into ``choices``; mutation adds the scaled difference of two other members to a
    third, crossover mixes it with the current member, the better of the two survives.  Values are rounded and clipped
    to the grid.  ``objective(tuple_of_band_counts) -> float``; returns (best_bands, best_value, evaluations)."""
    rnd = random.Random(seed)
    K = len(choices)
    cache = {}

    def value(vec):
        key = tuple(choices[i] for i in vec)
        if key not in cache:
            cache[key] = float(objective(key))
        return cache[key]

    pop = [[rnd.randrange(K) for _ in range(n_segments)] for _ in range(population)]
    if start is not None:
        pop[0] = [min(range(K), key=lambda i: abs(choices[i] - b)) for b in start]
    fit = [value(v) for v in pop]
    for _ in range(generations):
        for j in range(population):
            a, b, c = rnd.sample([k for k in range(population) if k != j], 3)
            force = rnd.randrange(n_segments)
            trial = []
            for d in range(n_segments):
                if d == force or rnd.random() < 0.7:
                    v = pop[a][d] + 0.8 * (pop[b][d] - pop[c][d])
                    trial.append(int(min(K - 1, max(0, round(v)))))
                else:
                    trial.append(pop[j][d])
            f = value(trial)
            if f <= fit[j]:
                pop[j], fit[j] = trial, f
    best = min(range(population), key=lambda k: fit[k])
    return tuple(choices[i] for i in pop[best]), fit[best], len(cache)


def measured(wl, bands, steps=30, warmup=5, device="cuda:0"):
    """Latency (us) of one pipelined request with ``bands[s]`` bands in segment ``s``, measured with CUDA events
    (L2 flushed between requests)."""
    import torch
    from .chain import DeviceChain
    dc = DeviceChain(wl, flags=B.LOP_FLAG_REUSE_HALO, device=device, n_bands=list(bands))
    x = dc.pinned_input()
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=device)
    stream = torch.cuda.Stream(device=device)
    times = []
    with torch.cuda.stream(stream):
        for k in range(warmup + steps):
            flush.zero_()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            dc.run_pipelined(x, stream)
            b.record(stream)
            stream.synchronize()
            if k >= warmup:
                times.append(a.elapsed_time(b) * 1e3)
    dc.check_device()
    times.sort()
    return times[len(times) // 2]


def choose(wl, measure_top=4, seed=0, machine=MACHINE, measure=measured):
    """Band counts for ``wl``: search on the model, then measure the best few candidates (and the workload's own band
    counts) on the device and return the fastest.  -> (bands, measured_us, report)"""
    own = tuple(seg.n_bands for seg in wl.segments)
    evaluated = {}

    def model(bands):
        evaluated[bands] = cost_model(wl, bands, machine)
        return evaluated[bands]

    search(model, len(wl.segments), seed=seed, start=own)
    ranked = sorted(evaluated, key=evaluated.get)[:measure_top]
    if own not in ranked:
        ranked.append(own)
    timed = {b: measure(wl, b) for b in ranked}
    best = min(timed, key=timed.get)
    return best, timed[best], {"model_us": {str(b): evaluated.get(b) for b in ranked}, "measured_us": {str(b): timed[b] for b in ranked},
                              "own": str(own), "candidates_modelled": len(evaluated)}

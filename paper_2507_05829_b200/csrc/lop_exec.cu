// Chain executor and band scheduler: lop_run_whole / lop_run_band / lop_run_banded /
// lop_copy_band / lop_run_pipelined.
//
// Sec. IV-B of the paper: a band's operations at every layer run in dependency order as soon
// as their inputs exist; the transfer of the next band's input overlaps the current band's
// computation.  Here the "transmission" is an asynchronous pinned-host -> device copy on a side
// stream, the dependency "input has arrived" is a CUDA event, and tensor "combining" is
// addressing: every band writes its rows straight into full-size tensors.
#include <cuda.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cmath>
#include <cstdio>
#include <map>
#include <tuple>
#include <vector>

#include "lop_internal.h"
#include "lop_kernels.cuh"
#include "lop_layerargs.h"
#include "lop_program.h"

namespace lop {

struct MapKey {
    int layer, TW, TR, TN, BN, BK;
    const void *x, *w;
    bool operator<(const MapKey &o) const
    {
        return std::tie(layer, TW, TR, TN, BN, BK, x, w) < std::tie(o.layer, o.TW, o.TR, o.TN, o.BN, o.BK, o.x, o.w);
    }
};

struct ProgKey {
    int kind;                        // -1 whole, -2 all bands, -3 pipelined, -4 pipelined with in-kernel fetch, -5 fetch alone,
                                     // >= 0 one band, <= -16: the block of bands [lo, hi) encoded as -16 - (lo * 65536 + hi)
    int sub;                         // fetch alone: the band, or -1 for all bands; 0 otherwise
    const void *src;                 // fetch source (host memory as the device addresses it) or nullptr
    // every plan of the chain the program spans: its input / output / workspace and its uid (new at creation and at
    // every lop_plan_set_params), so a program built from other plans, buffers or parameters is never reused
    std::vector<const void *> bound;
    bool operator<(const ProgKey &o) const { return std::tie(kind, sub, src, bound) < std::tie(o.kind, o.sub, o.src, o.bound); }
};

struct ExecState {
    std::map<ProgKey, Program *> programs;
    bool wavefront = false;
    cudaStream_t copy_stream = nullptr;                        // the side stream of the transfers
    cudaStream_t signal_stream = nullptr;                      // performs the arrival writes of the single-launch pipeline
    cudaEvent_t ev_signal_join = nullptr;
    cudaEvent_t ev_fork = nullptr, ev_begin = nullptr, ev_end = nullptr, ev_join = nullptr;
    unsigned *pinned_one = nullptr;                            // pinned host word holding 1: source of arrival flags
    std::vector<cudaEvent_t> ev_copy_start, ev_copy_end;       // [band]
    std::vector<cudaEvent_t> ev_arrive;                        // [band], no timing
    std::vector<cudaEvent_t> ev_layer;                         // [(band+1) * L + layer] * 2, slot 0 = whole
    std::vector<char> layer_timed;
    std::map<MapKey, ConvTcMaps> maps;
    const void *prepared_ws = nullptr;
    std::vector<const void *> prepared_w;                      // weight pointers the padded copies were made from
    cudaStream_t last_stream = nullptr;
    int launches = 0;                                          // kernels enqueued by the last execution call
    int copies = 0;                                            // async copies enqueued by it
    bool timing_valid = false;
    bool copies_timed = false;                                 // per-band copy events were recorded by the last pipelined run
    const void *mapped_host = nullptr, *mapped_dev = nullptr;  // last host buffer looked up and its device-side address (or nullptr)
    std::vector<char> copy_issued;
};

void exec_destroy(ExecState *e)
{
    if (!e) return;
    if (e->copy_stream) cudaStreamDestroy(e->copy_stream);
    if (e->signal_stream) cudaStreamDestroy(e->signal_stream);
    if (e->ev_signal_join) cudaEventDestroy(e->ev_signal_join);
    if (e->pinned_one) cudaFreeHost(e->pinned_one);
    for (cudaEvent_t ev : {e->ev_fork, e->ev_begin, e->ev_end, e->ev_join})
        if (ev) cudaEventDestroy(ev);
    for (auto &v : {&e->ev_copy_start, &e->ev_copy_end, &e->ev_layer, &e->ev_arrive})
        for (cudaEvent_t ev : *v)
            if (ev) cudaEventDestroy(ev);
    for (auto &kv : e->programs) program_destroy(kv.second);
    delete e;
}

void exec_invalidate(ExecState *e)
{
    if (!e) return;
    for (auto &kv : e->programs) program_destroy(kv.second);      // cudaFree waits for launches still in flight
    e->programs.clear();
    e->maps.clear();
    e->prepared_ws = nullptr;                                      // padded stem weights are rebuilt on the next call
}

namespace {

#define LOP_CUDA(call)                                                                  \
    do {                                                                                \
        cudaError_t e__ = (call);                                                       \
        if (e__ != cudaSuccess) {                                                       \
            set_error("%s failed: %s", #call, cudaGetErrorString(e__));                 \
            return LOP_ECUDA;                                                           \
        }                                                                               \
    } while (0)

// cuStreamWriteValue32 through the runtime's entry-point lookup: a stream-ordered 4-byte write with a fence in front of
// it, far cheaper than a 4-byte copy on the copy engine.  nullptr when the driver does not offer it.
typedef CUresult (*StreamWriteValue32Fn)(CUstream, CUdeviceptr, cuuint32_t, unsigned int);
StreamWriteValue32Fn stream_write_fn()
{
    static StreamWriteValue32Fn fn = nullptr;
    static bool looked = false;
    if (!looked) {
        looked = true;
        void *ptr = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuStreamWriteValue32", &ptr, cudaEnableDefault, &q) == cudaSuccess && q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<StreamWriteValue32Fn>(ptr);
    }
    return fn;
}

int ensure_exec(lop_plan_t *pl)
{
    if (pl->exec) return LOP_OK;
    ExecState *e = new (std::nothrow) ExecState();
    if (!e) { set_error("out of host memory"); return LOP_ENOMEM; }
    pl->exec = e;
    const int B = pl->n_bands, L = (int)pl->layers.size();
    LOP_CUDA(cudaStreamCreateWithFlags(&e->copy_stream, cudaStreamNonBlocking));
    LOP_CUDA(cudaEventCreateWithFlags(&e->ev_fork, cudaEventDisableTiming));
    LOP_CUDA(cudaEventCreateWithFlags(&e->ev_join, cudaEventDisableTiming));
    LOP_CUDA(cudaStreamCreateWithFlags(&e->signal_stream, cudaStreamNonBlocking));
    LOP_CUDA(cudaEventCreateWithFlags(&e->ev_signal_join, cudaEventDisableTiming));
    LOP_CUDA(cudaHostAlloc(reinterpret_cast<void **>(&e->pinned_one), 64, cudaHostAllocDefault));
    *e->pinned_one = 1u;
    LOP_CUDA(cudaEventCreate(&e->ev_begin));
    LOP_CUDA(cudaEventCreate(&e->ev_end));
    e->ev_copy_start.assign(B, nullptr);
    e->ev_copy_end.assign(B, nullptr);
    e->ev_arrive.assign(B, nullptr);
    e->copy_issued.assign(B, 0);
    for (int b = 0; b < B; ++b) {
        LOP_CUDA(cudaEventCreate(&e->ev_copy_start[b]));
        LOP_CUDA(cudaEventCreate(&e->ev_copy_end[b]));
        LOP_CUDA(cudaEventCreateWithFlags(&e->ev_arrive[b], cudaEventDisableTiming));
    }
    if (pl->flags & LOP_FLAG_TIME_LAYERS) {
        e->ev_layer.assign((size_t)(B + 1) * L * 2, nullptr);
        e->layer_timed.assign((size_t)(B + 1) * L, 0);
        for (auto &ev : e->ev_layer) LOP_CUDA(cudaEventCreate(&ev));
    }
    e->prepared_w.assign(L, nullptr);
    e->wavefront = program_supported(pl) && !(pl->flags & (LOP_FLAG_PER_LAYER | LOP_FLAG_TIME_LAYERS | LOP_FLAG_DEBUG_BOUNDS));
    return LOP_OK;
}

int check_common(lop_plan_t *pl, const void *in, const void *out, const void *ws)
{
    if (!pl) { set_error("plan is NULL"); return LOP_EINVAL; }
    if (!in || !out) { set_error("input/output pointer is NULL"); return LOP_EINVAL; }
    if (!ws || (reinterpret_cast<uintptr_t>(ws) & 255u)) { set_error("workspace is NULL or not 256-byte aligned"); return LOP_EWORKSPACE; }
    if ((reinterpret_cast<uintptr_t>(in) & 15u) || (reinterpret_cast<uintptr_t>(out) & 15u)) {
        set_error("input/output tensors must be 16-byte aligned");
        return LOP_EINVAL;
    }
    for (size_t i = 0; i < pl->layers.size(); ++i)
        if ((pl->layers[i].l.op == LOP_CONV2D || pl->layers[i].l.op == LOP_DWCONV2D) && !pl->layers[i].l.weight) {
            set_error("layer %zu has no weight pointer (lop_plan_set_params)", i);
            return LOP_EINVAL;
        }
    return ensure_exec(pl);
}

// One-time work per workspace: clear the status word, build the zero-padded weights of a gathered stem.
int prepare_workspace(lop_plan_t *pl, void *ws, cudaStream_t s)
{
    ExecState *e = pl->exec;
    char *base = static_cast<char *>(ws);
    bool fresh = e->prepared_ws != ws;
    if (fresh) {
        LOP_CUDA(cudaMemsetAsync(base + pl->status_off, 0, 1024, s));
    }
    for (size_t i = 0; i < pl->layers.size(); ++i) {
        LayerInfo &li = pl->layers[i];
        if (!li.stem_gather && !li.dw_transposed) continue;
        if (!fresh && e->prepared_w[i] == li.l.weight) continue;
        if (li.stem_gather) LOP_CUDA(launch_pad_weights(li.l.weight, base + li.wpad_off, li.l.cout, li.l.kh * li.l.kw * li.l.cin, li.cin_eff, s));
        else LOP_CUDA(launch_dw_transpose(li.l.weight, base + li.wpad_off, li.l.cin, li.l.kh * li.l.kw, s));
        e->prepared_w[i] = li.l.weight;
        e->launches++;
    }
    e->prepared_ws = ws;
    return LOP_OK;
}

// Rows [lo, hi) of layer i.  slot: index into the per-layer timing events, or -1.
int run_layer(lop_plan_t *pl, int i, int lo, int hi, const void *in, void *out, void *ws, cudaStream_t s, int slot)
{
    if (hi <= lo) return LOP_OK;
    ExecState *e = pl->exec;
    LayerInfo &li = pl->layers[i];
    const lop_layer &l = li.l;
    const bool timed = slot >= 0 && !e->ev_layer.empty();
    if (timed) {
        LOP_CUDA(cudaEventRecord(e->ev_layer[(size_t)slot * 2], s));
        e->layer_timed[slot] = 1;
    }
    if (l.op == LOP_MAXPOOL2D) {
        LOP_CUDA(launch_maxpool(pool_args(pl, i, in, out, ws, lo, hi), pl->dtype, s));
    } else if (li.kernel == K_DWCONV) {
        LOP_CUDA(launch_dwconv(conv_args(pl, i, in, out, ws, lo, hi), pl->dtype, li.dw_transposed ? static_cast<char *>(ws) + li.wpad_off : nullptr, s));
    } else if (li.kernel == K_LAYERNORM) {
        LOP_CUDA(launch_layernorm(conv_args(pl, i, in, out, ws, lo, hi), pl->dtype, s));
    } else if (li.kernel == K_CONCAT) {
        LOP_CUDA(launch_concat(conv_args(pl, i, in, out, ws, lo, hi), pl->dtype, s));
    } else {
        const ConvArgs a = conv_args(pl, i, in, out, ws, lo, hi);
        if (li.kernel == K_CONV_TC) {
            if (li.stem_gather) {                      // the band's patches first (the split step), same stream
                LOP_CUDA(launch_stem_gather(in, static_cast<char *>(ws) + pl->col_off, gather_geom(pl, i), lo, hi, s, a.dbg));
                e->launches++;
            }
            const ConvTcGeom g = conv_tc_geometry(a, hi - lo);
            const MapKey key{i, g.TW, g.TR, g.TN, g.BN, g.BK, a.x, a.w};
            auto it = e->maps.find(key);
            if (it == e->maps.end()) {
                if (e->maps.size() >= 4096) e->maps.clear();        // tensor maps are passed by value at launch: safe to drop
                ConvTcMaps m;
                int rc = conv_tc_encode(a, g, &m);
                if (rc != LOP_OK) { set_error("layer %d: tensor-map encoding failed", i); return rc; }
                it = e->maps.emplace(key, m).first;
            }
            LOP_CUDA(launch_conv_tc(a, g, it->second, reinterpret_cast<unsigned *>(static_cast<char *>(ws) + pl->status_off), s));
        } else {
            LOP_CUDA(launch_conv_simt(a, pl->dtype, s));
        }
    }
    e->launches++;
    if (timed) LOP_CUDA(cudaEventRecord(e->ev_layer[(size_t)slot * 2 + 1], s));
    return LOP_OK;
}

int run_band_impl(lop_plan_t *pl, int band, const void *in, void *out, void *ws, cudaStream_t s)
{
    const int L = (int)pl->layers.size();
    const bool reuse = (pl->flags & LOP_FLAG_REUSE_HALO) != 0;
    int rc = LOP_OK;
    for (int i = 0; i < L; ++i) {
        const lop_range &r = pl->ranges[(size_t)band * L + i];
        rc = run_layer(pl, i, reuse ? r.new_lo : r.out_lo, r.out_hi, in, out, ws, s, (band + 1) * L + i);
        if (rc != LOP_OK) return rc;
    }
    return LOP_OK;
}

// Requests of one band of plan `seg` in dependency order; a gathered stem is preceded by its patch-gather stage over
// the same rows.
// First row of layer i that band `band` computes when bands [block_lo, band) are the only ones that have run on this
// device: in reuse mode what the block has not produced yet (for block_lo = 0 that is the plan's new_lo).
int first_row(const lop_plan_t *pl, int block_lo, int band, int i)
{
    const int L = (int)pl->layers.size();
    const lop_range &r = pl->ranges[(size_t)band * L + i];
    if (!(pl->flags & LOP_FLAG_REUSE_HALO)) return r.out_lo;
    if (block_lo == 0) return r.new_lo;
    int done = 0;
    for (int b = block_lo; b < band; ++b) {
        const lop_range &q = pl->ranges[(size_t)b * L + i];
        if (q.out_hi > q.out_lo) done = std::max(done, (int)q.out_hi);
    }
    return std::min(std::max((int)r.out_lo, done), (int)r.out_hi);
}

// block_lo: the first band that runs on this device (0 unless the bands are sharded over devices).
void band_requests(const lop_plan_t *pl, int seg, int band, bool wait_arrival, std::vector<StageReq> &reqs, int block_lo = 0)
{
    const int L = (int)pl->layers.size();
    for (int i = 0; i < L; ++i) {
        const lop_range &r = pl->ranges[(size_t)band * L + i];
        const int lo = first_row(pl, block_lo, band, i);
        if (pl->layers[i].stem_gather) reqs.push_back(StageReq{seg, band, i, lo, r.out_hi, wait_arrival && seg == 0, true, 0});
        reqs.push_back(StageReq{seg, band, i, lo, r.out_hi, wait_arrival && seg == 0, false, 0});
    }
}

// Operation batching across thin bands (Sec. IV-C): deep in a network a band is a row or two of a small map, far less
// than the rows one tile covers, so every band would pay for a mostly empty tile -- and stream the layer's weights once
// more.  In reuse mode consecutive bands compute consecutive rows, so at a layer whose bands have fewer than eight rows
// the requests of g neighbouring bands are joined into one wherever their row ranges touch (g: about eight rows per
// group; a tile of a 16-pixel-wide map has eight).  The rows computed, and their bits, stay the same.
// keep_plan0: leave the first plan's bands alone (they are gated by the arrival of their input).
void merge_thin_bands(const std::vector<SegBind> &segs, std::vector<StageReq> &reqs, bool keep_plan0)
{
    for (int sg = keep_plan0 ? 1 : 0; sg < (int)segs.size(); ++sg) {
        const lop_plan_t *pl = segs[sg].pl;
        if (!(pl->flags & LOP_FLAG_REUSE_HALO) || pl->n_bands < 2) continue;
        const int L = (int)pl->layers.size();
        std::vector<int> group(L, 1);
        for (int i = 0; i < L; ++i) {
            const double rows_per_band = (double)pl->layers[i].Ho / pl->n_bands;
            if (rows_per_band < 8.0) group[i] = std::min(pl->n_bands, (int)std::ceil(8.0 / std::max(rows_per_band, 1.0 / 64)));
        }
        for (int i = 0; i + 1 < L; ++i) {
            // a convolution whose 2x2 pooling is folded into its epilogue must be cut like the pooling
            const lop_layer &q = pl->layers[i + 1].l;
            if (pl->layers[i].l.op == LOP_CONV2D && q.op == LOP_MAXPOOL2D && q.input_from == i && q.kh == 2 && q.kw == 2 && q.sh == 2 && q.sw == 2)
                group[i] = group[i + 1];
        }
        for (int layer = 0; layer < L; ++layer) {
            const int g = group[layer];
            if (g <= 1) continue;
            for (int gather = 0; gather < 2; ++gather) {
                int open = -1;                                        // request the following bands are joined into
                for (int b = 0; b < pl->n_bands; ++b) {
                    int found = -1;
                    for (size_t i = 0; i < reqs.size(); ++i)
                        if (reqs[i].seg == sg && reqs[i].layer == layer && (int)reqs[i].gather == gather && !reqs[i].fetch &&
                            reqs[i].band == b && reqs[i].hi > reqs[i].lo) { found = (int)i; break; }
                    if (b % g == 0) open = -1;
                    if (found < 0) continue;
                    if (open >= 0 && reqs[found].lo == reqs[open].hi) {
                        reqs[open].hi = reqs[found].hi;
                        reqs[found].hi = reqs[found].lo;                  // empty: dropped by the builder
                    } else {
                        open = found;
                    }
                }
            }
        }
    }
}

enum { PROG_WHOLE = -1, PROG_ALL_BANDS = -2, PROG_PIPELINED = -3, PROG_FETCHED = -4, PROG_FETCH_ALONE = -5, PROG_BLOCK0 = -16 };

// kind: PROG_WHOLE, PROG_ALL_BANDS, PROG_PIPELINED, PROG_FETCHED (fetch_src: the host input as the device addresses
// it), or b >= 0 for band b alone (single plan only).  segs: the plans of a chain with their buffers; the program is
// cached in the first plan.
int get_program(const std::vector<SegBind> &segs, int kind, Program **prog, const void *fetch_src = nullptr, int sub = 0)
{
    lop_plan_t *pl0 = segs[0].pl;
    ExecState *e = pl0->exec;
    ProgKey key{kind, sub, fetch_src, {}};
    for (const SegBind &sb : segs) {
        key.bound.push_back(sb.in);
        key.bound.push_back(sb.out);
        key.bound.push_back(sb.ws);
        key.bound.push_back(reinterpret_cast<const void *>(static_cast<uintptr_t>(sb.pl->uid)));
    }
    auto it = e->programs.find(key);
    if (it == e->programs.end()) {
        if (e->programs.size() >= 64) {
            // a caller that keeps changing buffers: start over rather than grow without bound (cudaFree waits for
            // launches still in flight)
            for (auto &kv : e->programs) program_destroy(kv.second);
            e->programs.clear();
        }
        std::vector<StageReq> reqs;
        long long next = 0;
        if (kind == PROG_WHOLE) {
            for (int sg = 0; sg < (int)segs.size(); ++sg) {
                const lop_plan_t *pl = segs[sg].pl;
                for (int i = 0; i < (int)pl->layers.size(); ++i) {
                    if (pl->layers[i].stem_gather) reqs.push_back(StageReq{sg, 0, i, 0, pl->layers[i].Ho, false, true, next++});
                    reqs.push_back(StageReq{sg, 0, i, 0, pl->layers[i].Ho, false, false, next++});
                }
            }
        } else if (kind == PROG_ALL_BANDS || kind == PROG_PIPELINED || kind == PROG_FETCHED) {
            // ALL_BANDS (input resident): the bands' operations of one layer do not depend on each other, so they are
            // batched layer by layer (operation batching, Sec. IV-C); dependencies stay per band row group.
            // PIPELINED: bands arrive one after the other and each band's stages form a dependency chain, so the
            // stages are ordered along the diagonals of the (band, stage) grid: while band b is at its first stage,
            // band b-1 is at its second, and so on -- the pipeline of Sec. IV-B -- and the plans of a chain follow
            // one another on the same diagonals (a later plan's band needs the previous plan's rows around it, so it
            // lags by a band; the builder moves a stage back wherever its producers come later still).  Inside a
            // diagonal the deeper stages come first, so a CTA does not sit on a band that has not arrived while
            // older bands have work.
            // FETCHED: the same, each band of plan 0 preceded by the fetch of its new input rows; the builder orders
            // these programs by earliest start.
            long long joff = 0;
            for (int sg = 0; sg < (int)segs.size(); ++sg) {
                const lop_plan_t *pl = segs[sg].pl;
                size_t per = 0;
                for (int b = 0; b < pl->n_bands; ++b) {
                    std::vector<StageReq> one;
                    if (kind == PROG_FETCHED && sg == 0) {
                        const lop_range &need = pl->in_need[b];
                        StageReq f{0, b, 0, need.new_lo, need.out_hi, false, false, (long long)b * 65536 - 1};
                        f.fetch = true;
                        reqs.push_back(f);
                    }
                    band_requests(pl, sg, b, kind == PROG_PIPELINED, one);
                    per = one.size();
                    for (size_t j = 0; j < one.size(); ++j) {
                        const long long depth = joff + (long long)j;
                        one[j].prio = kind == PROG_ALL_BANDS ? depth * 65536 + b : (b + depth + sg) * 65536 + (65534 - depth);
                        reqs.push_back(one[j]);
                    }
                }
                joff += (long long)per;
            }
            std::stable_sort(reqs.begin(), reqs.end(), [](const StageReq &x, const StageReq &y) { return x.prio < y.prio; });
        } else if (kind == PROG_FETCH_ALONE) {
            // the transfer step by itself: the fetch requests of one band (sub) or of all bands, no operator
            for (int b = 0; b < pl0->n_bands; ++b) {
                if (sub >= 0 && b != sub) continue;
                const lop_range &need = pl0->in_need[b];
                StageReq f{0, b, 0, need.new_lo, need.out_hi, false, false, (long long)b};
                f.fetch = true;
                reqs.push_back(f);
            }
        } else if (kind <= PROG_BLOCK0) {
            // a block of bands on a device that runs no other band: layer-major like ALL_BANDS, the first band whole
            const int code = PROG_BLOCK0 - kind, lo = code >> 16, hi = code & 0xFFFF;
            for (int b = lo; b < hi; ++b) {
                std::vector<StageReq> one;
                band_requests(pl0, 0, b, false, one, lo);
                for (size_t j = 0; j < one.size(); ++j) {
                    one[j].prio = (long long)j * 65536 + b;
                    reqs.push_back(one[j]);
                }
            }
            std::stable_sort(reqs.begin(), reqs.end(), [](const StageReq &x, const StageReq &y) { return x.prio < y.prio; });
        } else {
            band_requests(pl0, 0, kind, false, reqs);
            for (StageReq &r : reqs) r.prio = next++;
        }
        // pipelined: when each band should be on the device.  Measured on the copy stream: a command costs ~4.7 us and
        // overlaps the previous copy's transfer, which runs at ~64 GB/s; the flag write follows ~5 us behind.
        std::vector<double> arrival;
        if (kind == PROG_PIPELINED) {
            const double row_bytes = (double)pl0->W * pl0->C * elem_size(pl0->dtype) * pl0->N;
            double t = 5.0;
            std::vector<double> own(pl0->n_bands, 0.0);
            for (int b = 0; b < pl0->n_bands; ++b) {
                const lop_range &need = pl0->in_need[b];
                if (need.out_hi > need.new_lo) own[b] = (need.out_hi - need.new_lo) * row_bytes / 64e3;
            }
            for (int b0 = 0; b0 < pl0->n_bands; b0 += std::max(1, pl0->copy_group)) {
                const int b1 = std::min(pl0->n_bands, b0 + std::max(1, pl0->copy_group));
                double bytes_us = 0.0;
                for (int b = b0; b < b1; ++b) bytes_us += own[b];
                if (bytes_us > 0.0) t += std::max(4.7, bytes_us);
                for (int b = b0; b < b1; ++b) arrival.push_back(t + 5.0);       // the bands of one copy arrive together
            }
        }
        if (kind == PROG_ALL_BANDS || kind <= PROG_BLOCK0) merge_thin_bands(segs, reqs, false);
        // (also in the first plan, whose bands are gated by their arrival: a 12-layer stack cut into 32 one-row bands ran
        // 389 -> 352 us pipelined with its deep layers joined, the other configurations unchanged)
        else if (kind == PROG_PIPELINED || kind == PROG_FETCHED) merge_thin_bands(segs, reqs, false);
        Program *p = nullptr;
        int rc = program_build(segs, reqs, &p, (kind == PROG_PIPELINED || kind == PROG_ALL_BANDS) ? &arrival : nullptr, fetch_src);
        if (rc != LOP_OK) return rc;
        it = e->programs.emplace(key, p).first;
    }
    *prog = it->second;
    return LOP_OK;
}

int get_program(lop_plan_t *pl, int kind, const void *in, void *out, void *ws, Program **prog, const void *fetch_src = nullptr, int sub = 0)
{
    return get_program(std::vector<SegBind>{SegBind{pl, in, out, ws}}, kind, prog, fetch_src, sub);
}

// The address under which the device reads the host buffer, when it can (page-locked memory is mapped into the
// unified address space) and the plan does not insist on the copy engine; nullptr otherwise.
const void *fetchable(lop_plan_t *pl, const void *host)
{
    if (pl->flags & LOP_FLAG_COPY_ENGINE) return nullptr;
    ExecState *e = pl->exec;
    if (e->mapped_host == host) return e->mapped_dev;
    cudaPointerAttributes at{};
    const void *dev = nullptr;
    if (cudaPointerGetAttributes(&at, host) == cudaSuccess) {
        if (at.type == cudaMemoryTypeHost && at.devicePointer) dev = at.devicePointer;
    } else {
        cudaGetLastError();                                  // an unknown pointer is no error here: it gets copies
    }
    e->mapped_host = host;
    e->mapped_dev = dev;
    return dev;
}

int run_program(lop_plan_t *pl, int kind, const void *in, void *out, void *ws, cudaStream_t s)
{
    Program *p = nullptr;
    int rc = get_program(pl, kind, in, out, ws, &p);
    if (rc != LOP_OK) return rc;
    if (program_empty(p)) return LOP_OK;
    rc = program_launch(p, s);
    if (rc == LOP_OK) pl->exec->launches++;
    return rc;
}

void reset_layer_timing(lop_plan_t *pl)
{
    for (auto &c : pl->exec->layer_timed) c = 0;
}

int copy_rows_impl(lop_plan_t *pl, int lo, int hi, const void *host, void *staging, cudaStream_t s);

int copy_band_impl(lop_plan_t *pl, int band, const void *host, void *staging, cudaStream_t s)
{
    const lop_range &need = pl->in_need[band];
    return copy_rows_impl(pl, need.new_lo, need.out_hi, host, staging, s);
}

// Rows [lo, hi) of every image of the chain input, pinned host -> device, one asynchronous (2-D) copy.
int copy_rows_impl(lop_plan_t *pl, int lo, int hi, const void *host, void *staging, cudaStream_t s)
{
    if (hi <= lo) return LOP_OK;
    const size_t row = (size_t)pl->W * pl->C * elem_size(pl->dtype);
    const size_t img = row * pl->H;
    if (pl->N == 1)
        LOP_CUDA(cudaMemcpyAsync(static_cast<char *>(staging) + lo * row, static_cast<const char *>(host) + lo * row, (size_t)(hi - lo) * row,
                                 cudaMemcpyHostToDevice, s));
    else
        LOP_CUDA(cudaMemcpy2DAsync(static_cast<char *>(staging) + lo * row, img, static_cast<const char *>(host) + lo * row, img,
                                   (size_t)(hi - lo) * row, pl->N, cudaMemcpyHostToDevice, s));
    pl->exec->copies++;
    return LOP_OK;
}

// The single-launch band pipeline on stream s (which may be capturing): fork the side streams, launch the
// persistent kernel, enqueue every band's copy and arrival write, join.
// withheld: a band whose copy and arrival write are left out (lop_run_pipelined_withheld), or -1.
int enqueue_pipelined(lop_plan_t *pl, Program *p, const void *host, void *staging, cudaStream_t s, int withheld = -1)
{
    ExecState *e = pl->exec;
    int rc = LOP_OK;
    // the side streams start after everything already queued on the caller's stream
    LOP_CUDA(cudaEventRecord(e->ev_fork, s));
    LOP_CUDA(cudaStreamWaitEvent(e->copy_stream, e->ev_fork, 0));
    if (!program_empty(p)) {
        if ((rc = program_launch(p, s)) != LOP_OK) return rc;
        e->launches++;
    }
    // Every command on a stream costs a few microseconds whatever its size -- as much as a small band's copy, more
    // than its compute -- and commands of one stream run strictly one after the other.  So the copy stream carries,
    // per band, the copy and an event record and nothing else (no timing events), and a second stream waits for that
    // event and performs the 4-byte arrival write the kernel polls: the write of band b overlaps the copy of band b+1.
    StreamWriteValue32Fn write32 = stream_write_fn();
    LOP_CUDA(cudaStreamWaitEvent(e->signal_stream, e->ev_fork, 0));
    const int G = std::max(1, pl->copy_group);
    for (int b0 = 0; b0 < pl->n_bands; b0 += G) {
        // one copy for the bands [b0, b1): their new rows are one contiguous run; the arrival is written for the last band
        const int b1 = std::min(pl->n_bands, b0 + G), b = b1 - 1;
        int lo = 0, hi = 0;
        bool any = false;
        for (int q = b0; q < b1; ++q) {
            const lop_range &need = pl->in_need[q];
            e->copy_issued[q] = 0;
            if (need.out_hi <= need.new_lo) continue;
            lo = any ? std::min(lo, (int)need.new_lo) : (int)need.new_lo;
            hi = any ? std::max(hi, (int)need.out_hi) : (int)need.out_hi;
            any = true;
        }
        if (withheld >= b0 && withheld < b1) continue;
        e->copy_issued[b] = any;
        if (any && (rc = copy_rows_impl(pl, lo, hi, host, staging, e->copy_stream)) != LOP_OK) return rc;
        unsigned *flag = program_arrival_flag(p, b);
        if (!flag) continue;
        LOP_CUDA(cudaEventRecord(e->ev_arrive[b], e->copy_stream));
        LOP_CUDA(cudaStreamWaitEvent(e->signal_stream, e->ev_arrive[b], 0));
        if (write32) {
            if (write32(reinterpret_cast<CUstream>(e->signal_stream), reinterpret_cast<CUdeviceptr>(flag), 1u, 0u) != CUDA_SUCCESS) {
                set_error("cuStreamWriteValue32 failed");
                return LOP_ECUDA;
            }
        } else {
            LOP_CUDA(cudaMemcpyAsync(flag, e->pinned_one, sizeof(unsigned), cudaMemcpyHostToDevice, e->signal_stream));
        }
    }
    e->copies_timed = false;
    LOP_CUDA(cudaEventRecord(e->ev_signal_join, e->signal_stream));
    LOP_CUDA(cudaStreamWaitEvent(s, e->ev_signal_join, 0));
    LOP_CUDA(cudaEventRecord(e->ev_join, e->copy_stream));
    LOP_CUDA(cudaStreamWaitEvent(s, e->ev_join, 0));
    return LOP_OK;
}

}  // namespace
}  // namespace lop

using namespace lop;

extern "C" {

int lop_run_whole(lop_plan_t *pl, const void *in, void *out, void *ws, void *stream)
{
    int rc = check_common(pl, in, out, ws);
    if (rc != LOP_OK) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    pl->exec->launches = pl->exec->copies = 0;
    pl->exec->last_stream = s;
    reset_layer_timing(pl);
    if ((rc = prepare_workspace(pl, ws, s)) != LOP_OK) return rc;
    if (pl->exec->wavefront) return run_program(pl, PROG_WHOLE, in, out, ws, s);
    for (int i = 0; i < (int)pl->layers.size(); ++i)
        if ((rc = run_layer(pl, i, 0, pl->layers[i].Ho, in, out, ws, s, i)) != LOP_OK) return rc;
    return LOP_OK;
}

int lop_run_band(lop_plan_t *pl, int band, const void *in, void *out, void *ws, void *stream)
{
    int rc = check_common(pl, in, out, ws);
    if (rc != LOP_OK) return rc;
    if (band < 0 || band >= pl->n_bands) { set_error("band %d out of range", band); return LOP_EINVAL; }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    pl->exec->launches = pl->exec->copies = 0;
    pl->exec->last_stream = s;
    if ((rc = prepare_workspace(pl, ws, s)) != LOP_OK) return rc;
    if (pl->exec->wavefront) return run_program(pl, band, in, out, ws, s);
    return run_band_impl(pl, band, in, out, ws, s);
}

int lop_run_banded(lop_plan_t *pl, const void *in, void *out, void *ws, void *stream)
{
    int rc = check_common(pl, in, out, ws);
    if (rc != LOP_OK) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    pl->exec->launches = pl->exec->copies = 0;
    pl->exec->last_stream = s;
    reset_layer_timing(pl);
    if ((rc = prepare_workspace(pl, ws, s)) != LOP_OK) return rc;
    if (pl->exec->wavefront) return run_program(pl, PROG_ALL_BANDS, in, out, ws, s);
    if (pl->flags & LOP_FLAG_TIME_LAYERS) {                       // timed plans keep one launch per (band, layer)
        for (int b = 0; b < pl->n_bands; ++b)
            if ((rc = run_band_impl(pl, b, in, out, ws, s)) != LOP_OK) return rc;
        return LOP_OK;
    }
    // Operation batching (Sec. IV-C): with the whole input on the device, the bands' operations at a layer are one
    // contiguous run of rows (neighbouring bands' ranges touch or overlap), so each layer is ONE launch over the hull of
    // the bands' rows.  Every row is computed once, with the same bits as band by band.
    const int L = (int)pl->layers.size();
    for (int i = 0; i < L; ++i) {
        int lo = 0, hi = 0;
        bool any = false, contiguous = true;
        for (int b = 0; b < pl->n_bands; ++b) {
            const lop_range &r = pl->ranges[(size_t)b * L + i];
            if (r.out_hi <= r.out_lo) continue;
            if (any && r.out_lo > hi) contiguous = false;
            lo = any ? std::min(lo, (int)r.out_lo) : (int)r.out_lo;
            hi = any ? std::max(hi, (int)r.out_hi) : (int)r.out_hi;
            any = true;
        }
        if (!any) continue;
        if (contiguous) {
            if ((rc = run_layer(pl, i, lo, hi, in, out, ws, s, -1)) != LOP_OK) return rc;
        } else {
            for (int b = 0; b < pl->n_bands; ++b) {
                const lop_range &r = pl->ranges[(size_t)b * L + i];
                if ((rc = run_layer(pl, i, first_row(pl, 0, b, i), r.out_hi, in, out, ws, s, -1)) != LOP_OK) return rc;
            }
        }
    }
    return LOP_OK;
}

int lop_run_layer(lop_plan_t *pl, int layer, int row_lo, int row_hi, const void *in, void *out, void *ws, void *stream)
{
    int rc = check_common(pl, in, out, ws);
    if (rc != LOP_OK) return rc;
    const int L = (int)pl->layers.size();
    if (layer < 0 || layer >= L) { set_error("lop_run_layer: layer %d out of range", layer); return LOP_EINVAL; }
    if (row_lo < 0 || row_hi > pl->layers[layer].Ho || row_lo > row_hi) { set_error("lop_run_layer: rows [%d,%d) out of range", row_lo, row_hi); return LOP_EINVAL; }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    pl->exec->launches = pl->exec->copies = 0;
    pl->exec->last_stream = s;
    if ((rc = prepare_workspace(pl, ws, s)) != LOP_OK) return rc;
    return run_layer(pl, layer, row_lo, row_hi, in, out, ws, s, -1);
}

int lop_plan_shard(const lop_plan_t *pl, int rank, int world, int *band_lo, int *band_hi, int *row_lo, int *row_hi, int *in_lo,
                   int *in_hi)
{
    if (!pl || !band_lo || !band_hi || !row_lo || !row_hi || !in_lo || !in_hi) { set_error("lop_plan_shard: NULL argument"); return LOP_EINVAL; }
    if (world < 1 || rank < 0 || rank >= world) { set_error("lop_plan_shard: rank %d of %d", rank, world); return LOP_EINVAL; }
    const int B = pl->n_bands, L = (int)pl->layers.size();
    const int b0 = (int)((long long)rank * B / world), b1 = (int)((long long)(rank + 1) * B / world);
    *band_lo = b0; *band_hi = b1;
    *row_lo = *row_hi = *in_lo = *in_hi = 0;
    bool have_rows = false, have_in = false;
    for (int b = b0; b < b1; ++b) {
        const lop_range &r = pl->ranges[(size_t)b * L + (L - 1)];
        if (r.out_hi > r.out_lo) {
            if (!have_rows) { *row_lo = r.out_lo; have_rows = true; }
            *row_hi = r.out_hi;
        }
        const lop_range &n = pl->in_need[b];
        if (n.out_hi > n.out_lo) {
            if (!have_in || n.out_lo < *in_lo) *in_lo = n.out_lo;
            if (!have_in || n.out_hi > *in_hi) *in_hi = n.out_hi;
            have_in = true;
        }
    }
    return LOP_OK;
}

int lop_run_shard(lop_plan_t *pl, int band_lo, int band_hi, const void *in, void *out, void *ws, void *stream)
{
    int rc = check_common(pl, in, out, ws);
    if (rc != LOP_OK) return rc;
    if (band_lo < 0 || band_hi > pl->n_bands || band_lo > band_hi) { set_error("bands [%d,%d) out of range", band_lo, band_hi); return LOP_EINVAL; }
    if (pl->n_bands > 65535) { set_error("lop_run_shard: more than 65535 bands"); return LOP_EUNSUPPORTED; }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    pl->exec->launches = pl->exec->copies = 0;
    pl->exec->last_stream = s;
    reset_layer_timing(pl);
    if ((rc = prepare_workspace(pl, ws, s)) != LOP_OK) return rc;
    if (band_lo == band_hi) return LOP_OK;
    if (pl->exec->wavefront) return run_program(pl, PROG_BLOCK0 - (band_lo * 65536 + band_hi), in, out, ws, s);
    // per-layer launches
    const int L = (int)pl->layers.size();
    for (int b = band_lo; b < band_hi; ++b)
        for (int i = 0; i < L; ++i) {
            const lop_range &r = pl->ranges[(size_t)b * L + i];
            rc = run_layer(pl, i, first_row(pl, band_lo, b, i), r.out_hi, in, out, ws, s, (b + 1) * L + i);
            if (rc != LOP_OK) return rc;
        }
    return LOP_OK;
}

int lop_copy_band(lop_plan_t *pl, int band, const void *host, void *staging, void *stream)
{
    if (!pl || !host || !staging) { set_error("lop_copy_band: NULL argument"); return LOP_EINVAL; }
    if (band < 0 || band >= pl->n_bands) { set_error("band %d out of range", band); return LOP_EINVAL; }
    int rc = ensure_exec(pl);
    if (rc != LOP_OK) return rc;
    pl->exec->launches = pl->exec->copies = 0;
    return copy_band_impl(pl, band, host, staging, static_cast<cudaStream_t>(stream));
}

int lop_fetch_band(lop_plan_t *pl, int band, const void *host, void *staging, void *ws, void *stream)
{
    if (!pl || !host || !staging) { set_error("lop_fetch_band: NULL argument"); return LOP_EINVAL; }
    if (band < -1 || band >= pl->n_bands) { set_error("band %d out of range", band); return LOP_EINVAL; }
    int rc = check_common(pl, staging, staging, ws);
    if (rc != LOP_OK) return rc;
    ExecState *e = pl->exec;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    e->launches = e->copies = 0;
    e->last_stream = s;
    if (!e->wavefront) { set_error("lop_fetch_band: this plan does not run on the persistent kernel; use lop_copy_band"); return LOP_EUNSUPPORTED; }
    const void *src = fetchable(pl, host);
    if (!src || (reinterpret_cast<uintptr_t>(src) & 15) != (reinterpret_cast<uintptr_t>(staging) & 15)) {
        set_error("lop_fetch_band: the host buffer is not mapped into the device's address space, or differs from the staging tensor modulo 16 bytes");
        return LOP_EUNSUPPORTED;
    }
    if ((rc = prepare_workspace(pl, ws, s)) != LOP_OK) return rc;
    Program *p = nullptr;
    if ((rc = get_program(pl, PROG_FETCH_ALONE, staging, staging, ws, &p, src, band)) != LOP_OK) return rc;
    if (program_empty(p)) return LOP_OK;
    if ((rc = program_launch(p, s)) != LOP_OK) return rc;
    e->launches++;
    return LOP_OK;
}

int lop_run_pipelined(lop_plan_t *pl, const void *host, void *staging, void *out, void *ws, void *stream)
{
    int rc = check_common(pl, staging, out, ws);
    if (rc != LOP_OK) return rc;
    if (!host) { set_error("lop_run_pipelined: host input is NULL"); return LOP_EINVAL; }
    ExecState *e = pl->exec;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    e->launches = e->copies = 0;
    e->last_stream = s;
    e->timing_valid = false;
    reset_layer_timing(pl);
    // an event record is a stream command of its own (microseconds): only plans that ask for timing pay for them
    const bool timed = (pl->flags & LOP_FLAG_TIME_LAYERS) != 0;
    if (timed) LOP_CUDA(cudaEventRecord(e->ev_begin, s));
    if ((rc = prepare_workspace(pl, ws, s)) != LOP_OK) return rc;
    if (e->wavefront) {
        // One persistent launch for the whole request: it starts at once and every band's first stage waits
        // for that band's arrival flag, which a side stream sets right after the band's copy.  Plain stream
        // calls: replaying the same schedule from a CUDA graph was measured slower (and stalled for hundreds of
        // microseconds with 32 bands of 196 KB), so no graph is built here; a caller whose stream is capturing
        // simply gets these operations into its own graph.
        Program *p = nullptr;
        const void *src = fetchable(pl, host);
        if (src && (reinterpret_cast<uintptr_t>(src) & 15) == (reinterpret_cast<uintptr_t>(staging) & 15)) {
            // the kernel fetches the bands itself: nothing but the launch
            if ((rc = get_program(pl, PROG_FETCHED, staging, out, ws, &p, src)) != LOP_OK) return rc;
            for (int b = 0; b < pl->n_bands; ++b) e->copy_issued[b] = 0;
            e->copies_timed = false;
            if (!program_empty(p)) {
                if ((rc = program_launch(p, s)) != LOP_OK) return rc;
                e->launches++;
            }
        } else {
            if ((rc = get_program(pl, PROG_PIPELINED, staging, out, ws, &p)) != LOP_OK) return rc;
            if ((rc = enqueue_pipelined(pl, p, host, staging, s)) != LOP_OK) return rc;
        }
        if (timed) LOP_CUDA(cudaEventRecord(e->ev_end, s));
        e->timing_valid = timed;
        return LOP_OK;
    }
    // the side stream starts after everything already queued on the caller's stream; all transfers are queued
    // up front on it: band i+1 (and later) stream in while band i computes
    LOP_CUDA(cudaEventRecord(e->ev_fork, s));
    LOP_CUDA(cudaStreamWaitEvent(e->copy_stream, e->ev_fork, 0));
    e->copies_timed = true;
    for (int b = 0; b < pl->n_bands; ++b) {
        const lop_range &need = pl->in_need[b];
        e->copy_issued[b] = need.out_hi > need.new_lo;
        if (!e->copy_issued[b]) continue;
        LOP_CUDA(cudaEventRecord(e->ev_copy_start[b], e->copy_stream));
        if ((rc = copy_band_impl(pl, b, host, staging, e->copy_stream)) != LOP_OK) return rc;
        LOP_CUDA(cudaEventRecord(e->ev_copy_end[b], e->copy_stream));
    }
    bool joined = false;
    for (int b = 0; b < pl->n_bands; ++b) {
        if (e->copy_issued[b]) {
            LOP_CUDA(cudaStreamWaitEvent(s, e->ev_copy_end[b], 0));
            joined = true;
        }
        if ((rc = run_band_impl(pl, b, staging, out, ws, s)) != LOP_OK) return rc;
    }
    if (!joined) LOP_CUDA(cudaStreamWaitEvent(s, e->ev_fork, 0));
    if (timed) LOP_CUDA(cudaEventRecord(e->ev_end, s));
    e->timing_valid = timed;
    return LOP_OK;
}

int lop_plan_set_wait_limit(lop_plan_t *pl, unsigned polls)
{
    if (!pl) { set_error("plan is NULL"); return LOP_EINVAL; }
    pl->wait_limit = polls;
    return LOP_OK;
}

int lop_run_pipelined_withheld(lop_plan_t *pl, int band, const void *host, void *staging, void *out, void *ws, void *stream)
{
    int rc = check_common(pl, staging, out, ws);
    if (rc != LOP_OK) return rc;
    if (!host) { set_error("lop_run_pipelined_withheld: host input is NULL"); return LOP_EINVAL; }
    if (band < 0 || band >= pl->n_bands) { set_error("band %d out of range", band); return LOP_EINVAL; }
    ExecState *e = pl->exec;
    if (!e->wavefront) { set_error("lop_run_pipelined_withheld: this plan does not run on the persistent kernel"); return LOP_EUNSUPPORTED; }
    if (pl->wait_limit == 0 || pl->wait_limit > (1u << 16)) {
        set_error("lop_run_pipelined_withheld: set a wait limit of at most 65536 polls first (lop_plan_set_wait_limit)");
        return LOP_EINVAL;
    }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    e->launches = e->copies = 0;
    e->last_stream = s;
    e->timing_valid = false;
    if ((rc = prepare_workspace(pl, ws, s)) != LOP_OK) return rc;
    Program *p = nullptr;
    if ((rc = get_program(pl, PROG_PIPELINED, staging, out, ws, &p)) != LOP_OK) return rc;
    return enqueue_pipelined(pl, p, host, staging, s, band);
}

namespace {

// Validates a chain of plans (plan s+1 consumes plan s's output) and readies every plan for the persistent kernel.
int chain_prepare(lop_plan_t *const *plans, int n, const void *in0, void *const *outs, void *const *wss, cudaStream_t s,
                  std::vector<SegBind> &segs)
{
    if (!plans || !outs || !wss || n < 1) { set_error("chain: NULL argument or no plan"); return LOP_EINVAL; }
    const void *in = in0;
    for (int i = 0; i < n; ++i) {
        lop_plan_t *pl = plans[i];
        int rc = check_common(pl, in, outs[i], wss[i]);
        if (rc != LOP_OK) return rc;
        if (!pl->exec->wavefront) { set_error("chain: plan %d has a layer the persistent kernel does not take; run the plans one by one", i); return LOP_EUNSUPPORTED; }
        if (i > 0) {
            const lop_plan_t *pv = plans[i - 1];
            const LayerInfo &last = pv->layers.back();
            if (pl->N != pv->N || pl->H != last.Ho || pl->W != last.Wo || pl->C != last.Co || pl->dtype != pv->dtype ||
                (pl->flags & LOP_FLAG_REUSE_HALO) != (pv->flags & LOP_FLAG_REUSE_HALO)) {
                set_error("chain: plan %d does not take plan %d's output (shape, dtype or halo mode differ)", i, i - 1);
                return LOP_ESHAPE;
            }
        }
        pl->exec->launches = pl->exec->copies = 0;
        pl->exec->last_stream = s;
        if ((rc = prepare_workspace(pl, wss[i], s)) != LOP_OK) return rc;
        segs.push_back(SegBind{pl, in, outs[i], wss[i]});
        in = outs[i];
    }
    return LOP_OK;
}

}  // namespace

int lop_run_chain_banded(lop_plan_t *const *plans, int n_plans, const void *in_dev, void *const *outs_dev, void *const *workspaces,
                         void *stream)
{
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    std::vector<SegBind> segs;
    int rc = chain_prepare(plans, n_plans, in_dev, outs_dev, workspaces, s, segs);
    if (rc != LOP_OK) return rc;
    Program *p = nullptr;
    if ((rc = get_program(segs, PROG_ALL_BANDS, &p)) != LOP_OK) return rc;
    if (program_empty(p)) return LOP_OK;
    if ((rc = program_launch(p, s)) != LOP_OK) return rc;
    plans[0]->exec->launches++;
    return LOP_OK;
}

int lop_run_chain_pipelined(lop_plan_t *const *plans, int n_plans, const void *host, void *staging, void *const *outs_dev,
                            void *const *workspaces, void *stream)
{
    if (!host) { set_error("lop_run_chain_pipelined: host input is NULL"); return LOP_EINVAL; }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    std::vector<SegBind> segs;
    int rc = chain_prepare(plans, n_plans, staging, outs_dev, workspaces, s, segs);
    if (rc != LOP_OK) return rc;
    ExecState *e = plans[0]->exec;
    e->timing_valid = false;
    Program *p = nullptr;
    const void *src = fetchable(plans[0], host);
    if (src && (reinterpret_cast<uintptr_t>(src) & 15) == (reinterpret_cast<uintptr_t>(staging) & 15)) {
        if ((rc = get_program(segs, PROG_FETCHED, &p, src)) != LOP_OK) return rc;
        for (int b = 0; b < plans[0]->n_bands; ++b) e->copy_issued[b] = 0;
        e->copies_timed = false;
        if (!program_empty(p)) {
            if ((rc = program_launch(p, s)) != LOP_OK) return rc;
            e->launches++;
        }
    } else {
        if ((rc = get_program(segs, PROG_PIPELINED, &p)) != LOP_OK) return rc;
        if ((rc = enqueue_pipelined(plans[0], p, host, staging, s)) != LOP_OK) return rc;
    }
    return LOP_OK;
}

int lop_plan_last_timing(lop_plan_t *pl, lop_timing *out)
{
    if (!pl || !out) { set_error("lop_plan_last_timing: NULL argument"); return LOP_EINVAL; }
    if (!pl->exec || !pl->exec->timing_valid) { set_error("no timed pipelined run to report (the plan needs LOP_FLAG_TIME_LAYERS)"); return LOP_EINVAL; }
    ExecState *e = pl->exec;
    LOP_CUDA(cudaEventSynchronize(e->ev_end));
    lop_timing t = {0, 0, 0, 0, 0};
    LOP_CUDA(cudaEventElapsedTime(&t.total_ms, e->ev_begin, e->ev_end));
    bool first = true;
    for (int b = 0; b < pl->n_bands; ++b) {
        if (!e->copy_issued[b]) continue;
        float ms = 0;
        if (e->copies_timed) LOP_CUDA(cudaEventElapsedTime(&ms, e->ev_copy_start[b], e->ev_copy_end[b]));
        t.copy_ms += ms;
        if (first) { t.first_copy_ms = ms; first = false; }
        t.n_copies++;
    }
    *out = t;
    return LOP_OK;
}

int lop_plan_layer_time(lop_plan_t *pl, int band, int layer, float *ms)
{
    if (!pl || !ms) { set_error("lop_plan_layer_time: NULL argument"); return LOP_EINVAL; }
    const int L = (int)pl->layers.size();
    if (band < -1 || band >= pl->n_bands || layer < 0 || layer >= L) { set_error("band/layer out of range"); return LOP_EINVAL; }
    if (!pl->exec || pl->exec->ev_layer.empty()) { set_error("plan was not made with LOP_FLAG_TIME_LAYERS, or has not run"); return LOP_EINVAL; }
    ExecState *e = pl->exec;
    const size_t slot = (size_t)(band + 1) * L + layer;
    *ms = 0.0f;
    if (!e->layer_timed[slot]) return LOP_OK;
    LOP_CUDA(cudaEventSynchronize(e->ev_layer[slot * 2 + 1]));
    LOP_CUDA(cudaEventElapsedTime(ms, e->ev_layer[slot * 2], e->ev_layer[slot * 2 + 1]));
    return LOP_OK;
}

int lop_plan_layer_offset(const lop_plan_t *pl, int layer, size_t *offset)
{
    if (!pl || !offset) { set_error("lop_plan_layer_offset: NULL argument"); return LOP_EINVAL; }
    const int L = (int)pl->layers.size();
    if (layer < 0 || layer >= L - 1) { set_error("lop_plan_layer_offset: layer %d is not an intermediate layer", layer); return LOP_EINVAL; }
    *offset = pl->layers[layer].out_off;
    return LOP_OK;
}

int lop_plan_layer_stored(const lop_plan_t *pl, int layer)
{
    if (!pl) { set_error("plan is NULL"); return LOP_EINVAL; }
    const int L = (int)pl->layers.size();
    if (layer < 0 || layer >= L) { set_error("lop_plan_layer_stored: layer %d out of range", layer); return LOP_EINVAL; }
    const bool persistent = program_supported(pl) && !(pl->flags & (LOP_FLAG_PER_LAYER | LOP_FLAG_TIME_LAYERS | LOP_FLAG_DEBUG_BOUNDS));
    return (persistent && program_folds_pool(pl, layer)) ? 0 : 1;
}

int lop_plan_last_launches(const lop_plan_t *pl)
{
    if (!pl) { set_error("plan is NULL"); return LOP_EINVAL; }
    return pl->exec ? pl->exec->launches : 0;
}

int lop_plan_last_copies(const lop_plan_t *pl)
{
    if (!pl) { set_error("plan is NULL"); return LOP_EINVAL; }
    return pl->exec ? pl->exec->copies : 0;
}

int lop_plan_check_device(lop_plan_t *pl, void *ws)
{
    if (!pl || !ws) { set_error("lop_plan_check_device: NULL argument"); return LOP_EINVAL; }
    if (!pl->exec) return LOP_OK;
    LOP_CUDA(cudaStreamSynchronize(pl->exec->last_stream));
    unsigned status = 0;
    LOP_CUDA(cudaMemcpy(&status, static_cast<char *>(ws) + pl->status_off, sizeof(status), cudaMemcpyDeviceToHost));
    if (status) {
        // the run was abandoned half way: its row-group counters are meaningless now, so the programs (and their
        // counters) are dropped and rebuilt on the next call; the status word is cleared for that call
        for (auto &kv : pl->exec->programs) program_destroy(kv.second);
        pl->exec->programs.clear();
        cudaMemset(static_cast<char *>(ws) + pl->status_off, 0, sizeof(status));
        set_error(status & 0x100u ? "device status word 0x%x: a checked kernel computed an address outside its tensor (the access was skipped)"
                                 : "device status word 0x%x: a bounded wait ran out", status);
        return LOP_EDEVICE;
    }
    return LOP_OK;
}

}  // extern "C"

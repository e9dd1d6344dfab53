// Host side of the wavefront kernel: turns a list of (band, layer, row range) requests into a
// device-resident program (stages, item records, tensor maps, dependency lists, counters).
//
// Dependencies follow Sec. IV-B of the paper: a tile depends on a producer row group as soon as
// any row of that group lies inside the tile's receptive rows (for the residual: its own rows).
#include <cuda_runtime.h>

#include <algorithm>
#include <cmath>
#include <cstdio>
#include <vector>

#include "lop_internal.h"
#include "lop_kernels.cuh"
#include "lop_layerargs.h"
#include "lop_program.h"
#include "lop_rowops.cuh"
#include "lop_wavefront.cuh"

namespace lop {

struct Program {
    void *dev = nullptr;            // one allocation holding every table
    unsigned *counters = nullptr;
    WfParams params{};
    int grid = 0;
    int flag_base = 0, n_flags = 0;
    const lop_plan_t *owner = nullptr;  // the first plan: its wait limit applies to the launches
};

void program_destroy(Program *p)
{
    if (!p) return;
    if (p->dev) cudaFree(p->dev);
    delete p;
}

namespace {

#ifndef LOP_FETCH_ENTRY_BYTES
#define LOP_FETCH_ENTRY_BYTES 3072
#endif
#ifndef LOP_FETCH_WINDOW_BYTES
#define LOP_FETCH_WINDOW_BYTES (96 * 1024)
#endif
#ifndef LOP_FETCH_WINDOW_MAX_BYTES
#define LOP_FETCH_WINDOW_MAX_BYTES (256 * 1024)
#endif
#ifndef LOP_SA_MAX
#define LOP_SA_MAX 4
#endif
#ifndef LOP_SB_MAX
#define LOP_SB_MAX 8
#endif
#ifndef LOP_CPS_MAX
#define LOP_CPS_MAX 4
#endif
constexpr uint32_t A_BOX_MAX = 48u * 1024u;     // largest activation box a ring slot is sized for
constexpr uint32_t LOP_ROWOP_STAGING_BYTES = 64u * 1024u;    // largest receptive window a depth-wise item stages
constexpr uint32_t B_BOX_MAX = 32u * 1024u;     // largest weight box

int ilog2i(int v) { int l = 0; while ((1 << l) < v) ++l; return l; }
uint32_t round_up_u32(uint32_t v, uint32_t a) { return (v + a - 1) / a * a; }

// Tile geometry of one convolution stage.
struct Geom {
    int mode;
    int P, TR, TN;            // anchors: TN images x TR rows x P columns = 128
    int tw_valid;             // output columns per tile
    int RI;                   // rows of the activation box
    int BN, BK, tb, n_taps, n_chunks;
    uint32_t a_bytes, b_bytes, a_slot, b_slot;
};

// a: the convolution as its kernel sees it (a gathered stem already reduced to 1x1).
// even_tiles: tiles must hold whole 2x2 windows (rows and valid columns even, at least two rows).
Geom choose_geom(const ConvArgs &a, int rows, bool even_tiles)
{
    Geom g{};
    g.BK = a.Cin % 64 == 0 ? 64 : (a.Cin % 32 == 0 ? 32 : 16);
    g.BN = 16;
    for (int bn = 128; bn >= 16; bn -= 16)
        if (a.Cout % bn == 0) { g.BN = bn; break; }
    // A layer with few pixel tiles (a small map deep in the network) would occupy a handful of SMs, each streaming
    // all of K for a wide slice of the weights at what one SM can pull from L2 (~40 GB/s measured): narrower
    // output-channel tiles spread the same weight traffic over more SMs.  Not below 64: an MMA with N = 32 costs the
    // issuing thread as much as one with N = 64 (measured on a ResNet-50 of batch 8: 669 us with a floor of 64, 732 us with 32).
    const long long layer_tiles = ((long long)a.N * a.Ho * a.Wo + 127) / 128;
    while (g.BN > 64 && g.BN % 32 == 0 && layer_tiles * (a.Cout / g.BN) < 148) g.BN /= 2;
    g.n_taps = a.kh * a.kw;
    g.n_chunks = a.Cin / g.BK;
    const uint32_t row_bytes = (uint32_t)g.BK * 2u;
    const bool pointwise = a.kh == 1 && a.kw == 1;
    const int halo_w = (a.kw - 1) * a.dw, halo_h = (a.kh - 1) * a.dh;
    bool slab = false;
    if (!pointwise && a.sh == 1 && a.sw == 1 && g.BK == 64) {
        // pitch P: the split of 128 anchors into rows of P pixels that needs the fewest tiles, then the smallest box
        long long best_tiles = -1, best_box = 0;
        for (int P = 16; P <= 128; P <<= 1) {
            const int twv = P - halo_w, TR = 128 / P, RI = TR + halo_h;
            if (twv < 8 || RI > 256 || (even_tiles && (TR < 2 || (twv & 1)))) continue;
            const uint32_t box = (uint32_t)RI * P * row_bytes;
            if (box > A_BOX_MAX) continue;
            const long long tiles = (long long)((a.Wo + twv - 1) / twv) * ((rows + TR - 1) / TR);
            if (best_tiles < 0 || tiles < best_tiles || (tiles == best_tiles && box < best_box)) {
                best_tiles = tiles; best_box = box;
                g.P = P; g.TR = TR; g.TN = 1; g.tw_valid = twv; g.RI = RI;
                slab = true;
            }
        }
    }
    if (slab || pointwise) g.mode = WF_SLAB;
    else g.mode = WF_TAP;
    if (!slab) {
        // dense tile: the (TW, TR, TN) split of 128 pixels that needs the fewest tiles
        int nmax = 1;
        while (nmax * 2 <= a.N) nmax *= 2;
        long long best = -1;
        g.P = 128; g.TR = 1; g.TN = 1;
        for (int tw = 128; tw >= 1; tw >>= 1)
            for (int tr = 128 / tw; tr >= 1; tr >>= 1) {
                const int tn = 128 / (tw * tr);
                if (tn > nmax || (even_tiles && (tw < 2 || tr < 2))) continue;
                const long long tiles = (long long)((a.Wo + tw - 1) / tw) * ((rows + tr - 1) / tr) * ((a.N + tn - 1) / tn);
                if (best < 0 || tiles < best) { best = tiles; g.P = tw; g.TR = tr; g.TN = tn; }
            }
        g.tw_valid = g.P; g.RI = g.TR;
    }
    g.a_bytes = (uint32_t)g.RI * g.P * g.TN * row_bytes;
    // a shifted tap reads up to halo_w pixels past the box: the slot's padding takes that
    g.a_slot = round_up_u32(g.a_bytes + (slab ? (uint32_t)halo_w * row_bytes : 0u), 1024u);
    g.tb = 1;
    if (g.mode == WF_SLAB && g.n_taps > 1) {
        const int cap = std::max(1, (int)(B_BOX_MAX / ((uint32_t)g.BN * row_bytes)));
        const int nblk = (g.n_taps + cap - 1) / cap;
        g.tb = (g.n_taps + nblk - 1) / nblk;
    }
    g.b_bytes = (uint32_t)g.tb * g.BN * row_bytes;
    g.b_slot = round_up_u32(g.b_bytes, 1024u);
    return g;
}

struct MapSet { int seg, layer, P, RI, TN, BN, BK, tb, base; };

// Five tensor maps of a convolution stage: the activation seen through the (row parity, column parity)
// classes of its stride, and the weights as [tap][cout][cin].
int encode_maps(const ConvArgs &a, const Geom &g, CUtensorMap *out, int *valid_mask)
{
    TensorMapEncodeFn enc = tensor_map_encoder();
    if (!enc) return LOP_ECUDA;
    const CUtensorMapSwizzle swz = g.BK == 64 ? CU_TENSOR_MAP_SWIZZLE_128B
                                   : (g.BK == 32 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B);
    const cuuint32_t ones[4] = {1, 1, 1, 1};
    int mask = 0;
    for (int ph = 0; ph < a.sh; ++ph)
        for (int pw = 0; pw < a.sw; ++pw) {
            const int idx = ph * a.sw + pw;
            if (idx >= 4) continue;
            const long long Hp = (a.Hin - ph + a.sh - 1) / a.sh, Wp = (a.Win - pw + a.sw - 1) / a.sw;
            if (a.Hin - ph <= 0 || a.Win - pw <= 0 || Hp <= 0 || Wp <= 0) continue;
            const cuuint64_t dims[4] = {(cuuint64_t)a.Cin, (cuuint64_t)Wp, (cuuint64_t)Hp, (cuuint64_t)a.N};
            const cuuint64_t strides[3] = {(cuuint64_t)a.sw * a.Cin * 2, (cuuint64_t)a.sh * a.Win * a.Cin * 2,
                                           (cuuint64_t)a.Hin * a.Win * a.Cin * 2};
            const cuuint32_t box[4] = {(cuuint32_t)g.BK, (cuuint32_t)g.P, (cuuint32_t)g.RI, (cuuint32_t)g.TN};
            void *basep = (void *)(static_cast<const char *>(a.x) + ((size_t)ph * a.Win + pw) * a.Cin * 2);
            if (enc(&out[idx], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, basep, dims, strides, box, ones, CU_TENSOR_MAP_INTERLEAVE_NONE, swz,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
                return LOP_ECUDA;
            mask |= 1 << idx;
        }
    if (!mask) return LOP_ECUDA;
    for (int i = 0; i < 4; ++i)
        if (!((mask >> i) & 1))
            for (int j = 0; j < 4; ++j)
                if ((mask >> j) & 1) { out[i] = out[j]; break; }
    const cuuint64_t taps = (cuuint64_t)a.kh * a.kw;
    const cuuint64_t wd[3] = {(cuuint64_t)a.Cin, (cuuint64_t)a.Cout, taps};
    const cuuint64_t ws[2] = {taps * a.Cin * 2, (cuuint64_t)a.Cin * 2};
    const cuuint32_t wb[3] = {(cuuint32_t)g.BK, (cuuint32_t)g.BN, (cuuint32_t)g.tb};
    if (enc(&out[4], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(a.w), wd, ws, wb, ones, CU_TENSOR_MAP_INTERLEAVE_NONE, swz,
            CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return LOP_ECUDA;
    *valid_mask = mask;
    return LOP_OK;
}

// Layer i is a tensor-core convolution whose output is read by nothing but a 2x2 stride-2 unpadded max pooling
// right behind it: the persistent kernel can then pool inside the convolution's epilogue.
bool pool_fusable(const lop_plan_t *pl, int i)
{
    const int L = (int)pl->layers.size();
    if (i + 1 >= L) return false;
    const LayerInfo &c = pl->layers[i], &q = pl->layers[i + 1];
    if (c.l.op != LOP_CONV2D || c.kernel != K_CONV_TC || q.l.op != LOP_MAXPOOL2D || q.l.input_from != i) return false;
    if (q.l.kh != 2 || q.l.kw != 2 || q.l.sh != 2 || q.l.sw != 2 || q.l.ph != 0 || q.l.pw != 0) return false;
    for (int j = i + 2; j < L; ++j)
        if (pl->layers[j].l.input_from == i || pl->layers[j].l.residual_from == i) return false;
    return true;
}

}  // namespace

// Item shape of a depth-wise stage in the persistent kernel (rows, columns and channels of one tile).
static bool dw_tile(const lop_plan_t *pl, const LayerInfo &li, rowop::DwTile *t)
{
    const lop_layer &l = li.l;
    rowop::DwTile tmp;
    if (!li.dw_transposed) return false;
    return rowop::dw_choose_tile(l.kh, l.kw, l.sh, l.sw, l.dh, l.dw, pl->N, li.Ho, li.Wo, l.cin, LOP_ROWOP_STAGING_BYTES, 32 * WF_WORKER_WARPS,
                                 t ? t : &tmp);
}

bool program_folds_pool(const lop_plan_t *pl, int layer) { return pool_fusable(pl, layer); }

bool program_supported(const lop_plan_t *pl)
{
    if (pl->dtype != LOP_BF16) return false;
    for (const auto &li : pl->layers) {
        if (li.l.op == LOP_CONV2D && li.kernel != K_CONV_TC) return false;
        // the worker warps move these in 16-byte vectors of eight channels
        if (li.l.op == LOP_DWCONV2D && !dw_tile(pl, li, nullptr)) return false;
        if (li.l.op == LOP_LAYERNORM && (li.l.cin % 8 != 0 || li.l.cin > 1024)) return false;     // a lane keeps at most four vectors
        if (li.l.op == LOP_CONCAT && (li.l.cin % 8 != 0 || li.l.cout % 8 != 0)) return false;
        if (li.l.op == LOP_MAXPOOL2D && li.l.cin % 8 != 0) return false;
    }
    return true;
}

namespace {

// What a request reads: rows of tensors produced inside the program, and whether it touches the raw chain input
// (only plan 0 can: a later plan's "input" is the previous plan's last layer).
struct Need { int tensor, lo, hi; bool same_seg; };
struct Reads { Need need[3]; int n = 0; bool raw = false; };

struct Ctx {
    const std::vector<SegBind> &segs;
    std::vector<int> base;              // first tensor id of each plan; id base+layer, base+L = the stem's patches
    int raw = -1;                       // tensor id of the chain input when the program fetches it itself, else -1
    int tensor_id(int seg, int layer) const { return base[seg] + layer; }
    int patches_id(int seg) const { return base[seg] + (int)segs[seg].pl->layers.size(); }
    int input_id(int seg) const { return tensor_id(seg - 1, (int)segs[seg - 1].pl->layers.size() - 1); }
};

// A convolution's shortcut, a concatenation's second tensor: read at the rows that are computed.
bool has_second_input(const lop_layer &l)
{
    return (l.op == LOP_CONV2D || l.op == LOP_DWCONV2D || l.op == LOP_CONCAT) && l.residual_from != LOP_NO_RESIDUAL;
}

// Rows [o0, o1) of request rq: the tensors and rows they are computed from (Sec. IV-B: a dependency exists as soon as
// any part of a producer's output is used).
Reads reads_of(const Ctx &cx, const StageReq &rq, int o0, int o1)
{
    Reads r;
    const lop_plan_t *pl = cx.segs[rq.seg].pl;
    const LayerInfo &li = pl->layers[rq.layer];
    const lop_layer &l = li.l;
    auto window = [&](int &a_out, int &b_out) {
        long long a = (long long)o0 * l.sh - l.ph, b = (long long)(o1 - 1) * l.sh - l.ph + (long long)(l.kh - 1) * l.dh;
        a = std::max(a, 0LL); b = std::min(b, (long long)li.Hin - 1);
        a_out = (int)a; b_out = (int)b + 1;
        return a <= b;
    };
    int a = 0, b = 0;
    if (rq.fetch) return r;                                                   // reads host memory only
    if (rq.gather || (l.input_from == LOP_INPUT && !li.stem_gather)) {
        if (rq.seg == 0) {
            r.raw = true;
            if (cx.raw >= 0 && window(a, b)) r.need[r.n++] = Need{cx.raw, a, b, false};     // whichever band fetched them
        } else if (window(a, b)) r.need[r.n++] = Need{cx.input_id(rq.seg), a, b, false};
    } else if (li.stem_gather) {
        r.need[r.n++] = Need{cx.patches_id(rq.seg), o0, o1, true};            // the patches of exactly these rows
    } else if (window(a, b)) {
        r.need[r.n++] = Need{cx.tensor_id(rq.seg, l.input_from), a, b, true};
    }
    if (!rq.gather && has_second_input(l)) {
        if (l.residual_from >= 0) r.need[r.n++] = Need{cx.tensor_id(rq.seg, l.residual_from), o0, o1, true};
        else if (rq.seg == 0) {
            r.raw = true;
            if (cx.raw >= 0) r.need[r.n++] = Need{cx.raw, o0, o1, false};
        } else r.need[r.n++] = Need{cx.input_id(rq.seg), o0, o1, false};
    }
    return r;
}

// Rough shape of a stage for the ordering below: how many items it is cut into and how long one takes (microseconds;
// measured: ~1.2 us fixed per convolution tile plus ~0.035 us per tensor-core instruction and ~0.2 us per operand box, each
// issued by one thread; ~4 us more until the tile's epilogue has run and its rows are visible;
// ~2.5 us per pooling / gather row).  A fetch is not run by the CTAs: items = 0, item_us = its time on the host link.
struct StageShape { int items; double item_us; double tail_us; };   // tail_us: from an item's end on its CTA to its result being visible
StageShape stage_shape(const Ctx &cx, const StageReq &rq)
{
    const lop_plan_t *pl = cx.segs[rq.seg].pl;
    const LayerInfo &li = pl->layers[rq.layer];
    const double rows = rq.hi - rq.lo;
    if (rq.fetch) return StageShape{0, rows * pl->W * pl->C * 2.0 * pl->N / 24e3, 0.0};      // ~24 GB/s measured for SM-issued reads
    if (rq.gather || li.l.op == LOP_MAXPOOL2D || li.l.op == LOP_CONCAT) return StageShape{(int)rows * pl->N, 2.5, 0.5};
    if (li.l.op == LOP_LAYERNORM) return StageShape{(int)rows * pl->N, 4.0, 0.5};
    if (li.l.op == LOP_DWCONV2D) {
        rowop::DwTile t{1, 1, 8};
        dw_tile(pl, li, &t);
        return StageShape{(int)((rows + t.R - 1) / t.R) * pl->N * ((li.Wo + t.tw - 1) / t.tw) * (li.l.cin / t.cc), 4.0, 0.5};
    }
    const double tiles = std::ceil(rows * li.Wo * pl->N / 128.0) * std::max(1, li.l.cout / 128);
    // operand boxes, ~0.2 us each (issue, and the wait for a free ring slot): one per (tap, 64-channel chunk) and operand for strided windows, one
    // activation box and a few weight boxes per chunk otherwise
    const int taps = li.stem_gather ? 1 : li.l.kh * li.l.kw;
    const double chunks = std::ceil(li.cin_eff / 64.0);
    const bool per_tap = taps > 1 && (li.l.sh != 1 || li.l.sw != 1 || li.cin_eff % 64 != 0);
    const double boxes = per_tap ? 2.0 * taps * chunks : (1.0 + std::ceil(taps / 3.0)) * chunks;
    // a CTA overlaps a tile's epilogue with the next tile's loads and MMAs: the epilogue is latency, not occupancy
    return StageShape{(int)tiles, 1.2 + 0.2 * boxes + 0.035 * taps * (li.cin_eff / 16.0), 4.0};
}

// Puts the requests into program order.  Resident programs: ascending priority as far as dependencies allow (a
// stable topological order).  Programs whose input arrives while they run (arrival_us: when each band of plan 0 is
// expected on the device; or fetch requests): the order in which a model of the machine would start the stages.
int order_requests(const Ctx &cx, std::vector<StageReq> &reqs, bool reuse, const std::vector<double> *arrival_us)
{
    const size_t n = reqs.size();
    std::vector<int> produces(n);
    for (size_t i = 0; i < n; ++i)
        produces[i] = reqs[i].fetch ? cx.raw : (reqs[i].gather ? cx.patches_id(reqs[i].seg) : cx.tensor_id(reqs[i].seg, reqs[i].layer));
    const bool by_start = arrival_us != nullptr || cx.raw >= 0;
    bool sorted_already = !by_start;
    for (size_t i = 1; i < n; ++i)
        if (reqs[i].prio < reqs[i - 1].prio) sorted_already = false;
    std::vector<std::vector<int>> users(n), prods(n);
    std::vector<char> raw(n, 0);
    for (size_t i = 0; i < n; ++i) {
        const Reads r = reads_of(cx, reqs[i], reqs[i].lo, reqs[i].hi);
        raw[i] = r.raw;
        for (int q = 0; q < r.n; ++q)
            for (size_t j = 0; j < n; ++j) {
                if (j == i || produces[j] != r.need[q].tensor) continue;
                if (!reuse && r.need[q].same_seg && reqs[j].band != reqs[i].band) continue;
                if (std::max(r.need[q].lo, reqs[j].lo) >= std::min(r.need[q].hi, reqs[j].hi)) continue;
                users[j].push_back((int)i);
                prods[i].push_back((int)j);
                if (j > i) sorted_already = false;
            }
    }
    if (sorted_already) return LOP_OK;
    auto kahn = [&](std::vector<int> &order) {
        auto later = [&](int x, int y) { return reqs[x].prio != reqs[y].prio ? reqs[x].prio > reqs[y].prio : x > y; };
        std::vector<int> pending(n), heap;
        for (size_t i = 0; i < n; ++i) {
            pending[i] = (int)prods[i].size();
            if (!pending[i]) heap.push_back((int)i);
        }
        std::make_heap(heap.begin(), heap.end(), later);
        order.clear();
        while (!heap.empty()) {
            std::pop_heap(heap.begin(), heap.end(), later);
            const int i = heap.back();
            heap.pop_back();
            order.push_back(i);
            for (int u : users[i])
                if (--pending[u] == 0) { heap.push_back(u); std::push_heap(heap.begin(), heap.end(), later); }
        }
        return order.size() == n;
    };
    std::vector<int> order;
    if (!by_start) {
        if (!kahn(order)) { set_error("the stage requests depend on each other in a cycle"); return LOP_EINVAL; }
    } else {
        // A model of the machine as it really runs: items go round-robin to n_cta CTAs in program order and each
        // CTA takes its items in order, waiting for an item's stage to be ready; fetches queue on the host link.
        struct Machine {
            std::vector<double> cta_free;
            double link_free = 0.0, makespan = 0.0;
            long long rr = 0;                                   // items placed so far: the round-robin position
            explicit Machine(int n_cta) : cta_free(n_cta, 0.0) {}
            double run(const StageShape &sh, bool fetch, double ready)
            {
                double fin = ready;
                if (fetch) {
                    const double start = std::max(ready, link_free);
                    link_free = start + sh.item_us;
                    fin = link_free + 3.0;                      // + the link's latency
                } else {
                    for (int it = 0; it < sh.items; ++it, ++rr) {
                        double &f = cta_free[rr % (long long)cta_free.size()];
                        f = std::max(f, ready) + sh.item_us;
                        fin = std::max(fin, f + sh.tail_us);
                    }
                }
                makespan = std::max(makespan, fin);
                return fin;
            }
        };
        const int n_cta = 148;
        const double hop_us = 1.0;                              // producer's last store -> consumer sees the counter
        std::vector<StageShape> shape(n);
        for (size_t i = 0; i < n; ++i) shape[i] = stage_shape(cx, reqs[i]);
        auto arrival_of = [&](int i) {
            return (arrival_us && raw[i] && reqs[i].wait_arrival && reqs[i].band < (int)arrival_us->size()) ? (*arrival_us)[reqs[i].band] : 0.0;
        };
        // Candidate 1, greedy list scheduling: repeatedly append, among the stages whose producers are all placed,
        // the one that is ready first, and let the model run it.  While the machine waits for input this follows
        // each band down its layers (the pipeline of Sec. IV-B); once the machine is saturated, finish times slip,
        // stages of other bands become ready first and the order turns layer-major by itself.
        double span_greedy = 0.0;
        {
            Machine mc(n_cta);
            std::vector<double> ready(n, 0.0);
            std::vector<int> pending(n), heap;
            auto later = [&](int x, int y) {
                if (ready[x] != ready[y]) return ready[x] > ready[y];
                if (reqs[x].prio != reqs[y].prio) return reqs[x].prio > reqs[y].prio;
                return x > y;
            };
            for (size_t i = 0; i < n; ++i) {
                pending[i] = (int)prods[i].size();
                if (!pending[i]) { ready[i] = arrival_of((int)i); heap.push_back((int)i); }
            }
            std::make_heap(heap.begin(), heap.end(), later);
            while (!heap.empty()) {
                std::pop_heap(heap.begin(), heap.end(), later);
                const int i = heap.back();
                heap.pop_back();
                order.push_back(i);
                const double fin = mc.run(shape[i], reqs[i].fetch, ready[i]);
                for (int u : users[i]) {
                    ready[u] = std::max(ready[u], fin + hop_us);
                    if (--pending[u] == 0) {
                        ready[u] = std::max(ready[u], arrival_of(u));
                        heap.push_back(u);
                        std::push_heap(heap.begin(), heap.end(), later);
                    }
                }
            }
            if (order.size() != n) { set_error("the stage requests depend on each other in a cycle"); return LOP_EINVAL; }
            span_greedy = mc.makespan;
        }
        // Candidate 2, layer-major (operation batching, Sec. IV-C): all bands' stages of one depth together, the
        // way resident programs run; the input's transfer is then hidden only behind the first layers.  Deep
        // chains of many thin bands do better this way: their late stages have too few tiles to fill the machine
        // band by band.  The model decides.
        {
            std::vector<int> depth(n, 0);
            for (int i : order)
                for (int j : prods[i]) depth[i] = std::max(depth[i], depth[j] + 1);
            std::vector<long long> keep(n);
            for (size_t i = 0; i < n; ++i) { keep[i] = reqs[i].prio; reqs[i].prio = (long long)depth[i] * 65536 + reqs[i].band; }
            std::vector<int> batched;
            kahn(batched);
            for (size_t i = 0; i < n; ++i) reqs[i].prio = keep[i];
            Machine mc(n_cta);
            std::vector<double> fin(n, 0.0);
            for (int i : batched) {
                double ready = arrival_of(i);
                for (int j : prods[i]) ready = std::max(ready, fin[j] + hop_us);
                fin[i] = mc.run(shape[i], reqs[i].fetch, ready);
            }
#ifdef LOP_WF_TRACE
            fprintf(stderr, "order model: greedy %.1f us, layer-major %.1f us (%zu stages)\n", span_greedy, mc.makespan, n);
#endif
            // The model is too coarse to separate the two when they come out close, and measurements did: where the
            // input's transfer is a small part of the run (under a fifth), the layer-major order wins by running the
            // bulk of the work the way resident programs do (a ResNet-50 of batch 8: 836 vs 862 us); where the transfer is a large
            // part, following the arrivals wins (one 224x224 image through a VGG block: 38 vs 51 us).
            double transfer = 0.0;
            for (size_t i = 0; i < n; ++i)
                if (reqs[i].fetch) transfer += shape[i].item_us;
            if (arrival_us && !arrival_us->empty()) transfer = std::max(transfer, arrival_us->back());
            const bool compute_bound = transfer < 0.2 * mc.makespan;
            // (a resident program, nothing arriving: the greedy order unless the model clearly prefers layer-major --
            // it moves late layers of early bands in front of early layers of late bands where that shortens waits)
            const bool resident = transfer == 0.0;
            if (batched.size() == n && (resident ? mc.makespan < 0.98 * span_greedy
                                                 : (mc.makespan < 0.95 * span_greedy || (compute_bound && mc.makespan < 1.05 * span_greedy))))
                order.swap(batched);
        }
    }
    std::vector<StageReq> out;
    out.reserve(n);
    for (int i : order) out.push_back(reqs[i]);
    reqs.swap(out);
    return LOP_OK;
}

}  // namespace

int program_build(const std::vector<SegBind> &segs, std::vector<StageReq> reqs, Program **result, const std::vector<double> *arrival_us,
                  const void *fetch_src)
{
    *result = nullptr;
    if (segs.empty()) { set_error("program_build: no plan"); return LOP_EINVAL; }
    const bool reuse = (segs[0].pl->flags & LOP_FLAG_REUSE_HALO) != 0;
    Ctx cx{segs, {}};
    int n_tensors = 0;
    for (const SegBind &sb : segs) { cx.base.push_back(n_tensors); n_tensors += (int)sb.pl->layers.size() + 1; }
    for (const StageReq &rq : reqs)
        if (rq.fetch && rq.hi > rq.lo) cx.raw = n_tensors;
    if (cx.raw >= 0) {
        ++n_tensors;
        if (!fetch_src) { set_error("program_build: fetch requests without a source"); return LOP_EINVAL; }
        if ((reinterpret_cast<uintptr_t>(fetch_src) & 15) != (reinterpret_cast<uintptr_t>(segs[0].in) & 15) ||
            (reinterpret_cast<uintptr_t>(fetch_src) & 1)) {
            set_error("host input and staging tensor must agree in their address modulo 16");
            return LOP_EUNSUPPORTED;
        }
    }
    {
        std::vector<StageReq> live;
        for (const StageReq &rq : reqs)
            if (rq.hi > rq.lo) live.push_back(rq);
        reqs.swap(live);
    }
    int orc = order_requests(cx, reqs, reuse, arrival_us);
    if (orc != LOP_OK) return orc;

    std::vector<WfStage> stages;
    std::vector<int> stage_band, stage_rows_per_group;
    std::vector<int4> items, fetch_items;
    std::vector<CUtensorMap> maps;
    std::vector<MapSet> mapsets;
    std::vector<int2> deps;
    std::vector<std::vector<int>> by_tensor(n_tensors);   // stage indices per produced tensor
    std::vector<int> expected;                         // completions per row group, per stage
    int n_ctr = WF_CTR_FIRST;
    bool uses_flags = false;
    uint32_t a_slot = 1024, b_slot = 1024, stg_bytes = 1024;

    std::vector<char> consumed(reqs.size(), 0);            // pooling requests folded into their convolution's stage
    std::vector<int> prod_lo, prod_hi;                     // per stage: rows of the tensor it produces
    for (size_t ri = 0; ri < reqs.size(); ++ri) {
        const StageReq &rq = reqs[ri];
        if (consumed[ri]) continue;
        if (stages.size() >= 65535) { set_error("program has too many stages"); return LOP_EUNSUPPORTED; }
        lop_plan_t *pl = segs[rq.seg].pl;
        const void *in = segs[rq.seg].in;
        void *out = segs[rq.seg].out, *ws = segs[rq.seg].ws;
        char *wsb = static_cast<char *>(ws);
        const LayerInfo &li = pl->layers[rq.layer];
        const lop_layer &l = li.l;
        WfStage st{};
        st.oh_lo = rq.lo; st.oh_hi = rq.hi;
        const int rows = rq.hi - rq.lo;
        int group_rows = 1, tiles_r = rows, tiles_w = 1, tiles_n = pl->N, cout_tiles = 1;
        int produces = rq.fetch ? cx.raw : (rq.gather ? cx.patches_id(rq.seg) : cx.tensor_id(rq.seg, rq.layer));
        int out_lo = rq.lo, out_hi = rq.hi;                    // rows of the produced tensor
        if (rq.fetch) {
            // a stage only in the book-keeping sense (row-group counters its readers wait for): its work goes to the
            // fetch list.  Entries of about 3 KB, whole rows: a warp has that much in flight at a time.
            const long long row_b = (long long)pl->W * pl->C * 2;
            st.kind = WF_FETCH;
            st.x = fetch_src; st.y = const_cast<void *>(in);
            st.N = pl->N; st.Hin = pl->H; st.Win = pl->W; st.Cin = pl->C;
            group_rows = (int)std::max(1LL, std::min<long long>(rows, LOP_FETCH_ENTRY_BYTES / row_b));
            tiles_r = (rows + group_rows - 1) / group_rows;
            if (row_b * group_rows > 0x7fffffffLL) { set_error("input rows too long to fetch"); return LOP_EUNSUPPORTED; }
        } else if (rq.gather) {
            st.kind = WF_GATHER;
            st.x = in; st.y = wsb + pl->col_off;
            st.N = pl->N; st.Hin = pl->H; st.Win = pl->W; st.Cin = pl->C; st.Ho = li.Ho; st.Wo = li.Wo; st.Cout = li.cin_eff;
            st.kh = l.kh; st.kw = l.kw; st.sh = l.sh; st.sw = l.sw; st.ph = l.ph; st.pw = l.pw; st.dh = l.dh; st.dw = l.dw;
            // the kh image rows an output row reads are staged in shared memory when they fit (mode 0), else read in place
            const uint32_t pitch = ((uint32_t)pl->W * pl->C * 2u + 31u + 15u) & ~15u;
            const uint32_t need = round_up_u32((uint32_t)l.kh * pitch + 4u * (uint32_t)li.cin_eff, 1024u);
            if (need <= 48u * 1024u && l.kh <= 64) stg_bytes = std::max(stg_bytes, need);
            else st.mode = 1;
        } else if (l.op == LOP_MAXPOOL2D) {
            const PoolArgs a = pool_args(pl, rq.layer, in, out, ws, rq.lo, rq.hi);
            st.kind = WF_POOL;
            st.x = a.x; st.y = a.y;
            st.N = a.N; st.Hin = a.Hin; st.Win = a.Win; st.Cin = a.C; st.Ho = a.Ho; st.Wo = a.Wo; st.Cout = a.C;
            st.kh = a.kh; st.kw = a.kw; st.sh = a.sh; st.sw = a.sw; st.ph = a.ph; st.pw = a.pw; st.dh = a.dh; st.dw = a.dw;
        } else if (l.op == LOP_DWCONV2D || l.op == LOP_LAYERNORM || l.op == LOP_CONCAT) {
            const ConvArgs a = conv_args(pl, rq.layer, in, out, ws, rq.lo, rq.hi);
            st.kind = l.op == LOP_DWCONV2D ? WF_DWCONV : (l.op == LOP_LAYERNORM ? WF_LAYERNORM : WF_CONCAT);
            st.x = a.x; st.res = a.res; st.scale = a.scale; st.shift = a.shift; st.y = a.y;
            st.N = a.N; st.Hin = a.Hin; st.Win = a.Win; st.Cin = a.Cin; st.Ho = a.Ho; st.Wo = a.Wo; st.Cout = a.Cout;
            st.kh = a.kh; st.kw = a.kw; st.sh = a.sh; st.sw = a.sw; st.ph = a.ph; st.pw = a.pw; st.dh = a.dh; st.dw = a.dw;
            st.act = a.act; st.res_pos = a.res_pos;
            if (l.op == LOP_DWCONV2D) {
                rowop::DwTile t{1, 1, 8};
                if (!dw_tile(pl, li, &t)) { set_error("layer %d: depth-wise window does not fit the staging tile", rq.layer); return LOP_EUNSUPPORTED; }
                st.BN = t.cc; st.tw_valid = t.tw; st.tr_log = ilog2i(t.R);
                st.w_taps = wsb + li.wpad_off;
                group_rows = t.R;
                tiles_r = (rows + t.R - 1) / t.R;
                tiles_w = (li.Wo + t.tw - 1) / t.tw;
                cout_tiles = l.cin / t.cc;
                stg_bytes = std::max(stg_bytes, round_up_u32((uint32_t)rowop::dw_tile_bytes(l.kh, l.kw, l.sh, l.sw, l.dh, l.dw, t), 1024u));
            }
        } else {
            const ConvArgs a = conv_args(pl, rq.layer, in, out, ws, rq.lo, rq.hi);
            // a 2x2 pooling that is this convolution's only reader, asked for exactly the rows this stage feeds it
            size_t rj = reqs.size();
            if (pool_fusable(pl, rq.layer))
                for (size_t k = 0; k < reqs.size(); ++k)
                    if (!consumed[k] && !reqs[k].gather && reqs[k].seg == rq.seg && reqs[k].band == rq.band &&
                        reqs[k].layer == rq.layer + 1 && rq.lo == 2 * reqs[k].lo && rq.hi == 2 * reqs[k].hi) { rj = k; break; }
            const bool fuse = rj < reqs.size();
            const Geom g = choose_geom(a, rows, fuse);
            st.kind = WF_CONV;
            st.mode = g.mode;
            st.x = a.x; st.res = a.res; st.scale = a.scale; st.shift = a.shift; st.y = a.y;
            st.N = a.N; st.Hin = a.Hin; st.Win = a.Win; st.Cin = a.Cin; st.Ho = a.Ho; st.Wo = a.Wo; st.Cout = a.Cout;
            st.kh = a.kh; st.kw = a.kw; st.sh = a.sh; st.sw = a.sw; st.ph = a.ph; st.pw = a.pw; st.dh = a.dh; st.dw = a.dw;
            st.act = a.act; st.res_pos = a.res_pos;
            int base = -1;
            for (const MapSet &m : mapsets)
                if (m.seg == rq.seg && m.layer == rq.layer && m.P == g.P && m.RI == g.RI && m.TN == g.TN && m.BN == g.BN && m.BK == g.BK &&
                    m.tb == g.tb)
                    base = m.base;
            CUtensorMap cm[5];
            int mask = 0;
            const int rc = encode_maps(a, g, cm, &mask);            // also tells which parity classes exist
            if (rc != LOP_OK) { set_error("layer %d: tensor-map encoding failed", rq.layer); return rc; }
            if (base < 0) {
                base = (int)maps.size();
                for (int i = 0; i < 5; ++i) maps.push_back(cm[i]);
                mapsets.push_back(MapSet{rq.seg, rq.layer, g.P, g.RI, g.TN, g.BN, g.BK, g.tb, base});
            }
            st.map_base = base;
            st.a_valid_mask = mask;
            st.p_log = ilog2i(g.P); st.tr_log = ilog2i(g.TR); st.tw_valid = g.tw_valid;
            st.BN = g.BN; st.BK = g.BK; st.n_chunks = g.n_chunks; st.n_taps = g.n_taps; st.tb = g.tb;
            st.a_bytes = g.a_bytes; st.b_bytes = g.b_bytes;
            st.row_bytes = (uint32_t)g.BK * 2u;
            st.layout_code = g.BK == 64 ? 2u : (g.BK == 32 ? 4u : 6u);
            st.sbo_bytes = 8u * st.row_bytes;
            // instruction descriptor: fp32 accumulate, bf16 x bf16, both operands K-major, N = BN, M = 128
            st.idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(g.BN >> 3) << 17) | ((128u >> 4) << 24);
            a_slot = std::max(a_slot, g.a_slot);
            b_slot = std::max(b_slot, g.b_slot);
            stg_bytes = std::max(stg_bytes, round_up_u32(128u * (uint32_t)g.BN * 2u, 1024u));
            if (fuse) {
                const LayerInfo &pool = pl->layers[rq.layer + 1];
                consumed[rj] = 1;
                st.fuse_pool = 1; st.pool_Ho = pool.Ho; st.pool_Wo = pool.Wo;
                st.y = const_cast<void *>(tensor_of(pl, rq.layer + 1, in, out, ws));
                produces = cx.tensor_id(rq.seg, rq.layer + 1);
                out_lo = reqs[rj].lo; out_hi = reqs[rj].hi;
            }
            group_rows = g.TR;
            tiles_r = (rows + g.TR - 1) / g.TR;
            tiles_w = (a.Wo + g.tw_valid - 1) / g.tw_valid;
            tiles_n = (a.N + g.TN - 1) / g.TN;
            cout_tiles = a.Cout / g.BN;
        }
        if (tiles_w > 65535 || tiles_n > 65535 || cout_tiles > 65535 || tiles_r >= (1 << 20)) {
            set_error("layer %d: too many tiles for one stage", rq.layer);
            return LOP_EUNSUPPORTED;
        }
        st.ctr_base = n_ctr;
        n_ctr += tiles_r;
        const int exp_here = tiles_w * tiles_n * cout_tiles;
        const int sidx = (int)stages.size();

        // ---- dependencies of every row group of this stage on earlier stages of this program
        for (int tr = 0; tr < tiles_r; ++tr) {
            const int o0 = rq.lo + tr * group_rows, o1 = std::min(o0 + group_rows, rq.hi);
            const Reads rd = reads_of(cx, rq, o0, o1);
            const int first = (int)deps.size();
            if (rq.wait_arrival && rd.raw) {
                // every band whose transfer brings rows these output rows read (a request may span several bands where
                // thin bands were joined); no assumption is made about the order in which arrivals become visible
                long long a = (long long)o0 * l.sh - l.ph, b = (long long)(o1 - 1) * l.sh - l.ph + (long long)(l.kh - 1) * l.dh + 1;
                const bool main_raw = rq.gather || (l.input_from == LOP_INPUT && !li.stem_gather);
                if (!main_raw) { a = o0; b = o1; }                          // only the residual reads the chain input: its own rows
                else if (!rq.gather && has_second_input(l) && l.residual_from == LOP_INPUT) { a = std::min<long long>(a, o0); b = std::max<long long>(b, o1); }
                a = std::max(a, 0LL); b = std::min<long long>(b, pl->H);
                int last_leader = -1;
                for (int b2 = 0; b2 < pl->n_bands; ++b2) {
                    const lop_range &o = pl->in_need[b2];
                    if (o.out_hi <= o.new_lo || o.out_hi <= a || o.new_lo >= b) continue;
                    // the bands of one copy arrive together: the flag of the copy's last band stands for all of them
                    const int leader = std::min(pl->n_bands - 1, (b2 / pl->copy_group) * pl->copy_group + pl->copy_group - 1);
                    if (leader == last_leader) continue;
                    last_leader = leader;
                    deps.push_back(make_int2(-1 - leader, -1));         // patched below
                }
                uses_flags = true;
            }
            for (int q = 0; q < rd.n; ++q)
                for (int ps : by_tensor[rd.need[q].tensor]) {
                    if (!reuse && rd.need[q].same_seg && stage_band[ps] != rq.band) continue;
                    const WfStage &p = stages[ps];
                    const int lo = std::max(rd.need[q].lo, prod_lo[ps]), hi = std::min(rd.need[q].hi, prod_hi[ps]);
                    if (lo >= hi) continue;
                    const int gr = stage_rows_per_group[ps];
                    for (int g = (lo - prod_lo[ps]) / gr; g <= (hi - 1 - prod_lo[ps]) / gr; ++g)
                        deps.push_back(make_int2(p.ctr_base + g, expected[ps]));
                }
            const int count = (int)deps.size() - first;
            if (count > WF_MAX_DEPS) { set_error("layer %d: a tile depends on too many row groups", rq.layer); return LOP_EUNSUPPORTED; }
            if (rq.fetch) {
                const long long row_b = (long long)pl->W * pl->C * 2;
                for (int n = 0; n < pl->N; ++n) {
                    const unsigned long long off = (unsigned long long)(((long long)n * pl->H + o0) * row_b);
                    fetch_items.push_back(make_int4((int)(unsigned)(off & 0xffffffffu), (int)(unsigned)(off >> 32), (int)((o1 - o0) * row_b),
                                                    st.ctr_base + tr));
                }
                continue;
            }
            for (int tn = 0; tn < tiles_n; ++tn)
                for (int tw = 0; tw < tiles_w; ++tw)
                    for (int ct = 0; ct < cout_tiles; ++ct)
                        items.push_back(make_int4(sidx | (ct << 16), tw | (tn << 16), tr | (count << 20), first));
        }
        by_tensor[produces].push_back(sidx);
        stages.push_back(st);
        stage_band.push_back(rq.band);
        stage_rows_per_group.push_back(st.fuse_pool ? group_rows / 2 : group_rows);    // in rows of the produced tensor
        prod_lo.push_back(out_lo);
        prod_hi.push_back(out_hi);
        expected.push_back(exp_here);
    }

    lop_plan_t *pl0 = segs[0].pl;
    Program *p = new (std::nothrow) Program();
    if (!p) { set_error("out of host memory"); return LOP_ENOMEM; }
    if (uses_flags) {                                        // arrival flags live after the row-group counters
        p->flag_base = n_ctr;
        p->n_flags = pl0->n_bands;
        for (int2 &d : deps)
            if (d.x < 0) d.x = p->flag_base + (-1 - d.x);
        n_ctr += p->n_flags;
    }
    const int n_items = (int)items.size();
    if (n_items == 0 && fetch_items.empty()) { *result = p; return LOP_OK; }          // nothing to do: an empty program

    // ---- shared-memory rings: as many slots as fit beside the staging tile, weights first
    const size_t fixed = 1024 + stg_bytes + 8 * (2 * 8 + 2 * 8 + 4 + 2 * WF_PUBQ + 4) + 64 + 2048 + 1280 + 64;
    const size_t budget = 227 * 1024 - fixed;
    int sa = 2, sb = 2;
    if ((size_t)sa * a_slot + (size_t)sb * b_slot > budget) { delete p; set_error("tile buffers do not fit shared memory"); return LOP_EUNSUPPORTED; }
    for (bool grew = true; grew;) {
        grew = false;
        if (sb < LOP_SB_MAX && (size_t)sa * a_slot + (size_t)(sb + 1) * b_slot <= budget) { ++sb; grew = true; }
        if (sa < LOP_SA_MAX && (size_t)(sa + 1) * a_slot + (size_t)sb * b_slot <= budget) { ++sa; grew = true; }
    }

    // chunks per ring slot of the long pointwise stages (see WfStage::cps), now that the slot sizes are known
    for (WfStage &st : stages) {
        st.cps = 1;
        if (st.kind != WF_CONV) continue;
        const bool long_pointwise = st.mode == WF_SLAB && st.n_taps == 1 && st.BK == 64 && st.n_chunks > sb;
        if (!long_pointwise && st.mode != WF_TAP) continue;            // per-tap windows: cps consecutive taps per slot
        st.cps = std::max(1, std::min({(int)(a_slot / st.a_bytes), (int)(b_slot / st.b_bytes), LOP_CPS_MAX}));
    }

#ifdef LOP_WF_TRACE
    fprintf(stderr, "program: %zu stages, %d items, rings: %d x %u B activations, %d x %u B weights, staging %u B\n", stages.size(), n_items, sa, a_slot, sb, b_slot, stg_bytes);
#endif
    // ---- one device allocation for all tables
    auto al = [](size_t v) { return (v + 255) / 256 * 256; };
    const size_t o_stages = 0;
    const size_t o_items = o_stages + al(stages.size() * sizeof(WfStage));
    const size_t o_maps = o_items + al(items.size() * sizeof(int4));
    const size_t o_deps = o_maps + al(std::max<size_t>(maps.size(), 1) * sizeof(CUtensorMap));
    const size_t o_fetch = o_deps + al(std::max<size_t>(deps.size(), 1) * sizeof(int2));
    const size_t o_ctr = o_fetch + al(fetch_items.size() * sizeof(int4));
    const size_t total = o_ctr + al((size_t)n_ctr * sizeof(unsigned));
    cudaError_t e = cudaMalloc(&p->dev, total);
    if (e != cudaSuccess) { delete p; set_error("cudaMalloc(%zu) failed: %s", total, cudaGetErrorString(e)); return LOP_ECUDA; }
    char *d = static_cast<char *>(p->dev);
    auto up = [&](size_t off, const void *src, size_t bytes) {
        return bytes ? cudaMemcpy(d + off, src, bytes, cudaMemcpyHostToDevice) : cudaSuccess;
    };
    if ((e = cudaMemset(d, 0, total)) != cudaSuccess || (e = up(o_stages, stages.data(), stages.size() * sizeof(WfStage))) != cudaSuccess ||
        (e = up(o_items, items.data(), items.size() * sizeof(int4))) != cudaSuccess ||
        (e = up(o_maps, maps.data(), maps.size() * sizeof(CUtensorMap))) != cudaSuccess ||
        (e = up(o_deps, deps.data(), deps.size() * sizeof(int2))) != cudaSuccess ||
        (e = up(o_fetch, fetch_items.data(), fetch_items.size() * sizeof(int4))) != cudaSuccess) {
        program_destroy(p);
        set_error("program upload failed: %s", cudaGetErrorString(e));
        return LOP_ECUDA;
    }
    p->counters = reinterpret_cast<unsigned *>(d + o_ctr);
    WfParams &P = p->params;
    P.stages = reinterpret_cast<const WfStage *>(d + o_stages);
    P.items = reinterpret_cast<const int4 *>(d + o_items);
    P.maps = reinterpret_cast<const CUtensorMap *>(d + o_maps);
    P.deps = reinterpret_cast<const int2 *>(d + o_deps);
    P.counters = p->counters;
    P.status = reinterpret_cast<unsigned *>(static_cast<char *>(segs[0].ws) + pl0->status_off);
    P.flag_base = p->flag_base; P.n_flags = p->n_flags;
    P.n_stages = (int)stages.size();
    P.n_items = n_items;
    P.sa = sa; P.sb = sb;
    P.a_slot_bytes = a_slot; P.b_slot_bytes = b_slot; P.stg_bytes = stg_bytes;
    P.fetch_items = reinterpret_cast<const int4 *>(d + o_fetch);
    P.fetch_src = fetch_src;
    P.fetch_dst = const_cast<void *>(segs[0].in);
    P.n_fetch = (int)fetch_items.size();
    P.row_ops = 0;
    for (const WfStage &st : stages)
        if (st.kind == WF_DWCONV || st.kind == WF_LAYERNORM || st.kind == WF_CONCAT) P.row_ops = 1;
    // entries in flight: about the link's bandwidth-delay product (some 25 GB/s x 3 us), at least a few warps' worth
    if (P.n_fetch > 0) {
        long long bytes = 0;
        for (const int4 &f : fetch_items) bytes += f.z;
        // (a small input keeps the short window, which keeps its few bands in order; an input of megabytes is bound by
        // the link's rate, which needs more bytes on their way: measured 597 -> 577 us on a 2.4 MB batch)
        const long long window_bytes = std::min<long long>(LOP_FETCH_WINDOW_MAX_BYTES, std::max<long long>(LOP_FETCH_WINDOW_BYTES, bytes / 8));
        P.fetch_window = (int)std::max(8LL, window_bytes * P.n_fetch / std::max(1LL, bytes));
    }
    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    p->owner = pl0;
    p->grid = n_items > 0 ? std::min(n_items, sms) : std::min((int)fetch_items.size(), sms);   // (a fetch-only program: its fetch warps)
    // every CTA of a launch must be resident (see the kernel's deadlock-freedom argument); what the device can hold
    // with this kernel's shared memory and registers says whether that is possible at all -- whether the SMs are free
    // at launch time is the caller's business: the stream must have the GPU to itself while the kernel runs
    int resident = 0;
    e = wavefront_resident_ctas(P, &resident);
    if (e != cudaSuccess) { program_destroy(p); set_error("occupancy query failed: %s", cudaGetErrorString(e)); return LOP_ECUDA; }
    if (resident < p->grid) {
        program_destroy(p);
        set_error("the device holds %d CTAs of the persistent kernel at a time, the program needs %d", resident, p->grid);
        return LOP_EUNSUPPORTED;
    }
    *result = p;
    return LOP_OK;
}

int program_launch(Program *p, cudaStream_t s)
{
    if (!p || p->grid == 0) return LOP_OK;
    p->params.spin_limit = (p->owner && p->owner->wait_limit) ? p->owner->wait_limit : WF_SPIN_LIMIT_DEFAULT;
    cudaError_t e = launch_wavefront(p->params, p->grid, s);
    if (e != cudaSuccess) { set_error("wavefront launch failed: %s", cudaGetErrorString(e)); return LOP_ECUDA; }
    return LOP_OK;
}

bool program_empty(const Program *p) { return !p || p->grid == 0; }

unsigned *program_arrival_flag(Program *p, int band)
{
    if (!p || !p->counters || band < 0 || band >= p->n_flags) return nullptr;
    return p->counters + p->flag_base + band;
}

}  // namespace lop

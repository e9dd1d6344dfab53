// Host side of the wavefront kernel: turns a list of (band, layer, row range) requests into a
// device-resident program (stages, bound layers, tensor maps, dependency lists, counters).
//
// Dependencies follow Sec. IV-B of the paper: a tile depends on a producer row group as soon as
// any row of that group lies inside the tile's receptive rows (for the residual: its own rows).
#include <cuda_runtime.h>

#include <algorithm>
#include <vector>

#include "lop_internal.h"
#include "lop_kernels.cuh"
#include "lop_program.h"
#include "lop_wavefront.cuh"

namespace lop {

struct Program {
    void *dev = nullptr;            // one allocation holding every table
    unsigned *counters = nullptr;
    WfParams params{};
    int grid = 0;
    int flag_base = 0, n_flags = 0;
};

void program_destroy(Program *p)
{
    if (!p) return;
    if (p->dev) cudaFree(p->dev);
    delete p;
}

namespace {

#define PROG_CUDA(call)                                                                 \
    do {                                                                                \
        cudaError_t e__ = (call);                                                       \
        if (e__ != cudaSuccess) {                                                       \
            set_error("%s failed: %s", #call, cudaGetErrorString(e__));                 \
            return LOP_ECUDA;                                                           \
        }                                                                               \
    } while (0)

struct MapSet { int layer, TW, TR, TN, BN, BK, base; };

const void *tensor_ptr(const lop_plan_t *pl, int idx, const void *in, void *out, void *ws)
{
    if (idx == LOP_INPUT) return in;
    if (idx == (int)pl->layers.size() - 1) return out;
    return static_cast<char *>(ws) + pl->layers[idx].out_off;
}

int ilog2i(int v) { int l = 0; while ((1 << l) < v) ++l; return l; }

}  // namespace

bool program_supported(const lop_plan_t *pl)
{
    if (pl->dtype != LOP_BF16) return false;
    for (const auto &li : pl->layers) {
        if (li.l.op == LOP_CONV2D && li.kernel != K_CONV_TC) return false;
        if (li.l.op == LOP_MAXPOOL2D && li.l.cin % 8 != 0) return false;
    }
    return true;
}

int program_build(lop_plan_t *pl, const std::vector<StageReq> &reqs, const void *in, void *out, void *ws, Program **result)
{
    *result = nullptr;
    const int L = (int)pl->layers.size();
    const bool reuse = (pl->flags & LOP_FLAG_REUSE_HALO) != 0;
    char *wsb = static_cast<char *>(ws);

    // ---- bound layers; index L is the channel-padding pseudo-layer
    std::vector<WfLayer> layers(L + 1);
    for (int i = 0; i < L; ++i) {
        const LayerInfo &li = pl->layers[i];
        const lop_layer &l = li.l;
        WfLayer w{};
        w.x = (li.kernel == K_CONV_TC && li.reads_padded_input) ? wsb + pl->padin_off : tensor_ptr(pl, l.input_from, in, out, ws);
        w.res = (l.op == LOP_CONV2D && l.residual_from != LOP_NO_RESIDUAL) ? tensor_ptr(pl, l.residual_from, in, out, ws) : nullptr;
        w.scale = l.scale; w.shift = l.shift;
        w.y = const_cast<void *>(tensor_ptr(pl, i, in, out, ws));
        w.N = pl->N; w.Hin = li.Hin; w.Win = li.Win; w.Cin = l.op == LOP_CONV2D ? li.cin_eff : l.cin;
        w.Ho = li.Ho; w.Wo = li.Wo; w.Cout = l.cout;
        w.kh = l.kh; w.kw = l.kw; w.sh = l.sh; w.sw = l.sw; w.ph = l.ph; w.pw = l.pw; w.dh = l.dh; w.dw = l.dw;
        w.act = l.act; w.res_pos = w.res ? l.residual_pos : LOP_RES_NONE;
        layers[i] = w;
    }
    {
        WfLayer w{};
        w.x = in; w.y = wsb + pl->padin_off;
        w.N = pl->N; w.Hin = pl->H; w.Win = pl->W; w.Cin = pl->C; w.Ho = pl->H; w.Wo = pl->W; w.Cout = pl->Cpad;
        w.kh = w.kw = w.sh = w.sw = w.dh = w.dw = 1;
        layers[L] = w;
    }

    std::vector<WfStage> stages;
    std::vector<int> stage_band;
    std::vector<CUtensorMap> maps;
    std::vector<MapSet> mapsets;
    std::vector<int2> dep_index, deps;
    std::vector<std::vector<int>> by_layer(L + 1);      // stage indices per producing layer
    std::vector<int> expected;                         // completions per row group, per stage
    int n_items = 0, n_ctr = WF_CTR_FIRST;
    bool uses_flags = false;
    uint32_t slot_bytes = 1024;

    for (const StageReq &rq : reqs) {
        if (rq.hi <= rq.lo) continue;
        WfStage st{};
        const int lidx = rq.layer < 0 ? L : rq.layer;
        st.layer = lidx;
        st.oh_lo = rq.lo; st.oh_hi = rq.hi;
        st.first_item = n_items;
        const int rows = rq.hi - rq.lo;
        if (rq.layer >= 0 && pl->layers[rq.layer].l.op == LOP_CONV2D) {
            const LayerInfo &li = pl->layers[rq.layer];
            const lop_layer &l = li.l;
            st.kind = WF_CONV;
            ConvArgs a{};
            a.x = layers[lidx].x;
            a.w = li.reads_padded_input ? (const void *)(wsb + li.wpad_off) : l.weight;
            a.N = pl->N; a.Hin = li.Hin; a.Win = li.Win; a.Cin = li.cin_eff; a.Ho = li.Ho; a.Wo = li.Wo; a.Cout = l.cout;
            a.kh = l.kh; a.kw = l.kw; a.sh = l.sh; a.sw = l.sw; a.ph = l.ph; a.pw = l.pw; a.dh = l.dh; a.dw = l.dw;
            a.oh_lo = rq.lo; a.oh_hi = rq.hi;
            const ConvTcGeom g = conv_tc_geometry(a, rows, /*fill_sms=*/false);
            int base = -1;
            for (const MapSet &m : mapsets)
                if (m.layer == rq.layer && m.TW == g.TW && m.TR == g.TR && m.TN == g.TN && m.BN == g.BN && m.BK == g.BK) base = m.base;
            ConvTcMaps cm;
            const int rc = conv_tc_encode(a, g, &cm);               // also tells which parity classes exist
            if (rc != LOP_OK) { set_error("layer %d: tensor-map encoding failed", rq.layer); return rc; }
            if (base < 0) {
                base = (int)maps.size();
                for (int i = 0; i < 4; ++i) maps.push_back(cm.a[i]);
                maps.push_back(cm.w);
                mapsets.push_back(MapSet{rq.layer, g.TW, g.TR, g.TN, g.BN, g.BK, base});
            }
            st.map_base = base;
            st.a_valid_mask = cm.a_valid[0] | (cm.a_valid[1] << 1) | (cm.a_valid[2] << 2) | (cm.a_valid[3] << 3);
            st.tw_log = ilog2i(g.TW); st.tr_log = ilog2i(g.TR);
            st.tiles_w = (li.Wo + g.TW - 1) / g.TW;
            st.tiles_r = (rows + g.TR - 1) / g.TR;
            st.tiles_n = (pl->N + g.TN - 1) / g.TN;
            st.cout_tiles = l.cout / g.BN;
            st.BN = g.BN; st.BK = g.BK;
            st.k_iters = l.kh * l.kw * (li.cin_eff / g.BK);
            st.a_bytes = 128u * g.BK * 2u;
            st.b_bytes = (uint32_t)(g.BN * g.BK * 2);
            st.layout_code = g.BK == 64 ? 2u : (g.BK == 32 ? 4u : 6u);
            st.sbo_bytes = 8u * g.BK * 2u;
            st.idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(g.BN >> 3) << 17) | ((128u >> 4) << 24);
            slot_bytes = std::max(slot_bytes, st.a_bytes + (st.b_bytes + 1023u) / 1024u * 1024u);
        } else {
            // one output row of one image, cut into chunks of 128 pixels (padding) / 256 channel vectors (pooling)
            st.kind = rq.layer < 0 ? WF_PAD : WF_POOL;
            st.tw_log = 0; st.tr_log = 0;
            const int per_row = rq.layer < 0 ? pl->W : pl->layers[rq.layer].Wo * (pl->layers[rq.layer].l.cin / 8);
            const int per_item = rq.layer < 0 ? 128 : 256;
            st.tiles_w = (per_row + per_item - 1) / per_item;
            st.tiles_r = rows; st.tiles_n = pl->N; st.cout_tiles = 1;
        }
        st.n_items = st.tiles_w * st.tiles_r * st.tiles_n * st.cout_tiles;
        st.ctr_base = n_ctr;
        n_ctr += st.tiles_r;
        st.dep_base = (int)dep_index.size();
        const int exp_here = st.tiles_w * st.tiles_n * st.cout_tiles;

        // ---- dependencies of every row group of this stage on earlier stages of this program
        struct Need { int layer, lo, hi; };
        for (int tr = 0; tr < st.tiles_r; ++tr) {
            const int TR = 1 << st.tr_log;
            const int o0 = rq.lo + tr * TR, o1 = std::min(o0 + TR, rq.hi);
            Need needs[2];
            int nn = 0;
            if (rq.layer >= 0) {
                const LayerInfo &li = pl->layers[rq.layer];
                const lop_layer &l = li.l;
                int prod = l.input_from;
                if (prod == LOP_INPUT) prod = (li.kernel == K_CONV_TC && li.reads_padded_input) ? L : -1;
                if (prod >= 0) {
                    long long a = (long long)o0 * l.sh - l.ph, b = (long long)(o1 - 1) * l.sh - l.ph + (long long)(l.kh - 1) * l.dh;
                    a = std::max(a, 0LL); b = std::min(b, (long long)li.Hin - 1);
                    if (a <= b) needs[nn++] = Need{prod, (int)a, (int)b + 1};
                }
                if (l.op == LOP_CONV2D && l.residual_from >= 0) needs[nn++] = Need{l.residual_from, o0, o1};
            }
            const int first = (int)deps.size();
            if (rq.wait_arrival) {
                bool raw = rq.layer < 0;
                if (rq.layer >= 0) {
                    const LayerInfo &li = pl->layers[rq.layer];
                    raw = (li.l.input_from == LOP_INPUT && !(li.kernel == K_CONV_TC && li.reads_padded_input)) ||
                          (li.l.op == LOP_CONV2D && li.l.residual_from == LOP_INPUT);
                }
                if (raw) { deps.push_back(make_int2(-1 - rq.band, -1)); uses_flags = true; }   // patched below
            }
            for (int q = 0; q < nn; ++q)
                for (int ps : by_layer[needs[q].layer]) {
                    if (!reuse && stage_band[ps] != rq.band) continue;
                    const WfStage &p = stages[ps];
                    const int lo = std::max(needs[q].lo, p.oh_lo), hi = std::min(needs[q].hi, p.oh_hi);
                    if (lo >= hi) continue;
                    for (int g = (lo - p.oh_lo) >> p.tr_log; g <= (hi - 1 - p.oh_lo) >> p.tr_log; ++g)
                        deps.push_back(make_int2(p.ctr_base + g, expected[ps]));
                }
            dep_index.push_back(make_int2(first, (int)deps.size() - first));
        }
        by_layer[lidx].push_back((int)stages.size());
        stages.push_back(st);
        stage_band.push_back(rq.band);
        expected.push_back(exp_here);
        n_items += st.n_items;
    }

    Program *p = new (std::nothrow) Program();
    if (!p) { set_error("out of host memory"); return LOP_ENOMEM; }
    if (uses_flags) {                                        // arrival flags live after the row-group counters
        p->flag_base = n_ctr;
        p->n_flags = pl->n_bands;
        for (int2 &d : deps)
            if (d.x < 0) d.x = p->flag_base + (-1 - d.x);
        n_ctr += p->n_flags;
    }
    if (n_items == 0) { *result = p; return LOP_OK; }          // nothing to do: an empty program

    // ---- one device allocation for all tables
    auto al = [](size_t v) { return (v + 255) / 256 * 256; };
    const size_t o_stages = 0;
    const size_t o_layers = o_stages + al(stages.size() * sizeof(WfStage));
    const size_t o_maps = o_layers + al(layers.size() * sizeof(WfLayer));
    const size_t o_depi = o_maps + al(std::max<size_t>(maps.size(), 1) * sizeof(CUtensorMap));
    const size_t o_deps = o_depi + al(std::max<size_t>(dep_index.size(), 1) * sizeof(int2));
    const size_t o_ctr = o_deps + al(std::max<size_t>(deps.size(), 1) * sizeof(int2));
    const size_t total = o_ctr + al((size_t)n_ctr * sizeof(unsigned));
    cudaError_t e = cudaMalloc(&p->dev, total);
    if (e != cudaSuccess) { delete p; set_error("cudaMalloc(%zu) failed: %s", total, cudaGetErrorString(e)); return LOP_ECUDA; }
    char *d = static_cast<char *>(p->dev);
    auto up = [&](size_t off, const void *src, size_t bytes) {
        return bytes ? cudaMemcpy(d + off, src, bytes, cudaMemcpyHostToDevice) : cudaSuccess;
    };
    if ((e = cudaMemset(d, 0, total)) != cudaSuccess || (e = up(o_stages, stages.data(), stages.size() * sizeof(WfStage))) != cudaSuccess ||
        (e = up(o_layers, layers.data(), layers.size() * sizeof(WfLayer))) != cudaSuccess ||
        (e = up(o_maps, maps.data(), maps.size() * sizeof(CUtensorMap))) != cudaSuccess ||
        (e = up(o_depi, dep_index.data(), dep_index.size() * sizeof(int2))) != cudaSuccess ||
        (e = up(o_deps, deps.data(), deps.size() * sizeof(int2))) != cudaSuccess) {
        program_destroy(p);
        set_error("program upload failed: %s", cudaGetErrorString(e));
        return LOP_ECUDA;
    }
    p->counters = reinterpret_cast<unsigned *>(d + o_ctr);
    WfParams &P = p->params;
    P.stages = reinterpret_cast<const WfStage *>(d + o_stages);
    P.layers = reinterpret_cast<const WfLayer *>(d + o_layers);
    P.maps = reinterpret_cast<const CUtensorMap *>(d + o_maps);
    P.dep_index = reinterpret_cast<const int2 *>(d + o_depi);
    P.deps = reinterpret_cast<const int2 *>(d + o_deps);
    P.counters = p->counters;
    P.status = reinterpret_cast<unsigned *>(wsb + pl->status_off);
    P.flag_base = p->flag_base; P.n_flags = p->n_flags;
    P.n_stages = (int)stages.size();
    P.n_items = n_items;
    P.slot_bytes = slot_bytes;
    int ring = (int)((200u * 1024u) / slot_bytes);
    P.ring = std::max(2, std::min(8, ring));
    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    p->grid = std::min(n_items, sms);
    *result = p;
    return LOP_OK;
}

int program_launch(Program *p, cudaStream_t s)
{
    if (!p || p->grid == 0) return LOP_OK;
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

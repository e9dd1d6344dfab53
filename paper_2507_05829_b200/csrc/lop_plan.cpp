// Host-side band planner and plan accessors.  Pure integer arithmetic; no CUDA call, no device
// pointer is dereferenced here.
//
// Method: Sec. IV-A (block-wise local operators: the block an output needs is fixed by kernel
// size, padding, dilation -- and stride), Sec. IV-B (a dependency exists as soon as any part of
// an output is used) and the contiguous-interval rule of Sec. IV-C ("Computational Efficiency"):
// the operations one executor runs for an operator form one interval, so a band is one row
// interval per layer and one kernel launch.
#include <atomic>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <new>

#include "lop_internal.h"

namespace lop {

static thread_local char g_err[512] = "";

#ifndef LOP_MAX_BAND_COPIES
#define LOP_MAX_BAND_COPIES 8
#endif

unsigned long long next_plan_uid()
{
    static std::atomic<unsigned long long> counter{0};
    return ++counter;
}

void set_error(const char *fmt, ...)
{
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
}

static inline long long floor_div(long long a, long long b)      // b > 0
{
    long long q = a / b;
    return (a % b != 0 && a < 0) ? q - 1 : q;
}
static inline long long ceil_div(long long a, long long b) { return -floor_div(-a, b); }

static inline int window_out(int n, int k, int s, int p, int d)
{
    long long num = (long long)n + 2LL * p - (long long)d * (k - 1) - 1;
    if (num < 0) return 0;
    return (int)(num / s) + 1;
}

struct Span {
    long long lo = 0, hi = 0;                      // half-open; lo >= hi means empty
    bool empty() const { return lo >= hi; }
    void join(const Span &o)
    {
        if (o.empty()) return;
        if (empty()) { *this = o; return; }
        if (o.lo < lo) lo = o.lo;
        if (o.hi > hi) hi = o.hi;
    }
};

// Rows of an h_in-row input that output rows [o.lo, o.hi) read through a (k, s, p, d) window:
// per tap, the first/last output row whose tap lands inside the tensor gives one candidate.
static Span rows_read(const Span &o, int k, int s, int p, int d, int h_in, int *pad_top, int *pad_bot)
{
    const long long top = o.lo * s - p;
    const long long bot = (o.hi - 1) * s - p + (long long)(k - 1) * d;
    *pad_top = top < 0 ? (int)(-top) : 0;
    *pad_bot = bot > h_in - 1 ? (int)(bot - (h_in - 1)) : 0;
    bool any_lo = false, any_hi = false;
    long long lo = 0, hi = 0;
    for (int t = 0; t < k; ++t) {
        const long long off = (long long)t * d - p;            // row = o*s + off
        long long first = ceil_div(-off, s);
        if (first < o.lo) first = o.lo;
        if (first < o.hi) {
            const long long r = first * s + off;
            if (r < h_in && (!any_lo || r < lo)) { lo = r; any_lo = true; }
        }
        long long last = floor_div((long long)h_in - 1 - off, s);
        if (last > o.hi - 1) last = o.hi - 1;
        if (last >= o.lo) {
            const long long r = last * s + off;
            if (r >= 0 && (!any_hi || r > hi)) { hi = r; any_hi = true; }
        }
    }
    Span out;
    if (any_lo && any_hi && lo <= hi) { out.lo = lo; out.hi = hi + 1; }
    return out;
}

static int check_layers(lop_plan_t &pl)
{
    const int L = (int)pl.layers.size();
    for (int i = 0; i < L; ++i) {
        LayerInfo &li = pl.layers[i];
        if (li.l.op < LOP_CONV2D || li.l.op > LOP_CONCAT) { set_error("layer %d: unknown op %d", i, li.l.op); return LOP_EINVAL; }
        if (li.l.op == LOP_LINEAR || li.l.op == LOP_LAYERNORM || li.l.op == LOP_CONCAT) {
            const lop_layer &q = li.l;
            if (q.kh != 1 || q.kw != 1 || q.sh != 1 || q.sw != 1 || q.dh != 1 || q.dw != 1 || q.ph != 0 || q.pw != 0) {
                set_error("layer %d: a row-wise operator has no window (kh = kw = sh = sw = dh = dw = 1, ph = pw = 0)", i);
                return LOP_EINVAL;
            }
        }
        if (li.l.op == LOP_LINEAR) {
            // Y = X * W^T over the channel vectors of the pixels is the pointwise convolution with the same [cout][cin]
            // matrix: from here on the layer is planned and executed as one (rows map one to one, no halo)
            li.linear = true;
            li.l.op = LOP_CONV2D;
        }
        const lop_layer &l = li.l;
        if (l.kh < 1 || l.kw < 1 || l.sh < 1 || l.sw < 1 || l.dh < 1 || l.dw < 1 || l.ph < 0 || l.pw < 0 ||
            l.cin < 1 || l.cout < 1) {
            set_error("layer %d: kernel/stride/dilation must be >= 1, padding >= 0, channels >= 1", i);
            return LOP_ESHAPE;
        }
        if (l.act < LOP_ACT_NONE || l.act > LOP_ACT_GELU) { set_error("layer %d: unknown activation", i); return LOP_EINVAL; }
        if (l.input_from < LOP_INPUT || l.input_from >= i) {
            set_error("layer %d: input_from=%d must be LOP_INPUT or an earlier layer", i, l.input_from);
            return LOP_ESHAPE;
        }
        int hin, win, cin;
        if (l.input_from == LOP_INPUT) { hin = pl.H; win = pl.W; cin = pl.C; }
        else { const LayerInfo &s = pl.layers[l.input_from]; hin = s.Ho; win = s.Wo; cin = s.Co; }
        if (cin != l.cin) { set_error("layer %d: cin=%d but its input has %d channels", i, l.cin, cin); return LOP_ESHAPE; }
        if ((l.op == LOP_MAXPOOL2D || l.op == LOP_DWCONV2D || l.op == LOP_LAYERNORM) && l.cout != l.cin) {
            set_error("layer %d: pooling, depth-wise convolution and layer normalisation keep the channel count", i);
            return LOP_ESHAPE;
        }
        li.Hin = hin; li.Win = win;
        li.Ho = window_out(hin, l.kh, l.sh, l.ph, l.dh);
        li.Wo = window_out(win, l.kw, l.sw, l.pw, l.dw);
        li.Co = l.cout;
        if (li.Ho <= 0 || li.Wo <= 0) { set_error("layer %d: empty output (%d x %d)", i, li.Ho, li.Wo); return LOP_ESHAPE; }
        if (l.op == LOP_DWCONV2D && (long long)l.kh * l.kw > 1024) {
            set_error("layer %d: a depth-wise filter of more than 1024 taps is not supported", i);
            return LOP_EUNSUPPORTED;
        }
        if (l.residual_from != LOP_NO_RESIDUAL) {
            if (l.residual_from < LOP_INPUT || l.residual_from >= i) {
                set_error("layer %d: residual_from=%d must be LOP_INPUT or an earlier layer", i, l.residual_from);
                return LOP_ESHAPE;
            }
            const bool conv_like = l.op == LOP_CONV2D || l.op == LOP_DWCONV2D;
            if (l.op != LOP_CONCAT && (!conv_like || (l.residual_pos != LOP_RES_PRE_ACT && l.residual_pos != LOP_RES_POST_ACT))) {
                set_error("layer %d: a residual needs a convolution and residual_pos PRE_ACT or POST_ACT", i);
                return LOP_ESHAPE;
            }
            int rh, rw, rc;
            if (l.residual_from == LOP_INPUT) { rh = pl.H; rw = pl.W; rc = pl.C; }
            else { const LayerInfo &s = pl.layers[l.residual_from]; rh = s.Ho; rw = s.Wo; rc = s.Co; }
            const int want_c = l.op == LOP_CONCAT ? li.Co - l.cin : li.Co;
            if (rh != li.Ho || rw != li.Wo || rc != want_c || want_c < 1) {
                set_error(l.op == LOP_CONCAT ? "layer %d: the second input of a concatenation must have cout - cin channels and the main input's height and width"
                                             : "layer %d: residual shape mismatch", i);
                return LOP_ESHAPE;
            }
        } else if (l.op == LOP_CONCAT) {
            set_error("layer %d: a concatenation names its second input in residual_from", i);
            return LOP_ESHAPE;
        }
    }
    return LOP_OK;
}

static void plan_bands(lop_plan_t &pl)
{
    const int L = (int)pl.layers.size(), B = pl.n_bands;
    const long long HL = pl.layers[L - 1].Ho;
    pl.ranges.assign((size_t)B * L, lop_range{0, 0, 0, 0, 0, 0, 0, 0});
    pl.in_need.assign(B, lop_range{0, 0, 0, 0, 0, 0, 0, 0});
    std::vector<long long> produced(L + 1, 0);             // [0] = chain input, [i+1] = layer i
    std::vector<Span> need(L + 1);
    for (int b = 0; b < B; ++b) {
        for (auto &s : need) s = Span();
        need[L].lo = (long long)b * HL / B;
        need[L].hi = (long long)(b + 1) * HL / B;
        for (int i = L - 1; i >= 0; --i) {
            const Span o = need[i + 1];
            if (o.empty()) continue;
            const lop_layer &l = pl.layers[i].l;
            lop_range &r = pl.ranges[(size_t)b * L + i];
            int pt = 0, pb = 0;
            const Span in = rows_read(o, l.kh, l.sh, l.ph, l.dh, pl.layers[i].Hin, &pt, &pb);
            r.out_lo = (int)o.lo; r.out_hi = (int)o.hi;
            r.in_lo = (int)in.lo; r.in_hi = (int)in.hi;
            r.pad_top = pt; r.pad_bot = pb;
            need[l.input_from + 1].join(in);
            if (l.residual_from != LOP_NO_RESIDUAL) need[l.residual_from + 1].join(o);
        }
        for (int i = 0; i <= L; ++i) {
            lop_range &r = i == 0 ? pl.in_need[b] : pl.ranges[(size_t)b * L + (i - 1)];
            const Span &s = need[i];
            if (s.empty()) continue;
            if (i == 0) { r.out_lo = (int)s.lo; r.out_hi = (int)s.hi; }
            long long nl = s.lo > produced[i] ? s.lo : produced[i];
            if (nl > s.hi) nl = s.hi;
            r.new_lo = (int)nl;
            if (s.hi > produced[i]) produced[i] = s.hi;
        }
    }
}

// Decide which kernel serves each layer and lay the workspace out.
static void choose_kernels(lop_plan_t &pl)
{
    const int L = (int)pl.layers.size();
    const size_t es = elem_size(pl.dtype);
    pl.stem = -1;
    const bool tc_ok = pl.dtype == LOP_BF16 && !(pl.flags & LOP_FLAG_FORCE_SIMT);
    for (int i = 0; i < L; ++i) {
        LayerInfo &li = pl.layers[i];
        const lop_layer &l = li.l;
        li.cin_eff = l.cin;
        li.stem_gather = false;
        if (l.op == LOP_MAXPOOL2D) { li.kernel = K_POOL; continue; }
        li.dw_transposed = false;
        if (l.op == LOP_DWCONV2D) { li.kernel = K_DWCONV; li.dw_transposed = pl.dtype == LOP_BF16 && l.cin % 8 == 0; continue; }
        if (l.op == LOP_LAYERNORM) { li.kernel = K_LAYERNORM; continue; }
        if (l.op == LOP_CONCAT) { li.kernel = K_CONCAT; continue; }
        li.kernel = K_CONV_SIMT;
        if (!tc_ok) continue;
        if (l.cout % 16 != 0 || l.sh * l.sw > 4) continue;
        int cin = l.cin;
        if (cin % 16 != 0) {
            // a thin chain input (an image): gather each output pixel's kh*kw*cin patch, zero-padded to a multiple
            // of 16, and run the layer as a pointwise convolution over the patches
            const long long patch = (long long)l.kh * l.kw * cin;
            if (l.input_from != LOP_INPUT || cin > 16 || patch > 1024 || pl.stem >= 0) continue;
            cin = (int)align_up((size_t)patch, 16);
            li.stem_gather = true;
            pl.stem = i;
        }
        if ((long long)l.kh * l.kw * cin > (1LL << 20)) continue;
        li.cin_eff = cin;
        li.kernel = K_CONV_TC;
    }

    // Copy-engine band pipeline: every copy costs a few microseconds of stream commands whatever its size, so an input
    // of megabytes cut into many bands is moved a few neighbouring bands per copy (at most LOP_MAX_BAND_COPIES copies);
    // the bands of one copy arrive together.  Small inputs keep one copy per band.
    {
        const size_t in_bytes = (size_t)pl.N * pl.H * pl.W * pl.C * es;
        pl.copy_group = (in_bytes >= (1u << 20) && pl.n_bands > LOP_MAX_BAND_COPIES) ? (pl.n_bands + LOP_MAX_BAND_COPIES - 1) / LOP_MAX_BAND_COPIES : 1;
    }
    size_t off = 0;
    pl.status_off = off; off += 1024;
    for (int i = 0; i < L; ++i) {
        LayerInfo &li = pl.layers[i];
        if (li.stem_gather) {
            pl.col_off = off;
            off += align_up((size_t)pl.N * li.Ho * li.Wo * li.cin_eff * es, 1024);
            li.wpad_off = off;
            off += align_up((size_t)li.l.cout * li.cin_eff * es, 1024);
        }
        if (li.dw_transposed) {
            li.wpad_off = off;
            off += align_up((size_t)li.l.kh * li.l.kw * li.l.cin * es, 1024);
        }
        if (i != L - 1) {
            li.out_off = off;
            off += align_up((size_t)pl.N * li.Ho * li.Wo * li.Co * es, 1024);
        }
    }
    pl.ws_bytes = off;
    pl.flops = 0.0;
    for (auto &li : pl.layers)
        if (li.l.op == LOP_CONV2D)
            pl.flops += 2.0 * pl.N * li.Ho * li.Wo * li.Co * (double)li.l.kh * li.l.kw * li.l.cin;
        else if (li.l.op == LOP_DWCONV2D)
            pl.flops += 2.0 * pl.N * li.Ho * li.Wo * li.Co * (double)li.l.kh * li.l.kw;
}

}  // namespace lop

using namespace lop;

extern "C" {

int lop_plan(const lop_layer *layers, int n_layers, int N, int H, int W, int C, int dtype,
             int n_bands, unsigned flags, lop_plan_t **out)
{
    if (!out) { set_error("lop_plan: out is NULL"); return LOP_EINVAL; }
    *out = nullptr;
    if (!layers || n_layers < 1) { set_error("lop_plan: need at least one layer"); return LOP_EINVAL; }
    if (N < 1 || H < 1 || W < 1 || C < 1) { set_error("lop_plan: N, H, W, C must be >= 1"); return LOP_ESHAPE; }
    if (n_bands < 1) { set_error("lop_plan: n_bands must be >= 1"); return LOP_EINVAL; }
    if (dtype != LOP_F32 && dtype != LOP_BF16) { set_error("lop_plan: unknown dtype %d", dtype); return LOP_EINVAL; }
    if (flags & ~(LOP_FLAG_REUSE_HALO | LOP_FLAG_TIME_LAYERS | LOP_FLAG_FORCE_SIMT | LOP_FLAG_PER_LAYER | LOP_FLAG_COPY_ENGINE | LOP_FLAG_DEBUG_BOUNDS)) {
        set_error("lop_plan: unknown flag bits 0x%x", flags);
        return LOP_EINVAL;
    }
    lop_plan_t *pl = new (std::nothrow) lop_plan_t();
    if (pl) pl->uid = next_plan_uid();
    if (!pl) { set_error("lop_plan: out of host memory"); return LOP_ENOMEM; }
    try {
        pl->N = N; pl->H = H; pl->W = W; pl->C = C; pl->dtype = dtype; pl->n_bands = n_bands; pl->flags = flags;
        pl->layers.resize(n_layers);
        for (int i = 0; i < n_layers; ++i) pl->layers[i].l = layers[i];
        int rc = check_layers(*pl);
        if (rc != LOP_OK) { delete pl; return rc; }
        long long max_elems = 0;
        for (auto &li : pl->layers) {
            long long e = (long long)N * li.Ho * li.Wo * li.Co;
            if (e > max_elems) max_elems = e;
        }
        if (max_elems >= (1LL << 40)) { delete pl; set_error("lop_plan: tensor too large"); return LOP_EUNSUPPORTED; }
        plan_bands(*pl);
        choose_kernels(*pl);
    } catch (const std::bad_alloc &) {
        delete pl;
        set_error("lop_plan: out of host memory");
        return LOP_ENOMEM;
    }
    *out = pl;
    return LOP_OK;
}

void lop_plan_destroy(lop_plan_t *plan)
{
    if (!plan) return;
    if (plan->exec) exec_destroy(plan->exec);
    delete plan;
}

int lop_plan_num_bands(const lop_plan_t *plan)
{
    if (!plan) { set_error("plan is NULL"); return LOP_EINVAL; }
    return plan->n_bands;
}

int lop_plan_num_layers(const lop_plan_t *plan)
{
    if (!plan) { set_error("plan is NULL"); return LOP_EINVAL; }
    return (int)plan->layers.size();
}

int lop_plan_get_range(const lop_plan_t *plan, int band, int layer, lop_range *out)
{
    if (!plan || !out) { set_error("lop_plan_get_range: NULL argument"); return LOP_EINVAL; }
    const int L = (int)plan->layers.size();
    if (band < 0 || band >= plan->n_bands || layer < LOP_INPUT || layer >= L) {
        set_error("lop_plan_get_range: band %d / layer %d out of range", band, layer);
        return LOP_EINVAL;
    }
    *out = layer == LOP_INPUT ? plan->in_need[band] : plan->ranges[(size_t)band * L + layer];
    return LOP_OK;
}

int lop_plan_out_shape(const lop_plan_t *plan, int layer, int *H, int *W, int *C)
{
    if (!plan) { set_error("plan is NULL"); return LOP_EINVAL; }
    const int L = (int)plan->layers.size();
    if (layer < LOP_INPUT || layer >= L) { set_error("lop_plan_out_shape: layer %d out of range", layer); return LOP_EINVAL; }
    int h = plan->H, w = plan->W, c = plan->C;
    if (layer >= 0) { h = plan->layers[layer].Ho; w = plan->layers[layer].Wo; c = plan->layers[layer].Co; }
    if (H) *H = h;
    if (W) *W = w;
    if (C) *C = c;
    return LOP_OK;
}

int lop_plan_set_params(lop_plan_t *plan, int layer, const void *weight, const float *scale, const float *shift)
{
    if (!plan) { set_error("plan is NULL"); return LOP_EINVAL; }
    if (layer < 0 || layer >= (int)plan->layers.size()) { set_error("lop_plan_set_params: layer %d out of range", layer); return LOP_EINVAL; }
    lop_layer &l = plan->layers[layer].l;
    l.weight = weight; l.scale = scale; l.shift = shift;
    plan->uid = next_plan_uid();           // chain programs cached in another plan were built from the old pointers too
    exec_invalidate(plan->exec);           // device tables and tensor maps were built from the old pointers
    return LOP_OK;
}

size_t lop_plan_workspace_bytes(const lop_plan_t *plan) { return plan ? plan->ws_bytes : 0; }

size_t lop_plan_staging_bytes(const lop_plan_t *plan)
{
    return plan ? (size_t)plan->N * plan->H * plan->W * plan->C * elem_size(plan->dtype) : 0;
}

double lop_plan_flops(const lop_plan_t *plan) { return plan ? plan->flops : 0.0; }

int lop_plan_layer_kernel(const lop_plan_t *plan, int layer)
{
    if (!plan) { set_error("plan is NULL"); return LOP_EINVAL; }
    if (layer < 0 || layer >= (int)plan->layers.size()) { set_error("lop_plan_layer_kernel: layer %d out of range", layer); return LOP_EINVAL; }
    return plan->layers[layer].kernel;
}

const char *lop_strerror(int status)
{
    switch (status) {
    case LOP_OK: return "success";
    case LOP_EINVAL: return "invalid argument";
    case LOP_ESHAPE: return "layer list does not type-check";
    case LOP_EUNSUPPORTED: return "unsupported configuration";
    case LOP_ENOMEM: return "out of host memory";
    case LOP_ECUDA: return "CUDA error";
    case LOP_EWORKSPACE: return "workspace missing or misaligned";
    case LOP_EDEVICE: return "a kernel gave up on a bounded wait";
    default: return "unknown status";
    }
}

const char *lop_last_error(void) { return g_err; }

}  // extern "C"

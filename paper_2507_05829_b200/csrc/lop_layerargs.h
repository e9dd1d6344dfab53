// Kernel arguments of a planned layer, shared by the executors (host only).
#pragma once
#include "lop_gather.cuh"
#include "lop_internal.h"
#include "lop_kernels.cuh"

namespace lop {

// Full-size tensor a layer index refers to: the chain input, the caller's output (last layer), or workspace.
inline const void *tensor_of(const lop_plan_t *pl, int idx, const void *in, void *out, void *ws)
{
    if (idx == LOP_INPUT) return in;
    if (idx == (int)pl->layers.size() - 1) return out;
    return static_cast<char *>(ws) + pl->layers[idx].out_off;
}

inline GatherGeom gather_geom(const lop_plan_t *pl, int i)
{
    const LayerInfo &li = pl->layers[i];
    const lop_layer &l = li.l;
    GatherGeom g;
    g.N = pl->N; g.H = pl->H; g.W = pl->W; g.C = pl->C;
    g.Ho = li.Ho; g.Wo = li.Wo; g.Kcol = li.cin_eff;
    g.kh = l.kh; g.kw = l.kw; g.sh = l.sh; g.sw = l.sw; g.ph = l.ph; g.pw = l.pw; g.dh = l.dh; g.dw = l.dw;
    return g;
}

// Convolution layer i over output rows [lo, hi).  A tensor-core layer is described the way its kernel
// sees it: a gathered stem is a pointwise convolution over the patch tensor with zero-padded weights.
inline ConvArgs conv_args(const lop_plan_t *pl, int i, const void *in, void *out, void *ws, int lo, int hi)
{
    const LayerInfo &li = pl->layers[i];
    const lop_layer &l = li.l;
    ConvArgs a;
    a.x = tensor_of(pl, l.input_from, in, out, ws);
    a.w = l.weight;
    a.scale = l.scale; a.shift = l.shift;
    a.res = l.residual_from == LOP_NO_RESIDUAL ? nullptr : tensor_of(pl, l.residual_from, in, out, ws);
    a.y = const_cast<void *>(tensor_of(pl, i, in, out, ws));
    a.N = pl->N; a.Hin = li.Hin; a.Win = li.Win; a.Cin = l.cin; a.Ho = li.Ho; a.Wo = li.Wo; a.Cout = l.cout;
    a.kh = l.kh; a.kw = l.kw; a.sh = l.sh; a.sw = l.sw; a.ph = l.ph; a.pw = l.pw; a.dh = l.dh; a.dw = l.dw;
    a.act = l.act; a.res_pos = a.res ? l.residual_pos : LOP_RES_NONE;
    a.oh_lo = lo; a.oh_hi = hi;
    a.dbg = (pl->flags & LOP_FLAG_DEBUG_BOUNDS) ? reinterpret_cast<unsigned *>(static_cast<char *>(ws) + pl->status_off) : nullptr;
    if (li.kernel == K_CONV_TC) {
        a.Cin = li.cin_eff;
        if (li.stem_gather) {
            a.x = static_cast<char *>(ws) + pl->col_off;
            a.w = static_cast<char *>(ws) + li.wpad_off;
            a.Hin = li.Ho; a.Win = li.Wo;
            a.kh = a.kw = a.sh = a.sw = a.dh = a.dw = 1;
            a.ph = a.pw = 0;
        }
    }
    return a;
}

inline PoolArgs pool_args(const lop_plan_t *pl, int i, const void *in, void *out, void *ws, int lo, int hi)
{
    const LayerInfo &li = pl->layers[i];
    const lop_layer &l = li.l;
    PoolArgs a;
    a.x = tensor_of(pl, l.input_from, in, out, ws);
    a.y = const_cast<void *>(tensor_of(pl, i, in, out, ws));
    a.N = pl->N; a.Hin = li.Hin; a.Win = li.Win; a.C = l.cin; a.Ho = li.Ho; a.Wo = li.Wo;
    a.kh = l.kh; a.kw = l.kw; a.sh = l.sh; a.sw = l.sw; a.ph = l.ph; a.pw = l.pw; a.dh = l.dh; a.dw = l.dw;
    a.oh_lo = lo; a.oh_hi = hi;
    a.dbg = (pl->flags & LOP_FLAG_DEBUG_BOUNDS) ? reinterpret_cast<unsigned *>(static_cast<char *>(ws) + pl->status_off) : nullptr;
    return a;
}

}  // namespace lop

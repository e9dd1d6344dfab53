// Arithmetic shared by the two homes of the memory-bound local operators (depth-wise convolution, layer
// normalisation; Sec. IV-A of the paper): the stand-alone kernels of the per-layer executor and the worker warps of
// the persistent kernel.  Both walk a pixel's values in the same order through these functions, so a tensor's bits
// do not depend on which of the two produced it.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <cmath>
#include <cstdint>

#include "lop.h"

namespace lop {
namespace rowop {

constexpr float LAYERNORM_EPS = 1e-6f;

// Activation in its accurate form (library exp / erf): these operators are bound by memory, not by arithmetic.
__device__ __forceinline__ float activate(float t, int act)
{
    if (act == LOP_ACT_RELU) return fmaxf(t, 0.0f);
    if (act == LOP_ACT_SILU) return t / (1.0f + expf(-t));
    if (act == LOP_ACT_GELU) return 0.5f * t * (1.0f + erff(t * 0.70710678f));      // t * Phi(t)
    return t;
}

// scale * acc + shift, residual before or after the activation (res_pos is LOP_RES_NONE when there is none).
__device__ __forceinline__ float epilogue(float acc, float scale, float shift, float res, int res_pos, int act)
{
    float v = fmaf(scale, acc, shift);
    if (res_pos == LOP_RES_PRE_ACT) v += res;
    v = activate(v, act);
    if (res_pos == LOP_RES_POST_ACT) v += res;
    return v;
}

// Lanes that share a pixel in the layer normalisation: the smallest power of two that covers its V vectors, at most
// a warp.  Lane `sub` of the group owns vectors sub, sub + lanes, sub + 2 * lanes, ...
__host__ __device__ __forceinline__ int ln_lanes_log(int V)
{
    int l = 0;
    while ((1 << l) < V && l < 5) ++l;
    return l;
}

// Sum over the 2^lanes_log lanes of a pixel's group (every lane of the warp takes part; all get the total).
__device__ __forceinline__ float group_sum(float v, int lanes_log)
{
    for (int o = (1 << lanes_log) >> 1; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

__device__ __forceinline__ float ln_inv_std(float sum_sq, int C) { return 1.0f / sqrtf(sum_sq / (float)C + LAYERNORM_EPS); }
__device__ __forceinline__ float ln_value(float x, float mean, float inv, float gain, float offset) { return fmaf((x - mean) * inv, gain, offset); }

__device__ __forceinline__ void unpack_bf16x8(const uint4 &q, float (&f)[8])
{
    const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        f[2 * i] = __uint_as_float(w[i] << 16);
        f[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
    }
}

// Two fp32 values rounded to nearest-even bf16, lo in the low half of the word (one conversion instruction).
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi)
{
    const __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t *>(&h);
}

// ---------------------------------------------------------------------------------------------
// Layer normalisation of bf16 pixels with a multiple of eight channels, at most 1024: a group of 2^lanes_log lanes
// per pixel, lane `sub` owning vectors sub, sub + lanes, ... (VPL = 1, 2 or 4 of them, eight channels each).  A lane
// keeps four vectors in registers: the 4 / VPL pixels its group normalises at a time, all loaded before the first
// sum, so that a thread has 64 bytes on their way.  Per pixel: the lane's values summed in ascending order, the
// butterfly over the group, the centred squares likewise; the same order as the plain kernel's, so the bits agree.
// o[p]: element offset of pixel p, live[p]: whether the slot holds a pixel (dead slots still take part in the
// shuffles).  gain / offset may be null.
// ---------------------------------------------------------------------------------------------
template <bool THROUGH_L2, int VPL, int PPG>
__device__ __forceinline__ void ln_pixels(const uint16_t *x, uint16_t *y, int C, int lanes_log, int sub, const long long (&o)[PPG],
                                          const bool (&live)[PPG], const float *gain, const float *offset)
{
    const int nv = C >> 3, lanes = 1 << lanes_log;
    uint4 q[PPG][VPL];
    bool have[PPG][VPL];
#pragma unroll
    for (int p = 0; p < PPG; ++p)
#pragma unroll
        for (int k = 0; k < VPL; ++k) {
            have[p][k] = live[p] && sub + k * lanes < nv;
            q[p][k] = make_uint4(0u, 0u, 0u, 0u);
            if (have[p][k]) {
                const uint4 *src = reinterpret_cast<const uint4 *>(x + o[p]) + sub + k * lanes;
                q[p][k] = THROUGH_L2 ? __ldcg(src) : __ldg(src);
            }
        }
    // widened once; from the second pass on f holds the centred values
    float f[PPG][VPL][8], mean[PPG], inv[PPG];
#pragma unroll
    for (int p = 0; p < PPG; ++p) {
        float s1 = 0.0f;
#pragma unroll
        for (int k = 0; k < VPL; ++k) {
            unpack_bf16x8(q[p][k], f[p][k]);
            if (have[p][k]) {
#pragma unroll
                for (int j = 0; j < 8; ++j) s1 += f[p][k][j];
            }
        }
        mean[p] = group_sum(s1, lanes_log) / (float)C;
    }
#pragma unroll
    for (int p = 0; p < PPG; ++p) {
        float s2 = 0.0f;
#pragma unroll
        for (int k = 0; k < VPL; ++k)
            if (have[p][k]) {
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    f[p][k][j] -= mean[p];
                    s2 = fmaf(f[p][k][j], f[p][k][j], s2);
                }
            }
        inv[p] = ln_inv_std(group_sum(s2, lanes_log), C);
    }
#pragma unroll
    for (int k = 0; k < VPL; ++k) {
        const int v = sub + k * lanes;
        if (v >= nv) continue;
        float gn[8], of[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) { gn[j] = 1.0f; of[j] = 0.0f; }
        if (gain) {
            const float4 a = __ldg(reinterpret_cast<const float4 *>(gain + v * 8)), b = __ldg(reinterpret_cast<const float4 *>(gain + v * 8) + 1);
            gn[0] = a.x; gn[1] = a.y; gn[2] = a.z; gn[3] = a.w; gn[4] = b.x; gn[5] = b.y; gn[6] = b.z; gn[7] = b.w;
        }
        if (offset) {
            const float4 a = __ldg(reinterpret_cast<const float4 *>(offset + v * 8)), b = __ldg(reinterpret_cast<const float4 *>(offset + v * 8) + 1);
            of[0] = a.x; of[1] = a.y; of[2] = a.z; of[3] = a.w; of[4] = b.x; of[5] = b.y; of[6] = b.z; of[7] = b.w;
        }
#pragma unroll
        for (int p = 0; p < PPG; ++p)
            if (have[p][k]) {
                float r[8];
#pragma unroll
                for (int j = 0; j < 8; ++j) r[j] = fmaf(f[p][k][j] * inv[p], gn[j], of[j]);       // ln_value on the centred value
                *(reinterpret_cast<uint4 *>(y + o[p]) + v) =
                    make_uint4(pack_bf16x2(r[0], r[1]), pack_bf16x2(r[2], r[3]), pack_bf16x2(r[4], r[5]), pack_bf16x2(r[6], r[7]));
            }
    }
}
// Vectors per lane for a pixel of nv vectors (1, 2 or 4; nv <= 128).
__host__ __device__ inline int ln_vpl(int nv)
{
    const int lanes = 1 << ln_lanes_log(nv);
    return nv <= lanes ? 1 : (nv <= 2 * lanes ? 2 : 4);
}

// ---------------------------------------------------------------------------------------------
// Depth-wise convolution of one tile: R output rows x tw output columns x cc channels of one image, by `NTHREADS`
// threads that share a barrier.  With kh*kw multiply-adds per output and two bytes of input and output each, a 7x7
// filter is bound by the fp32 multiply-add rate, not by DRAM: what counts is the number of other instructions per
// multiply-add.  So the tile's receptive window and the filters of its channels are put into shared memory as fp32
// first (a value is widened once, not once per tap that reads it; taps outside the tensor read zeros, so the walk has
// no bounds checks), and the walk keeps a filter row's run of inputs in registers for several adjacent outputs and
// issues its multiply-adds two per instruction.  Every output sums its taps in the order a = 0..kh-1, b = 0..kw-1,
// whatever the tile: a pixel's bits do not depend on the tile or the band it is computed in.
// ---------------------------------------------------------------------------------------------
struct DwTile { int R, tw, cc; };

struct DwGeom {
    int Hin, Win, C, Ho, Wo;
    int kh, kw, sh, sw, ph, pw, dh, dw;
    int act, res_pos;                 // res_pos == LOP_RES_NONE when res is null
    DwTile t;
    const uint16_t *x;                // [N, Hin, Win, C] bf16
    const uint16_t *res;              // [N, Ho, Wo, C] or nullptr
    const uint16_t *w_taps;           // [kh*kw][C] bf16
    const float *scale, *shift;
    uint16_t *y;
    unsigned *dbg;                    // checked execution: status word that takes bit 0x100 on an address outside a tensor, else nullptr
    int N;                            // images (for the checks only)
};
// (the persistent kernel, THROUGH_L2, never runs checked: checked execution takes the stand-alone kernels)
template <bool THROUGH_L2>
__device__ __forceinline__ bool dw_in_bounds(const DwGeom &g, long long first, long long count, long long limit)
{
    if (THROUGH_L2 || !g.dbg || (first >= 0 && first + count <= limit)) return true;
    atomicOr(g.dbg, 0x100u);
    return false;
}

constexpr int DW_T = 8;               // adjacent output columns one thread computes on the sliding-window path

// The sliding-window path: stride 1 and dilation 1 along the width and a filter 3, 5 or 7 wide.  A thread then keeps a
// filter row's run of DW_T + kw - 1 input values in registers and uses each for up to kw outputs.
__host__ __device__ inline bool dw_slides(int kw, int sw, int dw) { return sw == 1 && dw == 1 && (kw == 3 || kw == 5 || kw == 7); }

// Columns of the staged window for ncol output columns.  On the sliding-window path the output columns are rounded up
// to whole groups of DW_T (the surplus outputs are computed from valid shared memory and dropped).
__host__ __device__ inline int dw_cols_in(int ncol, int kw, int sw, int dw)
{
    const int nc = dw_slides(kw, sw, dw) ? (ncol + DW_T - 1) / DW_T * DW_T : ncol;
    return (nc - 1) * sw + (kw - 1) * dw + 1;
}

// Pixels between the starts of two rows of the staged window (a pixel is cc fp32 values): the columns, padded so that
// a row's pitch in bytes is cc * 4 more than a multiple of 128.  The eight threads of one shared-memory access phase
// (16 bytes each) are the cc / 4 channel quads of 32 / cc consecutive rows (see dw_walk_sliding): with this pitch they
// read eight different groups of four banks.
__host__ __device__ inline int dw_pitch(int cols_in, int cc)
{
    const int m = 32 / cc;                                 // cc = 8, 16, 32: pitch = 1 modulo 4, 2, 1
    return m <= 1 ? cols_in : (cols_in + m - 2) / m * m + 1;
}

// Shared memory one tile needs (fp32 window + fp32 filters), in bytes.
__host__ __device__ inline long long dw_tile_bytes(int kh, int kw, int sh, int sw, int dh, int dw, const DwTile &t)
{
    const long long rows = (long long)(t.R - 1) * sh + (long long)(kh - 1) * dh + 1;
    const long long cols = dw_pitch(dw_cols_in(t.tw, kw, sw, dw), t.cc);
    return (rows * cols + (long long)kh * kw) * t.cc * 4;
}

// Tile shape for a layer: the one that re-reads the least input per output (rows and columns of halo) among those
// that fit `budget` bytes of shared memory, with enough (pixel, channel-quad) units to keep `threads` threads busy and
// enough tiles to give every SM one, where the layer is large enough for that.
inline bool dw_choose_tile(int kh, int kw, int sh, int sw, int dh, int dw, int N, int rows_out, int Wo, int C, long long budget,
                           int threads, DwTile *out)
{
    if (C % 8 != 0) return false;
    bool found = false;
    double best = 0.0;
    for (int cc = (C % 32 == 0 ? 32 : (C % 16 == 0 ? 16 : 8)); cc >= 8; cc /= 2)
        for (int R = 1; R <= 16; R *= 2)
            for (int div = 1; div <= 64; div *= 2) {
                const int tw = (Wo + div - 1) / div;
                if (div > 1 && tw < 4) break;
                const DwTile t{R, tw, cc};
                if (dw_tile_bytes(kh, kw, sh, sw, dh, dw, t) > budget) continue;
                const double rows_in = (R - 1) * sh + (kh - 1) * dh + 1, cols_in = (tw - 1) * sw + (kw - 1) * dw + 1;
                double cost = rows_in * cols_in / ((double)R * tw);                       // input values staged per output value
                const double units = (double)R * (dw_slides(kw, sw, dw) ? (tw + DW_T - 1) / DW_T : tw) * cc / 4;
                if (units < threads) cost *= threads / units;                             // idle threads
                const double tiles = (double)N * ((rows_out + R - 1) / R) * ((Wo + tw - 1) / tw) * (C / cc);
                cost *= std::ceil(tiles / 148.0) * 148.0 / tiles;                         // idle SMs in the last round of tiles
                if (!found || cost < best) { found = true; best = cost; *out = t; }
            }
    return found;
}

template <int BAR_ID, int NTHREADS>
__device__ __forceinline__ void tile_barrier()
{
    asm volatile("bar.sync %0, %1;" ::"n"(BAR_ID), "n"(NTHREADS) : "memory");
}

// Epilogue and store of four channels at element offset o of the output (scale / shift of those channels in sc / sf).
// SMOOTH: the activation is SiLU or GELU.  The caller picks the instantiation once per unit, so that the common
// kinds (none, ReLU) run a few instructions per value with no exp / erf code in their way.
template <bool THROUGH_L2, bool SMOOTH>
__device__ __forceinline__ void dw_store4(const DwGeom &g, long long o, const float4 &sc, const float4 &sf, const float (&acc)[4])
{
    if (!dw_in_bounds<THROUGH_L2>(g, o, 4, (long long)g.N * g.Ho * g.Wo * g.C)) return;
    float v[4] = {fmaf(sc.x, acc[0], sf.x), fmaf(sc.y, acc[1], sf.y), fmaf(sc.z, acc[2], sf.z), fmaf(sc.w, acc[3], sf.w)};
    float rf[4] = {0.0f, 0.0f, 0.0f, 0.0f};
    if (g.res) {
        const uint2 *src = reinterpret_cast<const uint2 *>(g.res + o);
        const uint2 rq = THROUGH_L2 ? __ldcg(src) : __ldg(src);
        rf[0] = __uint_as_float(rq.x << 16); rf[1] = __uint_as_float(rq.x & 0xFFFF0000u);
        rf[2] = __uint_as_float(rq.y << 16); rf[3] = __uint_as_float(rq.y & 0xFFFF0000u);
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        if (g.res_pos == LOP_RES_PRE_ACT) v[j] += rf[j];
        if (SMOOTH) v[j] = activate(v[j], g.act);
        else if (g.act == LOP_ACT_RELU) v[j] = fmaxf(v[j], 0.0f);
        if (g.res_pos == LOP_RES_POST_ACT) v[j] += rf[j];
    }
    *reinterpret_cast<uint2 *>(g.y + o) = make_uint2(pack_bf16x2(v[0], v[1]), pack_bf16x2(v[2], v[3]));
}
__device__ __forceinline__ float4 dw_load4(const float *p, int c, float dflt)
{
    return p ? __ldg(reinterpret_cast<const float4 *>(p + c)) : make_float4(dflt, dflt, dflt, dflt);
}

// Two fp32 values in one 64-bit register pair, and the packed fused multiply-add of sm_100: d = a * b + d on both
// halves, each rounded like a scalar fmaf (the results are the scalar ones; what is saved is issue slots).
typedef unsigned long long f32x2;
__device__ __forceinline__ f32x2 pack2(float lo, float hi)
{
    f32x2 r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(f32x2 v, float &lo, float &hi) { asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v)); }
__device__ __forceinline__ void fma2(f32x2 &d, f32x2 a, f32x2 b) { asm("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(d) : "l"(a), "l"(b)); }
// Sliding-window walk of a staged tile (stride 1, dilation 1 along the width; KW and the tile's channel count 2^CC_LOG
// known at compile time, so that every shared-memory offset is an immediate): a thread owns DW_T adjacent output
// columns of one row and four channels.  Per filter row it loads the DW_T + KW - 1 input vectors those outputs read
// once, then one weight vector per tap: DW_T + 2 * KW - 1 loads for 2 * DW_T * KW packed multiply-adds.  Every output
// still sums its taps in the order a = 0..kh-1, b = 0..KW-1, like the one-pixel walk.
// xs: the window, [row][pitch][cc] fp32; wsm: the filters, [tap][cc] fp32.
template <bool THROUGH_L2, int KW, int CC_LOG, int NTHREADS>
__device__ __forceinline__ void dw_walk_sliding(const DwGeom &g, int n, int oh0, int nrow, int ow0, int ncol, int c0, const float *xs,
                                                const float *wsm, int pitch, int tid)
{
    constexpr int CC = 1 << CC_LOG, Q4_LOG = CC_LOG - 2, Q4 = 1 << Q4_LOG;
    const int groups = (ncol + DW_T - 1) / DW_T;
    const int units = nrow * groups << Q4_LOG;
    const int row_step = g.dh * pitch * CC;                        // floats between two filter rows
    // unit order: channel quad fastest, then the row, then the column group.  The eight threads of a quarter warp (one
    // shared-memory access phase of 16-byte reads) are then the quads of 8 / Q4 consecutive rows; with the padded row
    // pitch they fall into eight different groups of four banks for a row stride of one.
    for (int i = tid; i < units; i += NTHREADS) {
        const int c4 = i & (Q4 - 1), gi = i >> Q4_LOG;
        const int grp = gi / nrow, r = gi - grp * nrow, owl = grp * DW_T;
        const float *xa = xs + ((size_t)(r * g.sh) * pitch + owl) * CC + c4 * 4;
        const float *wa = wsm + c4 * 4;
        f32x2 acc[DW_T][2];
#pragma unroll
        for (int t = 0; t < DW_T; ++t) acc[t][0] = acc[t][1] = 0ull;               // (+0, +0)
        for (int a = 0; a < g.kh; ++a, xa += row_step, wa += KW * CC) {
            f32x2 xw[DW_T + KW - 1][2];
#pragma unroll
            for (int j = 0; j < DW_T + KW - 1; ++j) {
                const float4 q = *reinterpret_cast<const float4 *>(xa + j * CC);
                xw[j][0] = pack2(q.x, q.y); xw[j][1] = pack2(q.z, q.w);
            }
#pragma unroll
            for (int b = 0; b < KW; ++b) {
                const float4 wv = *reinterpret_cast<const float4 *>(wa + b * CC);
                const f32x2 w0 = pack2(wv.x, wv.y), w1 = pack2(wv.z, wv.w);
#pragma unroll
                for (int t = 0; t < DW_T; ++t) {
                    fma2(acc[t][0], xw[t + b][0], w0);
                    fma2(acc[t][1], xw[t + b][1], w1);
                }
            }
        }
        const int c = c0 + c4 * 4;
        const float4 sc = dw_load4(g.scale, c, 1.0f), sf = dw_load4(g.shift, c, 0.0f);
        const long long o = (((long long)n * g.Ho + oh0 + r) * g.Wo + ow0 + owl) * g.C + c;
        const bool smooth = g.act > LOP_ACT_RELU;
#pragma unroll
        for (int t = 0; t < DW_T; ++t)
            if (owl + t < ncol) {
                float a4[4];
                unpack2(acc[t][0], a4[0], a4[1]);
                unpack2(acc[t][1], a4[2], a4[3]);
                if (smooth) dw_store4<THROUGH_L2, true>(g, o + (long long)t * g.C, sc, sf, a4);
                else dw_store4<THROUGH_L2, false>(g, o + (long long)t * g.C, sc, sf, a4);
            }
    }
}
template <bool THROUGH_L2, int KW, int NTHREADS>
__device__ __forceinline__ void dw_walk_sliding_cc(const DwGeom &g, int n, int oh0, int nrow, int ow0, int ncol, int c0, const float *xs,
                                                   const float *wsm, int pitch, int cc_log, int tid)
{
    if (cc_log == 3) dw_walk_sliding<THROUGH_L2, KW, 3, NTHREADS>(g, n, oh0, nrow, ow0, ncol, c0, xs, wsm, pitch, tid);
    else if (cc_log == 4) dw_walk_sliding<THROUGH_L2, KW, 4, NTHREADS>(g, n, oh0, nrow, ow0, ncol, c0, xs, wsm, pitch, tid);
    else dw_walk_sliding<THROUGH_L2, KW, 5, NTHREADS>(g, n, oh0, nrow, ow0, ncol, c0, xs, wsm, pitch, tid);
}

// Rows [oh0, oh0 + nrow), columns [ow0, ow0 + ncol), channels [c0, c0 + cc) of image n.  THROUGH_L2: the input and
// the residual may have been written by other SMs during this launch: read around L1.  sm: dw_tile_bytes() bytes,
// 16-byte aligned.
template <bool THROUGH_L2, int BAR_ID, int NTHREADS>
__device__ __forceinline__ void dwconv_tile(const DwGeom &g, int n, int oh0, int nrow, int ow0, int ncol, int c0, float *sm, int tid)
{
    const int cc = g.t.cc, cc_log = 31 - __clz(cc);
    const int rows_in = (nrow - 1) * g.sh + (g.kh - 1) * g.dh + 1, cols_in = dw_cols_in(ncol, g.kw, g.sw, g.dw);
    const int pitch = dw_pitch(cols_in, cc);
    const int ih0 = oh0 * g.sh - g.ph, iw0 = ow0 * g.sw - g.pw;
    float *xs = sm, *wsm = sm + ((size_t)rows_in * pitch << cc_log);
    const int v8_log = cc_log - 3, v8 = 1 << v8_log;                // 16-byte vectors of eight bf16 per pixel / per tap

    // filters of channels [c0, c0 + cc): [tap][cc] fp32
    for (int i = tid; i < (g.kh * g.kw << v8_log); i += NTHREADS) {
        const int t = i >> v8_log, v = i & (v8 - 1);
        float f[8];
        unpack_bf16x8(__ldg(reinterpret_cast<const uint4 *>(g.w_taps + (long long)t * g.C + c0) + v), f);
        float4 *d = reinterpret_cast<float4 *>(wsm + (t << cc_log) + v * 8);
        d[0] = make_float4(f[0], f[1], f[2], f[3]);
        d[1] = make_float4(f[4], f[5], f[6], f[7]);
    }
    // receptive window: [row][pitch][cc] fp32, zeros outside the tensor; four loads in flight per thread
    const int nvec = rows_in * cols_in << v8_log;
    for (int base = 0; base < nvec; base += 4 * NTHREADS) {
        uint4 q[4];
        int dst[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int i = base + u * NTHREADS + tid;
            q[u] = make_uint4(0u, 0u, 0u, 0u);
            dst[u] = -1;
            if (i < nvec) {
                const int v = i & (v8 - 1), pix = i >> v8_log;
                const int r = pix / cols_in, col = pix - r * cols_in;
                const int ih = ih0 + r, iw = iw0 + col;
                dst[u] = ((r * pitch + col) << cc_log) + v * 8;
                const long long xo = (((long long)n * g.Hin + ih) * g.Win + iw) * g.C + c0 + v * 8;
                if (ih >= 0 && ih < g.Hin && iw >= 0 && iw < g.Win && dw_in_bounds<THROUGH_L2>(g, xo, 8, (long long)g.N * g.Hin * g.Win * g.C)) {
                    const uint4 *src = reinterpret_cast<const uint4 *>(g.x + (((long long)n * g.Hin + ih) * g.Win + iw) * g.C + c0) + v;
                    q[u] = THROUGH_L2 ? __ldcg(src) : __ldg(src);
                }
            }
        }
#pragma unroll
        for (int u = 0; u < 4; ++u)
            if (dst[u] >= 0) {
                float f[8];
                unpack_bf16x8(q[u], f);
                float4 *d = reinterpret_cast<float4 *>(xs + dst[u]);
                d[0] = make_float4(f[0], f[1], f[2], f[3]);
                d[1] = make_float4(f[4], f[5], f[6], f[7]);
            }
    }
    tile_barrier<BAR_ID, NTHREADS>();

    if (dw_slides(g.kw, g.sw, g.dw)) {
        if (g.kw == 3) dw_walk_sliding_cc<THROUGH_L2, 3, NTHREADS>(g, n, oh0, nrow, ow0, ncol, c0, xs, wsm, pitch, cc_log, tid);
        else if (g.kw == 5) dw_walk_sliding_cc<THROUGH_L2, 5, NTHREADS>(g, n, oh0, nrow, ow0, ncol, c0, xs, wsm, pitch, cc_log, tid);
        else dw_walk_sliding_cc<THROUGH_L2, 7, NTHREADS>(g, n, oh0, nrow, ow0, ncol, c0, xs, wsm, pitch, cc_log, tid);
        return;
    }
    // any stride, dilation and filter width: one (pixel, four channels) at a time
    const int q4_log = cc_log - 2, q4 = 1 << q4_log;                // channel quads per pixel
    const int units = nrow * ncol << q4_log;
    const int tap_stride = g.dw << cc_log, row_stride = (g.dh * pitch) << cc_log;
    for (int i = tid; i < units; i += NTHREADS) {
        const int c4 = i & (q4 - 1), pix = i >> q4_log;
        const int r = pix / ncol, owl = pix - r * ncol;
        const float *xp = xs + (((size_t)(r * g.sh) * pitch + owl * g.sw) << cc_log) + c4 * 4;
        const float *wp = wsm + c4 * 4;
        float acc[4] = {0.0f, 0.0f, 0.0f, 0.0f};
        for (int a = 0; a < g.kh; ++a) {
            const float *xa = xp + (size_t)a * row_stride;
            const float *wa = wp + ((a * g.kw) << cc_log);
            for (int b = 0; b < g.kw; ++b) {
                const float4 xv = *reinterpret_cast<const float4 *>(xa + (size_t)b * tap_stride);
                const float4 wv = *reinterpret_cast<const float4 *>(wa + (b << cc_log));
                acc[0] = fmaf(xv.x, wv.x, acc[0]); acc[1] = fmaf(xv.y, wv.y, acc[1]);
                acc[2] = fmaf(xv.z, wv.z, acc[2]); acc[3] = fmaf(xv.w, wv.w, acc[3]);
            }
        }
        const int c = c0 + c4 * 4;
        const long long o = (((long long)n * g.Ho + oh0 + r) * g.Wo + ow0 + owl) * g.C + c;
        if (g.act > LOP_ACT_RELU) dw_store4<THROUGH_L2, true>(g, o, dw_load4(g.scale, c, 1.0f), dw_load4(g.shift, c, 0.0f), acc);
        else dw_store4<THROUGH_L2, false>(g, o, dw_load4(g.scale, c, 1.0f), dw_load4(g.shift, c, 0.0f), acc);
    }
}

}  // namespace rowop
}  // namespace lop

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

// Activation in its accurate form (library exp / erf): these operators are bound by memory, not by arithmetic.  The
// transcendental kinds are kept out of line: the tile routines run their epilogue a few times per thread, so what
// they cost is mostly the fetch of their instructions, and inlined copies of exp and erf multiply that.
static __device__ __noinline__ float activate_smooth(float t, int act)
{
    if (act == LOP_ACT_SILU) return t / (1.0f + expf(-t));
    return 0.5f * t * (1.0f + erff(t * 0.70710678f));       // GELU: t * Phi(t)
}
__device__ __forceinline__ float activate(float t, int act)
{
    if (act == LOP_ACT_NONE) return t;
    if (act == LOP_ACT_RELU) return fmaxf(t, 0.0f);
    return activate_smooth(t, act);
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

// ---------------------------------------------------------------------------------------------
// Depth-wise convolution of one tile: R output rows x tw output columns x cc channels of one image, by `NTHREADS`
// threads that share a barrier.  The tile's receptive window and the filters of its channels are put into shared
// memory as fp32 first (every input value is used by up to kh*kw taps: converting it once, not per tap, and leaving
// the bounds checks to the staging step -- taps outside the tensor read zeros -- more than halves the instructions
// per multiply-add), then every thread walks the taps of one (pixel, four channels) at a time, a = 0..kh-1,
// b = 0..kw-1, whatever the tile: a pixel's bits do not depend on the tile or the band it is computed in.
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
};

constexpr int DW_T = 4;               // adjacent output columns one thread computes on the sliding-window path

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

// Pixels between the starts of two rows of the staged window: the columns, padded so that a row's pitch in bytes is
// cc * 4 more than a multiple of 128.  Threads that differ in the row then read different shared-memory banks (see
// dw_walk_sliding).
__host__ __device__ inline int dw_pitch(int cols_in, int cc)
{
    const int m = 32 / cc;                                 // cc = 8, 16, 32: pitch = 1 modulo 4, 2, 1
    return m <= 1 ? cols_in : (cols_in + m - 2) / m * m + 1;
}

// Shared memory one tile needs (window + filters), in bytes.
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
        for (int R = 1; R <= 8; R *= 2)
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

// Epilogue and store of four channels c .. c+3 of output pixel (n, oh, ow).
template <bool THROUGH_L2>
__device__ __forceinline__ void dw_store4(const DwGeom &g, int n, int oh, int ow, int c, const float (&acc)[4])
{
    const long long o = (((long long)n * g.Ho + oh) * g.Wo + ow) * g.C + c;
    float rf[4] = {0.0f, 0.0f, 0.0f, 0.0f};
    if (g.res) {
        const uint2 *src = reinterpret_cast<const uint2 *>(g.res + o);
        const uint2 rq = THROUGH_L2 ? __ldcg(src) : __ldg(src);
        rf[0] = __uint_as_float(rq.x << 16); rf[1] = __uint_as_float(rq.x & 0xFFFF0000u);
        rf[2] = __uint_as_float(rq.y << 16); rf[3] = __uint_as_float(rq.y & 0xFFFF0000u);
    }
    const float4 sc = g.scale ? __ldg(reinterpret_cast<const float4 *>(g.scale + c)) : make_float4(1.0f, 1.0f, 1.0f, 1.0f);
    const float4 sf = g.shift ? __ldg(reinterpret_cast<const float4 *>(g.shift + c)) : make_float4(0.0f, 0.0f, 0.0f, 0.0f);
    const float v0 = epilogue(acc[0], sc.x, sf.x, rf[0], g.res_pos, g.act), v1 = epilogue(acc[1], sc.y, sf.y, rf[1], g.res_pos, g.act);
    const float v2 = epilogue(acc[2], sc.z, sf.z, rf[2], g.res_pos, g.act), v3 = epilogue(acc[3], sc.w, sf.w, rf[3], g.res_pos, g.act);
    uint2 out;
    out.x = (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(v0)) | ((uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(v1)) << 16);
    out.y = (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(v2)) | ((uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(v3)) << 16);
    *reinterpret_cast<uint2 *>(g.y + o) = out;
}

// Sliding-window walk of a staged tile (stride 1, dilation 1 along the width, KW known at compile time): a thread owns
// DW_T adjacent output columns of one row and four channels.  Per filter row it loads the DW_T + KW - 1 input values
// those outputs read once, then one weight vector per tap.  Every output still sums its taps in the order a = 0..kh-1,
// b = 0..KW-1, like the one-pixel walk.
template <bool THROUGH_L2, int KW, int NTHREADS>
__device__ __forceinline__ void dw_walk_sliding(const DwGeom &g, int n, int oh0, int nrow, int ow0, int ncol, int c0, const float *xs,
                                                const float *wsm, int pitch, int cc_log, int tid)
{
    const int q4_log = cc_log - 2, q4 = 1 << q4_log;
    const int groups = (ncol + DW_T - 1) / DW_T;
    const int units = nrow * groups << q4_log;
    // unit order: channel quad fastest, then the row, then the column group.  The eight threads of a quarter warp
    // (one shared-memory access phase) are then the quads of 8 / q4 consecutive rows; with the padded row pitch their
    // 16-byte reads fall into eight different bank groups for a row stride of one.
    for (int i = tid; i < units; i += NTHREADS) {
        const int c4 = i & (q4 - 1), gi = i >> q4_log;
        const int grp = gi / nrow, r = gi - grp * nrow, owl = grp * DW_T;
        const float *xp = xs + (((size_t)(r * g.sh) * pitch + owl) << cc_log) + c4 * 4;
        const float *wp = wsm + c4 * 4;
        float4 acc[DW_T];
#pragma unroll
        for (int t = 0; t < DW_T; ++t) acc[t] = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
        for (int a = 0; a < g.kh; ++a) {
            const float *xa = xp + (((size_t)a * g.dh * pitch) << cc_log);
            const float *wa = wp + ((a * KW) << cc_log);
            float4 xw[DW_T + KW - 1];
#pragma unroll
            for (int j = 0; j < DW_T + KW - 1; ++j) xw[j] = *reinterpret_cast<const float4 *>(xa + ((size_t)j << cc_log));
#pragma unroll
            for (int b = 0; b < KW; ++b) {
                const float4 wv = *reinterpret_cast<const float4 *>(wa + (b << cc_log));
#pragma unroll
                for (int t = 0; t < DW_T; ++t) {
                    acc[t].x = fmaf(xw[t + b].x, wv.x, acc[t].x); acc[t].y = fmaf(xw[t + b].y, wv.y, acc[t].y);
                    acc[t].z = fmaf(xw[t + b].z, wv.z, acc[t].z); acc[t].w = fmaf(xw[t + b].w, wv.w, acc[t].w);
                }
            }
        }
#pragma unroll
        for (int t = 0; t < DW_T; ++t)
            if (owl + t < ncol) {
                const float a4[4] = {acc[t].x, acc[t].y, acc[t].z, acc[t].w};
                dw_store4<THROUGH_L2>(g, n, oh0 + r, ow0 + owl + t, c0 + c4 * 4, a4);
            }
    }
}

// THROUGH_L2: the input (and the residual) may have been written by other SMs during this launch: read around L1.
// Rows [oh0, oh0 + nrow), columns [ow0, ow0 + ncol), channels [c0, c0 + cc) of image n.
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
    // receptive window: [row][column][cc] fp32, zeros outside the tensor; four loads in flight per thread
    const int nvec = rows_in * cols_in << v8_log;
    for (int base = 0; base < nvec; base += 4 * NTHREADS) {
        uint4 q[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int i = base + u * NTHREADS + tid;
            q[u] = make_uint4(0u, 0u, 0u, 0u);
            if (i < nvec) {
                const int v = i & (v8 - 1), pix = i >> v8_log;
                const int r = pix / cols_in, col = pix - r * cols_in;
                const int ih = ih0 + r, iw = iw0 + col;
                if (ih >= 0 && ih < g.Hin && iw >= 0 && iw < g.Win) {
                    const uint4 *src = reinterpret_cast<const uint4 *>(g.x + (((long long)n * g.Hin + ih) * g.Win + iw) * g.C + c0) + v;
                    q[u] = THROUGH_L2 ? __ldcg(src) : __ldg(src);
                }
            }
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int i = base + u * NTHREADS + tid;
            if (i < nvec) {
                float f[8];
                unpack_bf16x8(q[u], f);
                const int v = i & (v8 - 1), pix = i >> v8_log;
                const int r = pix / cols_in, col = pix - r * cols_in;
                float4 *d = reinterpret_cast<float4 *>(xs + (((size_t)r * pitch + col) << cc_log) + v * 8);
                d[0] = make_float4(f[0], f[1], f[2], f[3]);
                d[1] = make_float4(f[4], f[5], f[6], f[7]);
            }
        }
    }
    tile_barrier<BAR_ID, NTHREADS>();

    if (dw_slides(g.kw, g.sw, g.dw)) {
        if (g.kw == 3) dw_walk_sliding<THROUGH_L2, 3, NTHREADS>(g, n, oh0, nrow, ow0, ncol, c0, xs, wsm, pitch, cc_log, tid);
        else if (g.kw == 5) dw_walk_sliding<THROUGH_L2, 5, NTHREADS>(g, n, oh0, nrow, ow0, ncol, c0, xs, wsm, pitch, cc_log, tid);
        else dw_walk_sliding<THROUGH_L2, 7, NTHREADS>(g, n, oh0, nrow, ow0, ncol, c0, xs, wsm, pitch, cc_log, tid);
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
        dw_store4<THROUGH_L2>(g, n, oh0 + r, ow0 + owl, c0 + c4 * 4, acc);
    }
}

}  // namespace rowop
}  // namespace lop

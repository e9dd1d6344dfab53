// CUDA-core kernels: general convolution (any kernel/stride/padding/dilation/channel count),
// max pooling, patch gather of a thin chain input (the band "split" step), zero-padding of weight rows.
//
// The convolution here is the fp32 path and the fall-back for shapes the tensor-core kernel
// does not take; it is also the library's second on-GPU opinion (LOP_FLAG_FORCE_SIMT).
// Operators: Sec. IV-A of the paper (block-wise and element-wise local operators).
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "lop.h"
#include "lop_kernels.cuh"
#include "lop_gather.cuh"

namespace lop {

namespace {

__device__ __forceinline__ float to_f32(float v) { return v; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 v) { return __bfloat162float(v); }
__device__ __forceinline__ void from_f32(float &d, float v) { d = v; }
__device__ __forceinline__ void from_f32(__nv_bfloat16 &d, float v) { d = __float2bfloat16_rn(v); }

// idx = ((n * rows + r) * Wo + ow) * inner + g, taken apart with 32-bit divisions where the count allows it (a 64-bit
// division is a routine of several dozen instructions: four of them per thread outweigh a light kernel's real work).
__device__ __forceinline__ void split_index(long long idx, long long total, int inner, int Wo, int rows, int &g, int &ow, int &r, int &n)
{
    if (total < (1LL << 31)) {
        unsigned q = (unsigned)idx;
        const unsigned q1 = q / (unsigned)inner; g = (int)(q - q1 * (unsigned)inner);
        const unsigned q2 = q1 / (unsigned)Wo; ow = (int)(q1 - q2 * (unsigned)Wo);
        const unsigned q3 = q2 / (unsigned)rows; r = (int)(q2 - q3 * (unsigned)rows);
        n = (int)q3;
    } else {
        long long q = idx;
        g = (int)(q % inner); q /= inner;
        ow = (int)(q % Wo); q /= Wo;
        r = (int)(q % rows);
        n = (int)(q / rows);
    }
}

__device__ __forceinline__ float activate(float t, int act)
{
    if (act == LOP_ACT_RELU) return fmaxf(t, 0.0f);
    if (act == LOP_ACT_SILU) return t / (1.0f + expf(-t));
    if (act == LOP_ACT_GELU) return 0.5f * t * (1.0f + erff(t * 0.70710678f));
    return t;
}

// ---------------------------------------------------------------------------------------------
// Implicit-GEMM convolution on CUDA cores.  M = N*rows*Wo output pixels, N = Cout, K = kh*kw*Cin.
// 64x64 tile per 256-thread block, 16-wide K slabs staged through shared memory, 4x4 outputs per
// thread.  K is walked in one fixed order, so a pixel's value does not depend on the band it is in.
// ---------------------------------------------------------------------------------------------
constexpr int SM_BK = 16;

// TM: outputs per thread along each tile axis; the tile is (16*TM) pixels x (16*TM) output channels.  TM = 4 for
// layers with enough tiles to fill the machine, TM = 2 (four times as many CTAs) for small ones.  The next K slab's
// operands are loaded into registers while the current slab is multiplied, so a slab costs one barrier pair, not a
// global-memory round trip.  K is walked in ascending order whatever the tile, so a pixel's bits do not depend on it.
template <typename T, int TM>
__global__ void __launch_bounds__(256) conv_simt_kernel(ConvArgs p)
{
    constexpr int BM = 16 * TM, BN = 16 * TM;
    __shared__ float As[SM_BK][BM + 4];
    __shared__ float Bs[SM_BK][BN + 4];

    const T *__restrict__ x = static_cast<const T *>(p.x);
    const T *__restrict__ w = static_cast<const T *>(p.w);
    const int rows = p.oh_hi - p.oh_lo;
    const long long M = (long long)p.N * rows * p.Wo;
    const int K = p.kh * p.kw * p.Cin;
    const long long m0 = (long long)blockIdx.x * BM;
    const int n0 = blockIdx.y * BN;
    const int t = threadIdx.x;
    const long long x_elems = (long long)p.N * p.Hin * p.Win * p.Cin, y_elems = (long long)p.N * p.Ho * p.Wo * p.Cout;
    const int kk = t & 15;              // K index inside the slab this thread stages
    const int lr = t >> 4;              // 0..15: first of the TM tile rows (stride 16) this thread stages

    // the TM pixels / TM output channels whose operands this thread stages
    long long xbase[TM];
    int ih0[TM], iw0[TM];
    bool mvalid[TM];
#pragma unroll
    for (int e = 0; e < TM; ++e) {
        const long long m = m0 + lr + e * 16;
        mvalid[e] = m < M;
        const long long mm = mvalid[e] ? m : 0;
        const int ow = (int)(mm % p.Wo);
        const long long q = mm / p.Wo;
        const int oh = p.oh_lo + (int)(q % rows);
        const int n = (int)(q / rows);
        ih0[e] = oh * p.sh - p.ph;
        iw0[e] = ow * p.sw - p.pw;
        xbase[e] = (long long)n * p.Hin * p.Win * p.Cin;
    }

    const int tx = t & 15, ty = t >> 4;
    float acc[TM][TM];
#pragma unroll
    for (int i = 0; i < TM; ++i)
#pragma unroll
        for (int j = 0; j < TM; ++j) acc[i][j] = 0.0f;

    // this thread's operand values of the K slab starting at k0
    float av[TM], wv[TM];
    auto load_slab = [&](int k0) {
        const int k = k0 + kk;
        const bool kvalid = k < K;
        int ci = 0, a = 0, b = 0;
        if (kvalid) {
            ci = k % p.Cin;
            const int tap = k / p.Cin;
            b = tap % p.kw;
            a = tap / p.kw;
        }
#pragma unroll
        for (int e = 0; e < TM; ++e) {
            float v = 0.0f;
            if (kvalid && mvalid[e]) {
                const int ih = ih0[e] + a * p.dh, iw = iw0[e] + b * p.dw;
                if (ih >= 0 && ih < p.Hin && iw >= 0 && iw < p.Win) {
                    const long long xo = xbase[e] + ((long long)ih * p.Win + iw) * p.Cin + ci;
                    if (dbg_in_bounds(p.dbg, xo, 1, x_elems)) v = to_f32(x[xo]);
                }
            }
            av[e] = v;
            float u = 0.0f;
            const int co = n0 + lr + e * 16;
            if (kvalid && co < p.Cout && dbg_in_bounds(p.dbg, (long long)co * K + k, 1, (long long)p.Cout * K)) u = to_f32(w[(long long)co * K + k]);
            wv[e] = u;
        }
    };
    load_slab(0);
    for (int k0 = 0; k0 < K; k0 += SM_BK) {
#pragma unroll
        for (int e = 0; e < TM; ++e) {
            As[kk][lr + e * 16] = av[e];
            Bs[kk][lr + e * 16] = wv[e];
        }
        __syncthreads();
        if (k0 + SM_BK < K) load_slab(k0 + SM_BK);          // in flight while this slab is multiplied
#pragma unroll
        for (int q = 0; q < SM_BK; ++q) {
            float ar[TM], br[TM];
#pragma unroll
            for (int i = 0; i < TM; ++i) ar[i] = As[q][ty * TM + i];
#pragma unroll
            for (int j = 0; j < TM; ++j) br[j] = Bs[q][tx * TM + j];
#pragma unroll
            for (int i = 0; i < TM; ++i)
#pragma unroll
                for (int j = 0; j < TM; ++j) acc[i][j] = fmaf(ar[i], br[j], acc[i][j]);
        }
        __syncthreads();
    }

    T *__restrict__ y = static_cast<T *>(p.y);
    const T *__restrict__ res = static_cast<const T *>(p.res);
#pragma unroll
    for (int i = 0; i < TM; ++i) {
        const long long m = m0 + ty * TM + i;
        if (m >= M) continue;
        const int ow = (int)(m % p.Wo);
        const long long q = m / p.Wo;
        const int oh = p.oh_lo + (int)(q % rows);
        const int n = (int)(q / rows);
        const long long o = (((long long)n * p.Ho + oh) * p.Wo + ow) * p.Cout;
#pragma unroll
        for (int j = 0; j < TM; ++j) {
            const int co = n0 + tx * TM + j;
            if (co >= p.Cout) continue;
            // the element inside the tensor, the row inside the rows of this launch (tested as a one-row "tensor")
            if (!dbg_in_bounds(p.dbg, o + co, 1, y_elems) || !dbg_in_bounds(p.dbg, oh - p.oh_lo, 1, rows)) continue;
            float v = acc[i][j];
            v = fmaf(p.scale ? p.scale[co] : 1.0f, v, p.shift ? p.shift[co] : 0.0f);
            if (res && p.res_pos == LOP_RES_PRE_ACT) v += to_f32(res[o + co]);
            v = activate(v, p.act);
            if (res && p.res_pos == LOP_RES_POST_ACT) v += to_f32(res[o + co]);
            from_f32(y[o + co], v);
        }
    }
}

// ---------------------------------------------------------------------------------------------
// Max pooling, NHWC.  One thread per (output pixel, group of VEC channels); a warp covers
// consecutive channel groups of consecutive pixels, so loads and stores are 16-byte and coalesced.
// HBM-bound: bytes = rows read once + rows written once.
// ---------------------------------------------------------------------------------------------
template <typename T, int VEC>
struct alignas(sizeof(T) * VEC) Pack {
    T v[VEC];
};

template <typename T, int VEC>
__global__ void __launch_bounds__(256) maxpool_kernel(PoolArgs p)
{
    const int rows = p.oh_hi - p.oh_lo;
    const int cg = p.C / VEC;
    const long long total = (long long)p.N * rows * p.Wo * cg;
    const T *__restrict__ x = static_cast<const T *>(p.x);
    T *__restrict__ y = static_cast<T *>(p.y);
    for (long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
         idx += (long long)gridDim.x * blockDim.x) {
        int g, ow, r, n;
        split_index(idx, total, cg, p.Wo, rows, g, ow, r, n);
        const int oh = p.oh_lo + r;
        float m[VEC];
#pragma unroll
        for (int i = 0; i < VEC; ++i) m[i] = -INFINITY;
        for (int a = 0; a < p.kh; ++a) {
            const int ih = oh * p.sh - p.ph + a * p.dh;
            if (ih < 0 || ih >= p.Hin) continue;
            for (int b = 0; b < p.kw; ++b) {
                const int iw = ow * p.sw - p.pw + b * p.dw;
                if (iw < 0 || iw >= p.Win) continue;
                const long long xo = (((long long)n * p.Hin + ih) * p.Win + iw) * p.C + (long long)g * VEC;
                if (!dbg_in_bounds(p.dbg, xo, VEC, (long long)p.N * p.Hin * p.Win * p.C)) continue;
                const Pack<T, VEC> v = *reinterpret_cast<const Pack<T, VEC> *>(x + xo);
#pragma unroll
                for (int i = 0; i < VEC; ++i) m[i] = fmaxf(m[i], to_f32(v.v[i]));
            }
        }
        Pack<T, VEC> o;
#pragma unroll
        for (int i = 0; i < VEC; ++i) from_f32(o.v[i], m[i]);
        const long long yo = (((long long)n * p.Ho + oh) * p.Wo + ow) * p.C + (long long)g * VEC;
        if (dbg_in_bounds(p.dbg, yo, VEC, (long long)p.N * p.Ho * p.Wo * p.C)) *reinterpret_cast<Pack<T, VEC> *>(y + yo) = o;
    }
}

// bf16, channels a multiple of 8, a KH x KW window known at compile time: every tap's 16-byte load is issued
// before the first maximum is taken (four to nine independent loads in flight per thread), one thread per
// (output pixel, 8-channel group), as many blocks as there is work.
template <int KH, int KW>
__global__ void __launch_bounds__(256) maxpool_bf16x8_kernel(PoolArgs p)
{
    const int rows = p.oh_hi - p.oh_lo;
    const int cg = p.C >> 3;
    const long long total = (long long)p.N * rows * p.Wo * cg;
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= total) return;
    const uint4 *__restrict__ x = static_cast<const uint4 *>(p.x);
    int g, ow, r, n;
    split_index(idx, total, cg, p.Wo, rows, g, ow, r, n);
    const int oh = p.oh_lo + r;
    uint4 v[KH * KW];
    bool ok[KH * KW];
#pragma unroll
    for (int a = 0; a < KH; ++a) {
        const int ih = oh * p.sh - p.ph + a * p.dh;
#pragma unroll
        for (int b = 0; b < KW; ++b) {
            const int iw = ow * p.sw - p.pw + b * p.dw;
            ok[a * KW + b] = ih >= 0 && ih < p.Hin && iw >= 0 && iw < p.Win;
            const long long xo = (((long long)n * p.Hin + ih) * p.Win + iw) * cg + g;           // in 16-byte vectors
            ok[a * KW + b] = ok[a * KW + b] && dbg_in_bounds(p.dbg, xo, 1, (long long)p.N * p.Hin * p.Win * cg);
            if (ok[a * KW + b]) v[a * KW + b] = __ldg(x + xo);
        }
    }
    float m[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) m[i] = -INFINITY;
#pragma unroll
    for (int tpos = 0; tpos < KH * KW; ++tpos)
        if (ok[tpos]) {
            const uint32_t w4[4] = {v[tpos].x, v[tpos].y, v[tpos].z, v[tpos].w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                m[2 * i] = fmaxf(m[2 * i], __uint_as_float(w4[i] << 16));
                m[2 * i + 1] = fmaxf(m[2 * i + 1], __uint_as_float(w4[i] & 0xFFFF0000u));
            }
        }
    uint32_t o[4];
#pragma unroll
    for (int i = 0; i < 4; ++i)                      // the values are bf16 already: dropping the low half is exact
        o[i] = (__float_as_uint(m[2 * i]) >> 16) | (__float_as_uint(m[2 * i + 1]) & 0xFFFF0000u);
    const long long yo = (((long long)n * p.Ho + oh) * p.Wo + ow) * cg + g;
    if (dbg_in_bounds(p.dbg, yo, 1, (long long)p.N * p.Ho * p.Wo * cg)) static_cast<uint4 *>(p.y)[yo] = make_uint4(o[0], o[1], o[2], o[3]);
}

// ---------------------------------------------------------------------------------------------
// Patch gather for a thin chain input, rows [lo, hi) of the patch tensor (see lop_gather.cuh).
// One thread per 16-byte group of eight patch elements: consecutive threads write consecutive
// 16 bytes, reads hit the few image rows of the band in L1/L2.  HBM-bound on the write.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) stem_gather_kernel(const uint16_t *__restrict__ x, uint16_t *__restrict__ y,
                                                          GatherGeom g, int lo, int hi, unsigned *dbg)
{
    const int k8n = g.Kcol >> 3;
    const long long total = (long long)g.N * (hi - lo) * g.Wo * k8n;
    for (long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
         idx += (long long)gridDim.x * blockDim.x) {
        const int k8 = (int)(idx % k8n);
        long long q = idx / k8n;
        const int ow = (int)(q % g.Wo);
        q /= g.Wo;
        const int oh = lo + (int)(q % (hi - lo));
        const int n = (int)(q / (hi - lo));
        const uint4 v = gather8<false>(x, g, n, oh, ow, k8);        // reads in-bounds taps only, by construction of the patch
        const long long yo = (((long long)n * g.Ho + oh) * g.Wo + ow) * g.Kcol + k8 * 8;
        if (dbg_in_bounds(dbg, yo, 8, (long long)g.N * g.Ho * g.Wo * g.Kcol)) *reinterpret_cast<uint4 *>(y + yo) = v;
    }
}

__global__ void pad_weights_kernel(const uint16_t *__restrict__ w, uint16_t *__restrict__ wp, long long rows, int C,
                                   int Cpad)
{
    const long long total = rows * Cpad;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total;
         i += (long long)gridDim.x * blockDim.x) {
        const int c = (int)(i % Cpad);
        const long long r = i / Cpad;
        wp[i] = c < C ? w[r * C + c] : (uint16_t)0;
    }
}

inline int grid_for(long long work_items, int block, int max_blocks = 148 * 8)
{
    long long b = (work_items + block - 1) / block;
    if (b < 1) b = 1;
    if (b > max_blocks) b = max_blocks;
    return (int)b;
}

}  // namespace

cudaError_t launch_conv_simt(const ConvArgs &a, int dtype, cudaStream_t s)
{
    const int rows = a.oh_hi - a.oh_lo;
    if (rows <= 0) return cudaSuccess;
    const long long M = (long long)a.N * rows * a.Wo;
    const long long big_tiles = ((M + 63) / 64) * ((a.Cout + 63) / 64);
    if (big_tiles >= 2 * 148) {
        dim3 grid((unsigned)((M + 63) / 64), (unsigned)((a.Cout + 63) / 64));
        if (dtype == LOP_BF16) conv_simt_kernel<__nv_bfloat16, 4><<<grid, 256, 0, s>>>(a);
        else conv_simt_kernel<float, 4><<<grid, 256, 0, s>>>(a);
    } else {
        dim3 grid((unsigned)((M + 31) / 32), (unsigned)((a.Cout + 31) / 32));
        if (dtype == LOP_BF16) conv_simt_kernel<__nv_bfloat16, 2><<<grid, 256, 0, s>>>(a);
        else conv_simt_kernel<float, 2><<<grid, 256, 0, s>>>(a);
    }
    return cudaGetLastError();
}

cudaError_t launch_maxpool(const PoolArgs &a, int dtype, cudaStream_t s)
{
    const int rows = a.oh_hi - a.oh_lo;
    if (rows <= 0) return cudaSuccess;
    const long long pix = (long long)a.N * rows * a.Wo;
    if (dtype == LOP_BF16) {
        const long long vecs = pix * (a.C / 8);
        const bool aligned = (reinterpret_cast<uintptr_t>(a.x) & 15) == 0 && (reinterpret_cast<uintptr_t>(a.y) & 15) == 0;
        const unsigned blocks = (unsigned)((vecs + 255) / 256);
        if (a.C % 8 == 0 && aligned && vecs < (1LL << 38) && a.kh == 2 && a.kw == 2) maxpool_bf16x8_kernel<2, 2><<<blocks, 256, 0, s>>>(a);
        else if (a.C % 8 == 0 && aligned && vecs < (1LL << 38) && a.kh == 3 && a.kw == 3) maxpool_bf16x8_kernel<3, 3><<<blocks, 256, 0, s>>>(a);
        else if (a.C % 8 == 0) maxpool_kernel<__nv_bfloat16, 8><<<grid_for(pix * (a.C / 8), 256), 256, 0, s>>>(a);
        else maxpool_kernel<__nv_bfloat16, 1><<<grid_for(pix * a.C, 256), 256, 0, s>>>(a);
    } else {
        if (a.C % 4 == 0) maxpool_kernel<float, 4><<<grid_for(pix * (a.C / 4), 256), 256, 0, s>>>(a);
        else maxpool_kernel<float, 1><<<grid_for(pix * a.C, 256), 256, 0, s>>>(a);
    }
    return cudaGetLastError();
}

cudaError_t launch_stem_gather(const void *x, void *y, const GatherGeom &g, int lo, int hi, cudaStream_t s, unsigned *dbg)
{
    if (hi <= lo) return cudaSuccess;
    if (g.Kcol % 8 != 0) return cudaErrorInvalidValue;
    const long long work = (long long)g.N * (hi - lo) * g.Wo * (g.Kcol / 8);
    stem_gather_kernel<<<grid_for(work, 256), 256, 0, s>>>(static_cast<const uint16_t *>(x), static_cast<uint16_t *>(y), g, lo, hi, dbg);
    return cudaGetLastError();
}

cudaError_t launch_pad_weights(const void *w, void *wp, long long rows, int C, int Cpad, cudaStream_t s)
{
    pad_weights_kernel<<<grid_for(rows * Cpad, 256), 256, 0, s>>>(static_cast<const uint16_t *>(w),
                                                                  static_cast<uint16_t *>(wp), rows, C, Cpad);
    return cudaGetLastError();
}

}  // namespace lop

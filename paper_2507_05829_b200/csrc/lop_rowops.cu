// CUDA-core kernels of the local operators that are not dense contractions (Sec. IV-A of the paper): depth-wise
// convolution (block-wise, one small filter per channel), layer normalisation over the channels of a pixel
// (row-wise) and channel concatenation (row-wise, two inputs).  None has more than a few multiply-adds per byte, so
// they stay off the tensor cores: 16-byte vectors along the channels (the innermost, contiguous axis of NHWC),
// consecutive lanes on consecutive vectors, every tensor element read from DRAM once.  The depth-wise convolution in
// bf16 with a multiple of eight channels runs tile by tile out of shared memory (rowop::dwconv_tile, the routine the
// persistent kernel's worker warps run as well); other dtypes and channel counts take the plain kernel below.  Each
// kernel works on output rows [oh_lo, oh_hi) of all N images, like every other layer kernel, and a pixel's
// arithmetic does not depend on the band it is in.
#include <atomic>

#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "lop.h"
#include "lop_kernels.cuh"
#include "lop_rowops.cuh"

namespace lop {

namespace {

__device__ __forceinline__ float to_f32(float v) { return v; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 v) { return __bfloat162float(v); }
__device__ __forceinline__ void from_f32(float &d, float v) { d = v; }
__device__ __forceinline__ void from_f32(__nv_bfloat16 &d, float v) { d = __float2bfloat16_rn(v); }

template <typename T, int VEC>
struct alignas(sizeof(T) * VEC) Vec {
    T v[VEC];
};

// ---------------------------------------------------------------------------------------------
// Depth-wise convolution.  A block owns a chunk of CV*VEC channels and a run of output pixels; it first stages the
// chunk's filters in shared memory as fp32 [tap][channel] (so that the VEC weights a thread needs for a tap are
// contiguous), then every thread walks the taps of its pixels: one VEC-wide activation load and VEC multiply-adds
// per tap, in the fixed order a = 0..kh-1, b = 0..kw-1.
// ---------------------------------------------------------------------------------------------
constexpr int DW_THREADS = 256;

template <typename T, int VEC>
__global__ void __launch_bounds__(DW_THREADS) dwconv_kernel(ConvArgs p, int CV, int pix_per_thread)
{
    extern __shared__ float wsm[];                         // [kh*kw][CV*VEC]
    const int taps = p.kh * p.kw;
    const int CB = CV * VEC;
    const int c0 = blockIdx.y * CB;
    const T *__restrict__ w = static_cast<const T *>(p.w);
    for (int i = threadIdx.x; i < taps * CB; i += DW_THREADS) {
        const int c = i / taps, t = i - c * taps;          // weights are [C][kh][kw]: walk them in memory order
        wsm[t * CB + c] = (c0 + c < p.Cin) ? to_f32(w[(long long)(c0 + c) * taps + t]) : 0.0f;
    }
    __syncthreads();

    const int cv = threadIdx.x % CV;
    const int c = c0 + cv * VEC;
    if (c >= p.Cin) return;
    const int PP = DW_THREADS / CV;                        // pixels the block works on at a time
    const int rows = p.oh_hi - p.oh_lo;
    const long long M = (long long)p.N * rows * p.Wo;
    const T *__restrict__ x = static_cast<const T *>(p.x);
    const T *__restrict__ res = static_cast<const T *>(p.res);
    T *__restrict__ y = static_cast<T *>(p.y);
    const float *wc = wsm + cv * VEC;
    using V = Vec<T, VEC>;

    for (int it = 0; it < pix_per_thread; ++it) {
        const long long m = ((long long)blockIdx.x * pix_per_thread + it) * PP + threadIdx.x / CV;
        if (m >= M) return;
        const int ow = (int)(m % p.Wo);
        const long long q = m / p.Wo;
        const int oh = p.oh_lo + (int)(q % rows);
        const int n = (int)(q / rows);
        float acc[VEC];
#pragma unroll
        for (int j = 0; j < VEC; ++j) acc[j] = 0.0f;
        const int ih0 = oh * p.sh - p.ph, iw0 = ow * p.sw - p.pw;
        for (int a = 0; a < p.kh; ++a) {
            const int ih = ih0 + a * p.dh;
            if (ih < 0 || ih >= p.Hin) continue;
            const T *xr = x + ((long long)n * p.Hin + ih) * p.Win * p.Cin + c;
            const float *wr = wc + a * p.kw * CB;
            for (int b = 0; b < p.kw; ++b) {
                const int iw = iw0 + b * p.dw;
                if (iw < 0 || iw >= p.Win) continue;
                if (!dbg_in_bounds(p.dbg, (xr - x) + (long long)iw * p.Cin, VEC, (long long)p.N * p.Hin * p.Win * p.Cin)) continue;
                const V xv = *reinterpret_cast<const V *>(xr + (long long)iw * p.Cin);
#pragma unroll
                for (int j = 0; j < VEC; ++j) acc[j] = fmaf(to_f32(xv.v[j]), wr[b * CB + j], acc[j]);
            }
        }
        const long long o = (((long long)n * p.Ho + oh) * p.Wo + ow) * p.Cout + c;
        if (!dbg_in_bounds(p.dbg, o, VEC, (long long)p.N * p.Ho * p.Wo * p.Cout)) continue;
        V rv, out;
        if (res) rv = *reinterpret_cast<const V *>(res + o);
        const int res_pos = res ? p.res_pos : LOP_RES_NONE;
#pragma unroll
        for (int j = 0; j < VEC; ++j)
            from_f32(out.v[j], rowop::epilogue(acc[j], p.scale ? p.scale[c + j] : 1.0f, p.shift ? p.shift[c + j] : 0.0f,
                                               res ? to_f32(rv.v[j]) : 0.0f, res_pos, p.act));
        *reinterpret_cast<V *>(y + o) = out;
    }
}

// bf16 with a multiple of eight channels: one block per tile, the same tile routine the persistent kernel runs
// (rowop::dwconv_tile), so that both executors give the same bits.  w_taps: the filters as [tap][C].
constexpr int DW_TILE_THREADS = 256;
constexpr long long DW_TILE_SMEM = 64 * 1024;          // three blocks per SM (with at most 85 registers a thread): measured 6 % faster than two of 96 KB

__global__ void __launch_bounds__(DW_TILE_THREADS, 3) dwconv_tile_kernel(rowop::DwGeom g, int oh_lo, int oh_hi, int tiles_w)
{
    extern __shared__ float dw_sm[];
    const int tile_w = blockIdx.x % tiles_w, tile_c = blockIdx.x / tiles_w;
    const int oh0 = oh_lo + blockIdx.y * g.t.R, ow0 = tile_w * g.t.tw;
    rowop::dwconv_tile<false, 0, DW_TILE_THREADS>(g, blockIdx.z, oh0, min(g.t.R, oh_hi - oh0), ow0, min(g.t.tw, g.Wo - ow0), tile_c * g.t.cc,
                                                  dw_sm, threadIdx.x);
}

// ---------------------------------------------------------------------------------------------
// Layer normalisation: a group of lanes per pixel (a whole warp from 32 vectors per pixel on, a power-of-two part of
// it below), lane `sub` owning every lanes-th vector.  Mean, then the biased variance of the centred values (two
// passes, the numerically safe order), then the scaled and shifted result; the second and third pass re-read the
// pixel's channel vector from L1.  Partial sums are combined by a fixed butterfly, the same for every pixel.
// ---------------------------------------------------------------------------------------------
template <typename T, int VEC>
__global__ void __launch_bounds__(256) layernorm_kernel(ConvArgs p)
{
    const int rows = p.oh_hi - p.oh_lo;
    const long long M = (long long)p.N * rows * p.Wo;
    const int C = p.Cin, nvec = C / VEC;
    const int lanes_log = rowop::ln_lanes_log(nvec), lanes = 1 << lanes_log;
    const int sub = threadIdx.x & (lanes - 1);
    const long long m = (long long)blockIdx.x * (blockDim.x >> lanes_log) + (threadIdx.x >> lanes_log);
    const bool live0 = m < M;                              // dead lanes still take part in the group sums
    long long o = 0;
    if (live0) {
        const int ow = (int)(m % p.Wo);
        const long long q = m / p.Wo;
        const int oh = p.oh_lo + (int)(q % rows);
        const int n = (int)(q / rows);
        o = (((long long)n * p.Ho + oh) * p.Wo + ow) * C;
    }
    const bool live = live0 && dbg_in_bounds(p.dbg, o, C, (long long)p.N * p.Ho * p.Wo * C);
    const T *__restrict__ x = static_cast<const T *>(p.x) + o;
    T *__restrict__ y = static_cast<T *>(p.y) + o;
    using V = Vec<T, VEC>;

    float s = 0.0f;
    for (int v = sub; live && v < nvec; v += lanes) {
        const V xv = *reinterpret_cast<const V *>(x + v * VEC);
#pragma unroll
        for (int j = 0; j < VEC; ++j) s += to_f32(xv.v[j]);
    }
    const float mean = rowop::group_sum(s, lanes_log) / (float)C;
    float s2 = 0.0f;
    for (int v = sub; live && v < nvec; v += lanes) {
        const V xv = *reinterpret_cast<const V *>(x + v * VEC);
#pragma unroll
        for (int j = 0; j < VEC; ++j) {
            const float d = to_f32(xv.v[j]) - mean;
            s2 = fmaf(d, d, s2);
        }
    }
    const float inv = rowop::ln_inv_std(rowop::group_sum(s2, lanes_log), C);
    for (int v = sub; live && v < nvec; v += lanes) {
        const V xv = *reinterpret_cast<const V *>(x + v * VEC);
        V out;
#pragma unroll
        for (int j = 0; j < VEC; ++j) {
            const int c = v * VEC + j;
            from_f32(out.v[j], rowop::ln_value(to_f32(xv.v[j]), mean, inv, p.scale ? p.scale[c] : 1.0f, p.shift ? p.shift[c] : 0.0f));
        }
        *reinterpret_cast<V *>(y + v * VEC) = out;
    }
}

// ---------------------------------------------------------------------------------------------
// Channel concatenation: y[pixel] = x[pixel] (Ca channels) followed by second[pixel] (Cb channels).  One thread per
// VEC-wide vector of the output.
// ---------------------------------------------------------------------------------------------
template <typename T, int VEC>
__global__ void __launch_bounds__(256) concat_kernel(ConvArgs p)
{
    const int rows = p.oh_hi - p.oh_lo;
    const int Ca = p.Cin, Cb = p.Cout - p.Cin;
    const int va = Ca / VEC, vo = p.Cout / VEC;
    const long long total = (long long)p.N * rows * p.Wo * vo;
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= total) return;
    // vector v of band pixel m; the band's rows * Wo pixels of an image are contiguous in the tensors.  Divisions
    // in 32 bits where the counts are that small (64-bit division is a long routine).
    const long long band = (long long)rows * p.Wo;
    long long m, n, rem;
    int v;
    if (total < (1LL << 31)) {
        const unsigned m32 = (unsigned)i / (unsigned)vo, n32 = m32 / (unsigned)band;
        v = (int)((unsigned)i - m32 * (unsigned)vo);
        m = m32; n = n32; rem = m32 - n32 * (unsigned)band;
    } else {
        m = i / vo; v = (int)(i - m * vo);
        n = m / band; rem = m - n * band;
    }
    const long long pix = n * p.Ho * p.Wo + (long long)p.oh_lo * p.Wo + rem;
    const long long pixels = (long long)p.N * p.Ho * p.Wo;
    if (!dbg_in_bounds(p.dbg, pix, 1, pixels) || v < 0 || v >= vo) return;       // every offset below is pix * channels + v * VEC
    using V = Vec<T, VEC>;
    const V val = v < va ? *reinterpret_cast<const V *>(static_cast<const T *>(p.x) + pix * Ca + (long long)v * VEC)
                         : *reinterpret_cast<const V *>(static_cast<const T *>(p.res) + pix * Cb + (long long)(v - va) * VEC);
    *reinterpret_cast<V *>(static_cast<T *>(p.y) + pix * p.Cout + (long long)v * VEC) = val;
}

// [C][taps] -> [taps][C] (16-bit elements): the persistent kernel reads a tap's weights of eight channels as one vector.
__global__ void __launch_bounds__(256) dw_transpose_kernel(const uint16_t *__restrict__ w, uint16_t *__restrict__ wt, int C, int taps)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= C * taps) return;
    const int t = i / C, c = i - t * C;
    wt[i] = w[(long long)c * taps + t];
}

template <typename T>
constexpr int full_vec() { return 16 / (int)sizeof(T); }

template <typename T, int VEC>
cudaError_t dwconv_launch(const ConvArgs &a, cudaStream_t s)
{
    const int taps = a.kh * a.kw;
    int CV = 1;
    while (CV < 32 && CV * VEC < a.Cin && (size_t)taps * (CV * 2) * VEC * sizeof(float) <= 48u * 1024u) CV *= 2;
    const size_t smem = (size_t)taps * CV * VEC * sizeof(float);
    if (smem > 48u * 1024u) return cudaErrorInvalidValue;
    const int PP = DW_THREADS / CV;
    const long long M = (long long)a.N * (a.oh_hi - a.oh_lo) * a.Wo;
    // several pixels per thread pay the filter staging off, as long as that leaves a few blocks for every SM
    const unsigned chunks = (unsigned)((a.Cin + CV * VEC - 1) / (CV * VEC));
    long long ppt = M * chunks / ((long long)PP * 148 * 4);
    ppt = ppt < 1 ? 1 : (ppt > 8 ? 8 : ppt);
    const long long per_block = (long long)PP * ppt;
    dim3 grid((unsigned)((M + per_block - 1) / per_block), chunks);
    dwconv_kernel<T, VEC><<<grid, DW_THREADS, smem, s>>>(a, CV, (int)ppt);
    return cudaGetLastError();
}

template <typename T>
cudaError_t dwconv_dispatch(const ConvArgs &a, cudaStream_t s)
{
    if (a.Cin % full_vec<T>() == 0) return dwconv_launch<T, full_vec<T>()>(a, s);
    return dwconv_launch<T, 1>(a, s);
}

// bf16 with a multiple of eight channels, at most 1024: the routine the persistent kernel runs (rowop::ln_pixels),
// 4 / VPL pixels per lane group.
template <int VPL>
__global__ void __launch_bounds__(256) layernorm_bf16_kernel(ConvArgs p)
{
    constexpr int PPG = 4 / VPL;
    const int rows = p.oh_hi - p.oh_lo;
    const long long M = (long long)p.N * rows * p.Wo;
    const int C = p.Cin;
    const int lanes_log = rowop::ln_lanes_log(C >> 3);
    const int sub = threadIdx.x & ((1 << lanes_log) - 1);
    const long long group = (long long)blockIdx.x * (256 >> lanes_log) + (threadIdx.x >> lanes_log);
    long long o[PPG];
    bool live[PPG];
    // pixel m of the band is pixel (m mod band) of image m / band, band = rows * Wo pixels that are contiguous in the
    // tensor: one division per pixel, in 32 bits where the band is that small (64-bit division is a long routine)
    const long long band = (long long)rows * p.Wo, image = (long long)p.Ho * p.Wo, first = (long long)p.oh_lo * p.Wo;
#pragma unroll
    for (int q = 0; q < PPG; ++q) {
        const long long m = group * PPG + q;
        live[q] = m < M;
        o[q] = 0;
        if (live[q]) {
            long long n, rem;
            if (M < (1LL << 31)) {
                const unsigned n32 = (unsigned)m / (unsigned)band;
                n = n32; rem = (unsigned)m - n32 * (unsigned)band;
            } else {
                n = m / band; rem = m - n * band;
            }
            o[q] = (n * image + first + rem) * C;
            live[q] = dbg_in_bounds(p.dbg, o[q], C, (long long)p.N * image * C);
        }
    }
    rowop::ln_pixels<false, VPL, PPG>(static_cast<const uint16_t *>(p.x), static_cast<uint16_t *>(p.y), C, lanes_log, sub, o, live, p.scale, p.shift);
}

template <int VPL>
cudaError_t layernorm_bf16_launch(const ConvArgs &a, cudaStream_t s)
{
    const long long M = (long long)a.N * (a.oh_hi - a.oh_lo) * a.Wo;
    const long long per_block = (long long)(256 >> rowop::ln_lanes_log(a.Cin >> 3)) * (4 / VPL);
    layernorm_bf16_kernel<VPL><<<(unsigned)((M + per_block - 1) / per_block), 256, 0, s>>>(a);
    return cudaGetLastError();
}

template <typename T, int VEC>
cudaError_t layernorm_launch(const ConvArgs &a, cudaStream_t s)
{
    const long long M = (long long)a.N * (a.oh_hi - a.oh_lo) * a.Wo;
    const int per_block = 256 >> rowop::ln_lanes_log(a.Cin / VEC);
    layernorm_kernel<T, VEC><<<(unsigned)((M + per_block - 1) / per_block), 256, 0, s>>>(a);
    return cudaGetLastError();
}

template <typename T>
cudaError_t layernorm_dispatch(const ConvArgs &a, cudaStream_t s)
{
    if (a.Cin % full_vec<T>() == 0) return layernorm_launch<T, full_vec<T>()>(a, s);
    return layernorm_launch<T, 1>(a, s);
}

template <typename T, int VEC>
cudaError_t concat_launch(const ConvArgs &a, cudaStream_t s)
{
    const long long total = (long long)a.N * (a.oh_hi - a.oh_lo) * a.Wo * (a.Cout / VEC);
    concat_kernel<T, VEC><<<(unsigned)((total + 255) / 256), 256, 0, s>>>(a);
    return cudaGetLastError();
}

template <typename T>
cudaError_t concat_dispatch(const ConvArgs &a, cudaStream_t s)
{
    constexpr int FV = full_vec<T>();
    if (a.Cin % FV == 0 && a.Cout % FV == 0) return concat_launch<T, FV>(a, s);
    return concat_launch<T, 1>(a, s);
}

}  // namespace

cudaError_t launch_dwconv(const ConvArgs &a, int dtype, const void *w_taps, cudaStream_t s)
{
    if (a.oh_hi <= a.oh_lo) return cudaSuccess;
    rowop::DwTile t;
    if (dtype == LOP_BF16 && w_taps && a.N <= 65535 &&
        rowop::dw_choose_tile(a.kh, a.kw, a.sh, a.sw, a.dh, a.dw, a.N, a.oh_hi - a.oh_lo, a.Wo, a.Cin, DW_TILE_SMEM, DW_TILE_THREADS, &t)) {
        rowop::DwGeom g;
        g.Hin = a.Hin; g.Win = a.Win; g.C = a.Cin; g.Ho = a.Ho; g.Wo = a.Wo;
        g.kh = a.kh; g.kw = a.kw; g.sh = a.sh; g.sw = a.sw; g.ph = a.ph; g.pw = a.pw; g.dh = a.dh; g.dw = a.dw;
        g.act = a.act; g.res_pos = a.res ? a.res_pos : LOP_RES_NONE;
        g.t = t;
        g.x = static_cast<const uint16_t *>(a.x); g.res = static_cast<const uint16_t *>(a.res);
        g.w_taps = static_cast<const uint16_t *>(w_taps);
        g.scale = a.scale; g.shift = a.shift; g.y = static_cast<uint16_t *>(a.y);
        g.dbg = a.dbg; g.N = a.N;
        const int tiles_w = (a.Wo + t.tw - 1) / t.tw, tiles_r = (a.oh_hi - a.oh_lo + t.R - 1) / t.R;
        if (tiles_r <= 65535) {
            static std::atomic<bool> configured[64];     // the shared-memory limit is an attribute per device (set once; idempotent)
            int dev = 0;
            cudaError_t e = cudaGetDevice(&dev);
            if (e != cudaSuccess) return e;
            if (dev < 0 || dev >= 64 || !configured[dev].load(std::memory_order_acquire)) {
                e = cudaFuncSetAttribute(dwconv_tile_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)DW_TILE_SMEM);
                if (e != cudaSuccess) return e;
                if (dev >= 0 && dev < 64) configured[dev].store(true, std::memory_order_release);
            }
            dim3 grid((unsigned)(tiles_w * (a.Cin / t.cc)), (unsigned)tiles_r, (unsigned)a.N);
            dwconv_tile_kernel<<<grid, DW_TILE_THREADS, (size_t)rowop::dw_tile_bytes(a.kh, a.kw, a.sh, a.sw, a.dh, a.dw, t), s>>>(g, a.oh_lo, a.oh_hi, tiles_w);
            return cudaGetLastError();
        }
    }
    return dtype == LOP_BF16 ? dwconv_dispatch<__nv_bfloat16>(a, s) : dwconv_dispatch<float>(a, s);
}

cudaError_t launch_dw_transpose(const void *w, void *wt, int C, int taps, cudaStream_t s)
{
    dw_transpose_kernel<<<(unsigned)((C * taps + 255) / 256), 256, 0, s>>>(static_cast<const uint16_t *>(w), static_cast<uint16_t *>(wt), C, taps);
    return cudaGetLastError();
}

cudaError_t launch_layernorm(const ConvArgs &a, int dtype, cudaStream_t s)
{
    if (a.oh_hi <= a.oh_lo) return cudaSuccess;
    if (dtype == LOP_BF16 && a.Cin % 8 == 0 && a.Cin <= 1024) {
        const int vpl = rowop::ln_vpl(a.Cin >> 3);
        return vpl == 1 ? layernorm_bf16_launch<1>(a, s) : (vpl == 2 ? layernorm_bf16_launch<2>(a, s) : layernorm_bf16_launch<4>(a, s));
    }
    return dtype == LOP_BF16 ? layernorm_dispatch<__nv_bfloat16>(a, s) : layernorm_dispatch<float>(a, s);
}

cudaError_t launch_concat(const ConvArgs &a, int dtype, cudaStream_t s)
{
    if (a.oh_hi <= a.oh_lo) return cudaSuccess;
    return dtype == LOP_BF16 ? concat_dispatch<__nv_bfloat16>(a, s) : concat_dispatch<float>(a, s);
}

}  // namespace lop

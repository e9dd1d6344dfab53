// CUDA-core kernels of the local operators that are not dense contractions (Sec. IV-A of the paper): depth-wise
// convolution (block-wise, one small filter per channel), layer normalisation over the channels of a pixel
// (row-wise) and channel concatenation (row-wise, two inputs).  All three are bound by memory traffic -- a few
// multiply-adds per byte at most -- so they run on plain loads: 16-byte vectors along the channels (the innermost,
// contiguous axis of NHWC), consecutive lanes on consecutive vectors, every tensor element read from DRAM once
// (neighbouring windows of the depth-wise filter overlap in L1/L2).  Each works on output rows [oh_lo, oh_hi) of
// all N images, like every other layer kernel, and a pixel's arithmetic does not depend on the band it is in.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "lop.h"
#include "lop_kernels.cuh"

namespace lop {

namespace {

__device__ __forceinline__ float to_f32(float v) { return v; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 v) { return __bfloat162float(v); }
__device__ __forceinline__ void from_f32(float &d, float v) { d = v; }
__device__ __forceinline__ void from_f32(__nv_bfloat16 &d, float v) { d = __float2bfloat16_rn(v); }

__device__ __forceinline__ float activate(float t, int act)
{
    if (act == LOP_ACT_RELU) return fmaxf(t, 0.0f);
    if (act == LOP_ACT_SILU) return t / (1.0f + expf(-t));
    if (act == LOP_ACT_GELU) return 0.5f * t * (1.0f + erff(t * 0.70710678f));
    return t;
}

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
                const V xv = *reinterpret_cast<const V *>(xr + (long long)iw * p.Cin);
#pragma unroll
                for (int j = 0; j < VEC; ++j) acc[j] = fmaf(to_f32(xv.v[j]), wr[b * CB + j], acc[j]);
            }
        }
        const long long o = (((long long)n * p.Ho + oh) * p.Wo + ow) * p.Cout + c;
        V rv, out;
        if (res) rv = *reinterpret_cast<const V *>(res + o);
#pragma unroll
        for (int j = 0; j < VEC; ++j) {
            float v = fmaf(p.scale ? p.scale[c + j] : 1.0f, acc[j], p.shift ? p.shift[c + j] : 0.0f);
            if (res && p.res_pos == LOP_RES_PRE_ACT) v += to_f32(rv.v[j]);
            v = activate(v, p.act);
            if (res && p.res_pos == LOP_RES_POST_ACT) v += to_f32(rv.v[j]);
            from_f32(out.v[j], v);
        }
        *reinterpret_cast<V *>(y + o) = out;
    }
}

// ---------------------------------------------------------------------------------------------
// Layer normalisation: one warp per pixel.  Mean, then the biased variance of the centred values (two passes, the
// numerically safe order), then the scaled and shifted result; the second and third pass re-read the pixel's
// channel vector from L1.  Partial sums are combined lane-wise by a fixed butterfly, the same for every pixel.
// ---------------------------------------------------------------------------------------------
constexpr float LAYERNORM_EPS = 1e-6f;

__device__ __forceinline__ float warp_sum(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

template <typename T, int VEC>
__global__ void __launch_bounds__(256) layernorm_kernel(ConvArgs p)
{
    const int rows = p.oh_hi - p.oh_lo;
    const long long M = (long long)p.N * rows * p.Wo;
    const long long m = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (m >= M) return;
    const int lane = threadIdx.x & 31;
    const int C = p.Cin;
    const int ow = (int)(m % p.Wo);
    const long long q = m / p.Wo;
    const int oh = p.oh_lo + (int)(q % rows);
    const int n = (int)(q / rows);
    const long long o = (((long long)n * p.Ho + oh) * p.Wo + ow) * C;
    const T *__restrict__ x = static_cast<const T *>(p.x) + o;
    T *__restrict__ y = static_cast<T *>(p.y) + o;
    using V = Vec<T, VEC>;

    float s = 0.0f;
    for (int c = lane * VEC; c < C; c += 32 * VEC) {
        const V xv = *reinterpret_cast<const V *>(x + c);
#pragma unroll
        for (int j = 0; j < VEC; ++j) s += to_f32(xv.v[j]);
    }
    const float mean = warp_sum(s) / (float)C;
    float s2 = 0.0f;
    for (int c = lane * VEC; c < C; c += 32 * VEC) {
        const V xv = *reinterpret_cast<const V *>(x + c);
#pragma unroll
        for (int j = 0; j < VEC; ++j) {
            const float d = to_f32(xv.v[j]) - mean;
            s2 = fmaf(d, d, s2);
        }
    }
    const float inv = 1.0f / sqrtf(warp_sum(s2) / (float)C + LAYERNORM_EPS);
    for (int c = lane * VEC; c < C; c += 32 * VEC) {
        const V xv = *reinterpret_cast<const V *>(x + c);
        V out;
#pragma unroll
        for (int j = 0; j < VEC; ++j) {
            const float g = p.scale ? p.scale[c + j] : 1.0f, b = p.shift ? p.shift[c + j] : 0.0f;
            from_f32(out.v[j], fmaf((to_f32(xv.v[j]) - mean) * inv, g, b));
        }
        *reinterpret_cast<V *>(y + c) = out;
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
    const int v = (int)(i % vo);
    long long q = i / vo;
    const int ow = (int)(q % p.Wo); q /= p.Wo;
    const int oh = p.oh_lo + (int)(q % rows);
    const int n = (int)(q / rows);
    const long long pix = ((long long)n * p.Ho + oh) * p.Wo + ow;
    using V = Vec<T, VEC>;
    const V val = v < va ? *reinterpret_cast<const V *>(static_cast<const T *>(p.x) + pix * Ca + (long long)v * VEC)
                         : *reinterpret_cast<const V *>(static_cast<const T *>(p.res) + pix * Cb + (long long)(v - va) * VEC);
    *reinterpret_cast<V *>(static_cast<T *>(p.y) + pix * p.Cout + (long long)v * VEC) = val;
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

template <typename T>
cudaError_t layernorm_dispatch(const ConvArgs &a, cudaStream_t s)
{
    const long long M = (long long)a.N * (a.oh_hi - a.oh_lo) * a.Wo;
    const unsigned grid = (unsigned)((M + 7) / 8);
    if (a.Cin % full_vec<T>() == 0) layernorm_kernel<T, full_vec<T>()><<<grid, 256, 0, s>>>(a);
    else layernorm_kernel<T, 1><<<grid, 256, 0, s>>>(a);
    return cudaGetLastError();
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

cudaError_t launch_dwconv(const ConvArgs &a, int dtype, cudaStream_t s)
{
    if (a.oh_hi <= a.oh_lo) return cudaSuccess;
    return dtype == LOP_BF16 ? dwconv_dispatch<__nv_bfloat16>(a, s) : dwconv_dispatch<float>(a, s);
}

cudaError_t launch_layernorm(const ConvArgs &a, int dtype, cudaStream_t s)
{
    if (a.oh_hi <= a.oh_lo) return cudaSuccess;
    return dtype == LOP_BF16 ? layernorm_dispatch<__nv_bfloat16>(a, s) : layernorm_dispatch<float>(a, s);
}

cudaError_t launch_concat(const ConvArgs &a, int dtype, cudaStream_t s)
{
    if (a.oh_hi <= a.oh_lo) return cudaSuccess;
    return dtype == LOP_BF16 ? concat_dispatch<__nv_bfloat16>(a, s) : concat_dispatch<float>(a, s);
}

}  // namespace lop

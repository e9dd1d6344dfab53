// Launch interfaces of the device kernels (host-callable wrappers; each returns a cudaError_t).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <cstdint>

namespace lop {

struct ConvArgs {
    const void *x;          // [N, Hin, Win, Cin]
    const void *w;          // [Cout, kh, kw, Cin]
    const float *scale, *shift;
    const void *res;        // [N, Ho, Wo, Cout] or nullptr
    void *y;                // [N, Ho, Wo, Cout]
    int N, Hin, Win, Cin, Ho, Wo, Cout;
    int kh, kw, sh, sw, ph, pw, dh, dw;
    int act, res_pos;
    int oh_lo, oh_hi;       // rows to compute
    unsigned *dbg;          // checked execution: the status word that takes bit 0x100 on a violation, else nullptr
};

struct PoolArgs {
    const void *x;
    void *y;
    int N, Hin, Win, C, Ho, Wo;
    int kh, kw, sh, sw, ph, pw, dh, dw;
    int oh_lo, oh_hi;
    unsigned *dbg;          // as in ConvArgs
};

// Checked execution (LOP_FLAG_DEBUG_BOUNDS): elements [first, first + count) must lie inside a tensor of `limit`
// elements.  Without a status word the test costs one predictable branch.
#ifdef __CUDACC__
__device__ __forceinline__ bool dbg_in_bounds(unsigned *dbg, long long first, long long count, long long limit)
{
    if (!dbg || (first >= 0 && first + count <= limit)) return true;
    atomicOr(dbg, 0x100u);
    return false;
}
#endif

// CUDA-core convolution (fp32 accumulate); dtype: LOP_F32 / LOP_BF16 storage.
cudaError_t launch_conv_simt(const ConvArgs &a, int dtype, cudaStream_t s);
cudaError_t launch_maxpool(const PoolArgs &a, int dtype, cudaStream_t s);
// Depth-wise convolution (w: [C][kh][kw], Cout == Cin), layer normalisation over the channels (scale / shift = gain /
// offset; the window fields are unused) and channel concatenation (x: Cin channels, res: Cout - Cin channels).
// w_taps: the filters as [tap][C] (launch_dw_transpose), or nullptr -- the tiled bf16 kernel needs them.
cudaError_t launch_dwconv(const ConvArgs &a, int dtype, const void *w_taps, cudaStream_t s);
cudaError_t launch_layernorm(const ConvArgs &a, int dtype, cudaStream_t s);
cudaError_t launch_concat(const ConvArgs &a, int dtype, cudaStream_t s);
// depth-wise filters w[C][taps] -> wt[taps][C] (bf16 only), the layout the persistent kernel reads
cudaError_t launch_dw_transpose(const void *w, void *wt, int C, int taps, cudaStream_t s);
// rows [lo,hi) of the patch tensor y[N,Ho,Wo,Kcol] of a thin chain input x[N,H,W,C] (bf16 only).
struct GatherGeom;
// dbg: checked execution's status word (see ConvArgs), or nullptr
cudaError_t launch_stem_gather(const void *x, void *y, const GatherGeom &g, int lo, int hi, cudaStream_t s, unsigned *dbg = nullptr);
// w[rows][C] -> wp[rows][Cpad] zero-padded (bf16 only).
cudaError_t launch_pad_weights(const void *w, void *wp, long long rows, int C, int Cpad, cudaStream_t s);

// cuTensorMapEncodeTiled, looked up through the runtime (no link-time dependency on the driver library); nullptr if absent.
typedef CUresult (*TensorMapEncodeFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                      const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                      CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
TensorMapEncodeFn tensor_map_encoder();

// ---- tcgen05 tensor-core convolution ---------------------------------------------------------
struct ConvTcGeom {
    int TW, TR, TN;         // output tile = TN images x TR rows x TW columns, TW*TR*TN == 128 (powers of two)
    int BN;                 // output channels per CTA (multiple of 16, <= 256)
    int BK;                 // input channels per pipeline stage: 64, 32 or 16
    int stages;
};
struct ConvTcMaps {
    CUtensorMap a[4];       // activation maps, one per (row parity, column parity) of a strided window
    CUtensorMap w;          // weights as a [Cout][kh*kw*Cin] matrix
    int a_valid[4];
};
// Chooses the tile geometry for a layer and a number of rows.  fill_sms: a stand-alone launch prefers
// narrower channel tiles when there are too few pixel tiles to occupy every SM.
ConvTcGeom conv_tc_geometry(const ConvArgs &a, int rows, bool fill_sms = true);
// Encodes the tensor maps for a layer (x, w pointers and geometry are baked in).  Host only.
int conv_tc_encode(const ConvArgs &a, const ConvTcGeom &g, ConvTcMaps *maps);
cudaError_t launch_conv_tc(const ConvArgs &a, const ConvTcGeom &g, const ConvTcMaps &maps, unsigned *status,
                           cudaStream_t s);

}  // namespace lop

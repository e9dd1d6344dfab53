// Patch gather of a thin chain input (the tensor "split" an operator interceptor performs, Sec. III-B
// of the paper, combined with the block-wise operator's receptive field, Sec. IV-A): for every output
// pixel of the first convolution its kh*kw*C input values, in (kh, kw, channel) order, zero where a tap
// falls outside the image and in the tail up to Kcol.  The convolution then is a pointwise product of
// the [N, Ho, Wo, Kcol] patch tensor with the [Cout, Kcol] zero-padded weights.
#pragma once
#include <cuda_runtime.h>
#include <cstdint>

namespace lop {

struct GatherGeom {
    int N, H, W, C;           // chain input
    int Ho, Wo, Kcol;         // patch tensor
    int kh, kw, sh, sw, ph, pw, dh, dw;
};

// Eight consecutive patch elements k8*8 .. k8*8+7 of output pixel (n, oh, ow), as bf16 bit patterns.
// THROUGH_L2: read around L1 (for an input that another engine is still writing while the kernel runs,
// row band by row band; the caller has acquired the band's arrival flag).
template <bool THROUGH_L2>
__device__ __forceinline__ uint4 gather8(const uint16_t *__restrict__ x, const GatherGeom &g, int n, int oh, int ow, int k8)
{
    uint32_t h[8];
    const int klen = g.kh * g.kw * g.C;
    int k = k8 * 8;
    int tap = k / g.C, ci = k - tap * g.C;
    int a = tap / g.kw, b = tap - a * g.kw;
#pragma unroll
    for (int e = 0; e < 8; ++e, ++k) {
        uint32_t v = 0;
        if (k < klen) {
            const int ih = oh * g.sh - g.ph + a * g.dh, iw = ow * g.sw - g.pw + b * g.dw;
            if (ih >= 0 && ih < g.H && iw >= 0 && iw < g.W)
                v = THROUGH_L2 ? __ldcg(x + (((long long)n * g.H + ih) * g.W + iw) * g.C + ci)
                               : __ldg(x + (((long long)n * g.H + ih) * g.W + iw) * g.C + ci);
        }
        h[e] = v;
        if (++ci == g.C) { ci = 0; if (++b == g.kw) { b = 0; ++a; } }
    }
    return make_uint4(h[0] | (h[1] << 16), h[2] | (h[3] << 16), h[4] | (h[5] << 16), h[6] | (h[7] << 16));
}

}  // namespace lop

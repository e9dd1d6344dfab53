// Implicit-GEMM convolution on the 5th-generation tensor cores of sm_100a (bf16 x bf16 -> fp32).
//
// The block-wise local operator of Sec. IV-A of the paper, for one row band: GEMM view
// M = output pixels of the band, N = output channels, K = kh*kw*Cin.  One CTA owns a 128-pixel
// output tile (TN images x TR rows x TW columns) times BN output channels:
//
//   warp 0 (one lane)  TMA producer: per (tap, channel slab) one tiled 4-D box of the NHWC
//                      activation, shifted by the tap, plus one 2-D box of the KRSC weights, into
//                      a ring of shared-memory stages; out-of-bounds box elements are zero-filled
//                      by the TMA unit, which is exactly the convolution's zero padding.
//   warp 1 (one lane)  issues tcgen05.mma (M=128, N=BN, K=16) from the swizzled stages into a
//                      fp32 accumulator in tensor memory; tcgen05.commit hands stages back.
//   warps 2..5         epilogue: tcgen05.ld the accumulator rows (one pixel per thread), apply
//                      scale/shift, residual, activation, round to bf16, 16-byte stores.
//
// A strided window (stride 2) reads every other row/column: the activation is exposed through
// one tensor map per (row parity, column parity) whose base is offset by the parity and whose
// strides are doubled, so each tap is again a dense box.  K is always walked in the order
// (channel slab, kh, kw), whatever the tile position, so a pixel's value does not depend on the
// band that computes it.  Every wait is bounded; a wait that runs out sets the status word.
#include <cuda.h>
#include <atomic>

#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "lop.h"
#include "lop_kernels.cuh"
#include "lop_ptx.cuh"

namespace lop {

namespace {

struct TcParams {
    void *y;
    const void *res;
    const float *scale, *shift;
    unsigned *status;
    int N, Ho, Wo, Cout;
    int oh_lo, oh_hi;
    int tw_log, tr_log;            // TW = 1 << tw_log, TR = 1 << tr_log, TN = 128 >> (tw_log + tr_log)
    int tiles_w, tiles_r;
    int BN, BK, stages;
    int kh, kw, cin;
    int sh, sw, ph, pw, dh, dw;
    int act, res_pos;
    uint32_t a_stage_bytes, b_stage_bytes, tmem_cols;
    uint32_t layout_code, sbo_bytes;
    uint32_t idesc;
};

constexpr int TC_THREADS = 192;

using namespace ptx;

__global__ void __launch_bounds__(TC_THREADS) conv_tc_kernel(const __grid_constant__ ConvTcMaps maps, const TcParams p)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;            // swizzled stages need 1024-byte alignment
    uint8_t *smem = smem_raw + (base - raw);
    const uint32_t stage_bytes = p.a_stage_bytes + p.b_stage_bytes;
    const uint32_t bar_base = base + (uint32_t)p.stages * stage_bytes;
    // barrier area: full[stages], empty[stages], accum, then the TMEM address and the abort flag
    const uint32_t full0 = bar_base, empty0 = bar_base + 8u * p.stages, accum_bar = bar_base + 16u * p.stages;
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(smem + (size_t)p.stages * stage_bytes + 16u * p.stages + 8);
    volatile uint32_t *abort_flag = tmem_slot + 1;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) {
            mbar_init(full0 + 8u * s, 1);
            mbar_init(empty0 + 8u * s, 1);
        }
        mbar_init(accum_bar, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32((const void *)tmem_slot)),
                     "r"(p.tmem_cols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_acc = *tmem_slot;

    // which output tile
    const int TW = 1 << p.tw_log, TR = 1 << p.tr_log;
    const int tile = blockIdx.x;
    const int tile_w = tile % p.tiles_w;
    const int tile_r = (tile / p.tiles_w) % p.tiles_r;
    const int tile_n = tile / (p.tiles_w * p.tiles_r);
    const int ow0 = tile_w << p.tw_log;
    const int oh0 = p.oh_lo + (tile_r << p.tr_log);
    const int n0 = tile_n * (128 >> (p.tw_log + p.tr_log));
    const int co0 = blockIdx.y * p.BN;
    const int slabs = p.cin / p.BK;
    const int n_iter = p.kh * p.kw * slabs;

    if (warp == 0 && lane == 0) {
        // ---------------- TMA producer ----------------
        // K is walked as (channel slab, kh, kw): the order every executor of this library uses, so that a
        // pixel's value does not depend on which of them computed it
        int it = 0;
        for (int c = 0; c < slabs && !*abort_flag; ++c) {
            for (int a = 0; a < p.kh && !*abort_flag; ++a) {
                const int qh = a * p.dh - p.ph;
                const int offh = floor_div_i(qh, p.sh), parh = qh - offh * p.sh;
                for (int b = 0; b < p.kw; ++b, ++it) {
                    const int qw = b * p.dw - p.pw;
                    const int offw = floor_div_i(qw, p.sw), parw = qw - offw * p.sw;
                    const int mi = parh * p.sw + parw;
                    const CUtensorMap *amap = &maps.a[mi];
                    const bool have = maps.a_valid[mi] != 0;
                    const int s = it % p.stages;
                    const uint32_t round = (uint32_t)(it / p.stages);
                    if (round > 0 && !mbar_wait(empty0 + 8u * s, (round - 1) & 1)) {
                        atomicOr(p.status, 1u);
                        *abort_flag = 1;
                        break;
                    }
                    const uint32_t sa = base + (uint32_t)s * stage_bytes, sb = sa + p.a_stage_bytes;
                    const uint32_t fb = full0 + 8u * s;
                    mbar_expect_tx(fb, (uint32_t)(128 * p.BK * 2 + p.BN * p.BK * 2));
                    // a tap whose parity class holds no pixel at all reads only padding: fetch a box that lies
                    // wholly outside the tensor (zero-filled) so the schedule stays uniform
                    tma_load_4d(sa, amap, fb, c * p.BK, have ? ow0 + offw : -65536, have ? oh0 + offh : -65536, n0);
                    tma_load_2d(sb, &maps.w, fb, (a * p.kw + b) * p.cin + c * p.BK, co0);
                }
            }
        }
    } else if (warp == 1 && lane == 0) {
        // ---------------- MMA issuer ----------------
        for (int it = 0; it < n_iter; ++it) {
            const int s = it % p.stages;
            const uint32_t round = (uint32_t)(it / p.stages);
            if (*abort_flag || !mbar_wait(full0 + 8u * s, round & 1)) {
                atomicOr(p.status, 2u);
                *abort_flag = 1;
                break;
            }
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t sa = base + (uint32_t)s * stage_bytes, sb = sa + p.a_stage_bytes;
            for (int k = 0; k < p.BK / 16; ++k) {
                const uint64_t ad = smem_desc(sa + 32u * k, p.sbo_bytes, p.layout_code);
                const uint64_t bd = smem_desc(sb + 32u * k, p.sbo_bytes, p.layout_code);
                umma_bf16(tmem_acc, ad, bd, p.idesc, (it > 0 || k > 0) ? 1u : 0u);
            }
            umma_commit(empty0 + 8u * s);                     // stage reusable once these MMAs retire
        }
        umma_commit(accum_bar);                               // accumulator complete
    } else if (warp >= 2) {
        // ---------------- epilogue ----------------
        const int g = warp & 3;                               // TMEM lane group this warp may read
        const int m = g * 32 + lane;
        const int w_ = m & (TW - 1);
        const int r_ = (m >> p.tw_log) & (TR - 1);
        const int t_ = m >> (p.tw_log + p.tr_log);
        const int ow = ow0 + w_, oh = oh0 + r_, n = n0 + t_;
        const bool valid = ow < p.Wo && oh < p.oh_hi && n < p.N;
        const long long pix = (((long long)n * p.Ho + oh) * p.Wo + ow) * p.Cout + co0;
        bool ok = mbar_wait(accum_bar, 0);
        if (!ok) {
            atomicOr(p.status, 4u);
            *abort_flag = 1;
        }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        if (ok) {
            __nv_bfloat16 *y = static_cast<__nv_bfloat16 *>(p.y);
            const __nv_bfloat16 *res = static_cast<const __nv_bfloat16 *>(p.res);
            for (int j = 0; j < p.BN; j += 16) {
                uint32_t r[16];
                tmem_ld16(tmem_acc + ((uint32_t)(g * 32) << 16) + (uint32_t)j, r);
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                if (!valid) continue;
                float v[16];
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    const int co = co0 + j + i;
                    const float sc = p.scale ? __ldg(p.scale + co) : 1.0f;
                    const float sf = p.shift ? __ldg(p.shift + co) : 0.0f;
                    v[i] = fmaf(sc, __uint_as_float(r[i]), sf);
                }
                float rv[16];
                if (res) {
                    const uint4 q0 = *reinterpret_cast<const uint4 *>(res + pix + j);
                    const uint4 q1 = *reinterpret_cast<const uint4 *>(res + pix + j + 8);
                    const uint32_t rw[8] = {q0.x, q0.y, q0.z, q0.w, q1.x, q1.y, q1.z, q1.w};
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        rv[2 * i] = __uint_as_float(rw[i] << 16);
                        rv[2 * i + 1] = __uint_as_float(rw[i] & 0xFFFF0000u);
                    }
                }
                finish16(v, rv, res ? p.res_pos : LOP_RES_NONE, p.act);
                uint32_t o[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const __nv_bfloat162 h = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
                    o[i] = *reinterpret_cast<const uint32_t *>(&h);
                }
                *reinterpret_cast<uint4 *>(y + pix + j) = make_uint4(o[0], o[1], o[2], o[3]);
                *reinterpret_cast<uint4 *>(y + pix + j + 8) = make_uint4(o[4], o[5], o[6], o[7]);
            }
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_acc), "r"(p.tmem_cols) : "memory");
    }
}

typedef TensorMapEncodeFn EncodeTiledFn;

EncodeTiledFn encode_fn() { return tensor_map_encoder(); }

int ilog2(int v) { int l = 0; while ((1 << l) < v) ++l; return l; }

}  // namespace

TensorMapEncodeFn tensor_map_encoder()
{
    static TensorMapEncodeFn fn = nullptr;
    if (!fn) {
        void *ptr = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<TensorMapEncodeFn>(ptr);
    }
    return fn;
}

ConvTcGeom conv_tc_geometry(const ConvArgs &a, int rows, bool fill_sms)
{
    ConvTcGeom g;
    g.BK = a.Cin % 64 == 0 ? 64 : (a.Cin % 32 == 0 ? 32 : 16);
    g.BN = 16;
    for (int bn = 128; bn >= 16; bn -= 16)
        if (a.Cout % bn == 0) { g.BN = bn; break; }
    // output tile: the (TW, TR, TN) split of 128 pixels that needs the fewest tiles
    int nmax = 1;
    while (nmax * 2 <= a.N) nmax *= 2;
    long long best = -1;
    g.TW = 128; g.TR = 1; g.TN = 1;
    for (int tw = 128; tw >= 1; tw >>= 1)
        for (int tr = 128 / tw; tr >= 1; tr >>= 1) {
            const int tn = 128 / (tw * tr);
            if (tn > nmax) continue;
            const long long tiles = (long long)((a.Wo + tw - 1) / tw) * ((rows + tr - 1) / tr) * ((a.N + tn - 1) / tn);
            if (best < 0 || tiles < best) { best = tiles; g.TW = tw; g.TR = tr; g.TN = tn; }
        }
    // with few pixel tiles, narrower channel tiles give more CTAs to fill the 148 SMs
    while (fill_sms && best * (a.Cout / g.BN) < 148 && g.BN % 32 == 0 && g.BN > 32) g.BN /= 2;
    const int stage = 128 * g.BK * 2 + ((g.BN * g.BK * 2 + 1023) / 1024) * 1024;
    int stages = (100 * 1024) / stage;
    if (stages > 8) stages = 8;
    if (stages < 2) stages = 2;
    g.stages = stages;
    return g;
}

int conv_tc_encode(const ConvArgs &a, const ConvTcGeom &g, ConvTcMaps *maps)
{
    EncodeTiledFn enc = encode_fn();
    if (!enc) return LOP_ECUDA;
    const CUtensorMapSwizzle swz = g.BK == 64 ? CU_TENSOR_MAP_SWIZZLE_128B
                                   : (g.BK == 32 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B);
    const cuuint32_t ones[4] = {1, 1, 1, 1};
    for (int i = 0; i < 4; ++i) maps->a_valid[i] = 0;
    for (int ph = 0; ph < a.sh; ++ph)
        for (int pw = 0; pw < a.sw; ++pw) {
            const int idx = ph * a.sw + pw;
            const long long Hp = (a.Hin - ph + a.sh - 1) / a.sh, Wp = (a.Win - pw + a.sw - 1) / a.sw;
            if (a.Hin - ph <= 0 || a.Win - pw <= 0 || Hp <= 0 || Wp <= 0) continue;
            const cuuint64_t dims[4] = {(cuuint64_t)a.Cin, (cuuint64_t)Wp, (cuuint64_t)Hp, (cuuint64_t)a.N};
            const cuuint64_t strides[3] = {(cuuint64_t)a.sw * a.Cin * 2, (cuuint64_t)a.sh * a.Win * a.Cin * 2,
                                           (cuuint64_t)a.Hin * a.Win * a.Cin * 2};
            const cuuint32_t box[4] = {(cuuint32_t)g.BK, (cuuint32_t)g.TW, (cuuint32_t)g.TR, (cuuint32_t)g.TN};
            void *basep = (void *)(static_cast<const char *>(a.x) + ((size_t)ph * a.Win + pw) * a.Cin * 2);
            CUresult r = enc(&maps->a[idx], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, basep, dims, strides, box, ones,
                             CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
            if (r != CUDA_SUCCESS) return LOP_ECUDA;
            maps->a_valid[idx] = 1;
        }
    if (!(maps->a_valid[0] || maps->a_valid[1] || maps->a_valid[2] || maps->a_valid[3])) return LOP_ECUDA;
    for (int i = 0; i < 4; ++i)
        if (!maps->a_valid[i]) {
            for (int j = 0; j < 4; ++j)
                if (maps->a_valid[j]) { maps->a[i] = maps->a[j]; break; }
        }
    const cuuint64_t K = (cuuint64_t)a.kh * a.kw * a.Cin;
    const cuuint64_t wd[2] = {K, (cuuint64_t)a.Cout};
    const cuuint64_t ws[1] = {K * 2};
    const cuuint32_t wb[2] = {(cuuint32_t)g.BK, (cuuint32_t)g.BN};
    CUresult r = enc(&maps->w, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(a.w), wd, ws, wb, ones,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? LOP_OK : LOP_ECUDA;
}

cudaError_t launch_conv_tc(const ConvArgs &a, const ConvTcGeom &g, const ConvTcMaps &maps, unsigned *status,
                           cudaStream_t s)
{
    const int rows = a.oh_hi - a.oh_lo;
    if (rows <= 0) return cudaSuccess;
    TcParams p;
    p.y = a.y; p.res = a.res; p.scale = a.scale; p.shift = a.shift; p.status = status;
    p.N = a.N; p.Ho = a.Ho; p.Wo = a.Wo; p.Cout = a.Cout;
    p.oh_lo = a.oh_lo; p.oh_hi = a.oh_hi;
    p.tw_log = ilog2(g.TW); p.tr_log = ilog2(g.TR);
    p.tiles_w = (a.Wo + g.TW - 1) / g.TW;
    p.tiles_r = (rows + g.TR - 1) / g.TR;
    const int tiles_n = (a.N + g.TN - 1) / g.TN;
    p.BN = g.BN; p.BK = g.BK; p.stages = g.stages;
    p.kh = a.kh; p.kw = a.kw; p.cin = a.Cin;
    p.sh = a.sh; p.sw = a.sw; p.ph = a.ph; p.pw = a.pw; p.dh = a.dh; p.dw = a.dw;
    p.act = a.act; p.res_pos = a.res ? a.res_pos : LOP_RES_NONE;
    p.a_stage_bytes = 128u * g.BK * 2u;
    p.b_stage_bytes = ((uint32_t)(g.BN * g.BK * 2) + 1023u) / 1024u * 1024u;
    uint32_t cols = 32;
    while (cols < (uint32_t)g.BN) cols *= 2;
    p.tmem_cols = cols;
    p.layout_code = g.BK == 64 ? 2u : (g.BK == 32 ? 4u : 6u);
    p.sbo_bytes = 8u * g.BK * 2u;
    // instruction descriptor: fp32 accumulate, bf16 x bf16, both operands K-major, N = BN, M = 128
    p.idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(g.BN >> 3) << 17) | ((128u >> 4) << 24);
    const size_t smem = 1024 + (size_t)g.stages * (p.a_stage_bytes + p.b_stage_bytes) + 16 * g.stages + 32;
    // the attribute is per device: set it once on each device a launch is made from
    static std::atomic<bool> configured[64];            // set after the (idempotent) attribute call: plans on several host threads may race here
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64 || !configured[dev].load(std::memory_order_acquire)) {
        e = cudaFuncSetAttribute(conv_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(200 * 1024));
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) configured[dev].store(true, std::memory_order_release);
    }
    dim3 grid((unsigned)(p.tiles_w * p.tiles_r * tiles_n), (unsigned)(a.Cout / g.BN));
    conv_tc_kernel<<<grid, TC_THREADS, smem, s>>>(maps, p);
    return cudaGetLastError();
}

}  // namespace lop

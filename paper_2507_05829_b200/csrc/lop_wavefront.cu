// Persistent wavefront kernel (see lop_wavefront.cuh for the execution model).
//
// CTA layout (192 threads, one CTA per SM):
//   warp 0, one lane   waits for the item's producer row groups, then streams the item's activation and
//                      weight boxes by TMA into a shared-memory ring that lives across items
//   warp 1, one lane   tcgen05.mma into one of two fp32 accumulators in tensor memory, so the next
//                      item's main loop overlaps this item's epilogue
//   warps 2..5         epilogue of convolution items (TMEM -> scale/shift/residual/activation -> bf16),
//                      and the whole of pooling / channel-padding items; they publish each finished
//                      tile by a release increment of its row group's counter
// Deadlock freedom: items are numbered in a topological order, every CTA is resident and takes its
// items in increasing order, so the lowest unfinished item never waits on an unstarted one.  All
// waits are bounded all the same; one that runs out raises the status word and the abort flag.
#include <cuda_bf16.h>

#include "lop_ptx.cuh"
#include "lop_wavefront.cuh"

namespace lop {

namespace {

using namespace ptx;

constexpr uint32_t SPIN_LIMIT = 1u << 22;
constexpr int EPI_THREADS = 128;

struct RoleCtx {
    WfStage st;
    WfLayer ly;
};

__device__ __forceinline__ unsigned ld_acquire(const unsigned *p)
{
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ unsigned ld_relaxed(const unsigned *p)
{
    unsigned v;
    asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// Bounded wait until *ctr has reached target (counters only grow; compare modulo 2^32).
__device__ __forceinline__ bool wait_counter(const unsigned *ctr, unsigned target, const unsigned *abort_word)
{
    for (uint32_t i = 0; i < SPIN_LIMIT; ++i) {
        if ((int)(ld_acquire(ctr) - target) >= 0) return true;
        if ((i & 127u) == 127u && ld_relaxed(abort_word)) return false;
        __nanosleep(40);
    }
    return false;
}

__device__ __forceinline__ bool wait_deps(const WfParams &P, const WfStage &st, int tile_r, unsigned run)
{
    const int2 di = __ldg(&P.dep_index[st.dep_base + tile_r]);
    for (int j = di.x; j < di.x + di.y; ++j) {
        const int2 d = __ldg(&P.deps[j]);
        if (!wait_counter(P.counters + d.x, run * (unsigned)d.y, P.counters + 2)) return false;
    }
    return true;
}

__device__ __forceinline__ void copy_words(void *dst, const void *src, int words, int tid, int nthreads)
{
    const uint32_t *s = static_cast<const uint32_t *>(src);
    uint32_t *d = static_cast<uint32_t *>(dst);
    for (int i = tid; i < words; i += nthreads) d[i] = __ldg(s + i);
}

__device__ __forceinline__ void epi_bar() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

struct ConvTile {
    int cout_tile, tile_w, tile_n, tile_r;
};
__device__ __forceinline__ ConvTile decode_conv(const WfStage &st, int local)
{
    ConvTile t;
    t.cout_tile = local % st.cout_tiles;
    int q = local / st.cout_tiles;
    t.tile_w = q % st.tiles_w;
    q /= st.tiles_w;
    t.tile_n = q % st.tiles_n;
    t.tile_r = q / st.tiles_n;
    return t;
}

__global__ void __launch_bounds__(WF_THREADS, 1) wavefront_kernel(const WfParams P)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t *smem = smem_raw + (base - raw);
    const int S = P.ring;
    const uint32_t ring_bytes = (uint32_t)S * P.slot_bytes;
    const uint32_t full0 = base + ring_bytes, empty0 = full0 + 8u * S;
    const uint32_t accf0 = empty0 + 8u * S, acce0 = accf0 + 16u;
    volatile uint32_t *misc = reinterpret_cast<volatile uint32_t *>(smem + ring_bytes + 16u * S + 32u);
    // misc[0] TMEM base, misc[1] abort, misc[2] run number
    RoleCtx *ctx = reinterpret_cast<RoleCtx *>(smem + ring_bytes + 16u * S + 64u);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(full0 + 8u * s, 1);
            mbar_init(empty0 + 8u * s, 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(accf0 + 8u * b, 1);
            mbar_init(acce0 + 8u * b, 1);
        }
        misc[1] = 0;
        misc[2] = ld_acquire(P.counters) + 1u;                 // this launch is run number (completed runs + 1)
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32((const void *)&misc[0])),
                     "r"(512u)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = misc[0];
    const unsigned run = misc[2];
    volatile uint32_t *abort_flag = &misc[1];

    if (warp == 0) {
        if (lane == 0) {
            // ---------------- TMA producer ----------------
            RoleCtx &c = ctx[0];
            int sidx = 0, cur = -1;
            uint32_t it = 0;
            for (int item = blockIdx.x; item < P.n_items && !*abort_flag; item += gridDim.x) {
                while (item >= __ldg(&P.stages[sidx].first_item) + __ldg(&P.stages[sidx].n_items)) ++sidx;
                if (__ldg(&P.stages[sidx].kind) != WF_CONV) continue;
                if (sidx != cur) {
                    copy_words(&c.st, &P.stages[sidx], 32, 0, 1);
                    copy_words(&c.ly, &P.layers[c.st.layer], 32, 0, 1);
                    cur = sidx;
                }
                const WfStage &st = c.st;
                const WfLayer &ly = c.ly;
                const ConvTile t = decode_conv(st, item - st.first_item);
                if (!wait_deps(P, st, t.tile_r, run)) {
                    atomicOr(P.status, 0x10u);
                    atomicExch(P.counters + 2, 1u);
                    *abort_flag = 1;
                    break;
                }
                asm volatile("fence.proxy.async;" ::: "memory");       // producers' generic-proxy writes -> our TMA reads
                const int ow0 = t.tile_w << st.tw_log;
                const int oh0 = st.oh_lo + (t.tile_r << st.tr_log);
                const int n0 = t.tile_n * (128 >> (st.tw_log + st.tr_log));
                const int co0 = t.cout_tile * st.BN;
                const int slabs = ly.Cin / st.BK;
                const CUtensorMap *maps = P.maps + st.map_base;
                bool fail = false;
                for (int a = 0; a < ly.kh && !fail; ++a) {
                    const int qh = a * ly.dh - ly.ph;
                    const int offh = floor_div_i(qh, ly.sh), parh = qh - offh * ly.sh;
                    for (int b = 0; b < ly.kw && !fail; ++b) {
                        const int qw = b * ly.dw - ly.pw;
                        const int offw = floor_div_i(qw, ly.sw), parw = qw - offw * ly.sw;
                        const int mi = parh * ly.sw + parw;
                        const bool have = (st.a_valid_mask >> mi) & 1;
                        for (int cs = 0; cs < slabs; ++cs, ++it) {
                            const uint32_t s = it % (uint32_t)S, round = it / (uint32_t)S;
                            if (round > 0 && !mbar_wait(empty0 + 8u * s, (round - 1) & 1)) { fail = true; break; }
                            const uint32_t sa = base + s * P.slot_bytes, sb = sa + st.a_bytes;
                            const uint32_t fb = full0 + 8u * s;
                            mbar_expect_tx(fb, st.a_bytes + st.b_bytes);
                            tma_load_4d(sa, maps + mi, fb, cs * st.BK, have ? ow0 + offw : -65536, have ? oh0 + offh : -65536, n0);
                            tma_load_2d(sb, maps + 4, fb, (a * ly.kw + b) * ly.Cin + cs * st.BK, co0);
                        }
                    }
                }
                if (fail) {
                    atomicOr(P.status, 0x1u);
                    atomicExch(P.counters + 2, 1u);
                    *abort_flag = 1;
                    break;
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            // ---------------- MMA issuer ----------------
            RoleCtx &c = ctx[1];
            int sidx = 0, cur = -1;
            uint32_t it = 0, cnt = 0;
            bool fail = false;
            for (int item = blockIdx.x; item < P.n_items && !fail; item += gridDim.x) {
                while (item >= __ldg(&P.stages[sidx].first_item) + __ldg(&P.stages[sidx].n_items)) ++sidx;
                if (__ldg(&P.stages[sidx].kind) != WF_CONV) continue;
                if (sidx != cur) {
                    copy_words(&c.st, &P.stages[sidx], 32, 0, 1);
                    cur = sidx;
                }
                const WfStage &st = c.st;
                const uint32_t buf = cnt & 1u;
                if (cnt >= 2 && !mbar_wait(acce0 + 8u * buf, ((cnt >> 1) - 1) & 1)) { fail = true; break; }
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t acc = tmem_base + buf * 256u;
                for (int k = 0; k < st.k_iters; ++k, ++it) {
                    const uint32_t s = it % (uint32_t)S, round = it / (uint32_t)S;
                    if (*abort_flag || !mbar_wait(full0 + 8u * s, round & 1)) { fail = true; break; }
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint32_t sa = base + s * P.slot_bytes, sb = sa + st.a_bytes;
                    for (int kk = 0; kk < st.BK / 16; ++kk) {
                        const uint64_t ad = smem_desc(sa + 32u * kk, st.sbo_bytes, st.layout_code);
                        const uint64_t bd = smem_desc(sb + 32u * kk, st.sbo_bytes, st.layout_code);
                        umma_bf16(acc, ad, bd, st.idesc, (k > 0 || kk > 0) ? 1u : 0u);
                    }
                    umma_commit(empty0 + 8u * s);
                }
                if (fail) break;
                umma_commit(accf0 + 8u * buf);
                ++cnt;
            }
            if (fail) {
                atomicOr(P.status, 0x2u);
                atomicExch(P.counters + 2, 1u);
                *abort_flag = 1;
            }
        }
    } else {
        // ---------------- epilogue / SIMT warps ----------------
        RoleCtx &c = ctx[2];
        const int tid = threadIdx.x - 64;
        const int g = warp & 3;
        int sidx = 0, cur = -1;
        uint32_t cnt = 0;
        bool fail = false;
        for (int item = blockIdx.x; item < P.n_items; item += gridDim.x) {
            while (item >= __ldg(&P.stages[sidx].first_item) + __ldg(&P.stages[sidx].n_items)) ++sidx;
            if (sidx != cur) {
                epi_bar();                                           // everyone is done with the old context
                copy_words(&c.st, &P.stages[sidx], 32, tid, EPI_THREADS);
                epi_bar();
                copy_words(&c.ly, &P.layers[c.st.layer], 32, tid, EPI_THREADS);
                epi_bar();
                cur = sidx;
            }
            const WfStage &st = c.st;
            const WfLayer &ly = c.ly;
            const int local = item - st.first_item;
            int tile_r;
            if (st.kind == WF_CONV) {
                const ConvTile t = decode_conv(st, local);
                tile_r = t.tile_r;
                const uint32_t buf = cnt & 1u;
                const int TW = 1 << st.tw_log, TR = 1 << st.tr_log;
                const int m = g * 32 + lane;
                const int ow = (t.tile_w << st.tw_log) + (m & (TW - 1));
                const int oh = st.oh_lo + (t.tile_r << st.tr_log) + ((m >> st.tw_log) & (TR - 1));
                const int n = t.tile_n * (128 >> (st.tw_log + st.tr_log)) + (m >> (st.tw_log + st.tr_log));
                const bool valid = ow < ly.Wo && oh < st.oh_hi && n < ly.N;
                const int co0 = t.cout_tile * st.BN;
                const long long pix = (((long long)n * ly.Ho + oh) * ly.Wo + ow) * ly.Cout + co0;
                if (!mbar_wait(accf0 + 8u * buf, (cnt >> 1) & 1)) { fail = true; }
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                if (!fail) {
                    __nv_bfloat16 *y = static_cast<__nv_bfloat16 *>(ly.y);
                    const __nv_bfloat16 *res = static_cast<const __nv_bfloat16 *>(ly.res);
                    const uint32_t acc = tmem_base + buf * 256u + ((uint32_t)(g * 32) << 16);
                    for (int j = 0; j < st.BN; j += 16) {
                        uint32_t r[16];
                        tmem_ld16(acc + (uint32_t)j, r);
                        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                        if (!valid) continue;
                        float v[16];
#pragma unroll
                        for (int i = 0; i < 16; ++i) {
                            const int co = co0 + j + i;
                            const float sc = ly.scale ? __ldg(ly.scale + co) : 1.0f;
                            const float sf = ly.shift ? __ldg(ly.shift + co) : 0.0f;
                            v[i] = fmaf(sc, __uint_as_float(r[i]), sf);
                        }
                        if (res) {
                            // produced inside this launch by other SMs: read through L2, never a stale L1 line
                            const uint4 q0 = __ldcg(reinterpret_cast<const uint4 *>(res + pix + j));
                            const uint4 q1 = __ldcg(reinterpret_cast<const uint4 *>(res + pix + j + 8));
                            const uint32_t rw[8] = {q0.x, q0.y, q0.z, q0.w, q1.x, q1.y, q1.z, q1.w};
                            float rv[16];
#pragma unroll
                            for (int i = 0; i < 8; ++i) {
                                rv[2 * i] = __uint_as_float(rw[i] << 16);
                                rv[2 * i + 1] = __uint_as_float(rw[i] & 0xFFFF0000u);
                            }
                            if (ly.res_pos == LOP_RES_PRE_ACT) {
#pragma unroll
                                for (int i = 0; i < 16; ++i) v[i] = activate(v[i] + rv[i], ly.act);
                            } else {
#pragma unroll
                                for (int i = 0; i < 16; ++i) v[i] = activate(v[i], ly.act) + rv[i];
                            }
                        } else {
#pragma unroll
                            for (int i = 0; i < 16; ++i) v[i] = activate(v[i], ly.act);
                        }
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
                asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                __threadfence();
                epi_bar();
                if (tid == 0 && !fail)
                    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(acce0 + 8u * buf) : "memory");
                ++cnt;
            } else {
                // pooling or channel padding: one (row, image) per item, all 128 threads
                const int n = local % st.tiles_n;
                tile_r = local / st.tiles_n;
                const int oh = st.oh_lo + tile_r;
                if (!wait_deps(P, st, tile_r, run)) fail = true;
                if (!fail && st.kind == WF_POOL) {
                    const int cg = ly.Cin >> 3;
                    const __nv_bfloat16 *x = static_cast<const __nv_bfloat16 *>(ly.x);
                    __nv_bfloat16 *y = static_cast<__nv_bfloat16 *>(ly.y);
                    for (int idx = tid; idx < ly.Wo * cg; idx += EPI_THREADS) {
                        const int gch = idx % cg, ow = idx / cg;
                        float mx[8];
#pragma unroll
                        for (int i = 0; i < 8; ++i) mx[i] = -INFINITY;
                        for (int a = 0; a < ly.kh; ++a) {
                            const int ih = oh * ly.sh - ly.ph + a * ly.dh;
                            if (ih < 0 || ih >= ly.Hin) continue;
                            for (int b = 0; b < ly.kw; ++b) {
                                const int iw = ow * ly.sw - ly.pw + b * ly.dw;
                                if (iw < 0 || iw >= ly.Win) continue;
                                const uint4 q = __ldcg(reinterpret_cast<const uint4 *>(
                                    x + (((long long)n * ly.Hin + ih) * ly.Win + iw) * ly.Cin + gch * 8));
                                const uint32_t w4[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
                                for (int i = 0; i < 4; ++i) {
                                    mx[2 * i] = fmaxf(mx[2 * i], __uint_as_float(w4[i] << 16));
                                    mx[2 * i + 1] = fmaxf(mx[2 * i + 1], __uint_as_float(w4[i] & 0xFFFF0000u));
                                }
                            }
                        }
                        uint32_t o[4];
#pragma unroll
                        for (int i = 0; i < 4; ++i)          // values are bf16 already: truncation is exact
                            o[i] = (__float_as_uint(mx[2 * i]) >> 16) | (__float_as_uint(mx[2 * i + 1]) & 0xFFFF0000u);
                        *reinterpret_cast<uint4 *>(y + (((long long)n * ly.Ho + oh) * ly.Wo + ow) * ly.Cin + gch * 8) =
                            make_uint4(o[0], o[1], o[2], o[3]);
                    }
                } else if (!fail) {
                    // channel padding: ly.Cin real channels -> 16, one pixel per thread and step
                    const uint16_t *x = static_cast<const uint16_t *>(ly.x);
                    uint16_t *y = static_cast<uint16_t *>(ly.y);
                    const long long row = ((long long)n * ly.Hin + oh) * ly.Win;
                    for (int px = tid; px < ly.Win; px += EPI_THREADS) {
                        uint32_t o[8] = {0, 0, 0, 0, 0, 0, 0, 0};
                        const uint16_t *src = x + (row + px) * ly.Cin;
                        for (int ch = 0; ch < ly.Cin; ++ch) o[ch >> 1] |= (uint32_t)src[ch] << ((ch & 1) * 16);
                        uint4 *dst = reinterpret_cast<uint4 *>(y + (row + px) * 16);
                        dst[0] = make_uint4(o[0], o[1], o[2], o[3]);
                        dst[1] = make_uint4(o[4], o[5], o[6], o[7]);
                    }
                }
                __threadfence();
                epi_bar();
            }
            if (fail) {
                if (tid == 0) {
                    atomicOr(P.status, 0x4u);
                    atomicExch(P.counters + 2, 1u);
                    *abort_flag = 1;
                }
                break;
            }
            if (tid == 0) atomicAdd(P.counters + st.ctr_base + tile_r, 1u);   // release: stores fenced above
        }
    }

    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    if (warp == 1)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
    if (threadIdx.x == 0) {
        __threadfence();
        const unsigned done = atomicAdd(P.counters + 1, 1u);
        if (done == gridDim.x - 1) {                                  // last CTA out: this run is complete
            atomicExch(P.counters + 1, 0u);
            __threadfence();
            atomicAdd(P.counters, 1u);
        }
    }
}

}  // namespace

size_t wavefront_smem_bytes(int ring, uint32_t slot_bytes)
{
    return 1024 + (size_t)ring * slot_bytes + 16 * (size_t)ring + 64 + 3 * sizeof(RoleCtx) + 64;
}

cudaError_t launch_wavefront(const WfParams &p, int grid, cudaStream_t s)
{
    const size_t smem = wavefront_smem_bytes(p.ring, p.slot_bytes);
    static bool configured = false;
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(wavefront_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
        if (e != cudaSuccess) return e;
        configured = true;
    }
    if (smem > 227 * 1024) return cudaErrorInvalidValue;
    wavefront_kernel<<<grid, WF_THREADS, smem, s>>>(p);
    return cudaGetLastError();
}

}  // namespace lop

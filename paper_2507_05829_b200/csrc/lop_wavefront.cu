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

__device__ __forceinline__ bool wait_deps(const WfParams &P, int dep_slot, unsigned run)
{
    const int2 di = __ldg(&P.dep_index[dep_slot]);
    for (int j = di.x; j < di.x + di.y; ++j) {
        const int2 d = __ldg(&P.deps[j]);
        // d.y > 0: a row-group counter that grows by d.y per run; d.y < 0: an arrival flag set to >= -d.y
        const unsigned target = d.y > 0 ? run * (unsigned)d.y : (unsigned)(-d.y);
        if (!wait_counter(P.counters + d.x, target, P.counters + 2)) return false;
    }
    return true;
}

__device__ __forceinline__ void epi_bar() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

// Walks the stage list as the CTA's item index grows; touches global memory only on a stage change.
struct StageCursor {
    int sidx = -1, first = 0, end = 0, kind = -1;
    __device__ __forceinline__ bool advance(const WfParams &P, int item)      // true when the stage changed
    {
        if (item < end) return false;
        do {
            ++sidx;
            first = __ldg(&P.stages[sidx].first_item);
            end = first + __ldg(&P.stages[sidx].n_items);
        } while (item >= end);
        kind = __ldg(&P.stages[sidx].kind);
        return true;
    }
};

__global__ void __launch_bounds__(WF_THREADS, 1) wavefront_kernel(const WfParams P)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t *smem = smem_raw + (base - raw);
    const int S = P.ring;
    const uint32_t slot_bytes = P.slot_bytes;
    const uint32_t ring_bytes = (uint32_t)S * slot_bytes;
    const uint32_t full0 = base + ring_bytes, empty0 = full0 + 8u * S;
    const uint32_t accf0 = empty0 + 8u * S, acce0 = accf0 + 16u;
    volatile uint32_t *misc = reinterpret_cast<volatile uint32_t *>(smem + ring_bytes + 16u * S + 32u);
    // misc[0] TMEM base, misc[1] abort, misc[2] run number
    float *s_scale = reinterpret_cast<float *>(smem + ring_bytes + 16u * S + 64u);   // [256]
    float *s_shift = s_scale + 256;                                                   // [256]

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
    const int G = gridDim.x;

    if (warp == 0) {
        if (lane == 0) {
            // ---------------- TMA producer ----------------
            // Everything the inner loop needs lives in registers: the PTX wrappers clobber memory, so a field
            // left in shared or global memory would be re-read after every one of them.
            StageCursor cur;
            uint32_t slot = 0, phase = 0;
            int first_item = 0, oh_lo = 0, tw_log = 0, tr_log = 0, tiles_w = 1, tiles_n = 1, cout_tiles = 1, BN = 0, BK = 0,
                amask = 0, dep_base = 0, slabs = 1, kh = 1, kw = 1, sh = 1, sw = 1, ph = 0, pw = 0, dh = 1, dw = 1, cin = 0;
            uint32_t a_bytes = 0, tx_bytes = 0;
            const CUtensorMap *maps = nullptr;
            bool fail = false;
            for (int item = blockIdx.x; item < P.n_items && !fail; item += G) {
                if (cur.advance(P, item) && cur.kind == WF_CONV) {
                    const WfStage *sp = &P.stages[cur.sidx];
                    const WfLayer *lp = &P.layers[__ldg(&sp->layer)];
                    first_item = cur.first;
                    oh_lo = __ldg(&sp->oh_lo); tw_log = __ldg(&sp->tw_log); tr_log = __ldg(&sp->tr_log);
                    tiles_w = __ldg(&sp->tiles_w); tiles_n = __ldg(&sp->tiles_n); cout_tiles = __ldg(&sp->cout_tiles);
                    BN = __ldg(&sp->BN); BK = __ldg(&sp->BK); amask = __ldg(&sp->a_valid_mask); dep_base = __ldg(&sp->dep_base);
                    a_bytes = __ldg(&sp->a_bytes); tx_bytes = a_bytes + __ldg(&sp->b_bytes);
                    maps = P.maps + __ldg(&sp->map_base);
                    kh = __ldg(&lp->kh); kw = __ldg(&lp->kw); sh = __ldg(&lp->sh); sw = __ldg(&lp->sw);
                    ph = __ldg(&lp->ph); pw = __ldg(&lp->pw); dh = __ldg(&lp->dh); dw = __ldg(&lp->dw);
                    cin = __ldg(&lp->Cin);
                    slabs = cin / BK;
                }
                if (cur.kind != WF_CONV) continue;
                if (*abort_flag) break;
                int q = item - first_item;
                const int cout_tile = q % cout_tiles; q /= cout_tiles;
                const int tile_w = q % tiles_w; q /= tiles_w;
                const int tile_n = q % tiles_n;
                const int tile_r = q / tiles_n;
                if (!wait_deps(P, dep_base + tile_r, run)) {
                    atomicOr(P.status, 0x10u);
                    fail = true;
                    break;
                }
                asm volatile("fence.proxy.async;" ::: "memory");       // producers' generic-proxy writes -> our TMA reads
                const int ow0 = tile_w << tw_log;
                const int oh0 = oh_lo + (tile_r << tr_log);
                const int n0 = tile_n * (128 >> (tw_log + tr_log));
                const int co0 = cout_tile * BN;
                for (int a = 0; a < kh && !fail; ++a) {
                    const int qh = a * dh - ph;
                    const int offh = floor_div_i(qh, sh), parh = qh - offh * sh;
                    for (int b = 0; b < kw && !fail; ++b) {
                        const int qw = b * dw - pw;
                        const int offw = floor_div_i(qw, sw), parw = qw - offw * sw;
                        const int mi = parh * sw + parw;
                        const bool have = (amask >> mi) & 1;
                        const int cw = have ? ow0 + offw : -65536, chh = have ? oh0 + offh : -65536;
                        const int kbase = (a * kw + b) * cin;
                        for (int cs = 0; cs < slabs; ++cs) {
                            if (!mbar_wait(empty0 + 8u * slot, phase ^ 1u)) { atomicOr(P.status, 0x1u); fail = true; break; }
                            const uint32_t sa = base + slot * slot_bytes;
                            const uint32_t fb = full0 + 8u * slot;
                            mbar_expect_tx(fb, tx_bytes);
                            tma_load_4d(sa, maps + mi, fb, cs * BK, cw, chh, n0);
                            tma_load_2d(sa + a_bytes, maps + 4, fb, kbase + cs * BK, co0);
                            if (++slot == (uint32_t)S) { slot = 0; phase ^= 1u; }
                        }
                    }
                }
            }
            if (fail) {
                atomicExch(P.counters + 2, 1u);
                *abort_flag = 1;
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            // ---------------- MMA issuer ----------------
            StageCursor cur;
            uint32_t slot = 0, phase = 0, cnt = 0;
            int k_iters = 0, ksteps = 0;
            uint32_t a_bytes = 0, idesc = 0, layout_code = 0, sbo = 0;
            bool fail = false;
            for (int item = blockIdx.x; item < P.n_items && !fail; item += G) {
                if (cur.advance(P, item) && cur.kind == WF_CONV) {
                    const WfStage *sp = &P.stages[cur.sidx];
                    k_iters = __ldg(&sp->k_iters); ksteps = __ldg(&sp->BK) / 16;
                    a_bytes = __ldg(&sp->a_bytes); idesc = __ldg(&sp->idesc);
                    layout_code = __ldg(&sp->layout_code); sbo = __ldg(&sp->sbo_bytes);
                }
                if (cur.kind != WF_CONV) continue;
                const uint32_t buf = cnt & 1u;
                if (!mbar_wait(acce0 + 8u * buf, ((cnt >> 1) & 1u) ^ 1u)) { fail = true; break; }
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t acc = tmem_base + buf * 256u;
                for (int k = 0; k < k_iters; ++k) {
                    if (*abort_flag || !mbar_wait(full0 + 8u * slot, phase)) { fail = true; break; }
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint32_t sa = base + slot * slot_bytes, sb = sa + a_bytes;
                    for (int kk = 0; kk < ksteps; ++kk) {
                        const uint64_t ad = smem_desc(sa + 32u * kk, sbo, layout_code);
                        const uint64_t bd = smem_desc(sb + 32u * kk, sbo, layout_code);
                        umma_bf16(acc, ad, bd, idesc, (k > 0 || kk > 0) ? 1u : 0u);
                    }
                    umma_commit(empty0 + 8u * slot);
                    if (++slot == (uint32_t)S) { slot = 0; phase ^= 1u; }
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
        const int tid = threadIdx.x - 64;
        const int g = warp & 3;
        StageCursor cur;
        uint32_t cnt = 0;
        bool fail = false;
        int first_item = 0, oh_lo = 0, oh_hi = 0, tw_log = 0, tr_log = 0, tiles_w = 1, tiles_n = 1, cout_tiles = 1, BN = 0,
            dep_base = 0, ctr_base = 0;
        int N = 0, Hin = 0, Win = 0, Cin = 0, Ho = 0, Wo = 0, Cout = 0, kh = 1, kw = 1, sh = 1, sw = 1, ph = 0, pw = 0, dh = 1,
            dw = 1, act = 0, res_pos = 0;
        const void *xin = nullptr, *resp = nullptr;
        const float *scale = nullptr, *shift = nullptr;
        void *yout = nullptr;
        for (int item = blockIdx.x; item < P.n_items; item += G) {
            if (cur.advance(P, item)) {
                const WfStage *sp = &P.stages[cur.sidx];
                const WfLayer *lp = &P.layers[__ldg(&sp->layer)];
                first_item = cur.first;
                oh_lo = __ldg(&sp->oh_lo); oh_hi = __ldg(&sp->oh_hi); tw_log = __ldg(&sp->tw_log); tr_log = __ldg(&sp->tr_log);
                tiles_w = __ldg(&sp->tiles_w); tiles_n = __ldg(&sp->tiles_n); cout_tiles = __ldg(&sp->cout_tiles);
                BN = __ldg(&sp->BN); dep_base = __ldg(&sp->dep_base); ctr_base = __ldg(&sp->ctr_base);
                N = __ldg(&lp->N); Hin = __ldg(&lp->Hin); Win = __ldg(&lp->Win); Cin = __ldg(&lp->Cin);
                Ho = __ldg(&lp->Ho); Wo = __ldg(&lp->Wo); Cout = __ldg(&lp->Cout);
                kh = __ldg(&lp->kh); kw = __ldg(&lp->kw); sh = __ldg(&lp->sh); sw = __ldg(&lp->sw);
                ph = __ldg(&lp->ph); pw = __ldg(&lp->pw); dh = __ldg(&lp->dh); dw = __ldg(&lp->dw);
                act = __ldg(&lp->act); res_pos = __ldg(&lp->res_pos);
                xin = reinterpret_cast<const void *>(__ldg(reinterpret_cast<const unsigned long long *>(&lp->x)));
                resp = reinterpret_cast<const void *>(__ldg(reinterpret_cast<const unsigned long long *>(&lp->res)));
                scale = reinterpret_cast<const float *>(__ldg(reinterpret_cast<const unsigned long long *>(&lp->scale)));
                shift = reinterpret_cast<const float *>(__ldg(reinterpret_cast<const unsigned long long *>(&lp->shift)));
                yout = reinterpret_cast<void *>(__ldg(reinterpret_cast<const unsigned long long *>(&lp->y)));
            }
            int q = item - first_item;
            int tile_r;
            if (cur.kind == WF_CONV) {
                const int cout_tile = q % cout_tiles; q /= cout_tiles;
                const int tile_w = q % tiles_w; q /= tiles_w;
                const int tile_n = q % tiles_n;
                tile_r = q / tiles_n;
                const uint32_t buf = cnt & 1u;
                const int TW = 1 << tw_log, TR = 1 << tr_log;
                const int m = g * 32 + lane;
                const int ow = (tile_w << tw_log) + (m & (TW - 1));
                const int oh = oh_lo + (tile_r << tr_log) + ((m >> tw_log) & (TR - 1));
                const int n = tile_n * (128 >> (tw_log + tr_log)) + (m >> (tw_log + tr_log));
                const bool valid = ow < Wo && oh < oh_hi && n < N;
                const int co0 = cout_tile * BN;
                const long long pix = (((long long)n * Ho + oh) * Wo + ow) * Cout + co0;
                // this tile's scale/shift into shared memory while the main loop is still running
                epi_bar();                                           // previous item's readers are done
                for (int i = tid; i < BN; i += EPI_THREADS) {
                    s_scale[i] = scale ? __ldg(scale + co0 + i) : 1.0f;
                    s_shift[i] = shift ? __ldg(shift + co0 + i) : 0.0f;
                }
                epi_bar();
                if (!mbar_wait(accf0 + 8u * buf, (cnt >> 1) & 1u)) fail = true;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                if (!fail) {
                    __nv_bfloat16 *y = static_cast<__nv_bfloat16 *>(yout);
                    const __nv_bfloat16 *res = static_cast<const __nv_bfloat16 *>(resp);
                    const uint32_t acc = tmem_base + buf * 256u + ((uint32_t)(g * 32) << 16);
                    for (int j = 0; j < BN; j += 16) {
                        uint32_t r[16];
                        tmem_ld16(acc + (uint32_t)j, r);
                        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                        if (!valid) continue;
                        float v[16];
#pragma unroll
                        for (int i = 0; i < 16; ++i) v[i] = fmaf(s_scale[j + i], __uint_as_float(r[i]), s_shift[j + i]);
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
                            if (res_pos == LOP_RES_PRE_ACT) {
#pragma unroll
                                for (int i = 0; i < 16; ++i) v[i] = activate(v[i] + rv[i], act);
                            } else {
#pragma unroll
                                for (int i = 0; i < 16; ++i) v[i] = activate(v[i], act) + rv[i];
                            }
                        } else {
#pragma unroll
                            for (int i = 0; i < 16; ++i) v[i] = activate(v[i], act);
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
                // pooling or channel padding: a chunk of one output row of one image per item, all 128 threads
                const int chunk = q % tiles_w; q /= tiles_w;
                const int n = q % tiles_n;
                tile_r = q / tiles_n;
                const int oh = oh_lo + tile_r;
                if (!wait_deps(P, dep_base + tile_r, run)) fail = true;
                if (!fail && cur.kind == WF_POOL) {
                    // 2 channel-group vectors per thread, up to 3 taps of each in flight at once
                    const int cg = Cin >> 3;
                    const int total = Wo * cg;
                    const __nv_bfloat16 *x = static_cast<const __nv_bfloat16 *>(xin);
                    __nv_bfloat16 *y = static_cast<__nv_bfloat16 *>(yout);
                    int idx[2], gch[2], ow[2];
                    float mx[2][8];
#pragma unroll
                    for (int u = 0; u < 2; ++u) {
                        idx[u] = chunk * (2 * EPI_THREADS) + u * EPI_THREADS + tid;
                        gch[u] = idx[u] % cg;
                        ow[u] = idx[u] / cg;
#pragma unroll
                        for (int i = 0; i < 8; ++i) mx[u][i] = -INFINITY;
                    }
                    for (int a = 0; a < kh; ++a) {
                        const int ih = oh * sh - ph + a * dh;
                        if (ih < 0 || ih >= Hin) continue;
                        const long long rowbase = ((long long)n * Hin + ih) * Win;
                        for (int b0 = 0; b0 < kw; b0 += 3) {
                            uint4 q4[2][3];
                            bool ok[2][3];
#pragma unroll
                            for (int u = 0; u < 2; ++u)
#pragma unroll
                                for (int bb = 0; bb < 3; ++bb) {
                                    const int iw = ow[u] * sw - pw + (b0 + bb) * dw;
                                    ok[u][bb] = idx[u] < total && b0 + bb < kw && iw >= 0 && iw < Win;
                                    if (ok[u][bb])
                                        q4[u][bb] = __ldcg(reinterpret_cast<const uint4 *>(x + (rowbase + iw) * Cin + gch[u] * 8));
                                }
#pragma unroll
                            for (int u = 0; u < 2; ++u)
#pragma unroll
                                for (int bb = 0; bb < 3; ++bb)
                                    if (ok[u][bb]) {
                                        const uint32_t w4[4] = {q4[u][bb].x, q4[u][bb].y, q4[u][bb].z, q4[u][bb].w};
#pragma unroll
                                        for (int i = 0; i < 4; ++i) {
                                            mx[u][2 * i] = fmaxf(mx[u][2 * i], __uint_as_float(w4[i] << 16));
                                            mx[u][2 * i + 1] = fmaxf(mx[u][2 * i + 1], __uint_as_float(w4[i] & 0xFFFF0000u));
                                        }
                                    }
                        }
                    }
#pragma unroll
                    for (int u = 0; u < 2; ++u)
                        if (idx[u] < total) {
                            uint32_t o[4];
#pragma unroll
                            for (int i = 0; i < 4; ++i)      // values are bf16 already: truncation is exact
                                o[i] = (__float_as_uint(mx[u][2 * i]) >> 16) | (__float_as_uint(mx[u][2 * i + 1]) & 0xFFFF0000u);
                            *reinterpret_cast<uint4 *>(y + (((long long)n * Ho + oh) * Wo + ow[u]) * Cin + gch[u] * 8) =
                                make_uint4(o[0], o[1], o[2], o[3]);
                        }
                } else if (!fail) {
                    // channel padding: Cin real channels -> 16, one pixel per thread
                    const uint16_t *x = static_cast<const uint16_t *>(xin);
                    uint16_t *y = static_cast<uint16_t *>(yout);
                    const long long row = ((long long)n * Hin + oh) * Win;
                    const int px = chunk * EPI_THREADS + tid;
                    if (px < Win) {
                        const uint16_t *src = x + (row + px) * Cin;
                        uint32_t h[16];
#pragma unroll
                        for (int ch = 0; ch < 16; ++ch) h[ch] = ch < Cin ? (uint32_t)src[ch] : 0u;
                        uint4 *dst = reinterpret_cast<uint4 *>(y + (row + px) * 16);
                        dst[0] = make_uint4(h[0] | (h[1] << 16), h[2] | (h[3] << 16), h[4] | (h[5] << 16), h[6] | (h[7] << 16));
                        dst[1] = make_uint4(h[8] | (h[9] << 16), h[10] | (h[11] << 16), h[12] | (h[13] << 16), h[14] | (h[15] << 16));
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
            if (tid == 0) atomicAdd(P.counters + ctr_base + tile_r, 1u);      // release: stores fenced above
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
            for (int f = 0; f < P.n_flags; ++f) P.counters[P.flag_base + f] = 0u;   // arrival flags of the next run
            atomicExch(P.counters + 1, 0u);
            __threadfence();
            atomicAdd(P.counters, 1u);
        }
    }
}

}  // namespace

size_t wavefront_smem_bytes(int ring, uint32_t slot_bytes)
{
    return 1024 + (size_t)ring * slot_bytes + 16 * (size_t)ring + 64 + 2 * 256 * sizeof(float) + 64;
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

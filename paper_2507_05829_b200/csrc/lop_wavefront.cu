// Persistent wavefront kernel (see lop_wavefront.cuh for the execution model).
//
// CTA layout (three special warps + WF_WORKER_WARPS worker warps, one CTA per SM):
//   warp 0      all lanes poll the item's producer row groups in parallel (the dependency list of the
//               next item is prefetched while this one runs); lane 0 then streams the item's activation
//               and weight boxes by TMA into two shared-memory rings that live across items
//   warp 1      one lane issues tcgen05.mma into one of two fp32 accumulators in tensor memory, so the
//               next item's main loop overlaps this item's epilogue
//   warp 2      one lane publishes finished items: after the workers' barrier it fences and does the release
//               increment of the item's row-group counter, so that memory-fence latency is off the workers' path
//   workers     epilogue of convolution items: TMEM -> scale/shift/residual/activation -> bf16 rows in a
//               shared staging tile -> coalesced 16-byte stores; and the whole of pooling, patch-gather,
//               depth-wise convolution, layer-normalisation and concatenation items.
//               Many of them because straight-line per-element code needs several warps per scheduler to
//               hide its own latency; the four warps that share a TMEM lane group split a tile's columns.
//
// Convolution as implicit GEMM: accumulator row m is an *anchor*, a position in a flat list of pixels
// with a row pitch of P pixels.  In slab mode the activation box holds the tile's rows plus the halo of
// the filter, P pixels wide; filter tap (a, b) reads the same box starting (a*dh*P + b*dw) pixels later,
// so one TMA box per 64-channel chunk serves all taps (the shared-memory matrix descriptor simply starts
// later: the swizzle is a function of the address).  Anchors in the last (kw-1)*dw columns of a
// pitch would wrap into the next row; they are computed and dropped.  K is walked as (channel chunk, kh,
// kw, 16-channel step) whatever the tile, so a pixel's bits do not depend on who computes it.
//
// Deadlock freedom: items are numbered in a topological order, every CTA is resident and takes its
// items in increasing order, so the lowest unfinished item never waits on an unstarted one.  All
// waits are bounded all the same; one that runs out raises the status word and the abort flag.
#include <atomic>

#include <cuda_bf16.h>

#include "lop_gather.cuh"
#include "lop_ptx.cuh"
#include "lop_rowops.cuh"
#include "lop_wavefront.cuh"

namespace lop {

namespace {

using namespace ptx;

constexpr int EPI_THREADS = 32 * WF_WORKER_WARPS;
constexpr int COL_GROUPS = WF_WORKER_WARPS / 4;            // worker warps sharing a TMEM lane group split the columns

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

#ifdef LOP_WF_TRACE
// Developer build only: per-item time stamps (global timer, ns) of the three roles.
constexpr int TRACE_ITEMS = 1 << 15;
constexpr int TRACE_FETCH0 = 1 << 14;                       // fetch entry j is stamped at row TRACE_FETCH0 + j
__device__ unsigned long long g_wf_trace[TRACE_ITEMS * 16];
__device__ __forceinline__ void tr(int item, int slot)
{
    if (item < TRACE_ITEMS) {
        unsigned long long t;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
        g_wf_trace[item * 16 + slot] = t;
    }
}
__device__ __forceinline__ void trv(int item, int slot, unsigned long long v)
{
    if (item < TRACE_ITEMS) g_wf_trace[item * 16 + slot] = v;
}
#else
#define tr(item, slot) ((void)0)
#define trv(item, slot, v) ((void)0)
#endif

// ---- item records -------------------------------------------------------------------------------
__device__ __forceinline__ int rec_stage(const int4 &r) { return r.x & 0xFFFF; }
__device__ __forceinline__ int rec_cout(const int4 &r) { return (int)((unsigned)r.x >> 16); }
__device__ __forceinline__ int rec_tw(const int4 &r) { return r.y & 0xFFFF; }
__device__ __forceinline__ int rec_tn(const int4 &r) { return (int)((unsigned)r.y >> 16); }
__device__ __forceinline__ int rec_tr(const int4 &r) { return r.z & 0xFFFFF; }
__device__ __forceinline__ int rec_ndep(const int4 &r) { return (int)((unsigned)r.z >> 20); }
__device__ __forceinline__ int rec_dep0(const int4 &r) { return r.w; }

// Bounded wait of a whole warp for an item's dependencies: lane j polls entry j of the list (its first
// 32 entries were prefetched into `mine`).  Counters only grow (compare modulo 2^32).  The result is
// uniform across the warp.
__device__ __forceinline__ bool wait_deps_warp(const WfParams &P, int first, int count, int2 mine, unsigned run, int lane)
{
    for (int j0 = 0; j0 < count; j0 += 32) {
        const bool have = j0 + lane < count;
        int2 d = mine;
        if (j0 > 0 && have) d = __ldg(&P.deps[first + j0 + lane]);
        // d.y > 0: a row-group counter that grows by d.y per run; d.y < 0: an arrival flag set to >= -d.y
        const unsigned target = !have ? 0u : (d.y > 0 ? run * (unsigned)d.y : (unsigned)(-d.y));
        const unsigned *ctr = P.counters + (have ? d.x : 0);
        bool done = !have;
        for (uint32_t i = 0;; ++i) {
            if (!done) done = (int)(ld_acquire(ctr) - target) >= 0;
            if (__all_sync(0xffffffffu, done)) break;
            if (i >= P.spin_limit) return false;
            if ((i & 63u) == 63u && __any_sync(0xffffffffu, ld_relaxed(P.counters + 2) != 0u)) return false;
            __nanosleep(32);
        }
    }
    __syncwarp();            // every lane's acquire now orders the whole warp's later reads
    return true;
}

// Bounded mbarrier wait that also gives up when the CTA's abort flag is raised.
__device__ __forceinline__ bool mbar_wait_abortable(uint32_t bar, uint32_t parity, volatile uint32_t *abort_flag)
{
    for (uint32_t i = 0; i < WAIT_LIMIT; ++i) {
        uint32_t done;
        asm volatile(
            "{\n"
            ".reg .pred p;\n"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
            "selp.u32 %0, 1, 0, p;\n"
            "}\n"
            : "=r"(done)
            : "r"(bar), "r"(parity)
            : "memory");
        if (done) return true;
        if ((i & 255u) == 255u && *abort_flag) return false;
    }
    return false;
}

// The 16-channel MMA steps of one (tap, channel chunk): descriptors differ only in their start-address field.
// desc_hi: upper word of the operand descriptors (stride between 8-row groups, version, swizzle mode).
// la, lb: low words of the two descriptors (address >> 4 in the start field, leading-offset field 1).
template <int KSTEPS>
__device__ __forceinline__ void mma_ksteps_f(uint32_t acc, uint32_t la, uint32_t lb, uint32_t desc_hi, uint32_t idesc, uint32_t &accumulate)
{
#pragma unroll
    for (int kk = 0; kk < KSTEPS; ++kk) {
        const uint64_t ad = ((uint64_t)desc_hi << 32) | (uint64_t)(la + 2u * kk);
        const uint64_t bd = ((uint64_t)desc_hi << 32) | (uint64_t)(lb + 2u * kk);
        umma_bf16(acc, ad, bd, idesc, accumulate);
        accumulate = 1u;
    }
}
__device__ __forceinline__ uint32_t desc_lo(uint32_t smem_addr) { return ((smem_addr & 0x3FFFFu) >> 4) | (1u << 16); }
__device__ __forceinline__ void mma_tap_f(uint32_t acc, uint32_t la, uint32_t lb, uint32_t desc_hi, uint32_t idesc, int ksteps, uint32_t &accumulate)
{
    if (ksteps == 4) mma_ksteps_f<4>(acc, la, lb, desc_hi, idesc, accumulate);
    else if (ksteps == 2) mma_ksteps_f<2>(acc, la, lb, desc_hi, idesc, accumulate);
    else mma_ksteps_f<1>(acc, la, lb, desc_hi, idesc, accumulate);
}
__device__ __forceinline__ void mma_tap(uint32_t acc, uint32_t pa, uint32_t pb, uint32_t desc_hi, uint32_t idesc, int ksteps,
                                        uint32_t &accumulate)
{
    mma_tap_f(acc, desc_lo(pa), desc_lo(pb), desc_hi, idesc, ksteps, accumulate);
}

// One weight box of three taps of a 3x3 filter row over a 64-channel chunk: twelve MMAs whose descriptors differ
// from the first one by compile-time constants.  One thread issues every MMA of the CTA and each instruction it
// executes in between costs as much as a quarter of an N = 64 MMA, so the common case gets straight-line code.
// la, lb: start-address fields (address >> 4) of the slab row this filter row starts at and of the weight box;
// tap16: bytes of one tap's weights >> 4.
__device__ __forceinline__ void mma_row3x64(uint32_t acc, uint32_t la, uint32_t lb, uint32_t tap16, uint32_t desc_hi, uint32_t idesc,
                                            uint32_t &accumulate)
{
    const uint64_t hi = (uint64_t)desc_hi << 32;
#pragma unroll
    for (int tb = 0; tb < 3; ++tb)
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) {
            umma_bf16(acc, hi | (uint64_t)(la + 8u * tb + 2u * kk), hi | (uint64_t)(lb + tap16 * tb + 2u * kk), idesc, accumulate);
            accumulate = 1u;
        }
}

__device__ __forceinline__ void epi_bar() { asm volatile("bar.sync 1, %0;" ::"n"(EPI_THREADS) : "memory"); }

template <typename T>
__device__ __forceinline__ T ldg_ptr(const void *const *p)
{
    return reinterpret_cast<T>(__ldg(reinterpret_cast<const unsigned long long *>(p)));
}

// ---- the memory-bound operators, run by all worker threads (tid = 0 .. EPI_THREADS-1) on one item.  Kept out of line:
// they are rare and long, and inlined they cost the convolution roles registers.
// Depth-wise convolution item: 2^tr_log output rows x tw_valid columns x BN channels of image n (see
// rowop::dwconv_tile); the window is read through L2 -- other SMs produced it during this launch.
__device__ __noinline__ void dwconv_item(const WfStage *sp, int n, int tile_r, int tile_w, int tile_c, int tid, uint8_t *stg)
{
    rowop::DwGeom g;
    g.Hin = __ldg(&sp->Hin); g.Win = __ldg(&sp->Win); g.C = __ldg(&sp->Cin); g.Ho = __ldg(&sp->Ho); g.Wo = __ldg(&sp->Wo);
    g.kh = __ldg(&sp->kh); g.kw = __ldg(&sp->kw); g.sh = __ldg(&sp->sh); g.sw = __ldg(&sp->sw);
    g.ph = __ldg(&sp->ph); g.pw = __ldg(&sp->pw); g.dh = __ldg(&sp->dh); g.dw = __ldg(&sp->dw);
    g.act = __ldg(&sp->act);
    g.t.R = 1 << __ldg(&sp->tr_log); g.t.tw = __ldg(&sp->tw_valid); g.t.cc = __ldg(&sp->BN);
    g.x = ldg_ptr<const uint16_t *>(&sp->x);
    g.res = ldg_ptr<const uint16_t *>(&sp->res);
    g.res_pos = g.res ? __ldg(&sp->res_pos) : LOP_RES_NONE;
    g.w_taps = ldg_ptr<const uint16_t *>(&sp->w_taps);
    g.scale = ldg_ptr<const float *>(reinterpret_cast<const void *const *>(&sp->scale));
    g.shift = ldg_ptr<const float *>(reinterpret_cast<const void *const *>(&sp->shift));
    g.y = ldg_ptr<uint16_t *>(reinterpret_cast<const void *const *>(&sp->y));
    g.dbg = nullptr; g.N = __ldg(&sp->N);                     // checked execution runs the stand-alone kernels
    const int oh0 = __ldg(&sp->oh_lo) + tile_r * g.t.R, ow0 = tile_w * g.t.tw;
    rowop::dwconv_tile<true, 1, EPI_THREADS>(g, n, oh0, min(g.t.R, __ldg(&sp->oh_hi) - oh0), ow0, min(g.t.tw, g.Wo - ow0), tile_c * g.t.cc,
                                             reinterpret_cast<float *>(stg), tid);
}

// Layer normalisation over the channels of the pixels of output row oh of image n (rowop::ln_pixels: a group of
// lanes per pixel, four vectors in flight per lane).
template <int VPL>
__device__ __forceinline__ void layernorm_row(const uint16_t *x, uint16_t *y, const float *gain, const float *offset, int C, int Wo, long long row0,
                                              int tid)
{
    constexpr int PPG = 4 / VPL;
    const int lanes_log = rowop::ln_lanes_log(C >> 3);
    const int sub = tid & ((1 << lanes_log) - 1), slot = tid >> lanes_log, per_pass = (EPI_THREADS >> lanes_log) * PPG;
    for (int w0 = 0; w0 < Wo; w0 += per_pass) {               // the same trip count for every lane
        long long o[PPG];
        bool live[PPG];
#pragma unroll
        for (int q = 0; q < PPG; ++q) {
            const int ow = w0 + slot * PPG + q;
            live[q] = ow < Wo;
            o[q] = (row0 + ow) * C;
        }
        rowop::ln_pixels<true, VPL, PPG>(x, y, C, lanes_log, sub, o, live, gain, offset);
    }
}
__device__ __noinline__ void layernorm_item(const WfStage *sp, int n, int oh, int tid)
{
    const int C = __ldg(&sp->Cin), Ho = __ldg(&sp->Ho), Wo = __ldg(&sp->Wo);
    const uint16_t *x = ldg_ptr<const uint16_t *>(&sp->x);
    uint16_t *y = ldg_ptr<uint16_t *>(reinterpret_cast<const void *const *>(&sp->y));
    const float *gain = ldg_ptr<const float *>(reinterpret_cast<const void *const *>(&sp->scale));
    const float *offset = ldg_ptr<const float *>(reinterpret_cast<const void *const *>(&sp->shift));
    const long long row0 = ((long long)n * Ho + oh) * Wo;
    const int vpl = rowop::ln_vpl(C >> 3);
    if (vpl == 1) layernorm_row<1>(x, y, gain, offset, C, Wo, row0, tid);
    else if (vpl == 2) layernorm_row<2>(x, y, gain, offset, C, Wo, row0, tid);
    else layernorm_row<4>(x, y, gain, offset, C, Wo, row0, tid);
}

// Channel concatenation of output row oh of image n: the main input's Cin channels, then the second input's Cout - Cin.
__device__ __noinline__ void concat_item(const WfStage *sp, int n, int oh, int tid)
{
    const int Cin = __ldg(&sp->Cin), Cout = __ldg(&sp->Cout), Ho = __ldg(&sp->Ho), Wo = __ldg(&sp->Wo);
    const int va = Cin >> 3, vo = Cout >> 3;
    const long long row = ((long long)n * Ho + oh) * Wo;
    const uint4 *xa = reinterpret_cast<const uint4 *>(ldg_ptr<const __nv_bfloat16 *>(&sp->x) + row * Cin);
    const uint4 *xb = reinterpret_cast<const uint4 *>(ldg_ptr<const __nv_bfloat16 *>(&sp->res) + row * (Cout - Cin));
    uint4 *y = reinterpret_cast<uint4 *>(ldg_ptr<__nv_bfloat16 *>(reinterpret_cast<const void *const *>(&sp->y)) + row * Cout);
    for (int idx = tid; idx < Wo * vo; idx += EPI_THREADS) {
        const int ow = idx / vo, v = idx - ow * vo;
        y[idx] = v < va ? __ldcg(xa + (long long)ow * va + v) : __ldcg(xb + (long long)ow * (vo - va) + (v - va));
    }
}

// len bytes (a multiple of 2) from host memory the device can address to device memory, by the 32 lanes of a warp.
// Host lines are read around the caches (they change between launches without the device knowing); eight 16-byte
// loads per lane are in flight to cover the host link's latency.  src and dst agree modulo 16.
#ifndef LOP_FETCH_DEPTH
#define LOP_FETCH_DEPTH 8
#endif
constexpr int FETCH_DEPTH = LOP_FETCH_DEPTH;
__device__ __forceinline__ void fetch_bytes(const uint8_t *src, uint8_t *dst, int len, int lane)
{
    int head = (16 - (int)(reinterpret_cast<uintptr_t>(src) & 15)) & 15;
    if (head > len) head = len;
    for (int i = 2 * lane; i < head; i += 64)
        *reinterpret_cast<uint16_t *>(dst + i) = __ldcv(reinterpret_cast<const uint16_t *>(src + i));
    const int nvec = (len - head) >> 4;
    const uint4 *s4 = reinterpret_cast<const uint4 *>(src + head);
    uint4 *d4 = reinterpret_cast<uint4 *>(dst + head);
    for (int v0 = 0; v0 < nvec; v0 += FETCH_DEPTH * 32) {
        uint4 q[FETCH_DEPTH];
#pragma unroll
        for (int u = 0; u < FETCH_DEPTH; ++u) {
            const int v = v0 + u * 32 + lane;
            if (v < nvec) q[u] = __ldcv(s4 + v);
        }
#pragma unroll
        for (int u = 0; u < FETCH_DEPTH; ++u) {
            const int v = v0 + u * 32 + lane;
            if (v < nvec) d4[v] = q[u];
        }
    }
    for (int i = head + (nvec << 4) + 2 * lane; i < len; i += 64)
        *reinterpret_cast<uint16_t *>(dst + i) = __ldcv(reinterpret_cast<const uint16_t *>(src + i));
}

// FETCH: the program has a fetch list; the CTA then has one more warp, which walks it.
// FETCH: one more warp per CTA brings the chain input from host memory.  ROWOPS: the program has depth-wise /
// normalisation / concatenation stages; programs without them run an instantiation that does not carry their code.
template <bool FETCH, bool ROWOPS>
__global__ void __launch_bounds__(FETCH ? WF_THREADS + 32 : WF_THREADS, 1) wavefront_kernel(const WfParams P)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t *smem = smem_raw + (base - raw);
    const int SA = P.sa, SB = P.sb;
    const uint32_t a_slot_bytes = P.a_slot_bytes, b_slot_bytes = P.b_slot_bytes;
    const uint32_t a0 = base, b0 = a0 + (uint32_t)SA * a_slot_bytes, stg0 = b0 + (uint32_t)SB * b_slot_bytes;
    const uint32_t bars = stg0 + P.stg_bytes;
    const uint32_t full_a = bars, empty_a = full_a + 8u * SA, full_b = empty_a + 8u * SA, empty_b = full_b + 8u * SB;
    const uint32_t accf0 = empty_b + 8u * SB, acce0 = accf0 + 16u;
    const uint32_t pubf0 = acce0 + 16u, pube0 = pubf0 + 8u * WF_PUBQ;
    const uint32_t ssf0 = pube0 + 8u * WF_PUBQ, sse0 = ssf0 + 16u;      // scale/shift buffers of two tiles: full / empty
    uint8_t *tail = smem + (sse0 + 16u - base);
    volatile uint32_t *misc = reinterpret_cast<volatile uint32_t *>(tail);      // [0] TMEM base, [1] abort, [2] run, [3] epilogue failure
    float *s_scale = reinterpret_cast<float *>(tail + 64);                       // [2][128]: per-channel scale of this and the next tile
    float *s_shift = s_scale + 256;                                              // [2][128]
    long long *row_pix = reinterpret_cast<long long *>(tail + 64 + 2048);        // [128]: element offset of anchor m's output, or -1
    long long *pool_pix = row_pix + 128;                                         // [32]: element offset of a 2x2 window's pooled output, or -1
    uint8_t *stg = smem + (stg0 - base);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0 && blockIdx.x < 4) {
        tr(TRACE_ITEMS - 8 + (int)blockIdx.x, 0);
        trv(TRACE_ITEMS - 8 + (int)blockIdx.x, 4, (unsigned long long)clock64());
    }
    if (threadIdx.x == 0) {
        for (int s = 0; s < SA; ++s) {
            mbar_init(full_a + 8u * s, 1);
            mbar_init(empty_a + 8u * s, 1);
        }
        for (int s = 0; s < SB; ++s) {
            mbar_init(full_b + 8u * s, 1);
            mbar_init(empty_b + 8u * s, 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(accf0 + 8u * b, 1);
            mbar_init(acce0 + 8u * b, 1);
            mbar_init(ssf0 + 8u * b, 1);
            mbar_init(sse0 + 8u * b, 1);
        }
        for (int q = 0; q < WF_PUBQ; ++q) {
            mbar_init(pubf0 + 8u * q, 1);
            mbar_init(pube0 + 8u * q, 1);
        }
        misc[1] = 0;
        misc[2] = ld_acquire(P.counters) + 1u;                 // this launch is run number (completed runs + 1)
        misc[3] = 0;
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
    if (threadIdx.x == 0 && blockIdx.x < 4) tr(TRACE_ITEMS - 8 + (int)blockIdx.x, 1);
    const uint32_t tmem_base = misc[0];
    const unsigned run = misc[2];
    volatile uint32_t *abort_flag = &misc[1];
    volatile uint32_t *epi_fail = &misc[3];
    const int G = gridDim.x;
    const int NI = P.n_items;
    const int4 zero4 = make_int4(0, 0, 0, 0);

    if (warp == 0) {
        // ---------------- dependency wait (all lanes) + TMA producer (lane 0) ----------------
        int item = blockIdx.x;
        int4 cur = item < NI ? __ldg(&P.items[item]) : zero4;
        int4 nxt = item + G < NI ? __ldg(&P.items[item + G]) : zero4;
        int2 dep_cur = (item < NI && lane < rec_ndep(cur)) ? __ldg(&P.deps[rec_dep0(cur) + lane]) : make_int2(0, 0);
        int sidx = -1;
        int kind = -1, mode = 0, oh_lo = 0, tr_log = 0, p_log = 0, tw_valid = 0, BN = 0, BK = 0, n_chunks = 1, n_taps = 1, tbx = 1,
            amask = 0, kh = 1, kw = 1, sh = 1, sw = 1, ph = 0, pw = 0, dh = 1, dw = 1;
        uint32_t a_bytes = 0, b_bytes = 0;
        const CUtensorMap *maps = nullptr;
        const float *scale = nullptr, *shift = nullptr;
        int slab_offh = 0, slab_offw = 0, slab_mi = 0, n_boxes = 1, cps = 1;
        bool slab_have = true;
        uint32_t a_slot = 0, a_phase = 0, b_slot = 0, b_phase = 0, pc = 0;
        bool w_kept = false;                                   // (lane 0) the ring holds the weights of tile key w_key
        long long w_key = -1;
        for (; item < NI; item += G) {
            // two items ahead: the record; one item ahead: this lane's dependency entry
            const int4 nn = item + 2 * G < NI ? __ldg(&P.items[item + 2 * G]) : zero4;
            const int2 dep_nxt = (item + G < NI && lane < rec_ndep(nxt)) ? __ldg(&P.deps[rec_dep0(nxt) + lane]) : make_int2(0, 0);
            if (rec_stage(cur) != sidx) {
                sidx = rec_stage(cur);
                const WfStage *sp = &P.stages[sidx];
                kind = __ldg(&sp->kind); mode = __ldg(&sp->mode); oh_lo = __ldg(&sp->oh_lo);
                tr_log = __ldg(&sp->tr_log); p_log = __ldg(&sp->p_log); tw_valid = __ldg(&sp->tw_valid);
                BN = __ldg(&sp->BN); BK = __ldg(&sp->BK); n_chunks = __ldg(&sp->n_chunks); n_taps = __ldg(&sp->n_taps);
                tbx = __ldg(&sp->tb); amask = __ldg(&sp->a_valid_mask);
                a_bytes = __ldg(&sp->a_bytes); b_bytes = __ldg(&sp->b_bytes);
                maps = P.maps + __ldg(&sp->map_base);
                kh = __ldg(&sp->kh); kw = __ldg(&sp->kw); sh = __ldg(&sp->sh); sw = __ldg(&sp->sw);
                ph = __ldg(&sp->ph); pw = __ldg(&sp->pw); dh = __ldg(&sp->dh); dw = __ldg(&sp->dw);
                scale = ldg_ptr<const float *>(reinterpret_cast<const void *const *>(&sp->scale));
                shift = ldg_ptr<const float *>(reinterpret_cast<const void *const *>(&sp->shift));
                // slab mode: the box starts at the first tap's offset; which parity map that is and how far in
                const int offh = floor_div_i(-ph, sh), offw = floor_div_i(-pw, sw);
                slab_offh = offh; slab_offw = offw;
                slab_mi = (-ph - offh * sh) * sw + (-pw - offw * sw);
                slab_have = (amask >> slab_mi) & 1;
                n_boxes = n_chunks * ((n_taps + tbx - 1) / tbx);
                cps = __ldg(&sp->cps);
            }
            if (kind == WF_CONV) {
                if (lane == 0) tr(item, 0);
                // the tile's per-channel scale / shift go to shared memory from here, a tile ahead of the epilogue
                // that uses them: their load latency is off the workers' path
                bool ok = __all_sync(0xffffffffu, mbar_wait_abortable(sse0 + 8u * (pc & 1u), ((pc >> 1) & 1u) ^ 1u, abort_flag));
                if (ok) {
                    float *ds = s_scale + 128 * (pc & 1u), *dsh = s_shift + 128 * (pc & 1u);
                    const int c0 = rec_cout(cur) * BN;
                    for (int i = lane; i < BN; i += 32) {
                        ds[i] = scale ? __ldg(scale + c0 + i) : 1.0f;
                        dsh[i] = shift ? __ldg(shift + c0 + i) : 0.0f;
                    }
                    __syncwarp();
                }
                ok = ok && wait_deps_warp(P, rec_dep0(cur), rec_ndep(cur), dep_cur, run, lane);
                if (ok) {
                    // "scale / shift are in place AND the tile's producers (the residual's included) are done": the
                    // workers fetch the residual tile behind this barrier, while the operands are still on their way
                    if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(ssf0 + 8u * (pc & 1u)) : "memory");
                    ++pc;
                }
                int fail = 0;
                if (!ok) {
                    if (lane == 0) atomicOr(P.status, 0x10u);
                    fail = 1;
                } else if (lane == 0) {
                    tr(item, 1);
                    asm volatile("fence.proxy.async.global;" ::: "memory");       // producers' generic-proxy writes -> our TMA reads
                    const int ow0 = rec_tw(cur) * tw_valid;
                    const int oh0 = oh_lo + (rec_tr(cur) << tr_log);
                    const int n0 = rec_tn(cur) * (128 >> (p_log + tr_log));
                    const int co0 = rec_cout(cur) * BN;
                    // Weights stay in their ring slots from one tile to the next while consecutive tiles of this CTA
                    // use the same ones (same layer, same output channels) and all their boxes fit the ring: only the
                    // first such tile loads them.  The MMA issuer takes the same decisions from the same records and
                    // frees the slots when a tile with other weights comes up.
                    const long long wkey = (long long)(maps - P.maps) * 65536 + rec_cout(cur);
                    const bool can_keep = mode == WF_SLAB && n_boxes <= SB;
                    const bool reuse_w = w_kept && can_keep && wkey == w_key;
                    w_kept = reuse_w || can_keep;
                    w_key = wkey;
                    if (cps > 1 && mode == WF_SLAB) {
                        for (int ch = 0; ch < n_chunks && !fail; ch += cps) {
                            const int g = min(cps, n_chunks - ch);
                            if (!mbar_wait_abortable(empty_a + 8u * a_slot, a_phase ^ 1u, abort_flag) ||
                                !mbar_wait_abortable(empty_b + 8u * b_slot, b_phase ^ 1u, abort_flag)) { fail = 1; break; }
                            const uint32_t fa = full_a + 8u * a_slot, fb = full_b + 8u * b_slot;
                            mbar_expect_tx(fa, (uint32_t)g * a_bytes);
                            mbar_expect_tx(fb, (uint32_t)g * b_bytes);
                            for (int u = 0; u < g; ++u) {
                                tma_load_4d(a0 + a_slot * a_slot_bytes + (uint32_t)u * a_bytes, maps + slab_mi, fa, (ch + u) * BK,
                                            slab_have ? ow0 + slab_offw : -65536, slab_have ? oh0 + slab_offh : -65536, n0);
                                tma_load_3d(b0 + b_slot * b_slot_bytes + (uint32_t)u * b_bytes, maps + 4, fb, (ch + u) * BK, co0, 0);
                            }
                            if (++a_slot == (uint32_t)SA) { a_slot = 0; a_phase ^= 1u; }
                            if (++b_slot == (uint32_t)SB) { b_slot = 0; b_phase ^= 1u; }
                        }
                    } else {
                    int tap_u = 0, in_slot = 0;                        // per-tap mode: boxes issued so far, boxes in the open slot
                    for (int ch = 0; ch < n_chunks && !fail; ++ch) {
                        if (mode == WF_SLAB) {
                            // the whole receptive window of the tile in one box: its first tap's offset places it
                            const int mi = slab_mi, offh = slab_offh, offw = slab_offw;
                            const bool have = slab_have;
                            if (!mbar_wait_abortable(empty_a + 8u * a_slot, a_phase ^ 1u, abort_flag)) { fail = 1; break; }
                            const uint32_t fa = full_a + 8u * a_slot;
                            mbar_expect_tx(fa, a_bytes);
                            tma_load_4d(a0 + a_slot * a_slot_bytes, maps + mi, fa, ch * BK, have ? ow0 + offw : -65536,
                                        have ? oh0 + offh : -65536, n0);
                            if (++a_slot == (uint32_t)SA) { a_slot = 0; a_phase ^= 1u; }
                            for (int t0 = 0; t0 < n_taps && !reuse_w; t0 += tbx) {
                                if (!mbar_wait_abortable(empty_b + 8u * b_slot, b_phase ^ 1u, abort_flag)) { fail = 1; break; }
                                const uint32_t fb = full_b + 8u * b_slot;
                                mbar_expect_tx(fb, b_bytes);
                                tma_load_3d(b0 + b_slot * b_slot_bytes, maps + 4, fb, ch * BK, co0, t0);
                                if (++b_slot == (uint32_t)SB) { b_slot = 0; b_phase ^= 1u; }
                            }
                        } else {
                            // one activation and one weight box per (channel chunk, tap); `cps` consecutive taps share a
                            // slot of each ring and its barrier (strides are 1 or 2 almost always: no division then)
                            for (int a = 0; a < kh && !fail; ++a) {
                                const int qh = a * dh - ph;
                                const int offh = sh == 1 ? qh : (sh == 2 ? qh >> 1 : floor_div_i(qh, sh)), parh = qh - offh * sh;
                                for (int b = 0; b < kw; ++b, ++tap_u) {
                                    const int qw = b * dw - pw;
                                    const int offw = sw == 1 ? qw : (sw == 2 ? qw >> 1 : floor_div_i(qw, sw)), parw = qw - offw * sw;
                                    const int mi = parh * sw + parw;
                                    const bool have = (amask >> mi) & 1;
                                    if (in_slot == 0) {
                                        const int g = min(cps, n_chunks * n_taps - tap_u);
                                        if (!mbar_wait_abortable(empty_a + 8u * a_slot, a_phase ^ 1u, abort_flag) ||
                                            !mbar_wait_abortable(empty_b + 8u * b_slot, b_phase ^ 1u, abort_flag)) { fail = 1; break; }
                                        mbar_expect_tx(full_a + 8u * a_slot, (uint32_t)g * a_bytes);
                                        mbar_expect_tx(full_b + 8u * b_slot, (uint32_t)g * b_bytes);
                                    }
                                    tma_load_4d(a0 + a_slot * a_slot_bytes + (uint32_t)in_slot * a_bytes, maps + mi, full_a + 8u * a_slot, ch * BK,
                                                have ? ow0 + offw : -65536, have ? oh0 + offh : -65536, n0);
                                    tma_load_3d(b0 + b_slot * b_slot_bytes + (uint32_t)in_slot * b_bytes, maps + 4, full_b + 8u * b_slot, ch * BK, co0,
                                                a * kw + b);
                                    if (++in_slot == cps || tap_u + 1 == n_chunks * n_taps) {
                                        in_slot = 0;
                                        if (++a_slot == (uint32_t)SA) { a_slot = 0; a_phase ^= 1u; }
                                        if (++b_slot == (uint32_t)SB) { b_slot = 0; b_phase ^= 1u; }
                                    }
                                }
                            }
                        }
                    }
                    }
                    if (fail) atomicOr(P.status, 0x1u);
                    tr(item, 2);
                }
                if (__any_sync(0xffffffffu, fail | (int)*abort_flag)) {
                    if (lane == 0) {
                        atomicExch(P.counters + 2, 1u);
                        *abort_flag = 1;
                    }
                    break;
                }
            }
            cur = nxt; dep_cur = dep_nxt; nxt = nn;
        }
    } else if (warp == 1) {
        if (lane == 0) {
            // ---------------- MMA issuer ----------------
            int item = blockIdx.x;
            int4 cur = item < NI ? __ldg(&P.items[item]) : zero4;
            int sidx = -1;
            int kind = -1, mode = 0, n_chunks = 1, n_taps = 1, tbx = 1, kw = 1, dh = 1, dw = 1, p_log = 0, ksteps = 1;
            uint32_t idesc = 0, desc_hi = 0, row_bytes = 0, tap_bytes = 0;
            uint32_t a_slot = 0, a_phase = 0, b_slot = 0, b_phase = 0, cnt = 0;
            bool fail = false, row3x64 = false;
            bool w_kept = false;                               // weights kept in ring slots w_first .. w_first + w_n - 1 for key w_key
            long long w_key = -1;
            uint32_t w_first = 0, w_n = 0;
            int map_base = 0, nblk = 1, cps = 1;               // nblk: weight boxes per channel chunk; cps: chunks per ring slot
            uint32_t a_bytes = 0, b_bytes = 0;
            uint32_t tap16 = 0, step_w16 = 0, step_h16 = 0;    // descriptor start-field steps: next tap's weights, next filter column / row
#ifdef LOP_WF_TRACE
            long long dbg_c0 = 0, dbg_fence = 0, dbg_mma = 0;
#endif
            for (; item < NI && !fail; item += G) {
                const int4 nxt = item + G < NI ? __ldg(&P.items[item + G]) : zero4;
                if (rec_stage(cur) != sidx) {
                    sidx = rec_stage(cur);
                    const WfStage *sp = &P.stages[sidx];
                    kind = __ldg(&sp->kind); mode = __ldg(&sp->mode);
                    n_chunks = __ldg(&sp->n_chunks); n_taps = __ldg(&sp->n_taps); tbx = __ldg(&sp->tb);
                    kw = __ldg(&sp->kw); dh = __ldg(&sp->dh); dw = __ldg(&sp->dw); p_log = __ldg(&sp->p_log);
                    map_base = __ldg(&sp->map_base);
                    nblk = (n_taps + tbx - 1) / tbx;
                    ksteps = __ldg(&sp->BK) / 16;
                    idesc = __ldg(&sp->idesc);
                    desc_hi = ((__ldg(&sp->sbo_bytes) >> 4) & 0x3FFFu) | (1u << 14) | (__ldg(&sp->layout_code) << 29);
                    row_bytes = __ldg(&sp->row_bytes);
                    tap_bytes = (uint32_t)__ldg(&sp->BN) * row_bytes;
                    tap16 = tap_bytes >> 4;
                    step_w16 = ((uint32_t)dw * row_bytes) >> 4;
                    step_h16 = ((uint32_t)(dh << p_log) * row_bytes) >> 4;
                    row3x64 = mode == WF_SLAB && n_taps == 9 && kw == 3 && tbx == 3 && ksteps == 4 && dw == 1;
                    a_bytes = __ldg(&sp->a_bytes); b_bytes = __ldg(&sp->b_bytes);
                    cps = __ldg(&sp->cps);
                }
                if (kind == WF_CONV) {
                    const uint32_t buf = cnt & 1u;
                    if (!mbar_wait_abortable(acce0 + 8u * buf, ((cnt >> 1) & 1u) ^ 1u, abort_flag)) { fail = true; break; }
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    tr(item, 3);
                    const uint32_t acc = tmem_base + buf * 256u;
                    uint32_t accumulate = 0;
                    // kept weights (see the loader): used in place by tiles with the same key, freed -- once the MMAs
                    // that read them are done -- when a tile with another key comes up
                    // (this thread issues every MMA of the CTA and is bound by its own instruction latencies: no division
                    // or modulo in these loops)
                    const uint32_t n_boxes = (uint32_t)(n_chunks * nblk);
                    const long long wkey = (long long)map_base * 65536 + rec_cout(cur);
                    const bool can_keep = mode == WF_SLAB && n_boxes <= (uint32_t)SB;
                    const bool reuse_w = w_kept && can_keep && wkey == w_key;
                    if (w_kept && !reuse_w) {
                        for (uint32_t i = 0, sl = w_first; i < w_n; ++i) {
                            umma_commit(empty_b + 8u * sl);
                            if (++sl == (uint32_t)SB) sl = 0;
                        }
                        w_kept = false;
                    }
                    if (!reuse_w && can_keep) { w_kept = true; w_key = wkey; w_first = b_slot; w_n = n_boxes; }
                    uint32_t ws = w_first;                                  // kept box of the current (chunk, tap block)
                    if (reuse_w && row3x64 && n_chunks == 1) {
                        // the common tile of a 3x3 / 64-channel layer with its weights in place: 36 MMAs, nothing between
                        // them but the start addresses of the three filter rows
                        if (!mbar_wait_abortable(full_a + 8u * a_slot, a_phase, abort_flag)) { fail = true; break; }
                        tr(item, 13);
                        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                        const uint32_t la = (((a0 + a_slot * a_slot_bytes) & 0x3FFFFu) >> 4) | (1u << 16);
                        const uint32_t row16 = (uint32_t)(dh << p_log) * 8u;          // one filter row further down the slab, in 16-byte units
                        const uint32_t s0 = w_first, s1 = s0 + 1 == (uint32_t)SB ? 0u : s0 + 1, s2 = s1 + 1 == (uint32_t)SB ? 0u : s1 + 1;
                        mma_row3x64(acc, la, (((b0 + s0 * b_slot_bytes) & 0x3FFFFu) >> 4) | (1u << 16), tap_bytes >> 4, desc_hi, idesc, accumulate);
                        mma_row3x64(acc, la + row16, (((b0 + s1 * b_slot_bytes) & 0x3FFFFu) >> 4) | (1u << 16), tap_bytes >> 4, desc_hi, idesc, accumulate);
                        mma_row3x64(acc, la + 2u * row16, (((b0 + s2 * b_slot_bytes) & 0x3FFFFu) >> 4) | (1u << 16), tap_bytes >> 4, desc_hi, idesc, accumulate);
                        umma_commit(empty_a + 8u * a_slot);
                        if (++a_slot == (uint32_t)SA) { a_slot = 0; a_phase ^= 1u; }
                    } else if (cps > 1 && mode == WF_SLAB) {
                        for (int ch = 0; ch < n_chunks; ch += cps) {
                            const int g = min(cps, n_chunks - ch);
                            if (!mbar_wait_abortable(full_a + 8u * a_slot, a_phase, abort_flag) ||
                                !mbar_wait_abortable(full_b + 8u * b_slot, b_phase, abort_flag)) { fail = true; break; }
                            if (ch == 0) tr(item, 13);
                            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                            uint32_t la = desc_lo(a0 + a_slot * a_slot_bytes), lb = desc_lo(b0 + b_slot * b_slot_bytes);
                            for (int u = 0; u < g; ++u, la += a_bytes >> 4, lb += b_bytes >> 4) mma_ksteps_f<4>(acc, la, lb, desc_hi, idesc, accumulate);
                            umma_commit(empty_a + 8u * a_slot);
                            umma_commit(empty_b + 8u * b_slot);
                            if (++a_slot == (uint32_t)SA) { a_slot = 0; a_phase ^= 1u; }
                            if (++b_slot == (uint32_t)SB) { b_slot = 0; b_phase ^= 1u; }
                        }
                    } else {
                    int tap_u = 0, in_slot = 0;                        // per-tap mode: boxes consumed so far, boxes used of the open slot
                    for (int ch = 0; ch < n_chunks && !fail; ++ch) {
                        if (mode == WF_SLAB) {
                            if (!mbar_wait_abortable(full_a + 8u * a_slot, a_phase, abort_flag)) { fail = true; break; }
                            if (ch == 0) tr(item, 13);
                            const uint32_t sa = a0 + a_slot * a_slot_bytes;
                            int ta = 0, tb = 0;                             // filter position of tap t0
                            // start field of the tap's activation operand: one pixel further per filter column, one
                            // slab row further per filter row (kept incrementally: this thread pays for every instruction)
                            uint32_t la_row = desc_lo(sa), la = la_row;
                            for (int t0 = 0; t0 < n_taps; t0 += tbx) {
                                uint32_t bs = b_slot;
                                if (reuse_w) {
                                    bs = ws;
                                    if (++ws == (uint32_t)SB) ws = 0;
                                } else if (!mbar_wait_abortable(full_b + 8u * b_slot, b_phase, abort_flag)) { fail = true; break; }
                                if (ch == 0 && t0 == 0) tr(item, 14);
#ifdef LOP_WF_TRACE
                                const long long c0 = clock64();
                                if (t0 == 0) dbg_c0 = c0;
#endif
                                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#ifdef LOP_WF_TRACE
                                const long long c1 = clock64();
                                dbg_fence += c1 - c0;
#endif
                                const uint32_t sb = b0 + bs * b_slot_bytes;
                                if (row3x64) {
                                    // box = one row of a 3x3 filter: the slab row it starts at, then constants
                                    const uint32_t pa = sa + (uint32_t)((ta * dh) << p_log) * 128u;
                                    mma_row3x64(acc, ((pa & 0x3FFFFu) >> 4) | (1u << 16), ((sb & 0x3FFFFu) >> 4) | (1u << 16), tap_bytes >> 4,
                                                desc_hi, idesc, accumulate);
#ifdef LOP_WF_TRACE
                                    dbg_mma += clock64() - c1;
#endif
                                    ++ta;
                                } else {
                                    const int t1 = min(t0 + tbx, n_taps);
                                    uint32_t lb = desc_lo(sb);
                                    for (int t = t0; t < t1; ++t, lb += tap16) {
                                        // tap (ta, tb): the same box, read (ta*dh*P + tb*dw) pixels further on
                                        mma_tap_f(acc, la, lb, desc_hi, idesc, ksteps, accumulate);
                                        la += step_w16;
                                        if (++tb == kw) { tb = 0; la_row += step_h16; la = la_row; }
                                    }
                                }
                                if (!reuse_w) {
                                    if (!can_keep) umma_commit(empty_b + 8u * b_slot);
                                    if (++b_slot == (uint32_t)SB) { b_slot = 0; b_phase ^= 1u; }
                                }
                            }
                            umma_commit(empty_a + 8u * a_slot);
                            if (++a_slot == (uint32_t)SA) { a_slot = 0; a_phase ^= 1u; }
                        } else {
                            for (int t = 0; t < n_taps; ++t, ++tap_u) {
                                if (in_slot == 0) {
                                    if (!mbar_wait_abortable(full_a + 8u * a_slot, a_phase, abort_flag) ||
                                        !mbar_wait_abortable(full_b + 8u * b_slot, b_phase, abort_flag)) { fail = true; break; }
                                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                                }
                                mma_tap(acc, a0 + a_slot * a_slot_bytes + (uint32_t)in_slot * a_bytes, b0 + b_slot * b_slot_bytes + (uint32_t)in_slot * b_bytes,
                                        desc_hi, idesc, ksteps, accumulate);
                                if (++in_slot == cps || tap_u + 1 == n_chunks * n_taps) {
                                    in_slot = 0;
                                    umma_commit(empty_a + 8u * a_slot);
                                    umma_commit(empty_b + 8u * b_slot);
                                    if (++a_slot == (uint32_t)SA) { a_slot = 0; a_phase ^= 1u; }
                                    if (++b_slot == (uint32_t)SB) { b_slot = 0; b_phase ^= 1u; }
                                }
                            }
                        }
                    }
                    }
                    if (fail) break;
#ifdef LOP_WF_TRACE
                    trv(item, 8, (unsigned long long)dbg_fence);
                    trv(item, 9, (unsigned long long)dbg_mma);
                    trv(item, 10, (unsigned long long)(clock64() - dbg_c0));
                    dbg_fence = dbg_mma = 0;
#endif
                    tr(item, 15);
                    umma_commit(accf0 + 8u * buf);
                    tr(item, 4);
                    ++cnt;
                }
                cur = nxt;
            }
            if (fail) {
                atomicOr(P.status, 0x2u);
                atomicExch(P.counters + 2, 1u);
                *abort_flag = 1;
            }
        }
    } else if (warp == 2) {
        if (lane == 0) {
            // ---------------- publisher ----------------
            // Makes finished items visible: the workers' stores happen before their barrier and the arrive that
            // this thread waits for, so its fence orders them before the release increment of the counter.
            int item = blockIdx.x;
            int4 cur = item < NI ? __ldg(&P.items[item]) : zero4;
            int sidx = -1, ctr_base = 0;
            bool fail = false;
            for (uint32_t k = 0; item < NI; item += G, ++k) {
                const int4 nxt = item + G < NI ? __ldg(&P.items[item + G]) : zero4;
                if (rec_stage(cur) != sidx) {
                    sidx = rec_stage(cur);
                    ctr_base = __ldg(&P.stages[sidx].ctr_base);
                }
                const uint32_t q = k % WF_PUBQ, round = k / WF_PUBQ;
                if (!mbar_wait_abortable(pubf0 + 8u * q, round & 1u, abort_flag)) { fail = !*abort_flag; break; }
                __threadfence();
                atomicAdd(P.counters + ctr_base + rec_tr(cur), 1u);
                asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(pube0 + 8u * q) : "memory");
                cur = nxt;
            }
            if (fail) {
                atomicOr(P.status, 0x8u);
                atomicExch(P.counters + 2, 1u);
                *abort_flag = 1;
            }
        }
    } else if (FETCH && warp == WF_FIRST_WORKER + WF_WORKER_WARPS) {
        // ---------------- fetch warp: the chain input, host memory -> device, in list order ----------------
        const unsigned done_before = (run - 1u) * (unsigned)P.n_fetch;          // counters[3] never resets
        const uint8_t *src0 = static_cast<const uint8_t *>(P.fetch_src);
        uint8_t *dst0 = static_cast<uint8_t *>(P.fetch_dst);
        for (int j = blockIdx.x; j < P.n_fetch; j += G) {
            const int4 rec = __ldg(&P.fetch_items[j]);
            if (j >= P.fetch_window) {
                // the window keeps the link's queue short, so that early rows are not stuck behind late ones
                const unsigned target = done_before + (unsigned)(j - P.fetch_window + 1);
                int ok = 1;
                if (lane == 0) {
                    for (uint32_t i = 0; (int)(ld_acquire(P.counters + 3) - target) < 0; ++i) {
                        if (i >= P.spin_limit) { ok = 0; atomicOr(P.status, 0x20u); break; }
                        if ((i & 63u) == 63u && (ld_relaxed(P.counters + 2) != 0u || *abort_flag)) { ok = -1; break; }
                        __nanosleep(64);
                    }
                }
                ok = __shfl_sync(0xffffffffu, ok, 0);
                if (ok <= 0) {
                    if (ok == 0 && lane == 0) {
                        atomicExch(P.counters + 2, 1u);
                        *abort_flag = 1;
                    }
                    break;
                }
            }
            const long long off = (long long)(((unsigned long long)(unsigned)rec.y << 32) | (unsigned)rec.x);
            if (lane == 0) tr(TRACE_FETCH0 + j, 0);
            fetch_bytes(src0 + off, dst0 + off, rec.z, lane);
            __syncwarp();
            if (lane == 0) {
                tr(TRACE_FETCH0 + j, 1);
                __threadfence();                                   // the warp's stores, then the release increments
                atomicAdd(P.counters + rec.w, 1u);
                atomicAdd(P.counters + 3, 1u);
                tr(TRACE_FETCH0 + j, 2);
            }
        }
    } else {
        // ---------------- epilogue / SIMT warps ----------------
        const int tid = threadIdx.x - 32 * WF_FIRST_WORKER;
        const int g = warp & 3;                               // TMEM lane group this warp may read
        const int m = g * 32 + lane;                          // accumulator row = anchor of this thread
        const int cgrp = (warp - WF_FIRST_WORKER) >> 2;                     // which share of the tile's 16-column chunks is this warp's
        int item = blockIdx.x;
        int4 cur = item < NI ? __ldg(&P.items[item]) : zero4;
        int4 nxt = item + G < NI ? __ldg(&P.items[item + G]) : zero4;
        int2 dep_cur = (warp == WF_FIRST_WORKER && item < NI && lane < rec_ndep(cur)) ? __ldg(&P.deps[rec_dep0(cur) + lane]) : make_int2(0, 0);
        int sidx = -1;
        uint32_t cnt = 0, done_items = 0;
        int kind = -1, oh_lo = 0, oh_hi = 0, p_log = 0, tr_log = 0, tw_valid = 0, BN = 0, gather_direct = 0, fuse_pool = 0, pool_Ho = 0, pool_Wo = 0;
        int N = 0, Hin = 0, Win = 0, Cin = 0, Ho = 0, Wo = 0, Cout = 0, kh = 1, kw = 1, sh = 1, sw = 1, ph = 0, pw = 0, dh = 1,
            dw = 1, act = 0, res_pos = 0;
        const void *xin = nullptr, *resp = nullptr;
        const float *scale = nullptr, *shift = nullptr;
        void *yout = nullptr;
        for (; item < NI; item += G) {
            const int4 nn = item + 2 * G < NI ? __ldg(&P.items[item + 2 * G]) : zero4;
            const int2 dep_nxt =
                (warp == WF_FIRST_WORKER && item + G < NI && lane < rec_ndep(nxt)) ? __ldg(&P.deps[rec_dep0(nxt) + lane]) : make_int2(0, 0);
            if (rec_stage(cur) != sidx) {
                sidx = rec_stage(cur);
                const WfStage *sp = &P.stages[sidx];
                kind = __ldg(&sp->kind); gather_direct = __ldg(&sp->mode); oh_lo = __ldg(&sp->oh_lo); oh_hi = __ldg(&sp->oh_hi);
                p_log = __ldg(&sp->p_log); tr_log = __ldg(&sp->tr_log); tw_valid = __ldg(&sp->tw_valid);
                BN = __ldg(&sp->BN);
                N = __ldg(&sp->N); Hin = __ldg(&sp->Hin); Win = __ldg(&sp->Win); Cin = __ldg(&sp->Cin);
                Ho = __ldg(&sp->Ho); Wo = __ldg(&sp->Wo); Cout = __ldg(&sp->Cout);
                kh = __ldg(&sp->kh); kw = __ldg(&sp->kw); sh = __ldg(&sp->sh); sw = __ldg(&sp->sw);
                ph = __ldg(&sp->ph); pw = __ldg(&sp->pw); dh = __ldg(&sp->dh); dw = __ldg(&sp->dw);
                act = __ldg(&sp->act); res_pos = __ldg(&sp->res_pos);
                fuse_pool = __ldg(&sp->fuse_pool); pool_Ho = __ldg(&sp->pool_Ho); pool_Wo = __ldg(&sp->pool_Wo);
                xin = ldg_ptr<const void *>(&sp->x);
                resp = ldg_ptr<const void *>(&sp->res);
                scale = ldg_ptr<const float *>(reinterpret_cast<const void *const *>(&sp->scale));
                shift = ldg_ptr<const float *>(reinterpret_cast<const void *const *>(&sp->shift));
                yout = ldg_ptr<void *>(reinterpret_cast<const void *const *>(&sp->y));
            }
            const int tile_r = rec_tr(cur);
            if (tid == 0) tr(item, 7);
            if (kind == WF_CONV) {
                const uint32_t buf = cnt & 1u;
                const int c = m & ((1 << p_log) - 1);
                const int r = (m >> p_log) & ((1 << tr_log) - 1);
                const int ow = rec_tw(cur) * tw_valid + c;
                const int oh = oh_lo + (tile_r << tr_log) + r;
                const int n = rec_tn(cur) * (128 >> (p_log + tr_log)) + (m >> (p_log + tr_log));
                const bool valid = c < tw_valid && ow < Wo && oh < oh_hi && n < N;
                const int co0 = rec_cout(cur) * BN;
                if (cgrp == 0) row_pix[m] = valid ? (((long long)n * Ho + oh) * Wo + ow) * Cout + co0 : -1LL;
                if (fuse_pool && cgrp == 0 && !((r | c) & 1)) {
                    // top-left anchor of a 2x2 window: where its maximum goes, if the whole window is inside the stage
                    const int q = (((m >> (p_log + tr_log)) << (tr_log - 1)) + (r >> 1)) * ((1 << p_log) >> 1) + (c >> 1);
                    const bool ok = valid && c + 1 < tw_valid && ow + 1 < Wo && oh + 1 < oh_hi;
                    pool_pix[q] = ok ? (((long long)n * pool_Ho + (oh >> 1)) * pool_Wo + (ow >> 1)) * Cout + co0 : -1LL;
                }
                const float *t_scale = s_scale + 128 * buf, *t_shift = s_shift + 128 * buf;   // filled by warp 0 a tile ahead
                const int cpr = BN >> 3;                               // 16-byte chunks per staged row
                const int cpr_log = (cpr & (cpr - 1)) == 0 ? 31 - __clz(cpr) : -1;
                const uint32_t row_stride = (uint32_t)BN * 2u;
                const int swz = (cpr & 7) == 0 ? 7 : 0;                // chunk position = chunk ^ (row & 7): conflict-free columns
                __nv_bfloat16 *y = static_cast<__nv_bfloat16 *>(yout);
                // the loader warp arrives here once it has seen the tile's producers (the residual's included): the residual
                // tile is fetched now, under the operands' transfer and the main loop
                if (!mbar_wait_abortable(ssf0 + 8u * buf, (cnt >> 1) & 1u, abort_flag)) *epi_fail = 1;
                if (resp) {
                    epi_bar();                                         // row_pix of every anchor is written
                    // residual tile -> staging, coalesced; produced inside this launch by other SMs: read through L2
                    const __nv_bfloat16 *res = static_cast<const __nv_bfloat16 *>(resp);
#pragma unroll 4
                    for (int idx = tid; idx < 128 * cpr; idx += EPI_THREADS) {
                        const int row = cpr_log >= 0 ? idx >> cpr_log : idx / cpr, j = idx - row * cpr;
                        const long long rp = row_pix[row];
                        if (rp >= 0)
                            *reinterpret_cast<uint4 *>(stg + row * row_stride + ((j ^ (row & swz)) << 4)) =
                                __ldcg(reinterpret_cast<const uint4 *>(res + rp) + j);
                    }
                }
                if (!mbar_wait_abortable(accf0 + 8u * buf, (cnt >> 1) & 1u, abort_flag)) *epi_fail = 1;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                if (tid == 0) tr(item, 5);
                if (resp) epi_bar();                                   // the staged residual tile is complete
                {
                    const uint32_t acc = tmem_base + buf * 256u + ((uint32_t)(g * 32) << 16);
                    uint8_t *my_row = stg + m * row_stride;
                    for (int j = 16 * cgrp; j < BN; j += 16 * COL_GROUPS) {
                        uint32_t rr[16];
                        tmem_ld16(acc + (uint32_t)j, rr);
                        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                        if (!valid) continue;
                        float v[16];
#pragma unroll
                        for (int i = 0; i < 16; i += 4) {                  // 16-byte broadcast reads of the tile's scale / shift
                            const float4 sc = *reinterpret_cast<const float4 *>(t_scale + j + i);
                            const float4 sf = *reinterpret_cast<const float4 *>(t_shift + j + i);
                            v[i] = fmaf(sc.x, __uint_as_float(rr[i]), sf.x);
                            v[i + 1] = fmaf(sc.y, __uint_as_float(rr[i + 1]), sf.y);
                            v[i + 2] = fmaf(sc.z, __uint_as_float(rr[i + 2]), sf.z);
                            v[i + 3] = fmaf(sc.w, __uint_as_float(rr[i + 3]), sf.w);
                        }
                        uint4 *c0p = reinterpret_cast<uint4 *>(my_row + ((((j >> 3)) ^ (m & swz)) << 4));
                        uint4 *c1p = reinterpret_cast<uint4 *>(my_row + ((((j >> 3) + 1) ^ (m & swz)) << 4));
                        float rv[16];
                        if (resp) {
                            const uint4 q0 = *c0p, q1 = *c1p;
                            const uint32_t rw[8] = {q0.x, q0.y, q0.z, q0.w, q1.x, q1.y, q1.z, q1.w};
#pragma unroll
                            for (int i = 0; i < 8; ++i) {
                                rv[2 * i] = __uint_as_float(rw[i] << 16);
                                rv[2 * i + 1] = __uint_as_float(rw[i] & 0xFFFF0000u);
                            }
                        }
                        finish16(v, rv, resp ? res_pos : LOP_RES_NONE, act);
                        uint32_t o[8];
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            const __nv_bfloat162 h = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
                            o[i] = *reinterpret_cast<const uint32_t *>(&h);
                        }
                        *c0p = make_uint4(o[0], o[1], o[2], o[3]);
                        *c1p = make_uint4(o[4], o[5], o[6], o[7]);
                    }
                }
                asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                if (tid == 0) tr(item, 11);
                epi_bar();                                             // accumulator drained, staging tile complete
                if (tid == 0) {
                    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(acce0 + 8u * buf) : "memory");
                    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(sse0 + 8u * buf) : "memory");
                }
                ++cnt;
                if (!*epi_fail && fuse_pool) {
                    // 2x2 windows of staged rows -> their maxima (exact in bf16) -> the pooled tensor, 16 bytes per thread
                    const int P_ = 1 << p_log, half_p = P_ >> 1, half_tr = (1 << tr_log) >> 1;
                    for (int idx = tid; idx < 32 * cpr; idx += EPI_THREADS) {
                        const int q = cpr_log >= 0 ? idx >> cpr_log : idx / cpr, j = idx - q * cpr;
                        const long long pp = pool_pix[q];
                        if (pp < 0) continue;
                        const int pc = q % half_p, t = q / half_p;
                        const int m0 = ((t / half_tr) << (p_log + tr_log)) + ((2 * (t % half_tr)) << p_log) + 2 * pc;
                        const int rows4[4] = {m0, m0 + 1, m0 + P_, m0 + P_ + 1};
                        uint4 acc4 = *reinterpret_cast<const uint4 *>(stg + rows4[0] * row_stride + ((j ^ (rows4[0] & swz)) << 4));
#pragma unroll
                        for (int k = 1; k < 4; ++k) {
                            const uint4 v4 = *reinterpret_cast<const uint4 *>(stg + rows4[k] * row_stride + ((j ^ (rows4[k] & swz)) << 4));
                            __nv_bfloat162 *pa = reinterpret_cast<__nv_bfloat162 *>(&acc4);
                            const __nv_bfloat162 *pv = reinterpret_cast<const __nv_bfloat162 *>(&v4);
#pragma unroll
                            for (int e = 0; e < 4; ++e) pa[e] = __hmax2(pa[e], pv[e]);
                        }
                        *(reinterpret_cast<uint4 *>(y + pp) + j) = acc4;
                    }
                } else if (!*epi_fail) {
                    // staged rows -> global: consecutive threads write consecutive 16 bytes of a pixel's channels
#pragma unroll 4
                    for (int idx = tid; idx < 128 * cpr; idx += EPI_THREADS) {
                        const int row = cpr_log >= 0 ? idx >> cpr_log : idx / cpr, j = idx - row * cpr;
                        const long long rp = row_pix[row];
                        if (rp >= 0)
                            *(reinterpret_cast<uint4 *>(y + rp) + j) =
                                *reinterpret_cast<const uint4 *>(stg + row * row_stride + ((j ^ (row & swz)) << 4));
                    }
                }
                if (tid == 0) tr(item, 12);
            } else {
                // pooling or patch gather: one output row of one image per item, all worker threads
                if (warp == WF_FIRST_WORKER && !wait_deps_warp(P, rec_dep0(cur), rec_ndep(cur), dep_cur, run, lane) && lane == 0) *epi_fail = 1;
                epi_bar();
                if (tid == 0) tr(item, 1);
                const int n = rec_tn(cur);
                const int oh = oh_lo + tile_r;
                if (*epi_fail) {
                    // fall through to the common exit below
                } else if (kind == WF_POOL) {
                    const int cg = Cin >> 3;
                    const int total = Wo * cg;
                    const __nv_bfloat16 *x = static_cast<const __nv_bfloat16 *>(xin);
                    __nv_bfloat16 *y = static_cast<__nv_bfloat16 *>(yout);
                    // two channel-group vectors per thread
                    for (int idx0 = 0; idx0 < total; idx0 += 2 * EPI_THREADS) {
                        int gch[2], ow[2];
                        bool live[2];
                        float mx[2][8];
#pragma unroll
                        for (int u = 0; u < 2; ++u) {
                            const int idx = idx0 + u * EPI_THREADS + tid;
                            live[u] = idx < total;
                            ow[u] = idx / cg;
                            gch[u] = idx - ow[u] * cg;
#pragma unroll
                            for (int i = 0; i < 8; ++i) mx[u][i] = -INFINITY;
                        }
                        const int nt = kh * kw;
                        for (int t0 = 0; t0 < nt; t0 += 4) {                 // four filter taps of both vectors in flight
                            uint4 q4[2][4];
                            bool ok[2][4];
#pragma unroll
                            for (int tt = 0; tt < 4; ++tt) {
                                const int t = t0 + tt;
                                const int a = t / kw, b = t - a * kw;
                                const int ih = oh * sh - ph + a * dh;
                                const bool rowok = t < nt && ih >= 0 && ih < Hin;
                                const long long rowbase = ((long long)n * Hin + ih) * Win;
#pragma unroll
                                for (int u = 0; u < 2; ++u) {
                                    const int iw = ow[u] * sw - pw + b * dw;
                                    ok[u][tt] = live[u] && rowok && iw >= 0 && iw < Win;
                                    if (ok[u][tt]) q4[u][tt] = __ldcg(reinterpret_cast<const uint4 *>(x + (rowbase + iw) * Cin + gch[u] * 8));
                                }
                            }
#pragma unroll
                            for (int u = 0; u < 2; ++u)
#pragma unroll
                                for (int tt = 0; tt < 4; ++tt)
                                    if (ok[u][tt]) {
                                        const uint32_t w4[4] = {q4[u][tt].x, q4[u][tt].y, q4[u][tt].z, q4[u][tt].w};
#pragma unroll
                                        for (int i = 0; i < 4; ++i) {
                                            mx[u][2 * i] = fmaxf(mx[u][2 * i], __uint_as_float(w4[i] << 16));
                                            mx[u][2 * i + 1] = fmaxf(mx[u][2 * i + 1], __uint_as_float(w4[i] & 0xFFFF0000u));
                                        }
                                    }
                        }
#pragma unroll
                        for (int u = 0; u < 2; ++u)
                            if (live[u]) {
                                uint32_t o[4];
#pragma unroll
                                for (int i = 0; i < 4; ++i)      // values are bf16 already: truncation is exact
                                    o[i] = (__float_as_uint(mx[u][2 * i]) >> 16) | (__float_as_uint(mx[u][2 * i + 1]) & 0xFFFF0000u);
                                *reinterpret_cast<uint4 *>(y + (((long long)n * Ho + oh) * Wo + ow[u]) * Cin + gch[u] * 8) =
                                    make_uint4(o[0], o[1], o[2], o[3]);
                            }
                    }
                } else if (ROWOPS && kind == WF_DWCONV) {
                    dwconv_item(&P.stages[sidx], n, tile_r, rec_tw(cur), rec_cout(cur), tid, stg);
                } else if (ROWOPS && kind == WF_LAYERNORM) {
                    layernorm_item(&P.stages[sidx], n, oh, tid);
                } else if (ROWOPS && kind == WF_CONCAT) {
                    concat_item(&P.stages[sidx], n, oh, tid);
                } else {
                    // patch gather: Cout holds the patch length Kcol; x is the chain input, possibly still arriving
                    GatherGeom gg;
                    gg.N = N; gg.H = Hin; gg.W = Win; gg.C = Cin; gg.Ho = Ho; gg.Wo = Wo; gg.Kcol = Cout;
                    gg.kh = kh; gg.kw = kw; gg.sh = sh; gg.sw = sw; gg.ph = ph; gg.pw = pw; gg.dh = dh; gg.dw = dw;
                    const int k8n = Cout >> 3;
                    const int total = Wo * k8n;
                    const uint16_t *x = static_cast<const uint16_t *>(xin);
                    uint16_t *y = static_cast<uint16_t *>(yout);
                    if (gather_direct) {
                        for (int idx = tid; idx < total; idx += EPI_THREADS) {
                            const int ow = idx / k8n, k8 = idx - ow * k8n;
                            *reinterpret_cast<uint4 *>(y + (((long long)n * Ho + oh) * Wo + ow) * Cout + k8 * 8) =
                                gather8<true>(x, gg, n, oh, ow, k8);
                        }
                    } else {
                        // the kh image rows this output row reads, copied once into the staging tile with 16-byte
                        // loads (around L1: the rows may have arrived while the kernel was running), then the
                        // patches are put together from shared memory
                        const int row_bytes_in = Win * Cin * 2;
                        const int pitch = (row_bytes_in + 31 + 15) & ~15;
                        const long long tensor_bytes = (long long)N * Hin * row_bytes_in;
                        int *s_mis = reinterpret_cast<int *>(row_pix);       // per filter row: byte offset of the row's first element in staging, or -1
                        const uint8_t *xb = reinterpret_cast<const uint8_t *>(x);
                        const int nvec_max = (row_bytes_in + 30) >> 4;
                        for (int idx = tid; idx < kh * nvec_max; idx += EPI_THREADS) {
                            const int a = idx / nvec_max, v = idx - a * nvec_max;
                            const int ih = oh * sh - ph + a * dh;
                            const bool have = ih >= 0 && ih < Hin;
                            const long long off = ((long long)n * Hin + ih) * row_bytes_in;
                            const int mis = (int)(off & 15);
                            if (v == 0) s_mis[a] = have ? a * pitch + mis : -1;
                            if (!have || v >= ((mis + row_bytes_in + 15) >> 4)) continue;
                            const long long off_al = off - mis;
                            uint4 q;
                            if (off_al + 16LL * (v + 1) <= tensor_bytes) {
                                q = __ldcg(reinterpret_cast<const uint4 *>(xb + off_al) + v);
                            } else {                                          // the tensor ends inside this vector
                                uint32_t h[8];
#pragma unroll
                                for (int e = 0; e < 8; ++e) {
                                    const long long o = off_al + 16LL * v + 2 * e;
                                    h[e] = o < tensor_bytes ? (uint32_t)__ldcg(reinterpret_cast<const uint16_t *>(xb + o)) : 0u;
                                }
                                q = make_uint4(h[0] | (h[1] << 16), h[2] | (h[3] << 16), h[4] | (h[5] << 16), h[6] | (h[7] << 16));
                            }
                            *reinterpret_cast<uint4 *>(stg + a * pitch + 16 * v) = q;
                        }
                        // per patch element: filter row << 16 | element offset inside that row's run of kw*C values, or -1
                        int *tab = reinterpret_cast<int *>(stg + kh * pitch);
                        const int klen = kh * kw * Cin;
                        for (int k = tid; k < Cout; k += EPI_THREADS) {
                            int t = -1;
                            if (k < klen) {
                                const int tap = k / Cin, ci = k - tap * Cin;
                                const int a = tap / kw, b = tap - a * kw;
                                t = (a << 16) | (b * dw * Cin + ci);
                            }
                            tab[k] = t;
                        }
                        epi_bar();
                        const int row_elems = Win * Cin;
                        for (int idx = tid; idx < total; idx += EPI_THREADS) {
                            const int ow = idx / k8n, k8 = idx - ow * k8n;
                            const int base_e = (ow * sw - pw) * Cin;                  // first element of the pixel's runs
                            const int4 t0 = *reinterpret_cast<const int4 *>(tab + k8 * 8);
                            const int4 t1 = *reinterpret_cast<const int4 *>(tab + k8 * 8 + 4);
                            const int tt[8] = {t0.x, t0.y, t0.z, t0.w, t1.x, t1.y, t1.z, t1.w};
                            uint32_t h[8];
#pragma unroll
                            for (int e = 0; e < 8; ++e) {
                                const int fa = tt[e] >> 16, src = base_e + (tt[e] & 0xFFFF);
                                const int rowoff = s_mis[fa < 0 ? 0 : fa];          // byte offset of the row in staging, or -1
                                const bool ok = tt[e] >= 0 && rowoff >= 0 && src >= 0 && src < row_elems;
                                h[e] = ok ? (uint32_t)*reinterpret_cast<const uint16_t *>(stg + rowoff + src * 2) : 0u;
                            }
                            *reinterpret_cast<uint4 *>(y + (((long long)n * Ho + oh) * Wo + ow) * Cout + k8 * 8) =
                                make_uint4(h[0] | (h[1] << 16), h[2] | (h[3] << 16), h[4] | (h[5] << 16), h[6] | (h[7] << 16));
                        }
                    }
                }
            }
            if (kind != WF_CONV && tid == 0) tr(item, 12);
            epi_bar();                                                 // every worker's stores of this item are issued
            if (*epi_fail) {                                           // uniform: written only before a barrier
                if (tid == 0) {
                    atomicOr(P.status, 0x4u);
                    atomicExch(P.counters + 2, 1u);
                    *abort_flag = 1;
                }
                break;
            }
            if (tid == 0) {
                // hand the item to the publisher warp, which fences and increments the row group's counter while
                // the workers go on; it may lag WF_PUBQ items behind
                const uint32_t q = done_items % WF_PUBQ, round = done_items / WF_PUBQ;
                if (!mbar_wait_abortable(pube0 + 8u * q, (round & 1u) ^ 1u, abort_flag)) *epi_fail = 1;
                asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(pubf0 + 8u * q) : "memory");
                tr(item, 6);
            }
            ++done_items;
            cur = nxt; dep_cur = dep_nxt; nxt = nn;
        }
    }

    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    if (warp == 1)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
    if (threadIdx.x == 0 && blockIdx.x < 4) {
        tr(TRACE_ITEMS - 8 + (int)blockIdx.x, 2);
        trv(TRACE_ITEMS - 8 + (int)blockIdx.x, 5, (unsigned long long)clock64());
    }
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

#ifdef LOP_WF_TRACE
static WfParams g_last_params;
#endif

}  // namespace

#ifdef LOP_WF_TRACE
extern "C" int lop_debug_last_stages(void *host, int max_stages)
{
    const int n = g_last_params.n_stages < max_stages ? g_last_params.n_stages : max_stages;
    if (cudaMemcpy(host, g_last_params.stages, (size_t)n * sizeof(WfStage), cudaMemcpyDeviceToHost) != cudaSuccess) return -1;
    return n;
}
extern "C" int lop_debug_last_items(void *host, int max_items)
{
    const int n = g_last_params.n_items < max_items ? g_last_params.n_items : max_items;
    if (cudaMemcpy(host, g_last_params.items, (size_t)n * sizeof(int4), cudaMemcpyDeviceToHost) != cudaSuccess) return -1;
    return n;
}
extern "C" int lop_debug_trace_copy(void *host, size_t bytes, int clear)
{
    if (bytes > sizeof(unsigned long long) * TRACE_ITEMS * 16) bytes = sizeof(unsigned long long) * TRACE_ITEMS * 16;
    if (clear) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_wf_trace) != cudaSuccess) return -1;
        return cudaMemset(p, 0, sizeof(unsigned long long) * TRACE_ITEMS * 16) == cudaSuccess ? 0 : -1;
    }
    return cudaMemcpyFromSymbol(host, g_wf_trace, bytes) == cudaSuccess ? 0 : -1;
}
#endif

size_t wavefront_smem_bytes(const WfParams &p)
{
    return 1024 + (size_t)p.sa * p.a_slot_bytes + (size_t)p.sb * p.b_slot_bytes + p.stg_bytes + 8 * (size_t)(2 * p.sa + 2 * p.sb + 4 + 2 * WF_PUBQ + 4) + 64 +
           2 * 256 * sizeof(float) + (128 + 32) * sizeof(long long) + 64;
}

namespace {

typedef void (*WfKernel)(const WfParams);
WfKernel kernel_for(const WfParams &p)
{
    if (p.n_fetch > 0) return p.row_ops ? wavefront_kernel<true, true> : wavefront_kernel<true, false>;
    return p.row_ops ? wavefront_kernel<false, true> : wavefront_kernel<false, false>;
}

}  // namespace

// How many CTAs of the kernel this device can hold at once (the kernel's dependency waits assume that every CTA of
// a launch is resident: a CTA that has not started cannot produce what a running one waits for).
cudaError_t wavefront_resident_ctas(const WfParams &p, int *ctas)
{
    int dev = 0, sms = 0, per_sm = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
    const size_t smem = wavefront_smem_bytes(p);
    WfKernel k = kernel_for(p);
    if ((e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024)) != cudaSuccess) return e;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k, p.n_fetch > 0 ? WF_THREADS + 32 : WF_THREADS, smem);
    if (e != cudaSuccess) return e;
    *ctas = per_sm * sms;
    return cudaSuccess;
}

cudaError_t launch_wavefront(const WfParams &p, int grid, cudaStream_t s)
{
    const size_t smem = wavefront_smem_bytes(p);
    // the attribute is per device: set it once on each device a launch is made from
    static std::atomic<bool> configured[64];            // set after the (idempotent) attribute call: plans on several host threads may race here
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64 || !configured[dev].load(std::memory_order_acquire)) {
        WfKernel all[4] = {wavefront_kernel<false, false>, wavefront_kernel<false, true>, wavefront_kernel<true, false>, wavefront_kernel<true, true>};
        for (WfKernel k : all) {
            e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
            if (e != cudaSuccess) return e;
        }
        if (dev >= 0 && dev < 64) configured[dev].store(true, std::memory_order_release);
    }
    if (smem > 227 * 1024) return cudaErrorInvalidValue;
#ifdef LOP_WF_TRACE
    g_last_params = p;
#endif
    kernel_for(p)<<<grid, p.n_fetch > 0 ? WF_THREADS + 32 : WF_THREADS, smem, s>>>(p);
    return cudaGetLastError();
}

}  // namespace lop

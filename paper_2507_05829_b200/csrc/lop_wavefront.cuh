// The wavefront kernel: one persistent launch executes a whole list of (band, layer) stages.
//
// Sec. III-A / IV-B of the paper: the operations of later layers start as soon as the rows they
// depend on exist, without waiting for the whole earlier layer.  A *program* is the topologically
// ordered list of stages of one launch; every stage is cut into items (output tiles of a
// convolution, output rows of a pooling or patch-gather stage); resident CTAs take items
// round-robin in program order and an item waits -- with a bounded spin -- only for the producer
// row groups its receptive field touches.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <cstdint>

namespace lop {

// WF_FETCH: rows of the chain input brought from host memory by the CTAs' fetch warps.  Such a stage has row-group
// counters like any producer but no items in the main list: its work is the program's fetch list.
// WF_DWCONV / WF_LAYERNORM / WF_CONCAT: the memory-bound operators, run by the worker warps like pooling.  A depth-wise
// item is one output row of one image, tw_valid columns wide and BN channels deep (its receptive window is staged in
// shared memory); a normalisation or concatenation item is one whole output row of one image.
enum WfKind { WF_GATHER = 0, WF_CONV = 1, WF_POOL = 2, WF_FETCH = 3, WF_DWCONV = 4, WF_LAYERNORM = 5, WF_CONCAT = 6 };
// How a convolution stage feeds the tensor cores.
//   WF_SLAB  one activation box per channel chunk: the output tile's receptive window (tile plus halo),
//            laid out in shared memory as rows of P pixels; every filter tap is the same box read at a
//            shifted start address.  Weights arrive as boxes of several taps.
//   WF_TAP   one activation box and one weight box per (channel chunk, tap): strided windows and
//            channel chunks narrower than 64.
enum WfMode { WF_SLAB = 0, WF_TAP = 1 };

// One (band, layer) stage: rows [oh_lo, oh_hi) of a bound operator.
struct WfStage {
    int kind, mode;
    int oh_lo, oh_hi;
    int ctr_base;             // counters[ctr_base + tile_r]: finished items of that row group
    // convolution tile: accumulator row m is the anchor at column m & (P-1), row (m >> p_log) & (TR-1),
    // image m >> (p_log + tr_log) of the tile; columns >= tw_valid are the slab's halo gap and are dropped
    int p_log, tr_log, tw_valid;
    int BN, BK, n_chunks, n_taps, tb;     // tb: taps per weight box
    int map_base;             // first of 5 tensor maps (4 activation parity classes + weights)
    int a_valid_mask;
    uint32_t a_bytes, b_bytes;            // bytes of one activation / weight box
    uint32_t idesc, layout_code, sbo_bytes, row_bytes;
    // the operator, with its tensors bound (a gathered stem appears as the pointwise convolution it runs as)
    int N, Hin, Win, Cin, Ho, Wo, Cout;
    int kh, kw, sh, sw, ph, pw, dh, dw;
    int act, res_pos;
    const void *x;            // main input, full-size NHWC tensor
    const void *res;          // residual tensor or nullptr
    const float *scale, *shift;
    void *y;                  // full-size output (of the pooling layer when fuse_pool is set)
    // fuse_pool: the convolution's only consumer is a 2x2 stride-2 max pooling; the tile's epilogue takes the
    // maximum of each 2x2 window of staged rows and writes the pooled tensor [N, pool_Ho, pool_Wo, Cout] instead
    int fuse_pool, pool_Ho, pool_Wo;
    // cps > 1: a pointwise stage with a long walk over K puts `cps` consecutive channel chunks, a per-tap stage `cps`
    // consecutive taps, into one ring slot behind one barrier pair (activation boxes in the activation ring, weight
    // boxes in the weight ring), so that more bytes are on their way at a time: such a walk is bound by the loads'
    // latency, a few slots deep, not by their rate
    int cps;
    const void *w_taps;       // depth-wise stage: the filters as [tap][channel] bf16
    int pad_[10];
};
static_assert(sizeof(WfStage) == 256, "WfStage layout");

// One item, 16 bytes: x = stage | cout_tile << 16, y = tile_w | tile_n << 16, z = tile_r | dep_count << 20,
// w = first entry of its dependency list.
struct WfParams {
    const WfStage *stages;
    const int4 *items;
    const CUtensorMap *maps;
    const int2 *deps;         // (counter index, completions expected per run); y < 0: an arrival flag, target -y
    unsigned *counters;       // [0] runs completed, [1] CTAs finished, [2] abort, [3] fetch entries finished, [4..] row-group counters,
                              // then n_flags band-arrival flags (set by the copy stream, cleared at run end)
    int flag_base, n_flags;
    unsigned *status;
    int n_stages, n_items;
    int sa, sb;               // slots of the activation / weight ring
    uint32_t a_slot_bytes, b_slot_bytes, stg_bytes;
    // In-kernel input transfer (Sec. IV-B transmission, done by the kernel itself): every CTA has one more warp that
    // walks this list round-robin; entry j copies z bytes at byte offset (x | y << 32) from fetch_src (host memory
    // the device can address) to fetch_dst and then increments counters[w].  At most fetch_window entries are in
    // flight at a time (counters[3] counts finished ones), so the rows arrive in list order at the link's rate.
    uint32_t spin_limit;      // polls of a row-group counter, an arrival flag or the fetch window before the kernel gives up
    const int4 *fetch_items;
    const void *fetch_src;
    void *fetch_dst;
    int n_fetch, fetch_window;
    int row_ops;              // the program has WF_DWCONV / WF_LAYERNORM / WF_CONCAT stages
};

#ifndef LOP_WF_WORKER_WARPS
#define LOP_WF_WORKER_WARPS 8
#endif
constexpr int WF_WORKER_WARPS = LOP_WF_WORKER_WARPS;      // epilogue / SIMT warps (a multiple of 4)
constexpr int WF_FIRST_WORKER = 3;                         // warps 0..2: loader, MMA issuer, publisher
constexpr int WF_THREADS = 32 * (WF_FIRST_WORKER + WF_WORKER_WARPS);
constexpr int WF_PUBQ = 4;                                 // finished items the publisher may lag behind the workers
constexpr int WF_CTR_FIRST = 4;
constexpr int WF_MAX_DEPS = 4095;

size_t wavefront_smem_bytes(const WfParams &p);
cudaError_t launch_wavefront(const WfParams &p, int grid, cudaStream_t s);
cudaError_t wavefront_resident_ctas(const WfParams &p, int *ctas);
constexpr uint32_t WF_SPIN_LIMIT_DEFAULT = 1u << 22;

}  // namespace lop

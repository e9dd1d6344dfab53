// The wavefront kernel: one persistent launch executes a whole list of (band, layer) stages.
//
// Sec. III-A / IV-B of the paper: the operations of later layers start as soon as the rows they
// depend on exist, without waiting for the whole earlier layer.  A *program* is the topologically
// ordered list of stages of one launch; every stage is cut into items (output tiles); resident
// CTAs take items round-robin in program order and an item waits -- with a bounded spin -- only
// for the producer row groups its receptive field touches.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <cstdint>

namespace lop {

enum WfKind { WF_PAD = 0, WF_CONV = 1, WF_POOL = 2 };

// One operator instance with its tensors bound (device pointers).
struct WfLayer {
    const void *x;            // main input, full-size NHWC tensor
    const void *res;          // residual tensor or nullptr
    const float *scale, *shift;
    void *y;                  // full-size output
    int N, Hin, Win, Cin, Ho, Wo, Cout;
    int kh, kw, sh, sw, ph, pw, dh, dw;
    int act, res_pos;
    int pad_[5];
};
static_assert(sizeof(WfLayer) == 128, "WfLayer is copied as 32 words");

// One (band, layer) stage: rows [oh_lo, oh_hi) of a layer, cut into n_items tiles.
struct WfStage {
    int kind, layer;
    int oh_lo, oh_hi;
    int first_item, n_items;
    int tw_log, tr_log;       // conv tile = TN images x 2^tr_log rows x 2^tw_log columns (128 pixels)
    int tiles_w, tiles_r, tiles_n, cout_tiles;
    int BN, BK;
    int map_base;             // first of 5 tensor maps (4 activation parity classes + weights)
    int a_valid_mask;
    int dep_base;             // dep_index[dep_base + tile_r] = (first, count) into the dependency list
    int ctr_base;             // counters[ctr_base + tile_r]: completed tiles of that row group
    int k_iters;
    uint32_t a_bytes, b_bytes, idesc, layout_code, sbo_bytes;
    int pad_[8];
};
static_assert(sizeof(WfStage) == 128, "WfStage is copied as 32 words");

struct WfParams {
    const WfStage *stages;
    const WfLayer *layers;
    const CUtensorMap *maps;
    const int2 *dep_index;    // per (stage, tile_r): first, count
    const int2 *deps;         // (counter index, completions expected per run)
    unsigned *counters;       // [0] runs completed, [1] CTAs finished, [2] abort, [4..] row-group counters,
                              // then n_flags band-arrival flags (set by the copy stream, cleared at run end)
    int flag_base, n_flags;
    unsigned *status;
    int n_stages, n_items;
    int ring;                 // pipeline depth
    uint32_t slot_bytes;      // bytes of one ring slot (activation tile + weight tile)
};

constexpr int WF_THREADS = 192;
constexpr int WF_CTR_FIRST = 4;

size_t wavefront_smem_bytes(int ring, uint32_t slot_bytes);
cudaError_t launch_wavefront(const WfParams &p, int grid, cudaStream_t s);

}  // namespace lop

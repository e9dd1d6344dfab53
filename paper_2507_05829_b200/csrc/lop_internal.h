// Internal declarations shared by the library's translation units (not part of the ABI).
#pragma once
#include <cstdint>
#include <cstddef>
#include <string>
#include <vector>

#include "lop.h"

namespace lop {

enum KernelFamily { K_POOL = 0, K_CONV_SIMT = 1, K_CONV_TC = 2, K_DWCONV = 3, K_LAYERNORM = 4, K_CONCAT = 5 };

struct LayerInfo {
    lop_layer l;
    int Hin = 0, Win = 0;          // spatial extent of the main input
    int Ho = 0, Wo = 0, Co = 0;    // output shape
    int kernel = K_CONV_SIMT;
    int cin_eff = 0;               // channels the tensor-core kernel sees (= the patch length Kcol for a gathered stem)
    bool linear = false;           // given as the row-wise operator LOP_LINEAR (runs as the pointwise convolution it is)
    bool stem_gather = false;      // thin chain input: the layer's receptive patches are gathered into a
                                   // [N, Ho, Wo, Kcol] tensor first and the convolution runs as 1x1 over it
    size_t out_off = 0;            // workspace offset of the full-size output (unused for the last layer)
    size_t wpad_off = 0;           // workspace offset of the [cout][Kcol] zero-padded weights (if stem_gather), of the
                                   // [taps][C] transposed filters (if dw_transposed)
    bool dw_transposed = false;    // bf16 depth-wise convolution with C % 8 == 0: the workspace keeps its filters tap-major
};

struct ExecState;                  // CUDA-side resources, defined in lop_exec.cu

}  // namespace lop

struct lop_plan {
    std::vector<lop::LayerInfo> layers;
    int N = 0, H = 0, W = 0, C = 0, dtype = 0, n_bands = 0;
    unsigned flags = 0;
    int stem = -1;                 // index of the stem_gather layer, or -1
    std::vector<lop_range> ranges;     // [band][layer]
    std::vector<lop_range> in_need;    // [band]: chain-input rows (out_lo,out_hi,new_lo)
    size_t ws_bytes = 0, status_off = 0, col_off = 0;   // col_off: the gathered patch tensor
    double flops = 0.0;
    int copy_group = 1;                // bands moved by one copy-engine copy in pipelined runs (see lop_plan.cpp)
    unsigned wait_limit = 0;           // polls a device-side wait may take before the kernel gives up (0: the default)
    unsigned long long uid = 0;        // unique per plan and per state of its parameters (a new one at creation and at every
                                       // lop_plan_set_params): cached device programs name the plans they were built from by it
    lop::ExecState *exec = nullptr;
};

namespace lop {

void set_error(const char *fmt, ...);
unsigned long long next_plan_uid();
inline size_t elem_size(int dtype) { return dtype == LOP_BF16 ? 2 : 4; }
inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// lop_exec.cu
void exec_destroy(ExecState *e);
// Drops what was built from the layers' device pointers (programs, tensor maps, padded weights), after lop_plan_set_params.
void exec_invalidate(ExecState *e);

}  // namespace lop

// Programs for the wavefront kernel (host interface).
#pragma once
#include <cuda_runtime.h>

#include <vector>

#include "lop_internal.h"

namespace lop {

// One plan of a chain with its buffers bound: `in` is the plan's input tensor (for plan s > 0 the output of plan
// s-1), `out` its last layer's output, `ws` its workspace.
struct SegBind { lop_plan_t *pl; const void *in; void *out; void *ws; };

// Rows [lo, hi) of a layer of plan `seg` for one band.  gather: the patch-gather stage that precedes a gathered stem
// layer (same rows).  wait_arrival: stages of plan 0 that read the raw chain input wait for the arrival flags of the
// bands that bring their rows (single-launch pipelined programs).  prio: stages are put into the program in
// ascending priority, as far as their dependencies allow (a stage never precedes one it reads from).
// fetch: not an operator but the transfer of rows [lo, hi) of the chain input from host memory, done by the kernel
// itself (layer is ignored); the stages of plan 0 that read those rows then depend on it like on any producer.
struct StageReq { int seg, band, layer, lo, hi; bool wait_arrival; bool gather; long long prio; bool fetch = false; };
struct Program;

bool program_supported(const lop_plan_t *pl);
// The persistent kernel folds a 2x2 stride-2 pooling that is convolution `layer`'s only reader into that
// convolution's epilogue (its own output tensor is then never written).
bool program_folds_pool(const lop_plan_t *pl, int layer);
// arrival_us (optional): expected arrival time of each band of plan 0; stages are then ordered by their earliest
// possible start under that schedule instead of by prio.  fetch_src: the chain input in host memory as the device
// addresses it, source of the fetch requests (segs[0].in is their destination); programs with fetch requests are
// ordered by earliest start as well, the host link taken as a serial resource.
int program_build(const std::vector<SegBind> &segs, std::vector<StageReq> reqs, Program **result,
                  const std::vector<double> *arrival_us = nullptr, const void *fetch_src = nullptr);
int program_launch(Program *p, cudaStream_t s);
// Device address of band b's arrival flag (a 4-byte word a side stream sets non-zero), or nullptr.
unsigned *program_arrival_flag(Program *p, int band);
bool program_empty(const Program *p);
void program_destroy(Program *p);

}  // namespace lop

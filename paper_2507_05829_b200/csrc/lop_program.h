// Programs for the wavefront kernel (host interface).
#pragma once
#include <cuda_runtime.h>

#include <vector>

#include "lop_internal.h"

namespace lop {

// Rows [lo, hi) of a layer for one band.  gather: the patch-gather stage that precedes a gathered stem layer
// (same rows).  wait_arrival: stages that read the raw chain input wait for their band's arrival flag
// (single-launch pipelined programs).
struct StageReq { int band, layer, lo, hi; bool wait_arrival; bool gather; };
struct Program;

bool program_supported(const lop_plan_t *pl);
int program_build(lop_plan_t *pl, const std::vector<StageReq> &reqs, const void *in, void *out, void *ws, Program **result);
int program_launch(Program *p, cudaStream_t s);
// Device address of band b's arrival flag (a 4-byte word the copy stream sets non-zero), or nullptr.
unsigned *program_arrival_flag(Program *p, int band);
bool program_empty(const Program *p);
void program_destroy(Program *p);

}  // namespace lop

// Programs for the wavefront kernel (host interface).
#pragma once
#include <cuda_runtime.h>

#include <vector>

#include "lop_internal.h"

namespace lop {

struct StageReq { int band, layer, lo, hi; };     // layer -1: channel padding of the chain input
struct Program;

bool program_supported(const lop_plan_t *pl);
int program_build(lop_plan_t *pl, const std::vector<StageReq> &reqs, const void *in, void *out, void *ws, Program **result);
int program_launch(Program *p, cudaStream_t s);
bool program_empty(const Program *p);
void program_destroy(Program *p);

}  // namespace lop

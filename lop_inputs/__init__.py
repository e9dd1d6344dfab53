"""Seeded synthetic inputs for local-operator chains (layer lists, tensors, weights).

This package is shared by the CPU oracle's tests and by the CUDA library's tests and
benchmark.  It only *describes* workloads and draws random numbers: it holds no
convolution, pooling, planning or epilogue arithmetic of its own.
"""
from .rng import uniform, normal, round_to_bf16, bf16_bits, from_bf16_bits
from .workloads import (Layer, Segment, Workload, CONV, POOL, LINEAR, DWCONV, LAYERNORM, CONCAT, ACT_NONE, ACT_RELU, ACT_SILU, ACT_GELU,
                        RES_NONE, RES_PRE_ACT, RES_POST_ACT, build, WORKLOADS, conv, pool, linear, dwconv, layernorm, concat,
                        fill_parameters, make_input)

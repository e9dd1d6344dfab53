// PTX wrappers for sm_100a shared by the tensor-core kernels: mbarrier, TMA (cp.async.bulk.tensor),
// tcgen05 (alloc / mma / commit / ld) and the shared-memory matrix descriptor.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <cstdint>

#include "lop.h"

namespace lop {
namespace ptx {

constexpr uint32_t WAIT_LIMIT = 1u << 23;

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// Bounded wait on an mbarrier phase; false when the limit ran out.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity)
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
    }
    return false;
}

__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int c0, int c1, int c2,
                                            int c3)
{
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
        : "memory");
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int c0, int c1)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1)
        : "memory");
}

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int c0, int c1, int c2)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1), "r"(c2)
        : "memory");
}

// Shared-memory matrix descriptor of a K-major operand tile (rows of `row bytes` = swizzle span).
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t sbo_bytes, uint32_t layout_code)
{
    uint64_t d = 0;
    d |= (uint64_t)((addr & 0x3FFFFu) >> 4);               // start address, 16-byte units
    d |= (uint64_t)1 << 16;                                // leading-dimension offset: unused for swizzled K-major
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFF) << 32;      // stride between 8-row groups
    d |= (uint64_t)1 << 46;                                // descriptor version of this architecture
    // base-offset field (bits 49-51) stays 0: the swizzle is a function of the shared-memory address itself, so
    // an operand may start at any row of a 1024-byte-aligned box (the slab convolution's shifted taps rely on it)
    d |= (uint64_t)layout_code << 61;                      // swizzle mode
    return d;
}

__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n"
        "}\n" ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
}

__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}

// Activation with the kind fixed at compile time: selected once per tile, outside the per-element loops (a
// run-time `act` inside them makes the compiler evaluate the SiLU division for every element of every kind).
template <int ACT>
__device__ __forceinline__ float activate_t(float t)
{
    if (ACT == LOP_ACT_RELU) return fmaxf(t, 0.0f);
    if (ACT == LOP_ACT_SILU) return __fdividef(t, 1.0f + __expf(-t));
    if (ACT == LOP_ACT_GELU) return 0.5f * t * (1.0f + erff(t * 0.70710678f));     // t * Phi(t), the exact form
    return t;
}

// Last step of the fused epilogue on 16 channels: v = scale*acc + shift already; rv = residual values.
template <int ACT>
__device__ __forceinline__ void finish16_t(float (&v)[16], const float (&rv)[16], int res_pos)
{
    if (res_pos == LOP_RES_PRE_ACT) {
#pragma unroll
        for (int i = 0; i < 16; ++i) v[i] = activate_t<ACT>(v[i] + rv[i]);
    } else if (res_pos == LOP_RES_POST_ACT) {
#pragma unroll
        for (int i = 0; i < 16; ++i) v[i] = activate_t<ACT>(v[i]) + rv[i];
    } else {
#pragma unroll
        for (int i = 0; i < 16; ++i) v[i] = activate_t<ACT>(v[i]);
    }
}
// res_pos must be LOP_RES_NONE when there is no residual (rv is then not read).
__device__ __forceinline__ void finish16(float (&v)[16], const float (&rv)[16], int res_pos, int act)
{
    if (act == LOP_ACT_RELU) finish16_t<LOP_ACT_RELU>(v, rv, res_pos);
    else if (act == LOP_ACT_SILU) finish16_t<LOP_ACT_SILU>(v, rv, res_pos);
    else if (act == LOP_ACT_GELU) finish16_t<LOP_ACT_GELU>(v, rv, res_pos);
    else finish16_t<LOP_ACT_NONE>(v, rv, res_pos);
}

__device__ __forceinline__ int floor_div_i(int a, int b) { int q = a / b; return (a % b != 0 && a < 0) ? q - 1 : q; }


}  // namespace ptx
}  // namespace lop

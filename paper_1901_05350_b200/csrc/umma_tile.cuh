// Tile constants and the epilogue staging routine shared by the tcgen05 kernels (plain GEMM,
// implicit-GEMM convolution, fused depthwise + pointwise block).
#pragma once

#include <cuda_bf16.h>

#include "common.cuh"
#include "ptx_sm100.cuh"

namespace tfjsb {
namespace tile {

constexpr int BLOCK_M = 128;
constexpr int BLOCK_K = 32;  // fp32 elements: one 128-byte swizzle row
constexpr int UMMA_K = 8;    // tf32 elements per tcgen05.mma
constexpr int MAX_ACC_STAGES = 4;
constexpr int EPI_COLS = 32;
constexpr int A_STAGE_BYTES = BLOCK_M * BLOCK_K * 4;             // 16 KiB
constexpr int EPI_SLAB_BYTES = 32 * EPI_COLS * 4;                // 4 KiB: 32 rows x 128 B
constexpr int EPI_BYTES = 8 /*epilogue warps*/ * EPI_SLAB_BYTES;      // 32 KiB
constexpr int SMEM_LIMIT = 232448;                               // 227 KiB

// Fused epilogue of one 32-row x 32-column accumulator block held one row per lane: bias add,
// activation, and the swizzled store into the staging slab the bulk tensor store reads from
// (16-byte chunk j of row `lane` lives at chunk j ^ (lane % 8): the 128-byte swizzle).
template <int ACT>
__device__ __forceinline__ void stage_chunk(const uint32_t (&r)[32], const float* __restrict__ bias, int cols_left,
                                            uint32_t row_addr, int lane) {
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        float4 v;
        v.x = __uint_as_float(r[4 * j + 0]); v.y = __uint_as_float(r[4 * j + 1]);
        v.z = __uint_as_float(r[4 * j + 2]); v.w = __uint_as_float(r[4 * j + 3]);
        if (bias != nullptr && 4 * j < cols_left) {  // N % 4 == 0: a quad is all in or all out
            const float4 b = __ldg(reinterpret_cast<const float4*>(bias + 4 * j));
            v.x = v.x + b.x; v.y = v.y + b.y; v.z = v.z + b.z; v.w = v.w + b.w;
        }
        v.x = apply_act_t<ACT>(v.x); v.y = apply_act_t<ACT>(v.y);
        v.z = apply_act_t<ACT>(v.z); v.w = apply_act_t<ACT>(v.w);
        const uint32_t dst = row_addr + (uint32_t)((j ^ (lane & 7)) << 4);
        asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w)
                     : "memory");
    }
}

// ---- bfloat16 storage ------------------------------------------------------------------------------
// Instruction descriptor: fp32 accumulator, bfloat16 A and B (format 1), both K-major.
__device__ __forceinline__ uint32_t make_idesc_bf16(int m, int n) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}

// One 32-row x 32-column accumulator block, one row per lane: bias, activation, rounding to bfloat16,
// and the store into the staging slab in the 64-byte swizzle the bulk tensor store expects (rows of
// 64 bytes; 16-byte piece j of row r lives at piece j ^ ((r / 2) % 4)).
template <int ACT>
__device__ __forceinline__ void stage_chunk_bf16(const uint32_t (&r)[32], const float* __restrict__ bias, int cols_left,
                                                 uint32_t slab, int lane) {
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        float v[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) v[e] = __uint_as_float(r[8 * j + e]);
        if (bias != nullptr && 8 * j < cols_left) {  // N % 8 == 0: a group of eight is all in or all out
            const float4 b0 = __ldg(reinterpret_cast<const float4*>(bias + 8 * j));
            const float4 b1 = __ldg(reinterpret_cast<const float4*>(bias + 8 * j + 4));
            v[0] += b0.x; v[1] += b0.y; v[2] += b0.z; v[3] += b0.w;
            v[4] += b1.x; v[5] += b1.y; v[6] += b1.z; v[7] += b1.w;
        }
        uint32_t p[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const __nv_bfloat162 h = __floats2bfloat162_rn(apply_act_t<ACT>(v[2 * e]), apply_act_t<ACT>(v[2 * e + 1]));
            p[e] = *reinterpret_cast<const uint32_t*>(&h);
        }
        const uint32_t dst = slab + (uint32_t)lane * 64u + (uint32_t)((j ^ ((lane >> 1) & 3)) << 4);
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(p[0]), "r"(p[1]), "r"(p[2]), "r"(p[3])
                     : "memory");
    }
}

}  // namespace tile
}  // namespace tfjsb

// Tile constants and the epilogue staging routine shared by the tcgen05 kernels (plain GEMM,
// implicit-GEMM convolution, fused depthwise + pointwise block).
#pragma once

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

}  // namespace tile
}  // namespace tfjsb

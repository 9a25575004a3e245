// Tensor-core GEMM on bfloat16 storage (the narrow-storage mode), with the fused bias + activation
// epilogue:
//
//     C[M,N] = act( A[M,K] . Bt[N,K]^T + bias[N] )     A, Bt bfloat16; sums fp32; C bfloat16 or fp32
//
// The 16-bit analogue of the paper's half-float textures (Sec. 4.1.3): what is stored is 16 bits
// wide, the arithmetic stays wide.  Products of two bfloat16 are exact in fp32 and the tensor core
// accumulates them in fp32 in tensor memory; the result gets the fp32 bias, the activation, and one
// rounding (to nearest even) to bfloat16 when it is stored narrow.
//
// Same structure as the TF32 kernel (one persistent CTA per SM; a producer warp issuing bulk tensor
// copies into a ring of 128-byte-swizzled stages, an MMA warp, epilogue warps; two or four
// accumulator stages), and the same bytes per stage: a k-block is 64 bfloat16 = one 128-byte swizzle
// row, consumed by four `tcgen05.mma.kind::f16` of K = 16.  Half the bytes per element means half the
// k-blocks for the same K, and half the bytes of A and C to move.
//
// With half the bytes per tile the layers with one or two k-blocks per tile are bound by the epilogue's
// latency per 32 x 32 block (tcgen05.ld, bias, activation, rounding, staging, store), so those run with
// sixteen epilogue warps, four per lane quadrant, taking every fourth block; the layers with long K
// loops keep eight (the extra warps' polling costs them about 4 %).
//
// Every wait is bounded, as in the TF32 kernel.
#include <cuda_bf16.h>

#include <cstdlib>

#include "common.cuh"
#include "ptx_sm100.cuh"
#include "umma_tile.cuh"

namespace tfjsb {

using namespace ptx;
using namespace tile;

namespace {

constexpr int MAX_STAGES = 8;
constexpr int MAX_EPI_WARPS = 16;  // eight or sixteen epilogue warps: two or four per tensor-memory lane quadrant
constexpr int GEMM_THREADS = 64 + MAX_EPI_WARPS * 32;  // producer warp, MMA warp, the epilogue warps
constexpr int BK16 = 64;           // bfloat16 elements per k-block (128 bytes)
constexpr int UMMA_K16 = 16;       // elements per tcgen05.mma of kind::f16

// D[tmem] (+)= A[smem] . B[smem]^T, single CTA, bfloat16 operands, fp32 accumulate.
__device__ __forceinline__ void tc_mma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                            uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
struct KernelArgs {
    int M, N, K;
    int block_n;
    int stages;
    int n_tiles;
    int num_tiles;
    int acc_stages;
    int epi_warps;  // 8 or 16
    const float* bias;
    int act;
    unsigned int* dev_status;
};

template <bool OUT_BF16>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
gemm_bf16_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                 const __grid_constant__ CUtensorMap map_c, const KernelArgs args) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bar_full[MAX_STAGES];
    __shared__ __align__(8) uint64_t bar_empty[MAX_STAGES];
    __shared__ __align__(8) uint64_t bar_acc_full[MAX_ACC_STAGES];
    __shared__ __align__(8) uint64_t bar_acc_empty[MAX_ACC_STAGES];
    __shared__ __align__(8) uint64_t bar_drain;
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag_s;

    volatile int* abort_flag = &abort_flag_s;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int block_n = args.block_n, stages = args.stages, acc_stages = args.acc_stages;
    const int stage_bytes = A_STAGE_BYTES + block_n * 128;
    const int num_k_blocks = (args.K + BK16 - 1) / BK16;

    // dynamic shared memory, aligned to the 1024-byte swizzle pattern: [epilogue slabs][stage 0: A | B]...
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t epi_base = smem_base;
    constexpr uint32_t SLAB_BYTES = OUT_BF16 ? 2048u : 4096u;  // 32 rows x 32 columns of the output type
    const uint32_t stage_base = smem_base + (uint32_t)args.epi_warps * SLAB_BYTES;

    if (threadIdx.x == 0) {
        for (int s = 0; s < stages; ++s) {
            mbar_init(smem_u32(&bar_full[s]), 1);
            mbar_init(smem_u32(&bar_empty[s]), 1);
        }
        for (int s = 0; s < acc_stages; ++s) {
            mbar_init(smem_u32(&bar_acc_full[s]), 1);
            mbar_init(smem_u32(&bar_acc_empty[s]), (uint32_t)args.epi_warps);
        }
        mbar_init(smem_u32(&bar_drain), 1);
        abort_flag_s = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_a) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_b) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_c) : "memory");
    }
    uint32_t tmem_cols = 32;  // allocations are powers of two >= 32 columns
    while (tmem_cols < (uint32_t)(acc_stages * block_n)) tmem_cols <<= 1;
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                         smem_u32(&tmem_base_slot)),
                     "r"(tmem_cols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;
    pdl_launch_dependents();
    pdl_wait();

    if (warp == 0) {
        // ---------------------------------------------------------------- TMA producer
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            int armed[MAX_STAGES];  // parity of the last phase armed on each stage, -1 = never
#pragma unroll
            for (int s = 0; s < MAX_STAGES; ++s) armed[s] = -1;
            bool ok = true;
            for (int tile = blockIdx.x; ok && tile < args.num_tiles; tile += gridDim.x) {
                const int m0 = (tile / args.n_tiles) * BLOCK_M;
                const int n0 = (tile % args.n_tiles) * block_n;
                for (int kb = 0; kb < num_k_blocks; ++kb) {
                    if (!bounded_wait(smem_u32(&bar_empty[stage]), phase ^ 1u, abort_flag)) {
                        if (!*abort_flag) {
                            *abort_flag = 1;
                            atomicOr(args.dev_status, DEV_STATUS_TIMEOUT_PRODUCER);
                        }
                        ok = false;
                        break;
                    }
                    const uint32_t full = smem_u32(&bar_full[stage]);
                    const uint32_t a_dst = stage_base + (uint32_t)stage * (uint32_t)stage_bytes;
                    mbar_arrive_expect_tx(full, (uint32_t)stage_bytes);
                    tma_load_2d(a_dst, &map_a, full, kb * BK16, m0);
                    tma_load_2d(a_dst + A_STAGE_BYTES, &map_b, full, kb * BK16, n0);
#pragma unroll
                    for (int s = 0; s < MAX_STAGES; ++s)
                        if (s == stage) armed[s] = (int)phase;
                    if (++stage == stages) { stage = 0; phase ^= 1u; }
                }
            }
            if (!ok) {
                // wait (bounded) for the copies in flight so that nothing lands after the CTA has gone
#pragma unroll
                for (int s = 0; s < MAX_STAGES; ++s) {
                    if (s < stages && armed[s] >= 0) {
                        const unsigned long long t0 = global_ns();
                        while (!mbar_try_wait(smem_u32(&bar_full[s]), (uint32_t)armed[s])) {
                            if (global_ns() - t0 > WAIT_LIMIT_NS) {
                                atomicOr(args.dev_status, DEV_STATUS_TIMEOUT_DRAIN);
                                break;
                            }
                        }
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ---------------------------------------------------------------- MMA issuer
        if (lane == 0) {
            const uint32_t idesc = make_idesc_bf16(BLOCK_M, block_n);
            int stage = 0;
            uint32_t phase = 0;
            int acc = 0;
            uint32_t acc_phase = 0;
            bool ok = true;
            bool issued_any = false;
            for (int tile = blockIdx.x; ok && tile < args.num_tiles; tile += gridDim.x) {
                if (!bounded_wait(smem_u32(&bar_acc_empty[acc]), acc_phase ^ 1u, abort_flag)) { ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(acc * block_n);
                for (int kb = 0; kb < num_k_blocks; ++kb) {
                    if (!bounded_wait(smem_u32(&bar_full[stage]), phase, abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t a_addr = stage_base + (uint32_t)stage * (uint32_t)stage_bytes;
                    const uint64_t a_desc = make_kmajor_sw128_desc(a_addr);
                    const uint64_t b_desc = make_kmajor_sw128_desc(a_addr + A_STAGE_BYTES);
#pragma unroll
                    for (int k = 0; k < BK16 / UMMA_K16; ++k) {
                        // step along K inside the 128-byte swizzled row: 32 bytes = 2 descriptor units
                        tc_mma_bf16(d_tmem, a_desc + (uint64_t)(2 * k), b_desc + (uint64_t)(2 * k), idesc,
                                    (kb | k) != 0 ? 1u : 0u);
                    }
                    issued_any = true;
                    tc_commit(smem_u32(&bar_empty[stage]));
                    if (++stage == stages) { stage = 0; phase ^= 1u; }
                }
                if (!ok) break;
                tc_commit(smem_u32(&bar_acc_full[acc]));
                if (++acc == acc_stages) { acc = 0; acc_phase ^= 1u; }
            }
            if (!ok) {
                if (!*abort_flag) {
                    *abort_flag = 1;
                    atomicOr(args.dev_status, DEV_STATUS_TIMEOUT_MMA);
                }
                if (issued_any) {
                    // let the MMAs already issued finish before tensor memory is released
                    tc_commit(smem_u32(&bar_drain));
                    const unsigned long long t0 = global_ns();
                    while (!mbar_try_wait(smem_u32(&bar_drain), 0u)) {
                        if (global_ns() - t0 > WAIT_LIMIT_NS) {
                            atomicOr(args.dev_status, DEV_STATUS_TIMEOUT_DRAIN);
                            break;
                        }
                    }
                }
            }
        }
    } else {
        // ---------------------------------------------------------------- epilogue (warps 2..)
        // Two or four warps share each TMEM lane quadrant (a warp may only read lanes 32*(warp%4)..+31)
        // and take every second or fourth 32-column block, counted across tiles so that with one block
        // per tile they take tiles in turn.
        const int ew = warp - 2;
        const int quad = warp & 3;
        const int sub = ew >> 2;  // which of the quadrant's warps
        const int per_quad_mask = (args.epi_warps >> 2) - 1;  // 1 or 3
        const uint32_t slab = epi_base + (uint32_t)ew * SLAB_BYTES;
        int acc = 0;
        uint32_t acc_phase = 0;
        bool ok = true;
        const int chunks_per_tile = block_n / EPI_COLS;
        int chunk_base = 0;  // blocks of earlier tiles, modulo the quadrant's warps
        for (int tile = blockIdx.x; ok && tile < args.num_tiles; tile += gridDim.x) {
            const int m0 = (tile / args.n_tiles) * BLOCK_M;
            const int n0 = (tile % args.n_tiles) * block_n;
            const bool got = bounded_wait(smem_u32(&bar_acc_full[acc]), acc_phase, abort_flag);
            if (!__all_sync(0xffffffffu, got)) {
                if (lane == 0 && !*abort_flag) {
                    *abort_flag = 1;
                    atomicOr(args.dev_status, DEV_STATUS_TIMEOUT_EPILOGUE);
                }
                ok = false;
                break;
            }
            tc_fence_after();
            const int row0 = m0 + quad * 32;
            int n_chunks = block_n / EPI_COLS;
            const int live_cols = args.N - n0;
            if (live_cols < block_n) n_chunks = (live_cols + EPI_COLS - 1) / EPI_COLS;
            const bool rows_live = row0 < args.M;
            bool released = false;
            for (int ch = (sub - chunk_base) & per_quad_mask; ch < n_chunks; ch += per_quad_mask + 1) {
                uint32_t r[32];
                const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(acc * block_n + ch * EPI_COLS);
                tc_ld_32x32(taddr, r);
                tc_ld_wait();
                if (ch + per_quad_mask + 1 >= n_chunks) {
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&bar_acc_empty[acc]));
                    released = true;
                }
                if (!rows_live) continue;
                const int col0 = n0 + ch * EPI_COLS;
                if (lane == 0) tma_store_wait_read<0>();  // the slab is free once the previous store has read it
                __syncwarp();
                const float* bias = (args.bias != nullptr) ? args.bias + col0 : nullptr;
                const int cols_left = args.N - col0;
                if (OUT_BF16) {
                    if (args.act == TFJSB_ACT_RELU6) stage_chunk_bf16<TFJSB_ACT_RELU6>(r, bias, cols_left, slab, lane);
                    else if (args.act == TFJSB_ACT_RELU) stage_chunk_bf16<TFJSB_ACT_RELU>(r, bias, cols_left, slab, lane);
                    else stage_chunk_bf16<TFJSB_ACT_NONE>(r, bias, cols_left, slab, lane);
                } else {
                    const uint32_t row_addr = slab + (uint32_t)lane * 128u;
                    if (args.act == TFJSB_ACT_RELU6) stage_chunk<TFJSB_ACT_RELU6>(r, bias, cols_left, row_addr, lane);
                    else if (args.act == TFJSB_ACT_RELU) stage_chunk<TFJSB_ACT_RELU>(r, bias, cols_left, row_addr, lane);
                    else stage_chunk<TFJSB_ACT_NONE>(r, bias, cols_left, row_addr, lane);
                }
                fence_async_smem();
                __syncwarp();
                if (lane == 0) {
                    tma_store_2d(&map_c, slab, col0, row0);
                    tma_store_commit();
                }
            }
            if (!released) {  // no chunk of this tile fell to this warp
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&bar_acc_empty[acc]));
            }
            chunk_base = (chunk_base + chunks_per_tile) & per_quad_mask;
            if (++acc == acc_stages) { acc = 0; acc_phase ^= 1u; }
        }
        if (lane == 0) tma_store_wait_all();
        __syncwarp();
    }

    // ---------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols)
                     : "memory");
    }
}

int choose_block_n(int64_t M, int64_t N, int sm_count) {
    int bn = 32;
    while (bn < 256 && bn < N) bn <<= 1;
    const int64_t m_tiles = (M + BLOCK_M - 1) / BLOCK_M;
    while (bn > 32 && m_tiles * ((N + bn - 1) / bn) < sm_count) bn >>= 1;
    if (bn == 256 && N > 256) {
        // every tile of a launch costs the same, so the launch takes ceil(tiles / SMs) rounds; 192-wide
        // tiles sometimes fill the last round where 256-wide ones leave most SMs idle
        auto rounds = [&](int w) { return (m_tiles * ((N + w - 1) / w) + sm_count - 1) / sm_count; };
        if (rounds(192) * 192 < rounds(256) * 256) bn = 192;
    }
    return bn;
}

tfjsb_status encode(tfjsb_ctx* ctx, CUtensorMap* map, CUtensorMapDataType type, int elem_bytes, const void* base,
                    int64_t inner, int64_t outer, int box_inner, int box_outer, CUtensorMapSwizzle swizzle,
                    const char* what) {
    cuuint64_t dims[2] = {(cuuint64_t)inner, (cuuint64_t)outer};
    cuuint64_t strides[1] = {(cuuint64_t)inner * (cuuint64_t)elem_bytes};
    cuuint32_t box[2] = {(cuuint32_t)box_inner, (cuuint32_t)box_outer};
    cuuint32_t elem[2] = {1u, 1u};
    CUresult r = ctx->encode_tiled(map, type, 2, const_cast<void*>(base), dims, strides, box, elem,
                                   CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS)
        return fail(ctx, TFJSB_ERR_CUDA,
                    std::string("cuTensorMapEncodeTiled failed for ") + what + " (CUresult " + std::to_string((int)r) + ")");
    return TFJSB_OK;
}

}  // namespace

bool gemm_bf16_supported(int64_t M, int64_t N, int64_t K) {
    // row pitches of A, Bt (K bfloat16) and C (N bfloat16) must be multiples of 16 bytes; coordinates are 32-bit
    return M >= 1 && N >= 8 && K >= 8 && (K % 8 == 0) && (N % 8 == 0) && M < (1LL << 31) - 256 && N < (1LL << 31) - 256 &&
           K < (1LL << 31) - 256 && ((M + BLOCK_M - 1) / BLOCK_M) * ((N + 31) / 32) < (1LL << 31);
}

tfjsb_status gemm_bf16_plan(tfjsb_ctx* ctx, const void* a, const void* bt, void* c, bool c_is_bf16, int64_t M, int64_t N,
                            int64_t K, GemmBf16Plan* plan) {
    if (!gemm_bf16_supported(M, N, K)) return fail(ctx, TFJSB_ERR_UNSUPPORTED, "shape not supported by the bfloat16 GEMM");
    if (!ctx->encode_tiled) return fail(ctx, TFJSB_ERR_CUDA, "cuTensorMapEncodeTiled is not available");
    if (c_is_bf16) {
        const char* pair_env = getenv("TFJSB_GEMM_PAIR");
        const bool use_pair = pair_env ? (pair_env[0] == '1' && N >= 64) : gemm_bf16_pair_preferred(M, N, K, ctx->sm_count);
        if (use_pair) return gemm_bf16_pair_plan(ctx, a, bt, c, M, N, K, plan);
    }
    plan->M = M; plan->N = N; plan->K = K;
    plan->c_is_bf16 = c_is_bf16;
    plan->pair = false;
    plan->block_n = choose_block_n(M, N, ctx->sm_count);
    plan->acc_stages = plan->block_n > 128 ? 2 : MAX_ACC_STAGES;
    const int stage_bytes = A_STAGE_BYTES + plan->block_n * 128;
    plan->epi_warps = (K + BK16 - 1) / BK16 <= 4 ? 16 : 8;
    const int epi_bytes = plan->epi_warps * (c_is_bf16 ? 2048 : 4096);
    int stages = (SMEM_LIMIT - 1024 - epi_bytes - 512) / stage_bytes;
    if (stages > MAX_STAGES) stages = MAX_STAGES;
    plan->stages = stages;
    plan->smem_bytes = (size_t)1024 + epi_bytes + (size_t)stages * stage_bytes;
    const int64_t n_tiles = (N + plan->block_n - 1) / plan->block_n;
    const int64_t tiles = ((M + BLOCK_M - 1) / BLOCK_M) * n_tiles;
    if (tiles >= (1LL << 31)) return fail(ctx, TFJSB_ERR_UNSUPPORTED, "too many tiles");
    plan->num_tiles = (int)tiles;
    plan->grid = (int)(tiles < ctx->sm_count ? tiles : ctx->sm_count);
    tfjsb_status st;
    if ((st = encode(ctx, &plan->map_a, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, a, K, M, BK16, BLOCK_M,
                     CU_TENSOR_MAP_SWIZZLE_128B, "A")) != TFJSB_OK) return st;
    if ((st = encode(ctx, &plan->map_b, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, bt, K, N, BK16, plan->block_n,
                     CU_TENSOR_MAP_SWIZZLE_128B, "B")) != TFJSB_OK) return st;
    if (c_is_bf16)
        return encode(ctx, &plan->map_c, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, c, N, M, EPI_COLS, 32,
                      CU_TENSOR_MAP_SWIZZLE_64B, "C");
    return encode(ctx, &plan->map_c, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, c, N, M, EPI_COLS, 32, CU_TENSOR_MAP_SWIZZLE_128B,
                  "C");
}

cudaError_t launch_gemm_bf16(const GemmBf16Plan& plan, const float* bias, int act, unsigned int* dev_status,
                             cudaStream_t s, int64_t* launches) {
    if (plan.pair) return launch_gemm_bf16_pair(plan, bias, act, dev_status, s, launches);
    {
        cudaError_t ae = cudaSuccess;
        if (ae == cudaSuccess) ae = smem_attr_once(reinterpret_cast<const void*>(&gemm_bf16_kernel<false>), SMEM_LIMIT - 2048);
        if (ae == cudaSuccess) ae = smem_attr_once(reinterpret_cast<const void*>(&gemm_bf16_kernel<true>), SMEM_LIMIT - 2048);
        if (ae != cudaSuccess) return ae;
    }
    KernelArgs args;
    args.M = (int)plan.M; args.N = (int)plan.N; args.K = (int)plan.K;
    args.block_n = plan.block_n;
    args.stages = plan.stages;
    args.n_tiles = (int)((plan.N + plan.block_n - 1) / plan.block_n);
    args.num_tiles = plan.num_tiles;
    args.acc_stages = plan.acc_stages;
    args.epi_warps = plan.epi_warps;
    args.bias = bias;
    args.act = act;
    args.dev_status = dev_status;
    cudaError_t e;
    if (plan.c_is_bf16)
        e = launch_k(gemm_bf16_kernel<true>, dim3(plan.grid), dim3(64 + 32 * plan.epi_warps), plan.smem_bytes, s, plan.map_a, plan.map_b,
                     plan.map_c, args);
    else
        e = launch_k(gemm_bf16_kernel<false>, dim3(plan.grid), dim3(64 + 32 * plan.epi_warps), plan.smem_bytes, s, plan.map_a, plan.map_b,
                     plan.map_c, args);
    ++*launches;
    return e;
}

}  // namespace tfjsb

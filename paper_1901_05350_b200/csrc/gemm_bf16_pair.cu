// Tensor-core GEMM on CTA pairs (tcgen05 cta_group::2) for bfloat16 storage:
//
//     C[M,N] = act( A[M,K] . Bt[N,K]^T + bias[N] )      A, Bt, C bfloat16; sums fp32 in tensor memory
//
// The CTA-pair kernel of the fp32-storage path (gemm_tf32_pair.cu) with bfloat16 operands: a k-block is
// 64 elements (the same 128-byte swizzled rows and the same bytes per stage), consumed by four
// `tcgen05.mma.cta_group::2.kind::f16` of K = 16; the epilogue rounds to bfloat16 and stores through
// 64-byte-swizzled slabs.  For the layers whose time is set by the K loop: with 16-bit operands a
// 128 x 256 tile per SM needs 48 KB of operands from L2 for every 4.2 MFLOP, more than L2 and the
// shared memories deliver at the tensor core's rate; a pair shares one 256 x 256 tile, each CTA
// loading its own 128 rows of A and half of the Bt rows, which halves the Bt traffic per multiply-add.
//
// Structure, roles, barriers and bounded waits are those of gemm_tf32_pair.cu.
#include "common.cuh"
#include "ptx_sm100.cuh"
#include "umma_tile.cuh"

namespace tfjsb {

using namespace ptx;
using namespace tile;

namespace {

constexpr int BK16 = 64;      // bfloat16 elements per k-block (128 bytes)
constexpr int UMMA_K16 = 16;  // elements per tcgen05.mma of kind::f16

// D[tmem of both CTAs] (+)= A . B^T over the pair, bfloat16 operands: M = 256, issued by the even CTA.
__device__ __forceinline__ void tc_mma_bf16_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                                 uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}

constexpr int P_THREADS = 320;      // producer warp, MMA warp, 8 epilogue warps
constexpr int P_MAX_STAGES = 8;
constexpr int P_ACC_STAGES = 2;     // 2 x 256 columns = all of tensor memory
constexpr int P_TILE_M = 2 * BLOCK_M;

struct PairArgs16 {
    int M, N, K;
    int block_n;    // columns of the pair's tile: a multiple of 32, 64..256
    int stages;
    int n_tiles;    // tiles along N
    int num_tiles;  // total
    const float* bias;
    int act;
    unsigned int* dev_status;
};

__global__ void __launch_bounds__(P_THREADS, 1)
gemm_bf16_pair_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                      const __grid_constant__ CUtensorMap map_c, const PairArgs16 args) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bar_full[P_MAX_STAGES];        // used in the even CTA only
    __shared__ __align__(8) uint64_t bar_empty[P_MAX_STAGES];       // one per CTA
    __shared__ __align__(8) uint64_t bar_acc_full[P_ACC_STAGES];    // one per CTA
    __shared__ __align__(8) uint64_t bar_acc_empty[P_ACC_STAGES];   // used in the even CTA only
    __shared__ __align__(8) uint64_t bar_drain;
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag_s;

    volatile int* abort_flag = &abort_flag_s;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();    // 0 = even CTA (issues the MMAs), 1 = its partner
    const bool leader = rank == 0;
    const int block_n = args.block_n, stages = args.stages;
    const int half_n = block_n >> 1;
    const int stage_bytes = A_STAGE_BYTES + half_n * 128;
    const int num_k_blocks = (args.K + BK16 - 1) / BK16;
    const int pair = blockIdx.x >> 1, num_pairs = gridDim.x >> 1;

    // dynamic shared memory, identical in both CTAs (the MMA descriptors address both by offset):
    //   [epilogue slabs: 32 KiB][stage 0: A | B half][stage 1] ...
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t epi_base = smem_base;
    const uint32_t stage_base = smem_base + EPI_BYTES;

    if (threadIdx.x == 0) {
        for (int s = 0; s < stages; ++s) {
            mbar_init(smem_u32(&bar_full[s]), 1);
            mbar_init(smem_u32(&bar_empty[s]), 1);
        }
        for (int s = 0; s < P_ACC_STAGES; ++s) {
            mbar_init(smem_u32(&bar_acc_full[s]), 1);
            mbar_init(smem_u32(&bar_acc_empty[s]), 16);  // the eight epilogue warps of both CTAs
        }
        mbar_init(smem_u32(&bar_drain), 1);
        abort_flag_s = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_a) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_b) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_c) : "memory");
    }
    const uint32_t tmem_cols = 512;
    if (warp == 1) {
        // the same warp of both CTAs, writing the address to the same shared-memory slot
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)),
                     "r"(tmem_cols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    // the partner's barriers must be initialised before anything of this CTA can signal them
    cluster_arrive();
    cluster_wait();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;
    pdl_launch_dependents();
    pdl_wait();

    if (warp == 0) {
        // ---------------------------------------------------------------- TMA producer (both CTAs)
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            int issued = 0;
            bool ok = true;
            for (int tile = pair; ok && tile < args.num_tiles; tile += num_pairs) {
                const int m0 = (tile / args.n_tiles) * P_TILE_M + (int)rank * BLOCK_M;
                const int n0 = (tile % args.n_tiles) * block_n + (int)rank * half_n;
                for (int kb = 0; kb < num_k_blocks; ++kb) {
                    if (!bounded_wait(smem_u32(&bar_empty[stage]), phase ^ 1u, abort_flag)) {
                        if (!*abort_flag) {
                            *abort_flag = 1;
                            atomicOr(args.dev_status, DEV_STATUS_TIMEOUT_PRODUCER);
                        }
                        ok = false;
                        break;
                    }
                    // the bytes of both CTAs' copies of this stage are counted on the even CTA's barrier
                    const uint32_t full = map_to_cta(smem_u32(&bar_full[stage]), 0u);
                    if (leader) mbar_arrive_expect_tx(smem_u32(&bar_full[stage]), (uint32_t)(2 * stage_bytes));
                    const uint32_t a_dst = stage_base + (uint32_t)stage * (uint32_t)stage_bytes;
                    tma_load_2d_pair(a_dst, &map_a, full, kb * BK16, m0);
                    tma_load_2d_pair(a_dst + A_STAGE_BYTES, &map_b, full, kb * BK16, n0);
                    ++issued;
                    if (++stage == stages) { stage = 0; phase ^= 1u; }
                }
            }
            if (!ok) {
                // Copies in flight must land before this CTA's shared memory goes away.  The even CTA
                // can watch its "full" barriers (a phase completes when both CTAs' bytes are in); the
                // partner has no barrier of its own to watch and waits out the longest a copy can take.
                const unsigned long long t0 = global_ns();
                if (leader) {
                    for (int k = (issued > stages ? issued - stages : 0); k < issued; ++k) {
                        while (!mbar_try_wait(smem_u32(&bar_full[k % stages]), (uint32_t)((k / stages) & 1))) {
                            if (global_ns() - t0 > WAIT_LIMIT_NS) {
                                atomicOr(args.dev_status, DEV_STATUS_TIMEOUT_DRAIN);
                                break;
                            }
                        }
                    }
                } else {
                    while (global_ns() - t0 < 2000000ull) {}  // 2 ms
                }
            }
        }
    } else if (warp == 1) {
        // ---------------------------------------------------------------- MMA issuer (even CTA only)
        if (lane == 0 && leader) {
            const uint32_t idesc = make_idesc_bf16(P_TILE_M, block_n);
            const uint16_t both = 3;
            int stage = 0;
            uint32_t phase = 0;
            int acc = 0;
            uint32_t acc_phase = 0;
            bool ok = true;
            bool issued_any = false;
            for (int tile = pair; ok && tile < args.num_tiles; tile += num_pairs) {
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
                    for (int k = 0; k < BK16 / UMMA_K16; ++k)
                        tc_mma_bf16_pair(d_tmem, a_desc + (uint64_t)(2 * k), b_desc + (uint64_t)(2 * k), idesc,
                                         (kb | k) != 0 ? 1u : 0u);
                    issued_any = true;
                    tc_commit_pair(smem_u32(&bar_empty[stage]), both);
                    if (++stage == stages) { stage = 0; phase ^= 1u; }
                }
                if (!ok) break;
                tc_commit_pair(smem_u32(&bar_acc_full[acc]), both);
                if (++acc == P_ACC_STAGES) { acc = 0; acc_phase ^= 1u; }
            }
            if (!ok) {
                if (!*abort_flag) {
                    *abort_flag = 1;
                    atomicOr(args.dev_status, DEV_STATUS_TIMEOUT_MMA);
                }
                if (issued_any) {
                    // let the MMAs already issued finish before tensor memory is released
                    tc_commit_pair(smem_u32(&bar_drain), (uint16_t)1);
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
        // ---------------------------------------------------------------- epilogue (warps 2..9, both CTAs)
        // As in the single-CTA kernel: two warps per tensor-memory lane quadrant take alternate
        // 32-column chunks of this CTA's 128 rows.
        const int ew = warp - 2;
        const int quad = warp & 3;
        const int half = ew >> 2;
        const uint32_t slab = epi_base + (uint32_t)ew * EPI_SLAB_BYTES;
        int acc = 0;
        uint32_t acc_phase = 0;
        bool ok = true;
        const int chunks_per_tile = block_n / EPI_COLS;
        int first_chunk = half;
        for (int tile = pair; ok && tile < args.num_tiles; tile += num_pairs) {
            const int m0 = (tile / args.n_tiles) * P_TILE_M + (int)rank * BLOCK_M;
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
            const uint32_t acc_empty = map_to_cta(smem_u32(&bar_acc_empty[acc]), 0u);
            const int row0 = m0 + quad * 32;
            int n_chunks = chunks_per_tile;
            const int live_cols = args.N - n0;
            if (live_cols < block_n) n_chunks = (live_cols + EPI_COLS - 1) / EPI_COLS;
            const bool rows_live = row0 < args.M;
            bool released = false;
            for (int ch = first_chunk; ch < n_chunks; ch += 2) {
                uint32_t r[32];
                const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(acc * block_n + ch * EPI_COLS);
                tc_ld_32x32(taddr, r);
                tc_ld_wait();
                if (ch + 2 >= n_chunks) {
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive_cluster(acc_empty);
                    released = true;
                }
                if (!rows_live) continue;
                const int col0 = n0 + ch * EPI_COLS;
                if (lane == 0) tma_store_wait_read<0>();
                __syncwarp();
                const float* bias = (args.bias != nullptr) ? args.bias + col0 : nullptr;
                const int cols_left = args.N - col0;
                if (args.act == TFJSB_ACT_RELU6) stage_chunk_bf16<TFJSB_ACT_RELU6>(r, bias, cols_left, slab, lane);
                else if (args.act == TFJSB_ACT_RELU) stage_chunk_bf16<TFJSB_ACT_RELU>(r, bias, cols_left, slab, lane);
                else stage_chunk_bf16<TFJSB_ACT_NONE>(r, bias, cols_left, slab, lane);
                fence_async_smem();
                __syncwarp();
                if (lane == 0) {
                    tma_store_2d(&map_c, slab, col0, row0);
                    tma_store_commit();
                }
            }
            if (!released) {
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster(acc_empty);
            }
            if (chunks_per_tile & 1) first_chunk ^= 1;
            if (++acc == P_ACC_STAGES) { acc = 0; acc_phase ^= 1u; }
        }
        if (lane == 0) tma_store_wait_all();
        __syncwarp();
    }

    // ---------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    cluster_arrive();
    cluster_wait();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
    }
}

tfjsb_status encode_pair16(tfjsb_ctx* ctx, CUtensorMap* map, const void* base, int64_t inner, int64_t outer, int box_inner,
                           int box_outer, CUtensorMapSwizzle swizzle, const char* what) {
    cuuint64_t dims[2] = {(cuuint64_t)inner, (cuuint64_t)outer};
    cuuint64_t strides[1] = {(cuuint64_t)inner * 2u};
    cuuint32_t box[2] = {(cuuint32_t)box_inner, (cuuint32_t)box_outer};
    cuuint32_t elem[2] = {1u, 1u};
    CUresult r = ctx->encode_tiled(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, elem,
                                   CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS)
        return fail(ctx, TFJSB_ERR_CUDA,
                    std::string("cuTensorMapEncodeTiled failed for ") + what + " (CUresult " + std::to_string((int)r) + ")");
    return TFJSB_OK;
}

}  // namespace

// Where the pair pays: nowhere yet.  On the shape it was written for (25088 x 512 x 512, the 14 x 14
// pointwise layers at batch 128) it measures 19.6 us alone against 19.7 us for the single-CTA kernel,
// and 23 us against 21.5 us inside the model: with 16-bit operands that GEMM is eight k-blocks per
// tile and three rounds of tiles, and its fixed costs (first loads, last epilogue, 52 MB of HBM
// traffic in 8 us) outweigh the K loop the pair shortens.  The planner therefore never picks it by
// itself; TFJSB_GEMM_PAIR=1 selects it wherever the shape allows (the parity tests do), for shapes
// with long K loops and many tiles, where its fp32-storage sibling wins 6-10 %.
bool gemm_bf16_pair_preferred(int64_t M, int64_t N, int64_t K, int sm_count) {
    (void)M; (void)N; (void)K; (void)sm_count;
    return false;
}

tfjsb_status gemm_bf16_pair_plan(tfjsb_ctx* ctx, const void* a, const void* bt, void* c, int64_t M, int64_t N, int64_t K,
                                 GemmBf16Plan* plan) {
    if (!gemm_bf16_supported(M, N, K)) return fail(ctx, TFJSB_ERR_UNSUPPORTED, "shape not supported by the bfloat16 GEMM");
    if (!ctx->encode_tiled) return fail(ctx, TFJSB_ERR_CUDA, "cuTensorMapEncodeTiled is not available");
    plan->M = M; plan->N = N; plan->K = K;
    plan->c_is_bf16 = true;
    plan->pair = true;
    int bn = 256;
    while (bn > 64 && bn / 2 >= N) bn >>= 1;
    plan->block_n = bn;
    plan->acc_stages = P_ACC_STAGES;
    const int stage_bytes = A_STAGE_BYTES + (bn / 2) * 128;
    int stages = (SMEM_LIMIT - 1024 - EPI_BYTES - 512) / stage_bytes;
    if (stages > P_MAX_STAGES) stages = P_MAX_STAGES;
    plan->stages = stages;
    plan->smem_bytes = (size_t)1024 + EPI_BYTES + (size_t)stages * stage_bytes;
    const int64_t n_tiles = (N + bn - 1) / bn;
    const int64_t tiles = ((M + P_TILE_M - 1) / P_TILE_M) * n_tiles;
    if (tiles >= (1LL << 31)) return fail(ctx, TFJSB_ERR_UNSUPPORTED, "too many tiles");
    plan->num_tiles = (int)tiles;
    const int64_t pairs = ctx->sm_count / 2;
    plan->grid = 2 * (int)(tiles < pairs ? tiles : pairs);
    tfjsb_status st;
    if ((st = encode_pair16(ctx, &plan->map_a, a, K, M, BK16, BLOCK_M, CU_TENSOR_MAP_SWIZZLE_128B, "A")) != TFJSB_OK) return st;
    if ((st = encode_pair16(ctx, &plan->map_b, bt, K, N, BK16, bn / 2, CU_TENSOR_MAP_SWIZZLE_128B, "B")) != TFJSB_OK) return st;
    return encode_pair16(ctx, &plan->map_c, c, N, M, EPI_COLS, 32, CU_TENSOR_MAP_SWIZZLE_64B, "C");
}

cudaError_t launch_gemm_bf16_pair(const GemmBf16Plan& plan, const float* bias, int act, unsigned int* dev_status,
                                  cudaStream_t s, int64_t* launches) {
    {
        cudaError_t ae = cudaSuccess;
        if (ae == cudaSuccess) ae = smem_attr_once(reinterpret_cast<const void*>(&gemm_bf16_pair_kernel), SMEM_LIMIT - 2048);
        if (ae != cudaSuccess) return ae;
    }
    PairArgs16 args;
    args.M = (int)plan.M; args.N = (int)plan.N; args.K = (int)plan.K;
    args.block_n = plan.block_n;
    args.stages = plan.stages;
    args.n_tiles = (int)((plan.N + plan.block_n - 1) / plan.block_n);
    args.num_tiles = plan.num_tiles;
    args.bias = bias;
    args.act = act;
    args.dev_status = dev_status;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(plan.grid);
    cfg.blockDim = dim3(P_THREADS);
    cfg.dynamicSmemBytes = plan.smem_bytes;
    cfg.stream = s;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = g_launch_pdl ? 2 : 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, gemm_bf16_pair_kernel, plan.map_a, plan.map_b, plan.map_c, args);
    ++*launches;
    return e;
}

}  // namespace tfjsb

// Tensor-core GEMM on CTA pairs (tcgen05 cta_group::2) with the fused bias + activation epilogue:
//
//     C[M,N] = act( A[M,K] . Bt[N,K]^T + bias[N] )
//
// One kernel template, two element types: fp32 in and out with TF32 multiplies (the fp32-storage path), and
// bfloat16 in and out (the narrow-storage path: a k-block is 64 elements in the same 128-byte swizzled rows,
// consumed by four `kind::f16` MMAs of K = 16; the epilogue rounds to bfloat16 and stores through
// 64-byte-swizzled slabs).  Sums are fp32 in tensor memory in both.
//
// Same contract as the single-CTA kernels (gemm_cta.cu); this one is for the shapes whose
// time is set by the K loop (large K and N, many tiles).  With fp32 operands a single CTA must bring
// 128 + 256 operand rows of 128 bytes into shared memory for every 128 x 256 x 32 block of
// multiply-adds and read them back out for the tensor core, which saturates the shared memory's
// bandwidth before the tensor pipe.  A CTA pair shares one 256 x block_n tile: each CTA loads its own
// 128 rows of A and only HALF of the Bt rows; the tensor cores of the two SMs read each other's half.
// Bytes written into each shared memory per multiply-add fall by a third.
//
// Structure: clusters of two CTAs, one cluster per SM pair, persistent, static round-robin over
// 256 x block_n tiles.  Per CTA, 10 warps as in the single-CTA kernel:
//   warp 0      producer: waits for its own stage to be free, then issues the bulk tensor copies of
//               its A rows and its half of Bt; their bytes are counted on the EVEN CTA's "full"
//               barrier, which that CTA's producer arms for the bytes of both.
//   warp 1      allocates tensor memory (both CTAs); in the even CTA one thread issues the pair MMAs
//               (M 256, N block_n, K 8) and signals, through tcgen05.commit to both CTAs at once, the
//               stage free ("empty") and the accumulator ready ("acc_full").
//   warps 2-9   epilogue of the CTA's own 128 rows out of its own tensor memory; an accumulator
//               stage is handed back by arriving on the even CTA's "acc_empty" barrier.
// Every wait is bounded and reports through the device status word.  A CTA never leaves before its
// partner has finished (cluster barrier before tensor memory is released), so no signal or operand
// read ever targets a CTA that has gone.
#include "common.cuh"
#include "ptx_sm100.cuh"
#include "umma_tile.cuh"

namespace tfjsb {

using namespace ptx;
using namespace tile;

namespace {

constexpr int P_THREADS = 320;      // producer warp, MMA warp, 8 epilogue warps
constexpr int P_MAX_STAGES = 8;
constexpr int P_ACC_STAGES = 2;     // 2 x 256 columns = all of tensor memory
constexpr int P_TILE_M = 2 * BLOCK_M;

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

// elements per k-block (one 128-byte swizzled row) and per MMA, by element type
template <bool BF16> struct PairElem { static constexpr int BK = BLOCK_K, MMA_K = UMMA_K; };
template <> struct PairElem<true> { static constexpr int BK = 64, MMA_K = 16; };

struct PairArgs {
    int M, N, K;
    int block_n;    // columns of the pair's tile: a multiple of 32, 64..256
    int stages;
    int n_tiles;    // tiles along N
    int num_tiles;  // total
    const float* bias;
    int act;
    unsigned int* dev_status;
};

template <bool BF16>
__global__ void __launch_bounds__(P_THREADS, 1)
gemm_pair_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                      const __grid_constant__ CUtensorMap map_c, const PairArgs args) {
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
    constexpr int BK = PairElem<BF16>::BK, MMA_K = PairElem<BF16>::MMA_K;
    const int stage_bytes = A_STAGE_BYTES + half_n * 128;  // rows of 128 bytes whatever the element type
    const int num_k_blocks = (args.K + BK - 1) / BK;
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
                    tma_load_2d_pair(a_dst, &map_a, full, kb * BK, m0);
                    tma_load_2d_pair(a_dst + A_STAGE_BYTES, &map_b, full, kb * BK, n0);
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
            const uint32_t idesc = BF16 ? make_idesc_bf16(P_TILE_M, block_n) : make_idesc_tf32(P_TILE_M, block_n);
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
                    for (int k = 0; k < BK / MMA_K; ++k) {  // 32 bytes along K per MMA: 2 descriptor units
                        if (BF16) tc_mma_bf16_pair(d_tmem, a_desc + (uint64_t)(2 * k), b_desc + (uint64_t)(2 * k), idesc, (kb | k) != 0 ? 1u : 0u);
                        else tc_mma_tf32_pair(d_tmem, a_desc + (uint64_t)(2 * k), b_desc + (uint64_t)(2 * k), idesc, (kb | k) != 0 ? 1u : 0u);
                    }
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
                const uint32_t row_addr = slab + (uint32_t)lane * 128u;
                const float* bias = (args.bias != nullptr) ? args.bias + col0 : nullptr;
                const int cols_left = args.N - col0;
                if (BF16) {
                    if (args.act == TFJSB_ACT_RELU6) stage_chunk_bf16<TFJSB_ACT_RELU6>(r, bias, cols_left, slab, lane);
                    else if (args.act == TFJSB_ACT_RELU) stage_chunk_bf16<TFJSB_ACT_RELU>(r, bias, cols_left, slab, lane);
                    else stage_chunk_bf16<TFJSB_ACT_NONE>(r, bias, cols_left, slab, lane);
                } else if (args.act == TFJSB_ACT_RELU6) stage_chunk<TFJSB_ACT_RELU6>(r, bias, cols_left, row_addr, lane);
                else if (args.act == TFJSB_ACT_RELU) stage_chunk<TFJSB_ACT_RELU>(r, bias, cols_left, row_addr, lane);
                else stage_chunk<TFJSB_ACT_NONE>(r, bias, cols_left, row_addr, lane);
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

tfjsb_status encode_pair_2d(tfjsb_ctx* ctx, CUtensorMap* map, const void* base, int64_t inner, int64_t outer, int box_inner,
                            int box_outer, const char* what, bool bf16 = false, CUtensorMapSwizzle swizzle = CU_TENSOR_MAP_SWIZZLE_128B) {
    cuuint64_t dims[2] = {(cuuint64_t)inner, (cuuint64_t)outer};
    cuuint64_t strides[1] = {(cuuint64_t)inner * (bf16 ? 2u : 4u)};
    cuuint32_t box[2] = {(cuuint32_t)box_inner, (cuuint32_t)box_outer};
    cuuint32_t elem[2] = {1u, 1u};
    CUresult r = ctx->encode_tiled(map, bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2,
                                   const_cast<void*>(base), dims, strides, box, elem, CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle,
                                   CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS)
        return fail(ctx, TFJSB_ERR_CUDA,
                    std::string("cuTensorMapEncodeTiled failed for ") + what + " (CUresult " + std::to_string((int)r) + ")");
    return TFJSB_OK;
}

}  // namespace

// Where the pair kernel pays.  Both kernels turn out to be bound by shared-memory bandwidth, not by the
// tensor pipe: per 128 x 256 x 32 block of multiply-adds a single CTA's shared memory takes 48 KB of
// copy-engine writes and gives the tensor core 48 KB of operand reads (768 cycles at 128 B/cycle against
// 512 cycles of MMA work); in a pair each CTA's memory takes 32 KB and gives 48 KB.  Measured, the pair
// is 6-10 % faster once the K loop dominates (K >= 512) and there are at least two and a half rounds of
// 256 x 256 tiles for the SM pairs; with fewer tiles its coarser tiling loses more than that.
bool gemm_tf32_pair_preferred(int64_t M, int64_t N, int64_t K, int sm_count) {
    if (!gemm_tf32_supported(M, N, K)) return false;
    if (K < 512 || N < 512) return false;
    const int64_t tiles = ((M + P_TILE_M - 1) / P_TILE_M) * ((N + 255) / 256);
    const int64_t pairs = sm_count / 2;
    return 2 * tiles >= 5 * pairs;
}

tfjsb_status gemm_tf32_pair_plan(tfjsb_ctx* ctx, const float* a, const float* bt, float* c, int64_t M, int64_t N, int64_t K,
                                 GemmTf32Plan* plan) {
    if (!gemm_tf32_supported(M, N, K)) return fail(ctx, TFJSB_ERR_UNSUPPORTED, "shape not supported by the TF32 GEMM");
    if (!ctx->encode_tiled) return fail(ctx, TFJSB_ERR_CUDA, "cuTensorMapEncodeTiled is not available");
    plan->M = M; plan->N = N; plan->K = K;
    plan->gather = false;
    plan->x = nullptr;
    plan->pair = true;
    plan->cluster_split = false;
    plan->splits = 1;
    plan->c = c;
    plan->batches = 1;
    int bn = 256;
    while (bn > 64 && bn / 2 >= N) bn >>= 1;
    plan->block_n = bn;
    plan->acc_stages = P_ACC_STAGES;
    const int stage_bytes = A_STAGE_BYTES + (bn / 2) * BLOCK_K * 4;
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
    if ((st = encode_pair_2d(ctx, &plan->map_a, a, K, M, BLOCK_K, BLOCK_M, "A")) != TFJSB_OK) return st;
    if ((st = encode_pair_2d(ctx, &plan->map_b, bt, K, N, BLOCK_K, bn / 2, "B")) != TFJSB_OK) return st;
    return encode_pair_2d(ctx, &plan->map_c, c, N, M, EPI_COLS, 32, "C");
}

namespace {

template <bool BF16>
cudaError_t launch_pair(const CUtensorMap& map_a, const CUtensorMap& map_b, const CUtensorMap& map_c, int64_t M, int64_t N, int64_t K,
                        int block_n, int stages, int num_tiles, int grid, size_t smem_bytes, const float* bias, int act,
                        unsigned int* dev_status, cudaStream_t s, int64_t* launches) {
    cudaError_t ae = smem_attr_once(reinterpret_cast<const void*>(&gemm_pair_kernel<BF16>), SMEM_LIMIT - 2048);
    if (ae != cudaSuccess) return ae;
    PairArgs args;
    args.M = (int)M; args.N = (int)N; args.K = (int)K;
    args.block_n = block_n;
    args.stages = stages;
    args.n_tiles = (int)((N + block_n - 1) / block_n);
    args.num_tiles = num_tiles;
    args.bias = bias;
    args.act = act;
    args.dev_status = dev_status;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(P_THREADS);
    cfg.dynamicSmemBytes = smem_bytes;
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
    cudaError_t e = cudaLaunchKernelEx(&cfg, gemm_pair_kernel<BF16>, map_a, map_b, map_c, args);
    ++*launches;
    return e;
}

}  // namespace

cudaError_t launch_gemm_tf32_pair(const GemmTf32Plan& plan, const float* bias, int act, unsigned int* dev_status,
                                  cudaStream_t s, int64_t* launches) {
    return launch_pair<false>(plan.map_a, plan.map_b, plan.map_c, plan.M, plan.N, plan.K, plan.block_n, plan.stages, plan.num_tiles,
                              plan.grid, plan.smem_bytes, bias, act, dev_status, s, launches);
}

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
    if ((st = encode_pair_2d(ctx, &plan->map_a, a, K, M, PairElem<true>::BK, BLOCK_M, "A", true)) != TFJSB_OK) return st;
    if ((st = encode_pair_2d(ctx, &plan->map_b, bt, K, N, PairElem<true>::BK, bn / 2, "B", true)) != TFJSB_OK) return st;
    return encode_pair_2d(ctx, &plan->map_c, c, N, M, EPI_COLS, 32, "C", true, CU_TENSOR_MAP_SWIZZLE_64B);
}

cudaError_t launch_gemm_bf16_pair(const GemmBf16Plan& plan, const float* bias, int act, unsigned int* dev_status,
                                  cudaStream_t s, int64_t* launches) {
    return launch_pair<true>(plan.map_a, plan.map_b, plan.map_c, plan.M, plan.N, plan.K, plan.block_n, plan.stages, plan.num_tiles,
                             plan.grid, plan.smem_bytes, bias, act, dev_status, s, launches);
}

}  // namespace tfjsb

// Split-K tensor-core GEMM whose slices meet in distributed shared memory:
//
//     C[M,N] = act( A[M,K] . Bt[N,K]^T + bias[N] )        fp32 in, fp32 out, TF32 multiplies
//
// For GEMMs with few output tiles and a long K loop (the dense layer; every pointwise layer at small
// batch), where the persistent kernel would leave most SMs idle while a few walk all the k-blocks
// one after the other.  A cluster of S CTAs (2, 4 or 8) owns one 128 x block_n tile; CTA r
// accumulates the r-th slice of the k-blocks in its tensor memory and then sends every band of 128/S
// rows of its partial tile to the shared memory of the CTA that owns the band (stores into the
// partner's shared memory); after one cluster barrier every CTA finds the S partial copies of its
// band in its own shared memory, adds them in slice order, adds the bias, applies the activation and
// stores its band of C.  No workspace in global memory, no second kernel, no access to a partner's
// memory after the barrier (so a CTA may leave as soon as it is done), and the result does not
// depend on which slice finishes first.
//
// Per CTA, 6 warps: warp 0 producer (bulk tensor copies into a ring of stages), warp 1 tensor-memory
// allocation and MMA issue, warps 2-5 one per tensor-memory lane quadrant: accumulator -> shared
// memory, then the reduction.  Each CTA processes exactly one work item.
//
// Two cluster barriers order the remote accesses.  The first ("started") is arrived at by every
// thread right after the CTA's own set-up and waited for before the first store into a partner: the
// shared memory of a CTA may only be touched once that CTA is known to be executing, and being
// launched as one cluster does not by itself order a fast CTA's store after a slow partner's start.
// The second ("delivered") separates the remote stores from the reduction.  Every mbarrier wait is
// bounded; a CTA whose wait gave up still takes part in both cluster barriers, so its partners never
// wait for it (the barriers themselves have no limit: every path below reaches them).
#include <cstdlib>

#include "common.cuh"
#include "ptx_sm100.cuh"
#include "umma_tile.cuh"

namespace tfjsb {

using namespace ptx;
using namespace tile;

namespace {

constexpr int S_THREADS = 192;
constexpr int S_MAX_STAGES = 8;
constexpr int S_MAX_BLOCK_N = 128;
constexpr int S_MIN_KB = 4;        // k-blocks per slice at least
constexpr int S_MAX_SPLITS = 8;    // portable cluster size

struct SplitArgs {
    int M, N, K;
    int block_n;       // 32, 64 or 128
    int stages;
    int n_tiles;       // tiles along N
    int splits;        // = cluster size
    int kb_per_split;
    const float* bias;
    int act;
    float* c;
    unsigned int* dev_status;
};

__device__ __forceinline__ void st_cluster_v4(uint32_t cluster_addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    asm volatile("st.shared::cluster.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(cluster_addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
__device__ __forceinline__ float4 ld_shared_v4(uint32_t addr) {
    float4 v;
    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr) : "memory");
    return v;
}

__global__ void __launch_bounds__(S_THREADS, 1)
gemm_tf32_splitk_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                        const SplitArgs args) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bar_full[S_MAX_STAGES];
    __shared__ __align__(8) uint64_t bar_empty[S_MAX_STAGES];
    __shared__ __align__(8) uint64_t bar_acc_full;
    __shared__ __align__(8) uint64_t bar_drain;
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag_s;

    volatile int* abort_flag = &abort_flag_s;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int splits = args.splits;
    const uint32_t rank = cluster_ctarank();              // = slice of the K loop
    const int tile = blockIdx.x / splits;                 // the cluster's tile
    const int block_n = args.block_n, stages = args.stages;
    const int chunks = block_n / EPI_COLS;
    const int stage_bytes = A_STAGE_BYTES + block_n * BLOCK_K * 4;
    const int num_k_blocks = (args.K + BLOCK_K - 1) / BLOCK_K;
    const int kb_begin = (int)rank * args.kb_per_split;
    const int kb_end = min(num_k_blocks, kb_begin + args.kb_per_split);
    const int m0 = (tile / args.n_tiles) * BLOCK_M;
    const int n0 = (tile % args.n_tiles) * block_n;

    // dynamic shared memory, the same layout in every CTA of the cluster:
    //   [this CTA's band of every slice: S x (128/S rows) x chunks x 128 B, 16-byte pieces swizzled by row][stage 0: A | B] ...
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t partial_base = smem_base;
    const uint32_t stage_base = smem_base + (uint32_t)(BLOCK_M * block_n * 4);

    if (threadIdx.x == 0) {
        for (int s = 0; s < stages; ++s) {
            mbar_init(smem_u32(&bar_full[s]), 1);
            mbar_init(smem_u32(&bar_empty[s]), 1);
        }
        mbar_init(smem_u32(&bar_acc_full), 1);
        mbar_init(smem_u32(&bar_drain), 1);
        abort_flag_s = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_a) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_b) : "memory");
    }
    const uint32_t tmem_cols = block_n < 32 ? 32u : (uint32_t)block_n;  // 32, 64 or 128: a power of two
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)),
                     "r"(tmem_cols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;
    // barrier "started", arrive half: this CTA is running and its shared memory may be written by the
    // partners.  Each thread completes it (cluster_wait) where it next needs it: warps 2-5 before
    // their first remote store, warps 0-1 at the end of their role, before arriving at the second barrier.
    cluster_arrive();
    pdl_launch_dependents();
    pdl_wait();

    if (warp == 0) {
        // ---------------------------------------------------------------- TMA producer
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            int issued = 0;
            bool ok = true;
            for (int kb = kb_begin; kb < kb_end; ++kb) {
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
                tma_load_2d(a_dst, &map_a, full, kb * BLOCK_K, m0);
                tma_load_2d(a_dst + A_STAGE_BYTES, &map_b, full, kb * BLOCK_K, n0);
                ++issued;
                if (++stage == stages) { stage = 0; phase ^= 1u; }
            }
            if (!ok) {
                // wait (bounded) for the copies in flight so that nothing lands after the CTA has gone
                const unsigned long long t0 = global_ns();
                for (int k = (issued > stages ? issued - stages : 0); k < issued; ++k) {
                    while (!mbar_try_wait(smem_u32(&bar_full[k % stages]), (uint32_t)((k / stages) & 1))) {
                        if (global_ns() - t0 > WAIT_LIMIT_NS) {
                            atomicOr(args.dev_status, DEV_STATUS_TIMEOUT_DRAIN);
                            break;
                        }
                    }
                }
            }
        }
        cluster_wait();
    } else if (warp == 1) {
        // ---------------------------------------------------------------- MMA issuer
        if (lane == 0) {
            const uint32_t idesc = make_idesc_tf32(BLOCK_M, block_n);
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            bool issued_any = false;
            for (int kb = kb_begin; kb < kb_end; ++kb) {
                if (!bounded_wait(smem_u32(&bar_full[stage]), phase, abort_flag)) { ok = false; break; }
                tc_fence_after();
                const uint32_t a_addr = stage_base + (uint32_t)stage * (uint32_t)stage_bytes;
                const uint64_t a_desc = make_kmajor_sw128_desc(a_addr);
                const uint64_t b_desc = make_kmajor_sw128_desc(a_addr + A_STAGE_BYTES);
#pragma unroll
                for (int k = 0; k < BLOCK_K / UMMA_K; ++k)
                    tc_mma_tf32(tmem_base, a_desc + (uint64_t)(2 * k), b_desc + (uint64_t)(2 * k), idesc,
                                (kb != kb_begin || k != 0) ? 1u : 0u);
                issued_any = true;
                tc_commit(smem_u32(&bar_empty[stage]));
                if (++stage == stages) { stage = 0; phase ^= 1u; }
            }
            if (ok) {
                tc_commit(smem_u32(&bar_acc_full));
            } else {
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
        cluster_wait();
    } else {
        // ---------------------------------------------------------------- accumulator -> the band owners' shared memory (warps 2..5)
        const int quad = warp & 3;  // the tensor-memory lanes this warp may read: 32*quad ..
        cluster_wait();             // every partner has started: its shared memory exists and may be written
        const bool got = bounded_wait(smem_u32(&bar_acc_full), 0u, abort_flag);
        if (__all_sync(0xffffffffu, got)) {
            tc_fence_after();
            const int rows_per = BLOCK_M / splits;
            const int row = quad * 32 + lane;            // this lane's row of the tile
            const int owner = row / rows_per, i = row - owner * rows_per;
            for (int ch = 0; ch < chunks; ++ch) {
                uint32_t r[32];
                tc_ld_32x32(tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(ch * EPI_COLS), r);
                tc_ld_wait();
                // slot of (slice = this CTA, band row i, chunk ch) in the owner's shared memory
                const uint32_t dst = map_to_cta(partial_base + (uint32_t)((((int)rank * rows_per + i) * chunks + ch) * 128), (uint32_t)owner);
#pragma unroll
                for (int j = 0; j < 8; ++j)
                    st_cluster_v4(dst + (uint32_t)((j ^ (i & 7)) << 4), r[4 * j], r[4 * j + 1], r[4 * j + 2], r[4 * j + 3]);
            }
        } else if (lane == 0 && !*abort_flag) {
            *abort_flag = 1;
            atomicOr(args.dev_status, DEV_STATUS_TIMEOUT_EPILOGUE);
        }
    }

    // ---------------------------------------------------------------- reduction of this CTA's band
    tc_fence_before();
    __syncthreads();
    cluster_arrive();   // this CTA's stores into its partners' shared memory are done ...
    cluster_wait();     // ... and every partner's stores into this one are visible
    if (warp >= 2) {
        const int rows_per = BLOCK_M / splits;
        const int total = rows_per * chunks * 8;         // 16-byte pieces in the band (a multiple of 128)
        for (int e = (int)threadIdx.x - 64; e < total; e += S_THREADS - 64) {
            const int j = e & 7;                          // consecutive threads, consecutive bytes of C
            const int ch = (e >> 3) % chunks;
            const int i = (e >> 3) / chunks;
            const int grow = m0 + (int)rank * rows_per + i, gcol = n0 + ch * EPI_COLS + 4 * j;
            const bool live = grow < args.M && gcol < args.N;   // N % 4 == 0: a quad is all in or all out
            float4 bq = make_float4(0.f, 0.f, 0.f, 0.f);
            if (args.bias != nullptr && live) bq = __ldg(reinterpret_cast<const float4*>(args.bias + gcol));
            const uint32_t piece = partial_base + (uint32_t)((i * chunks + ch) * 128) + (uint32_t)((j ^ (i & 7)) << 4);
            const uint32_t slice_pitch = (uint32_t)(rows_per * chunks * 128);
            float4 v = ld_shared_v4(piece);
            for (int sl = 1; sl < splits; ++sl) {
                const float4 p = ld_shared_v4(piece + (uint32_t)sl * slice_pitch);
                v.x += p.x; v.y += p.y; v.z += p.z; v.w += p.w;
            }
            if (live) {
                v.x = apply_act(v.x + bq.x, args.act); v.y = apply_act(v.y + bq.y, args.act);
                v.z = apply_act(v.z + bq.z, args.act); v.w = apply_act(v.w + bq.w, args.act);
                *reinterpret_cast<float4*>(args.c + (int64_t)grow * args.N + gcol) = v;
            }
        }
    }
    // nothing touches a partner's shared memory after the barrier above: no second barrier before leaving
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
    }
}

tfjsb_status encode_split_2d(tfjsb_ctx* ctx, CUtensorMap* map, const void* base, int64_t inner, int64_t outer, int box_inner,
                             int box_outer, const char* what) {
    cuuint64_t dims[2] = {(cuuint64_t)inner, (cuuint64_t)outer};
    cuuint64_t strides[1] = {(cuuint64_t)inner * 4u};
    cuuint32_t box[2] = {(cuuint32_t)box_inner, (cuuint32_t)box_outer};
    cuuint32_t elem[2] = {1u, 1u};
    CUresult r = ctx->encode_tiled(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<void*>(base), dims, strides, box, elem,
                                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                   CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS)
        return fail(ctx, TFJSB_ERR_CUDA,
                    std::string("cuTensorMapEncodeTiled failed for ") + what + " (CUresult " + std::to_string((int)r) + ")");
    return TFJSB_OK;
}

}  // namespace

// Shared memory of one CTA: alignment slack, the partial tile, the stage ring (at most four stages, so
// that two CTAs with narrow tiles fit one SM).
int splitk_stages(int kb_per_split) { return kb_per_split < 4 ? kb_per_split : 4; }
size_t splitk_smem_bytes(int block_n, int stages) {
    return (size_t)1024 + (size_t)BLOCK_M * block_n * 4 + (size_t)stages * (A_STAGE_BYTES + block_n * BLOCK_K * 4);
}

// Tile width and number of slices for a GEMM whose tiles cannot occupy the SMs; false: do not split.
// Slices come in powers of two up to the portable cluster size, at least four k-blocks each.  Each
// CTA runs a single work item, so everything should be resident at once (a second, partly filled
// wave would cost a whole kernel's fixed latency again): the choice is the (width, slices) pair that
// puts the most CTAs on the chip within what fits (one or two CTAs per SM, by shared memory); among
// equals the wider tile, whose MMAs are the more efficient.
bool gemm_tf32_splitk_choice(int64_t M, int64_t N, int64_t K, int sm_count, int* block_n, int* splits) {
    if (!gemm_tf32_supported(M, N, K)) return false;
    const int64_t m_tiles = (M + BLOCK_M - 1) / BLOCK_M;
    const int64_t nkb = (K + BLOCK_K - 1) / BLOCK_K;
    if (m_tiles * ((N + 31) / 32) >= sm_count) return false;  // enough 32-wide tiles without cutting K
    int max_s = 1;
    while (max_s * 2 <= S_MAX_SPLITS && nkb / (max_s * 2) >= S_MIN_KB) max_s *= 2;
    if (max_s < 2) return false;
    int64_t best = 0;
    for (int bn = S_MAX_BLOCK_N; bn >= 32; bn >>= 1) {
        if (bn >= 2 * N && bn > 32) continue;  // wider than the matrix
        const int64_t tiles = m_tiles * ((N + bn - 1) / bn);
        for (int s = max_s; s >= 2; s >>= 1) {
            const int kbs = (int)((nkb + s - 1) / s);
            if ((int64_t)(s - 1) * kbs >= nkb) continue;  // the last slice would be empty
            const size_t smem = splitk_smem_bytes(bn, splitk_stages(kbs));
            const int64_t capacity = (int64_t)sm_count * (2 * smem + 2048 <= (size_t)SMEM_LIMIT ? 2 : 1);
            if (tiles * s > capacity) continue;
            if (tiles * s > best) {
                best = tiles * s;
                *block_n = bn;
                *splits = s;
            }
            break;  // fewer slices of the same width only lower the count
        }
    }
    return best > 0;
}

tfjsb_status gemm_tf32_splitk_plan(tfjsb_ctx* ctx, const float* a, const float* bt, float* c, int64_t M, int64_t N, int64_t K,
                                   int block_n, int splits, GemmTf32Plan* plan) {
    if (!ctx->encode_tiled) return fail(ctx, TFJSB_ERR_CUDA, "cuTensorMapEncodeTiled is not available");
    plan->M = M; plan->N = N; plan->K = K;
    plan->gather = false;
    plan->pair = false;
    plan->x = nullptr;
    plan->c = c;
    plan->batches = 1;
    plan->cluster_split = true;
    const int64_t nkb = (K + BLOCK_K - 1) / BLOCK_K;
    const int kbs = (int)((nkb + splits - 1) / splits);
    if ((int64_t)(splits - 1) * kbs >= nkb) return fail(ctx, TFJSB_ERR_UNSUPPORTED, "a split-K slice would be empty");
    plan->block_n = block_n;
    plan->splits = splits;
    plan->kb_per_split = kbs;
    plan->acc_stages = 1;
    plan->stages = splitk_stages(kbs);
    plan->smem_bytes = splitk_smem_bytes(block_n, plan->stages);
    const int64_t tiles = ((M + BLOCK_M - 1) / BLOCK_M) * ((N + block_n - 1) / block_n);
    if (tiles * splits >= (1LL << 31)) return fail(ctx, TFJSB_ERR_UNSUPPORTED, "too many tiles");
    plan->num_tiles = (int)tiles;
    plan->grid = (int)(tiles * splits);
    tfjsb_status st;
    if ((st = encode_split_2d(ctx, &plan->map_a, a, K, M, BLOCK_K, BLOCK_M, "A")) != TFJSB_OK) return st;
    if ((st = encode_split_2d(ctx, &plan->map_b, bt, K, N, BLOCK_K, block_n, "B")) != TFJSB_OK) return st;
    plan->map_c = plan->map_b;  // unused: C is stored directly
    return TFJSB_OK;
}

cudaError_t launch_gemm_tf32_splitk(const GemmTf32Plan& plan, const float* bias, int act, unsigned int* dev_status,
                                    cudaStream_t s, int64_t* launches) {
    {
        cudaError_t ae = cudaSuccess;
        if (ae == cudaSuccess) ae = smem_attr_once(reinterpret_cast<const void*>(&gemm_tf32_splitk_kernel), SMEM_LIMIT - 2048);
        if (ae != cudaSuccess) return ae;
    }
    SplitArgs args;
    args.M = (int)plan.M; args.N = (int)plan.N; args.K = (int)plan.K;
    args.block_n = plan.block_n;
    args.stages = plan.stages;
    args.n_tiles = (int)((plan.N + plan.block_n - 1) / plan.block_n);
    args.splits = plan.splits;
    args.kb_per_split = plan.kb_per_split;
    args.bias = bias;
    args.act = act;
    args.c = plan.c;
    args.dev_status = dev_status;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(plan.grid);
    cfg.blockDim = dim3(S_THREADS);
    cfg.dynamicSmemBytes = plan.smem_bytes;
    cfg.stream = s;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)plan.splits;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = g_launch_pdl ? 2 : 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, gemm_tf32_splitk_kernel, plan.map_a, plan.map_b, args);
    ++*launches;
    return e;
}

}  // namespace tfjsb

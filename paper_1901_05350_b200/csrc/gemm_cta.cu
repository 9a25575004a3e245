// Tensor-core GEMM for sm_100a with the fused bias + activation epilogue:
//
//     C[M,N] = act( A[M,K] . Bt[N,K]^T + bias[N] )        fp32 in, fp32 out
//
// A and Bt are row-major with K contiguous ("K-major"), which is what a pointwise convolution
// over NHWC activations gives for A (rows = pixels, columns = input channels) and what the
// model builder / the matMul entry point produce for the weights.  Operands are fed to the
// tensor cores as they lie in memory (`kind::tf32` reads the fp32 bit pattern and uses its top
// 19 bits); products are accumulated in fp32 in tensor memory.
//
// Structure (one persistent CTA per SM, 10 warps, static round-robin over 128 x block_n tiles):
//   warp 0      producer: one thread issues the bulk tensor copies (TMA, 128-byte swizzle) of the
//               A tile [128 x 32] and the Bt tile [block_n x 32] of each k-block into a ring of
//               shared-memory stages, signalling a "full" mbarrier per stage.
//   warp 1      allocates tensor memory; one thread issues tcgen05.mma (M=128, N=block_n, K=8,
//               four per k-block) into one of two accumulator stages, frees shared-memory stages
//               with tcgen05.commit -> "empty" mbarrier, and hands a finished accumulator to the
//               epilogue with tcgen05.commit -> "acc_full".
//   warps 2-9   epilogue: each warp reads the 32 accumulator rows (TMEM lanes) its warp id allows
//               it to read, 32 columns at a time (tcgen05.ld); the two warps of a lane quadrant
//               take alternate column chunks.  A chunk gets bias and activation in registers, goes
//               into the warp's own swizzled staging slab and leaves with a bulk tensor store
//               (clipped at the matrix edge by the hardware).  One warp per scheduler cannot hide
//               its own instruction latency, hence eight.
//               The two accumulator stages let the epilogue of tile i overlap the MMAs of tile i+1.
// Ragged edges need no special code: rows/columns past M, N or K are zero-filled on load and
// clipped on store by the tensor maps.  A batch of independent products of one shape (rank-3 matMul)
// is one launch: the tensor maps carry the batch as a third dimension, and a tile is (batch, rows,
// columns), so the tiles of all products share the SMs.
//
// Every wait is bounded: a wait that exceeds WAIT_LIMIT_NS raises an abort flag that all roles
// poll, ORs a code into the context's device status word, and the CTA drains its copies, frees
// its tensor memory and returns.
//
// The same pipeline serves bfloat16 storage (the narrow-storage mode, the 16-bit analogue of the
// paper's half-float textures, Sec. 4.1.3): `gemm_pipeline` is a template on the element format and
// `gemm_tf32_kernel` / `gemm_bf16_kernel` are its instances.  With bfloat16 a k-block is 64 elements
// (still one 128-byte swizzle row, consumed by four `kind::f16` MMAs of K = 16), products of two
// bfloat16 are exact in fp32, the sums are fp32 in tensor memory, and the result gets the fp32 bias,
// the activation and one rounding (to nearest even) when it is stored as bfloat16.  Half the bytes per
// tile leave the layers with one or two k-blocks per tile bound by the epilogue's latency per 32 x 32
// block, so those run with sixteen epilogue warps, four per lane quadrant, taking every fourth block;
// long K loops keep eight (the extra warps' polling costs them about 4 %).
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
constexpr int MAX_EPI_WARPS = 16;    // eight or sixteen epilogue warps: two or four per tensor-memory lane quadrant
constexpr int GEMM_MAX_THREADS = 64 + MAX_EPI_WARPS * 32;  // producer warp, MMA warp, the epilogue warps
constexpr int GATHER_EPI_WARPS = 8;
constexpr int GATHER_GROUPS = 3;     // implicit-GEMM convolution: groups of 4 warps that build A tiles
constexpr int CONV_THREADS = 64 + GATHER_EPI_WARPS * 32 + GATHER_GROUPS * 128;

// element formats of the pipeline: what A and Bt are stored as, and what C is stored as
constexpr int IO_F32 = 0;        // fp32 in (multiplied as TF32), fp32 out
constexpr int IO_BF16 = 1;       // bfloat16 in, bfloat16 out
constexpr int IO_BF16_F32 = 2;   // bfloat16 in, fp32 out

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

// ---- A-row gathers of the implicit-GEMM convolution ---------------------------------------------
// Each fills v[0..31] with columns k0..k0+31 of one row of the im2col matrix: k = (ky*fw + kx)*Cin + ci
// -> x[iy0 + ky*dh, ix0 + kx*dw, ci], zero outside the image, for k >= k_total and for dead rows.

// Window and channel count known at compile time and fh*fw*Cin <= 32 (one k-block): no index
// arithmetic is left at run time beyond three row pointers and six bounds flags.
template <int FH, int FW, int CIN>
__device__ __forceinline__ void gather_small(float (&v)[BLOCK_K], const float* __restrict__ xn, const ConvGeom& g,
                                             int iy0, int ix0, bool live) {
    static_assert(FH * FW * CIN <= BLOCK_K, "one k-block only");
    const float* rowp[FH];
    bool vy[FH], vx[FW];
#pragma unroll
    for (int ky = 0; ky < FH; ++ky) {
        const int iy = iy0 + ky * g.dh;
        vy[ky] = live && iy >= 0 && iy < g.H;
        rowp[ky] = xn + ((int64_t)iy * g.W + ix0) * CIN;
    }
#pragma unroll
    for (int kx = 0; kx < FW; ++kx) {
        const int ix = ix0 + kx * g.dw;
        vx[kx] = ix >= 0 && ix < g.W;
    }
    const int dwc = g.dw * CIN;
#pragma unroll
    for (int e = 0; e < BLOCK_K; ++e) {
        if (e < FH * FW * CIN) {
            const int ky = e / (FW * CIN), kx = (e / CIN) % FW, ci = e % CIN;
            v[e] = (vy[ky] && vx[kx]) ? __ldg(rowp[ky] + kx * dwc + ci) : 0.0f;
        } else {
            v[e] = 0.0f;
        }
    }
}

// Cin % 4 == 0: four consecutive k share a tap, so each quad is one float4 load.
__device__ __forceinline__ void gather_vec4(float (&v)[BLOCK_K], const float* __restrict__ xn, const ConvGeom& g,
                                            int iy0, int ix0, bool live, int k0, int k_total) {
    int tap = k0 / g.C;
    int ci = k0 - tap * g.C;
    int ky = tap / g.fw;
    int kx = tap - ky * g.fw;
#pragma unroll
    for (int e = 0; e < BLOCK_K; e += 4) {
        float4 q = make_float4(0.f, 0.f, 0.f, 0.f);
        const int iy = iy0 + ky * g.dh, ix = ix0 + kx * g.dw;
        if (live && k0 + e < k_total && iy >= 0 && iy < g.H && ix >= 0 && ix < g.W)
            q = __ldg(reinterpret_cast<const float4*>(xn + ((int64_t)iy * g.W + ix) * g.C + ci));
        v[e] = q.x; v[e + 1] = q.y; v[e + 2] = q.z; v[e + 3] = q.w;
        ci += 4;
        if (ci == g.C) { ci = 0; if (++kx == g.fw) { kx = 0; ++ky; } }
    }
}

// Any window and channel count: a pointer walks the tap, re-based when the tap column or row changes.
__device__ __forceinline__ void gather_scalar(float (&v)[BLOCK_K], const float* __restrict__ xn, const ConvGeom& g,
                                              int iy0, int ix0, bool live, int k0, int k_total) {
    int tap = k0 / g.C;
    int ci = k0 - tap * g.C;
    int ky = tap / g.fw;
    int kx = tap - ky * g.fw;
    int iy = iy0 + ky * g.dh, ix = ix0 + kx * g.dw;
    const float* p = xn + ((int64_t)iy * g.W + ix) * g.C + ci;
    bool ok = live && iy >= 0 && iy < g.H && ix >= 0 && ix < g.W;
    const int left = k_total - k0;
#pragma unroll
    for (int e = 0; e < BLOCK_K; ++e) {
        v[e] = (ok && e < left) ? __ldg(p) : 0.0f;
        ++p;
        if (++ci == g.C) {
            ci = 0;
            if (++kx == g.fw) { kx = 0; ++ky; }
            iy = iy0 + ky * g.dh;
            ix = ix0 + kx * g.dw;
            p = xn + ((int64_t)iy * g.W + ix) * g.C;
            ok = live && iy >= 0 && iy < g.H && ix >= 0 && ix < g.W;
        }
    }
}

struct KernelArgs {
    int M, N, K;
    int block_n;
    int stages;
    int n_tiles;    // tiles along N
    int tiles_per_batch;  // tiles of one product (rows x columns)
    int num_tiles;  // total, over all products of the batch
    int acc_stages;  // accumulator stages in tensor memory: 2 (block_n 256) or 4
    int epi_warps;   // 8 or 16
    const float* bias;
    int act;
    unsigned int* dev_status;
    // implicit-GEMM convolution only: the input tensor and its geometry (A is gathered, not copied)
    const float* x;
    ConvGeom g;
};

template <bool GATHER, int IO, bool BATCHED>
__device__ __forceinline__ void gemm_pipeline(const CUtensorMap& map_a, const CUtensorMap& map_b, const CUtensorMap& map_c,
                                              const KernelArgs& args) {
    static_assert(!GATHER || IO == IO_F32, "the gathering producer builds fp32 tiles");
    constexpr bool IN_BF16 = IO != IO_F32;
    constexpr bool OUT_BF16 = IO == IO_BF16;
    constexpr int BK = IN_BF16 ? 64 : BLOCK_K;        // elements per k-block: 128 bytes either way
    constexpr int MMAS_PER_KB = 4;                    // 32 bytes of K per tcgen05.mma in both formats
    constexpr uint32_t SLAB_BYTES = OUT_BF16 ? 2048u : (uint32_t)EPI_SLAB_BYTES;  // 32 rows x 32 columns of the output type
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
    const int epi_warps = GATHER ? GATHER_EPI_WARPS : args.epi_warps;
    const int stage_bytes = A_STAGE_BYTES + block_n * 128;
    const int num_k_blocks = (args.K + BK - 1) / BK;

    // dynamic shared memory, aligned to the 1024-byte swizzle pattern:
    //   [epilogue slabs, one per epilogue warp][stage 0: A | B][stage 1] ...
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t epi_base = smem_base;
    const uint32_t stage_base = smem_base + (uint32_t)epi_warps * SLAB_BYTES;

    if (threadIdx.x == 0) {
        for (int s = 0; s < stages; ++s) {
            // a stage is full when the copy engine has delivered its bytes and, for the convolution,
            // the four warps of one gather group have written the A tile
            mbar_init(smem_u32(&bar_full[s]), GATHER ? 5 : 1);
            mbar_init(smem_u32(&bar_empty[s]), 1);
        }
        for (int s = 0; s < acc_stages; ++s) {
            mbar_init(smem_u32(&bar_acc_full[s]), 1);
            mbar_init(smem_u32(&bar_acc_empty[s]), (uint32_t)epi_warps);
        }
        mbar_init(smem_u32(&bar_drain), 1);
        abort_flag_s = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        if (!GATHER) asm volatile("prefetch.tensormap [%0];" ::"l"(&map_a) : "memory");
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
    // everything above touched only this CTA's shared and tensor memory; the inputs come from the
    // previous kernel in the stream
    pdl_launch_dependents();
    pdl_wait();

    if (warp == 0) {
        // ---------------------------------------------------------------- TMA producer
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            int armed[MAX_STAGES];      // parity of the last phase armed on each stage, -1 = never
#pragma unroll
            for (int s = 0; s < MAX_STAGES; ++s) armed[s] = -1;
            bool ok = true;
            for (int tile = blockIdx.x; ok && tile < args.num_tiles; tile += gridDim.x) {
                const int batch = BATCHED ? tile / args.tiles_per_batch : 0;
                const int in_batch = tile - batch * args.tiles_per_batch;
                const int m0 = (in_batch / args.n_tiles) * BLOCK_M;
                const int n0 = (in_batch % args.n_tiles) * block_n;
                (void)m0;
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
                    if (GATHER) {
                        mbar_arrive_expect_tx(full, (uint32_t)(stage_bytes - A_STAGE_BYTES));
                    } else {
                        mbar_arrive_expect_tx(full, (uint32_t)stage_bytes);
                        if (BATCHED) tma_load_3d(a_dst, &map_a, full, kb * BK, m0, batch);
                        else tma_load_2d(a_dst, &map_a, full, kb * BK, m0);
                    }
                    if (BATCHED) tma_load_3d(a_dst + A_STAGE_BYTES, &map_b, full, kb * BK, n0, batch);
                    else tma_load_2d(a_dst + A_STAGE_BYTES, &map_b, full, kb * BK, n0);
#pragma unroll
                    for (int s = 0; s < MAX_STAGES; ++s)
                        if (s == stage) armed[s] = (int)phase;
                    if (++stage == stages) { stage = 0; phase ^= 1u; }
                }
            }
            if (!ok) {
                // Another role may never consume what was armed: wait (bounded) for the copies in
                // flight so that nothing lands in shared memory after the CTA has gone.
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
            const uint32_t idesc = IN_BF16 ? make_idesc_bf16(BLOCK_M, block_n) : make_idesc_tf32(BLOCK_M, block_n);
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
                    for (int k = 0; k < MMAS_PER_KB; ++k) {
                        // step along K inside the 128-byte swizzled row: 32 bytes = 2 descriptor units
                        if (IN_BF16)
                            tc_mma_bf16(d_tmem, a_desc + (uint64_t)(2 * k), b_desc + (uint64_t)(2 * k), idesc,
                                        (kb | k) != 0 ? 1u : 0u);
                        else
                            tc_mma_tf32(d_tmem, a_desc + (uint64_t)(2 * k), b_desc + (uint64_t)(2 * k), idesc,
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
    } else if (warp < 2 + epi_warps) {
        // ---------------------------------------------------------------- epilogue (warps 2..)
        // Two or four warps share each TMEM lane quadrant (a warp may only read lanes 32*(warp%4)..+31)
        // and take every second or fourth 32-column chunk, counted across tiles so that with one chunk
        // per tile they take tiles in turn.
        const int ew = warp - 2;
        const int quad = warp & 3;
        const int sub = ew >> 2;  // which of the quadrant's warps
        const int per_quad_mask = (epi_warps >> 2) - 1;  // 1 or 3
        const uint32_t slab = epi_base + (uint32_t)ew * SLAB_BYTES;
        int acc = 0;
        uint32_t acc_phase = 0;
        bool ok = true;
        const int chunks_per_tile = block_n / EPI_COLS;
        int chunk_base = 0;  // chunks of earlier tiles, modulo the quadrant's warps
        for (int tile = blockIdx.x; ok && tile < args.num_tiles; tile += gridDim.x) {
            const int batch = BATCHED ? tile / args.tiles_per_batch : 0;
            const int in_batch = tile - batch * args.tiles_per_batch;
            const int m0 = (in_batch / args.n_tiles) * BLOCK_M;
            const int n0 = (in_batch % args.n_tiles) * block_n;
            // every lane polls (each needs the acquire), the vote keeps the warp uniform
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
            // chunks whose first column is past N hold nothing to store
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
                    // this warp has read its share of the accumulator: hand it back to the MMA issuer
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&bar_acc_empty[acc]));
                    released = true;
                }
                if (!rows_live) continue;
                const int col0 = n0 + ch * EPI_COLS;
                // the slab is free once the previous store issued from it has read it
                if (lane == 0) tma_store_wait_read<0>();
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
                    if (BATCHED) tma_store_3d(&map_c, slab, col0, row0, batch);
                    else tma_store_2d(&map_c, slab, col0, row0);
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

    else if (GATHER) {
        // ---------------------------------------------------------------- A-tile gather (warps 10..)
        // Implicit GEMM: row p of A is output pixel p = (n, oy, ox); column k = (ky*fw + kx)*Cin + ci
        // is the input sample that pixel sees through filter tap (ky, kx) at channel ci, zero outside
        // the image and for k >= fh*fw*Cin.  One thread builds one row of a 128 x 32 tile (32 loads in
        // flight) and writes it in the 128-byte-swizzled layout the tensor core reads; the groups take
        // k-blocks in turn so that several tiles' loads are outstanding at once.
        const ConvGeom& g = args.g;
        const int gw = warp - (2 + GATHER_EPI_WARPS);
        const int group = gw >> 2;
        const int row = ((gw & 3) << 5) + lane;
        const bool vec4 = (g.C & 3) == 0;
        const bool small333 = g.fh == 3 && g.fw == 3 && g.C == 3;  // the usual RGB stem: everything compile-time
        const int k_total = g.fh * g.fw * g.C;
        int stage = 0;
        uint32_t phase = 0;
        int turn = 0;  // which group's turn the next k-block is
        bool ok = true;
        for (int tile = blockIdx.x; ok && tile < args.num_tiles; tile += gridDim.x) {
            const int m0 = (tile / args.n_tiles) * BLOCK_M;
            const int p = m0 + row;
            const bool live = p < args.M;
            int iy0 = 0, ix0 = 0;
            const float* xn = args.x;
            if (live) {
                const int hw = g.Ho * g.Wo;
                const int n = p / hw;
                const int rem = p - n * hw;
                const int oy = rem / g.Wo, ox = rem - oy * g.Wo;
                iy0 = oy * g.sh - g.pt;
                ix0 = ox * g.sw - g.pl;
                xn = args.x + (int64_t)n * g.H * g.W * g.C;
            }
            for (int kb = 0; kb < num_k_blocks; ++kb) {
                if (turn == group) {
                    const bool got = bounded_wait(smem_u32(&bar_empty[stage]), phase ^ 1u, abort_flag);
                    if (!__all_sync(0xffffffffu, got)) {
                        if (lane == 0 && !*abort_flag) {
                            *abort_flag = 1;
                            atomicOr(args.dev_status, DEV_STATUS_TIMEOUT_PRODUCER);
                        }
                        ok = false;
                        break;
                    }
                    float v[BLOCK_K];
                    if (small333) gather_small<3, 3, 3>(v, xn, g, iy0, ix0, live);
                    else if (vec4) gather_vec4(v, xn, g, iy0, ix0, live, kb * BLOCK_K, k_total);
                    else gather_scalar(v, xn, g, iy0, ix0, live, kb * BLOCK_K, k_total);
                    const uint32_t row_addr = stage_base + (uint32_t)stage * (uint32_t)stage_bytes + (uint32_t)row * 128u;
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const uint32_t dst = row_addr + (uint32_t)((j ^ (row & 7)) << 4);
                        asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "f"(v[4 * j]), "f"(v[4 * j + 1]),
                                     "f"(v[4 * j + 2]), "f"(v[4 * j + 3])
                                     : "memory");
                    }
                    fence_async_smem();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&bar_full[stage]));
                }
                if (++turn == GATHER_GROUPS) turn = 0;
                if (++stage == stages) { stage = 0; phase ^= 1u; }
            }
        }
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

// The instances.  The tensor maps stay kernel parameters (`__grid_constant__`): the copy unit reads them
// from parameter space, and the pipeline, inlined, takes their addresses there.
template <bool GATHER>
__global__ void __launch_bounds__(GATHER ? CONV_THREADS : GEMM_MAX_THREADS, 1)
gemm_tf32_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                 const __grid_constant__ CUtensorMap map_c, const KernelArgs args) {
    gemm_pipeline<GATHER, IO_F32, false>(map_a, map_b, map_c, args);
}

// A batch of independent products of one shape (rank-3 matMul): the tensor maps carry the batch as a third
// dimension and a tile is (product, rows, columns).
__global__ void __launch_bounds__(GEMM_MAX_THREADS, 1)
gemm_tf32_batched_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                         const __grid_constant__ CUtensorMap map_c, const KernelArgs args) {
    gemm_pipeline<false, IO_F32, true>(map_a, map_b, map_c, args);
}

template <bool OUT_BF16>
__global__ void __launch_bounds__(GEMM_MAX_THREADS, 1)
gemm_bf16_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                 const __grid_constant__ CUtensorMap map_c, const KernelArgs args) {
    gemm_pipeline<false, OUT_BF16 ? IO_BF16 : IO_BF16_F32, false>(map_a, map_b, map_c, args);
}

int choose_block_n(int64_t M, int64_t N, int sm_count, int64_t batches) {
    int bn = 32;
    while (bn < 256 && bn < N) bn <<= 1;
    const int64_t m_tiles = batches * ((M + BLOCK_M - 1) / BLOCK_M);  // row tiles of all products
    while (bn > 32 && m_tiles * ((N + bn - 1) / bn) < sm_count) bn >>= 1;
    if (bn == 256 && N > 256) {
        // Wave quantisation: every tile of a launch costs the same, so the launch takes
        // ceil(tiles / SMs) rounds of one tile each.  192-wide tiles (six 32-column chunks) sometimes
        // fill the last round where 256-wide ones leave most SMs idle (196 tiles on 148 SMs).
        auto rounds = [&](int w) { return (m_tiles * ((N + w - 1) / w) + sm_count - 1) / sm_count; };
        if (rounds(192) * 192 < rounds(256) * 256) bn = 192;
    }
    return bn;
}

// A row-major matrix [outer, inner], or (batches > 1: a rank-3 map) that many of them stored one after the other;
// box = one tile of one matrix.  fp32 elements with the 128-byte swizzle unless `bf16` (then bfloat16, and `swizzle` as given: 128 bytes for
// the operand tiles, 64 for the 32-column output slab).
tfjsb_status encode_2d(tfjsb_ctx* ctx, CUtensorMap* map, const void* base, int64_t inner, int64_t outer,
                       int box_inner, int box_outer, const char* what, int64_t batches = 1, bool bf16 = false,
                       CUtensorMapSwizzle swizzle = CU_TENSOR_MAP_SWIZZLE_128B) {
    const cuuint64_t eb = bf16 ? 2u : 4u;
    cuuint64_t dims[3] = {(cuuint64_t)inner, (cuuint64_t)outer, (cuuint64_t)batches};
    cuuint64_t strides[2] = {(cuuint64_t)inner * eb, (cuuint64_t)inner * (cuuint64_t)outer * eb};
    cuuint32_t box[3] = {(cuuint32_t)box_inner, (cuuint32_t)box_outer, 1u};
    cuuint32_t elem[3] = {1u, 1u, 1u};
    CUresult r = ctx->encode_tiled(map, bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, batches > 1 ? 3 : 2,
                                   const_cast<void*>(base), dims, strides, box, elem, CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle,
                                   CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS)
        return fail(ctx, TFJSB_ERR_CUDA,
                    std::string("cuTensorMapEncodeTiled failed for ") + what + " (CUresult " + std::to_string((int)r) + ")");
    return TFJSB_OK;
}

}  // namespace

bool gemm_tf32_supported(int64_t M, int64_t N, int64_t K) {
    // row pitches of A, Bt (K floats) and C (N floats) must be multiples of 16 bytes; coordinates are 32-bit
    return M >= 1 && N >= 4 && K >= 4 && (K % 4 == 0) && (N % 4 == 0) && M < (1LL << 31) - 256 && N < (1LL << 31) - 256 &&
           K < (1LL << 31) - 256 && ((M + BLOCK_M - 1) / BLOCK_M) * ((N + 31) / 32) < (1LL << 31);
}

namespace {

// tile choice, pipeline depth and the B / C tensor maps shared by the GEMM and the convolution
tfjsb_status plan_common(tfjsb_ctx* ctx, const float* bt, int64_t k_pitch, float* c, GemmTf32Plan* plan, int64_t batches = 1) {
    const int64_t M = plan->M, N = plan->N;
    plan->batches = batches;
    plan->block_n = choose_block_n(M, N, ctx->sm_count, batches);
    plan->acc_stages = plan->block_n > 128 ? 2 : MAX_ACC_STAGES;
    const int stage_bytes = A_STAGE_BYTES + plan->block_n * BLOCK_K * 4;
    int stages = (SMEM_LIMIT - 1024 - EPI_BYTES - 512) / stage_bytes;
    if (stages > MAX_STAGES) stages = MAX_STAGES;
    plan->stages = stages;
    plan->smem_bytes = (size_t)1024 + EPI_BYTES + (size_t)stages * stage_bytes;
    const int64_t n_tiles = (N + plan->block_n - 1) / plan->block_n;
    const int64_t tiles = batches * ((M + BLOCK_M - 1) / BLOCK_M) * n_tiles;
    if (tiles >= (1LL << 31)) return fail(ctx, TFJSB_ERR_UNSUPPORTED, "too many tiles");
    plan->num_tiles = (int)tiles;
    plan->grid = (int)(tiles < ctx->sm_count ? tiles : ctx->sm_count);
    tfjsb_status st;
    if ((st = encode_2d(ctx, &plan->map_b, bt, k_pitch, N, BLOCK_K, plan->block_n, "B", batches)) != TFJSB_OK) return st;
    if ((st = encode_2d(ctx, &plan->map_c, c, N, M, EPI_COLS, 32, "C", batches)) != TFJSB_OK) return st;
    return TFJSB_OK;
}

}  // namespace

tfjsb_status gemm_tf32_plan(tfjsb_ctx* ctx, const float* a, const float* bt, float* c, int64_t M, int64_t N,
                            int64_t K, GemmTf32Plan* plan, int64_t batches) {
    if (!gemm_tf32_supported(M, N, K) || batches < 1 || batches >= (1LL << 31))
        return fail(ctx, TFJSB_ERR_UNSUPPORTED, "shape not supported by the TF32 GEMM");
    if (!ctx->encode_tiled) return fail(ctx, TFJSB_ERR_CUDA, "cuTensorMapEncodeTiled is not available");
    const char* pair_env = getenv("TFJSB_GEMM_PAIR");
    const bool use_pair = pair_env ? (pair_env[0] == '1' && N >= 64) : gemm_tf32_pair_preferred(M, N, K, ctx->sm_count);
    if (batches == 1 && use_pair) return gemm_tf32_pair_plan(ctx, a, bt, c, M, N, K, plan);
    if (batches == 1) {
        // few tiles and a long K loop: the K loop is cut across the CTAs of a cluster (gemm_tf32_splitk.cu)
        int split_bn = 0, split_s = 0;
        if (!getenv("TFJSB_NO_SPLIT_K") && gemm_tf32_splitk_choice(M, N, K, ctx->sm_count, &split_bn, &split_s))
            return gemm_tf32_splitk_plan(ctx, a, bt, c, M, N, K, split_bn, split_s, plan);
    }
    plan->M = M; plan->N = N; plan->K = K;
    plan->pair = false;
    plan->cluster_split = false;
    plan->gather = false;
    plan->x = nullptr;
    tfjsb_status st;
    if ((st = plan_common(ctx, bt, K, c, plan, batches)) != TFJSB_OK) return st;
    return encode_2d(ctx, &plan->map_a, a, K, M, BLOCK_K, BLOCK_M, "A", batches);
}

int64_t conv_igemm_k_pad(const ConvGeom& g) {
    const int64_t k = (int64_t)g.fh * g.fw * g.C;
    return (k + BLOCK_K - 1) / BLOCK_K * BLOCK_K;
}

bool conv_igemm_supported(const ConvGeom& g) {
    const int64_t M = g.N * g.Ho * g.Wo;
    const int64_t K = (int64_t)g.fh * g.fw * g.C;
    return M >= 1 && g.Co >= 4 && (g.Co % 4 == 0) && K >= 1 && K < (1 << 24) && M < (1LL << 31) - 256 &&
           (int64_t)g.H * g.W * g.C < (1LL << 31) && ((M + BLOCK_M - 1) / BLOCK_M) * ((g.Co + 31) / 32) < (1LL << 31);
}

tfjsb_status conv_igemm_plan(tfjsb_ctx* ctx, const float* x, const float* bt, float* y, const ConvGeom& g,
                             GemmTf32Plan* plan) {
    if (!conv_igemm_supported(g)) return fail(ctx, TFJSB_ERR_UNSUPPORTED, "shape not supported by the implicit-GEMM convolution");
    if (!ctx->encode_tiled) return fail(ctx, TFJSB_ERR_CUDA, "cuTensorMapEncodeTiled is not available");
    plan->M = g.N * g.Ho * g.Wo;
    plan->N = g.Co;
    plan->K = (int64_t)g.fh * g.fw * g.C;
    plan->gather = true;
    plan->pair = false;
    plan->cluster_split = false;
    plan->x = x;
    plan->g = g;
    tfjsb_status st = plan_common(ctx, bt, conv_igemm_k_pad(g), y, plan);
    if (st != TFJSB_OK) return st;
    plan->map_a = plan->map_b;  // unused by the gathering kernel; kept initialised
    return TFJSB_OK;
}

cudaError_t launch_gemm_tf32(const GemmTf32Plan& plan, const float* bias, int act, unsigned int* dev_status,
                             cudaStream_t s, int64_t* launches) {
    if (plan.pair) return launch_gemm_tf32_pair(plan, bias, act, dev_status, s, launches);
    if (plan.cluster_split) return launch_gemm_tf32_splitk(plan, bias, act, dev_status, s, launches);
    {
        cudaError_t ae = cudaSuccess;
        if (ae == cudaSuccess) ae = smem_attr_once(reinterpret_cast<const void*>(&gemm_tf32_kernel<false>), SMEM_LIMIT - 2048);
        if (ae == cudaSuccess) ae = smem_attr_once(reinterpret_cast<const void*>(&gemm_tf32_kernel<true>), SMEM_LIMIT - 2048);
        if (ae == cudaSuccess) ae = smem_attr_once(reinterpret_cast<const void*>(&gemm_tf32_batched_kernel), SMEM_LIMIT - 2048);
        if (ae != cudaSuccess) return ae;
    }
    cudaError_t e;
    KernelArgs args;
    args.M = (int)plan.M; args.N = (int)plan.N; args.K = (int)plan.K;
    args.block_n = plan.block_n;
    args.stages = plan.stages;
    args.n_tiles = (int)((plan.N + plan.block_n - 1) / plan.block_n);
    args.tiles_per_batch = (int)(plan.num_tiles / (plan.batches > 0 ? plan.batches : 1));
    args.num_tiles = plan.num_tiles;
    args.acc_stages = plan.acc_stages;
    args.epi_warps = GATHER_EPI_WARPS;  // sixteen measured slower with fp32 tiles
    args.bias = bias;
    args.act = act;
    args.dev_status = dev_status;
    args.x = plan.x;
    args.g = plan.g;
    if (plan.gather)
        e = launch_k(gemm_tf32_kernel<true>, dim3(plan.grid), dim3(CONV_THREADS), plan.smem_bytes, s, plan.map_a, plan.map_b,
                     plan.map_c, args);
    else if (plan.batches > 1)
        e = launch_k(gemm_tf32_batched_kernel, dim3(plan.grid), dim3(64 + 32 * args.epi_warps), plan.smem_bytes, s, plan.map_a,
                     plan.map_b, plan.map_c, args);
    else
        e = launch_k(gemm_tf32_kernel<false>, dim3(plan.grid), dim3(64 + 32 * args.epi_warps), plan.smem_bytes, s, plan.map_a, plan.map_b,
                     plan.map_c, args);
    ++*launches;
    return e;
}

// ---- bfloat16 storage ------------------------------------------------------------------------------
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
    constexpr int BK16 = 64;  // bfloat16 elements per k-block
    plan->M = M; plan->N = N; plan->K = K;
    plan->c_is_bf16 = c_is_bf16;
    plan->pair = false;
    plan->block_n = choose_block_n(M, N, ctx->sm_count, 1);
    plan->acc_stages = plan->block_n > 128 ? 2 : MAX_ACC_STAGES;
    const int stage_bytes = A_STAGE_BYTES + plan->block_n * 128;
    plan->epi_warps = (K + BK16 - 1) / BK16 <= 4 ? 16 : 8;
    const int epi_bytes = plan->epi_warps * (c_is_bf16 ? 2048 : EPI_SLAB_BYTES);
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
    if ((st = encode_2d(ctx, &plan->map_a, a, K, M, BK16, BLOCK_M, "A", 1, true)) != TFJSB_OK) return st;
    if ((st = encode_2d(ctx, &plan->map_b, bt, K, N, BK16, plan->block_n, "B", 1, true)) != TFJSB_OK) return st;
    if (c_is_bf16) return encode_2d(ctx, &plan->map_c, c, N, M, EPI_COLS, 32, "C", 1, true, CU_TENSOR_MAP_SWIZZLE_64B);
    return encode_2d(ctx, &plan->map_c, c, N, M, EPI_COLS, 32, "C");
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
    KernelArgs args{};
    args.M = (int)plan.M; args.N = (int)plan.N; args.K = (int)plan.K;
    args.block_n = plan.block_n;
    args.stages = plan.stages;
    args.n_tiles = (int)((plan.N + plan.block_n - 1) / plan.block_n);
    args.tiles_per_batch = plan.num_tiles;
    args.num_tiles = plan.num_tiles;
    args.acc_stages = plan.acc_stages;
    args.epi_warps = plan.epi_warps;
    args.bias = bias;
    args.act = act;
    args.dev_status = dev_status;
    const dim3 block(64 + 32 * plan.epi_warps);
    cudaError_t e;
    if (plan.c_is_bf16)
        e = launch_k(gemm_bf16_kernel<true>, dim3(plan.grid), block, plan.smem_bytes, s, plan.map_a, plan.map_b, plan.map_c, args);
    else
        e = launch_k(gemm_bf16_kernel<false>, dim3(plan.grid), block, plan.smem_bytes, s, plan.map_a, plan.map_b, plan.map_c, args);
    ++*launches;
    return e;
}

}  // namespace tfjsb

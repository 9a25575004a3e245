// Fused depthwise-separable block for sm_100a:
//
//     y = act2( pointwise( act1( depthwise3x3(x) + b1 ) ) + b2 )      stride 1, NHWC fp32
//
// The depthwise output never goes to global memory.  A persistent CTA walks tiles of 8 x 16 output
// pixels (= the 128 rows of one tensor-core tile) and, per block of 32 channels (= one k-block):
//   warp 0       producer: bulk tensor copies (TMA) of the input patch (10 x 18 pixels x 32 channels,
//                zero-filled outside the image = the 'same' padding) and of the matching 32-column
//                slice of the pointwise weights Bt[Cout, Cin], each into its own ring of stages;
//   warps 10-25  depthwise: two groups of eight warps take alternate k-blocks (two are in flight, so
//                one group's load and FMA latency hides behind the other's); a thread computes
//                2 channels x 2 columns x 4 rows from the patch on CUDA cores (each value it loads
//                serves up to six outputs; the same FMA order as the stand-alone kernel), adds
//                bias, applies the activation and writes the result as the A operand in the
//                128-byte-swizzled K-major layout;
//   warp 1       issues tcgen05.mma (TF32, M 128, N = block_n, K 8, four per k-block) on A and Bt,
//                accumulating over the channel blocks in tensor memory;
//   warps 2-9    epilogue: tcgen05.ld, pointwise bias + activation, swizzled staging slab, 4-D bulk
//                tensor store of 2 image rows x 16 pixels x 32 channels (clipped at the image edge).
// The kernel is bound by shared-memory bandwidth (patch written once and read by the depthwise
// threads, A written and read back by the tensor core, Bt slices, output staging), so the pointwise
// weights stay resident in shared memory for the whole kernel when all their k-blocks fit (up to
// four), instead of being fetched again for every tile.
// Every wait is bounded (see ptx_sm100.cuh); a timeout raises the abort flag all roles poll and is
// reported through the context's device status word.
//
// Small-window convolution mode (template parameter CONV): a conv2d whose whole im2col row fits one
// k-block (fh*fw*Cin <= 32, e.g. a 3x3 stem on RGB input) runs on the same pipeline.  The producer
// brings the input patch of a tile in by one 3-D copy over x viewed as [N, H, W*Cin], four warps
// rearrange it into the A operand (thread = pixel), the packed filter [Cout, 32] stays resident as
// B, and the block is 14 warps so that two CTAs share an SM: per tile every role costs mostly its
// own synchronisation, and two CTAs double each of them.
#include <cstdlib>

#include "common.cuh"
#include "ptx_sm100.cuh"
#include "umma_tile.cuh"

namespace tfjsb {

using namespace ptx;
using namespace tile;

namespace {

constexpr int F_THREADS = 832;        // 26 warps: producer, MMA, 8 epilogue, 16 depthwise; one CTA per SM
constexpr int F_DW_WARPS = 16;
constexpr int F_DW_GROUPS = 2;        // groups of depthwise warps that take alternate k-blocks
constexpr int F_DW_GROUP_WARPS = F_DW_WARPS / F_DW_GROUPS;
constexpr int F_CONV_THREADS = 448;   // 14 warps: producer, MMA, 8 epilogue, 4 im2col; two CTAs per SM
constexpr int F_CONV_CMP_WARPS = 4;
constexpr int F_CONV_SMEM = 112 * 1024;  // per-CTA dynamic budget that lets two CTAs share an SM's 228 KiB
constexpr int F_TH = 8, F_TW = 16;    // output pixels per tile (8 rows x 16 columns = 128 GEMM rows)
constexpr int F_PH = F_TH + 2, F_PW = F_TW + 2;
constexpr int F_PATCH_FLOATS = F_PH * F_PW * BLOCK_K;
constexpr int F_PATCH_BYTES = F_PATCH_FLOATS * 4;              // 23040
constexpr int F_PATCH_STRIDE = 23 * 1024;                      // stage pitch, keeps stages 1024-aligned
constexpr int F_MAX_RING = 12;
constexpr int F_MAX_ACC = 8;           // accumulator stages (32-column tiles of the small-window mode use all)

struct FusedArgs {
    int C, Co;                // depthwise channels (= K of the GEMM), pointwise output channels (= N)
    int Ho, Wo;               // = input H, W (stride 1, 'same') or the 'valid' output size
    int pt, pl;               // padding before
    int tiles_x, tiles_y;
    int num_tiles;
    int block_n;              // accumulator columns per MMA group (<= 256)
    int n_sub;                // MMA groups per k-block: 1, or 2 when 256 < Cout <= 512 (they share the A tile)
    int acc_stages;
    int patch_stages, a_stages, b_stages;
    int b_resident;           // the B ring holds every k-block's slice: loaded during the first tile, never released
    int patch_bytes, patch_stride;   // bytes of one input patch and pitch of the patch ring
    // small-window convolution mode (CONV): the patch holds (8-1)*sh+fh rows of row_floats floats
    int cin, fw_cin, sh, sw, row_floats, k_total;
    int rows9;                // 3 x 3 window on 3 channels with even offsets: the rows are read with 8-byte loads
    int koff[32];             // patch offset of im2col column k relative to the pixel's window origin
    const float* dw_filter;   // [3,3,C,1]
    const float* dw_bias;     // [C] or null
    int dw_act;
    const float* pw_bias;     // [Co] or null
    int pw_act;
    unsigned int* dev_status;
};

__device__ __forceinline__ float4 ld4s(const float* p) { return *reinterpret_cast<const float4*>(p); }
__device__ __forceinline__ void fma4s(float4& acc, const float4& a, const float4& b) {
    acc.x = fmaf(a.x, b.x, acc.x); acc.y = fmaf(a.y, b.y, acc.y);
    acc.z = fmaf(a.z, b.z, acc.z); acc.w = fmaf(a.w, b.w, acc.w);
}

// Bias, activation and the swizzled store of one depthwise thread's 4 rows x 2 columns x 2 channels
// into the A operand (GEMM row of a pixel = row*16 + column).  The activation is a template parameter:
// the kernel is close to instruction-issue bound, and a run-time choice costs two extra instructions
// per value.
template <int ACT, bool ROUND_BF16 = false>
__device__ __forceinline__ void store_depthwise_block(const float2 (&acc)[F_TH / 2][2], const float2 b, uint32_t a_stage,
                                                      int rg, int colg, int c2) {
    constexpr int R = F_TH / 2;
#pragma unroll
    for (int r = 0; r < R; ++r) {
#pragma unroll
        for (int cc = 0; cc < 2; ++cc) {
            float vx = apply_act_t<ACT>(acc[r][cc].x + b.x);
            float vy = apply_act_t<ACT>(acc[r][cc].y + b.y);
            if (ROUND_BF16) {  // narrow storage: the depthwise layer's output is a bfloat16 (an exact TF32 operand)
                vx = __bfloat162float(__float2bfloat16_rn(vx));
                vy = __bfloat162float(__float2bfloat16_rn(vy));
            }
            const int p = (rg * R + r) * F_TW + colg * 2 + cc;
            const uint32_t dst = a_stage + (uint32_t)p * 128u + (uint32_t)(((c2 >> 1) ^ (p & 7)) << 4) + (uint32_t)((c2 & 1) << 3);
            asm volatile("st.shared.v2.f32 [%0], {%1, %2};" ::"r"(dst), "f"(vx), "f"(vy) : "memory");
        }
    }
}

// NARROW: the narrow-storage forms.  Depthwise + pointwise: the block input is bfloat16 (the patch is copied as
// such and widened by the depthwise threads), the depthwise result is rounded to bfloat16 before it becomes the
// A operand, the pointwise filter holds bfloat16 values, the output is stored as bfloat16.  Small-window mode: the
// narrow-storage form of the convolution.  The fp32 input is rounded to
// bfloat16 as it is rearranged into the A operand and the filter holds bfloat16 values, so every TF32
// product is the exact product of two bfloat16 values (8 significand bits fit TF32's 11); the sum is fp32
// and the result is stored as bfloat16 (rounded to nearest even after bias and activation).
// STREAM_B: the weight slices do not stay resident (more k-blocks than the ring has stages) and are fetched
// again for every tile; the producer then feeds two rings that drain at different rates and must not block on
// either (a kernel instance of its own, so that the common case keeps its register allocation).
// WIDE_EPI: blocks with few input channels (one k-block per tile) are paced by the epilogue, not by the
// depthwise stage: sixteen epilogue warps (four per tensor-memory lane quarter, taking tiles in turn) and a
// single group of eight depthwise warps, instead of eight and two groups of eight.
template <bool CONV, bool NARROW = false, bool STREAM_B = false, bool WIDE_EPI = false>
__global__ void __launch_bounds__(CONV ? F_CONV_THREADS : F_THREADS, CONV ? 2 : 1)
dwpw_fused_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_b,
                  const __grid_constant__ CUtensorMap map_y, const FusedArgs args) {
    extern __shared__ uint8_t smem_raw[];
    constexpr int RING = CONV ? F_MAX_RING : 4;       // deepest ring of this mode (the patch ring)
    constexpr int ACCS = CONV ? F_MAX_ACC : MAX_ACC_STAGES;
    __shared__ __align__(8) uint64_t bar_patch_full[RING], bar_patch_empty[RING];
    __shared__ __align__(8) uint64_t bar_a_full[4], bar_a_empty[4];
    __shared__ __align__(8) uint64_t bar_b_full[4], bar_b_empty[4];
    __shared__ __align__(8) uint64_t bar_acc_full[ACCS], bar_acc_empty[ACCS];
    __shared__ __align__(8) uint64_t bar_drain;
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag_s;

    // Role split of the warps after the producer and the MMA issuer.  The small-window mode has
    // little arithmetic per tile: what bounds a tile there is the fixed cost of each role's
    // synchronisation (barrier waits, fences, MMA issue), so it runs as two small CTAs per SM, which
    // doubles every role, instead of one large CTA.
    static_assert(!(WIDE_EPI && CONV), "the wide epilogue belongs to the depthwise + pointwise mode");
    constexpr int EPI_WARPS = WIDE_EPI ? 16 : 8;
    constexpr int DW_GROUPS = WIDE_EPI ? 1 : F_DW_GROUPS;
    constexpr int CMP_WARPS = CONV ? F_CONV_CMP_WARPS : DW_GROUPS * F_DW_GROUP_WARPS;
    constexpr int GROUP_WARPS = CONV ? F_CONV_CMP_WARPS : F_DW_GROUP_WARPS;  // warps that fill one A stage
    constexpr int CMP_WARP0 = 2 + EPI_WARPS;
    constexpr int EPI_GROUPS = EPI_WARPS / 4;
    static_assert((CMP_WARP0 + CMP_WARPS) * 32 == (CONV ? F_CONV_THREADS : F_THREADS), "role split must cover the block");

    volatile int* abort_flag = &abort_flag_s;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int block_n = args.block_n;
    const int num_k_blocks = CONV ? 1 : args.C / BLOCK_K;
    const int b_stage_bytes = block_n * BLOCK_K * 4;

    // dynamic shared memory (1024-aligned): [epilogue slabs][patch ring][A ring][B ring]
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t epi_base = smem_base;
    const uint32_t patch_base = epi_base + (uint32_t)(EPI_WARPS * EPI_SLAB_BYTES);
    const uint32_t a_base = patch_base + (uint32_t)(args.patch_stages * args.patch_stride);
    const uint32_t b_base = a_base + (uint32_t)args.a_stages * A_STAGE_BYTES;
    const float* patch_ptr = reinterpret_cast<const float*>(smem_raw + (patch_base - smem_u32(smem_raw)));

    if (threadIdx.x == 0) {
        for (int s = 0; s < RING; ++s) {
            mbar_init(smem_u32(&bar_patch_full[s]), 1);
            mbar_init(smem_u32(&bar_patch_empty[s]), GROUP_WARPS);
        }
        for (int s = 0; s < 4; ++s) {
            mbar_init(smem_u32(&bar_a_full[s]), GROUP_WARPS);
            mbar_init(smem_u32(&bar_a_empty[s]), 1);
            mbar_init(smem_u32(&bar_b_full[s]), 1);
            mbar_init(smem_u32(&bar_b_empty[s]), 1);
        }
        // only the groups that have a chunk of a tile wait for its accumulator and hand it back: with fewer chunks
        // per tile than groups, the others skip the tile (the groups' first chunks are a permutation of
        // 0 .. EPI_GROUPS-1 that shifts by the same amount every tile, so the number of takers is constant)
        int nch = (args.Co + EPI_COLS - 1) / EPI_COLS;
        if (nch > block_n * args.n_sub / EPI_COLS) nch = block_n * args.n_sub / EPI_COLS;
        const int epi_arrivals = 4 * (nch < EPI_GROUPS ? nch : EPI_GROUPS);
        for (int s = 0; s < ACCS; ++s) {
            mbar_init(smem_u32(&bar_acc_full[s]), 1);
            mbar_init(smem_u32(&bar_acc_empty[s]), (uint32_t)epi_arrivals);
        }
        mbar_init(smem_u32(&bar_drain), 1);
        abort_flag_s = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_x) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_b) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_y) : "memory");
    }
    const int acc_cols = block_n * args.n_sub;  // accumulator columns per tile
    const uint32_t tmem_cols = (uint32_t)(args.acc_stages * acc_cols);
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
    const int tiles_per_image = args.tiles_x * args.tiles_y;
    pdl_launch_dependents();
    pdl_wait();  // the block input is the previous kernel's output

    if (warp == 0) {
        // ---------------------------------------------------------------- producer
        if (STREAM_B && lane == 0) {
            // One thread, two rings (input patches for the depthwise warps, weight slices for the tensor core):
            // it probes both "empty" barriers in turn and issues whichever copy has room.  Issued in program
            // order, a full weight ring held back the next patch and the depthwise warps spent half their
            // time waiting for input (28x28x256 -> 256 at batch 128: 78 -> 71 us).
            int ps = 0, bs = 0;
            uint32_t pphase = 0, bphase = 0;
            const int my_tiles = (int)blockIdx.x < args.num_tiles ? (args.num_tiles - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x : 0;
            const int total_p = my_tiles * num_k_blocks, total_b = total_p * args.n_sub;
            int pk = 0, bk = 0;                  // copies issued so far
            int p_tile = blockIdx.x, p_kb = 0;   // next patch: tile and k-block
            int p_n = 0, p_ty = 0, p_tx = 0;
            bool p_coords = false;
            int b_kb = 0, b_h = 0;               // next weight slice: k-block and column half
            bool ok = true;
            unsigned long long idle_since = 0;
            while (ok && (pk < total_p || bk < total_b)) {
                bool progressed = false;
                // a single ring left to feed: sleep on its barrier instead of probing
                if (bk == total_b && !bounded_wait(smem_u32(&bar_patch_empty[ps]), pphase ^ 1u, abort_flag)) { ok = false; break; }
                if (pk == total_p && !bounded_wait(smem_u32(&bar_b_empty[bs]), bphase ^ 1u, abort_flag)) { ok = false; break; }
                if (pk < total_p && mbar_test_wait(smem_u32(&bar_patch_empty[ps]), pphase ^ 1u)) {
                    if (!p_coords) {
                        p_n = p_tile / tiles_per_image;
                        const int rem = p_tile - p_n * tiles_per_image;
                        p_ty = rem / args.tiles_x;
                        p_tx = rem - p_ty * args.tiles_x;
                        p_coords = true;
                    }
                    const uint32_t pf = smem_u32(&bar_patch_full[ps]);
                    mbar_arrive_expect_tx(pf, (uint32_t)args.patch_bytes);
                    tma_load_4d(patch_base + (uint32_t)(ps * args.patch_stride), &map_x, pf, p_kb * BLOCK_K,
                                p_tx * F_TW - args.pl, p_ty * F_TH - args.pt, p_n);
                    if (++ps == args.patch_stages) { ps = 0; pphase ^= 1u; }
                    if (++p_kb == num_k_blocks) { p_kb = 0; p_tile += gridDim.x; p_coords = false; }
                    ++pk;
                    progressed = true;
                }
                if (bk < total_b && mbar_test_wait(smem_u32(&bar_b_empty[bs]), bphase ^ 1u)) {
                    const uint32_t bf = smem_u32(&bar_b_full[bs]);
                    mbar_arrive_expect_tx(bf, (uint32_t)b_stage_bytes);
                    tma_load_2d(b_base + (uint32_t)bs * (uint32_t)b_stage_bytes, &map_b, bf, b_kb * BLOCK_K, b_h * block_n);
                    if (++bs == args.b_stages) { bs = 0; bphase ^= 1u; }
                    if (++b_h == args.n_sub) { b_h = 0; if (++b_kb == num_k_blocks) b_kb = 0; }
                    ++bk;
                    progressed = true;
                }
                if (progressed) { idle_since = 0; continue; }
                __nanosleep(32);
                if (*abort_flag) ok = false;
                else if (idle_since == 0) idle_since = global_ns();
                else if (global_ns() - idle_since > WAIT_LIMIT_NS) ok = false;
            }
            if (!ok || *abort_flag) {
                if (!*abort_flag) {
                    *abort_flag = 1;
                    atomicOr(args.dev_status, DEV_STATUS_TIMEOUT_PRODUCER);
                }
                // copies in flight must land before the CTA's shared memory is released
                const unsigned long long t0 = global_ns();
                bool all = true;
                for (int k = (pk > args.patch_stages ? pk - args.patch_stages : 0); k < pk; ++k)
                    while (!mbar_try_wait(smem_u32(&bar_patch_full[k % args.patch_stages]), (uint32_t)((k / args.patch_stages) & 1)))
                        if (global_ns() - t0 > WAIT_LIMIT_NS) { all = false; break; }
                for (int k = (bk > args.b_stages ? bk - args.b_stages : 0); k < bk; ++k)
                    while (!mbar_try_wait(smem_u32(&bar_b_full[k % args.b_stages]), (uint32_t)((k / args.b_stages) & 1)))
                        if (global_ns() - t0 > WAIT_LIMIT_NS) { all = false; break; }
                if (!all) atomicOr(args.dev_status, DEV_STATUS_TIMEOUT_DRAIN);
            }
        }
        if (!STREAM_B && lane == 0) {
            int ps = 0, bs = 0;
            uint32_t pphase = 0, bphase = 0;
            int issued = 0;
            bool ok = true;
            for (int tile = blockIdx.x; ok && tile < args.num_tiles; tile += gridDim.x) {
                const int n = tile / tiles_per_image;
                const int rem = tile - n * tiles_per_image;
                const int ty = rem / args.tiles_x, tx = rem - ty * args.tiles_x;
                for (int kb = 0; kb < num_k_blocks; ++kb) {
                    if (!bounded_wait(smem_u32(&bar_patch_empty[ps]), pphase ^ 1u, abort_flag)) { ok = false; break; }
                    const uint32_t pf = smem_u32(&bar_patch_full[ps]);
                    mbar_arrive_expect_tx(pf, (uint32_t)args.patch_bytes);
                    if (CONV)
                        tma_load_3d(patch_base + (uint32_t)(ps * args.patch_stride), &map_x, pf,
                                    (tx * F_TW * args.sw - args.pl) * args.cin, ty * F_TH * args.sh - args.pt, n);
                    else
                        tma_load_4d(patch_base + (uint32_t)(ps * args.patch_stride), &map_x, pf, kb * BLOCK_K,
                                    tx * F_TW - args.pl, ty * F_TH - args.pt, n);
                    if (++ps == args.patch_stages) { ps = 0; pphase ^= 1u; }
                    // resident weights (and the packed filter of the small-window mode) are loaded during
                    // the first tile only and never released
                    const int b_loads = (args.b_resident && issued >= num_k_blocks) ? 0 : args.n_sub;
                    for (int h = 0; ok && h < b_loads; ++h) {
                        if (!bounded_wait(smem_u32(&bar_b_empty[bs]), bphase ^ 1u, abort_flag)) { ok = false; break; }
                        const uint32_t bf = smem_u32(&bar_b_full[bs]);
                        mbar_arrive_expect_tx(bf, (uint32_t)b_stage_bytes);
                        tma_load_2d(b_base + (uint32_t)bs * (uint32_t)b_stage_bytes, &map_b, bf, kb * BLOCK_K, h * block_n);
                        if (++bs == args.b_stages) { bs = 0; bphase ^= 1u; }
                    }
                    if (!ok) break;
                    ++issued;
                }
            }
            if (!ok || *abort_flag) {
                if (!*abort_flag) {
                    *abort_flag = 1;
                    atomicOr(args.dev_status, DEV_STATUS_TIMEOUT_PRODUCER);
                }
                // give the copies in flight time to land before the CTA's shared memory is released:
                // every armed phase completes within the copy latency unless the device is wedged
                const unsigned long long t0 = global_ns();
                bool all = false;
                while (!all && global_ns() - t0 < WAIT_LIMIT_NS) {
                    all = true;
                    for (int k = (issued > RING ? issued - RING : 0); k < issued; ++k) {
                        if (!mbar_try_wait(smem_u32(&bar_patch_full[k % args.patch_stages]),
                                           (uint32_t)((k / args.patch_stages) & 1)) &&
                            k >= issued - args.patch_stages)
                            all = false;
                        for (int h = 0; h < (args.b_resident ? 0 : args.n_sub); ++h) {
                            const int kk = k * args.n_sub + h;  // index of the B copy in its own ring
                            if (kk >= issued * args.n_sub - args.b_stages &&
                                !mbar_try_wait(smem_u32(&bar_b_full[kk % args.b_stages]), (uint32_t)((kk / args.b_stages) & 1)))
                                all = false;
                        }
                    }
                }
                if (args.b_resident && all) {
                    const int loaded = issued < num_k_blocks ? issued : num_k_blocks;
                    for (int k = 0; all && k < loaded; ++k)
                        while (!(all = mbar_try_wait(smem_u32(&bar_b_full[k]), 0u)) && global_ns() - t0 < WAIT_LIMIT_NS) {}
                }
                if (!all) atomicOr(args.dev_status, DEV_STATUS_TIMEOUT_DRAIN);
            }
        }
    } else if (warp == 1) {
        // ---------------------------------------------------------------- MMA issuer
        if (lane == 0) {
            const uint32_t idesc = make_idesc_tf32(BLOCK_M, block_n);
            int as = 0, bs = 0, acc = 0;
            uint32_t aphase = 0, bphase = 0, acc_phase = 0;
            bool ok = true, issued_any = false;
            bool first_tile = true;
            for (int tile = blockIdx.x; ok && tile < args.num_tiles; tile += gridDim.x) {
                if (!bounded_wait(smem_u32(&bar_acc_empty[acc]), acc_phase ^ 1u, abort_flag)) { ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(acc * acc_cols);
                for (int kb = 0; kb < num_k_blocks; ++kb) {
                    if (!bounded_wait(smem_u32(&bar_a_full[as]), aphase, abort_flag)) { ok = false; break; }
                    const uint64_t a_desc = make_kmajor_sw128_desc(a_base + (uint32_t)as * A_STAGE_BYTES);
                    for (int h = 0; h < args.n_sub; ++h) {
                        if (!args.b_resident || first_tile) {
                            if (!bounded_wait(smem_u32(&bar_b_full[bs]), bphase, abort_flag)) { ok = false; break; }
                        }
                        tc_fence_after();
                        const uint64_t b_desc = make_kmajor_sw128_desc(b_base + (uint32_t)bs * (uint32_t)b_stage_bytes);
#pragma unroll
                        for (int k = 0; k < BLOCK_K / UMMA_K; ++k)
                            tc_mma_tf32(d_tmem + (uint32_t)(h * block_n), a_desc + (uint64_t)(2 * k), b_desc + (uint64_t)(2 * k),
                                        idesc, (kb | k) != 0 ? 1u : 0u);
                        issued_any = true;
                        if (!args.b_resident) tc_commit(smem_u32(&bar_b_empty[bs]));
                        // resident: stage kb again for the next tile, its first phase (parity 0) long complete
                        if (++bs == args.b_stages) { bs = 0; if (!args.b_resident) bphase ^= 1u; }
                    }
                    if (!ok) break;
                    tc_commit(smem_u32(&bar_a_empty[as]));
                    if (++as == args.a_stages) { as = 0; aphase ^= 1u; }
                }
                if (!ok) break;
                tc_commit(smem_u32(&bar_acc_full[acc]));
                first_tile = false;
                if (++acc == args.acc_stages) { acc = 0; acc_phase ^= 1u; }
            }
            if (!ok) {
                if (!*abort_flag) {
                    *abort_flag = 1;
                    atomicOr(args.dev_status, DEV_STATUS_TIMEOUT_MMA);
                }
                if (issued_any) {
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
    } else if (warp < CMP_WARP0) {
        // ---------------------------------------------------------------- epilogue (warps 2..)
        // Groups of four warps (one per TMEM lane quarter) take the 32-column chunks round-robin,
        // across tile boundaries.
        const int ew = warp - 2;
        const int quad = warp & 3;   // TMEM lanes 32*quad.. = image rows 2*quad, 2*quad+1 of the tile
        const int group = ew >> 2;
        const uint32_t slab = epi_base + (uint32_t)ew * EPI_SLAB_BYTES;
        const int chunks_per_tile = acc_cols / EPI_COLS;
        int n_chunks = (args.Co + EPI_COLS - 1) / EPI_COLS;
        if (n_chunks > chunks_per_tile) n_chunks = chunks_per_tile;
        int acc = 0;
        uint32_t acc_phase = 0;
        int first_chunk = group;
        // round-robin over tile boundaries: a tile of n_chunks chunks moves every group's first chunk
        const int chunk_shift = EPI_GROUPS - (n_chunks & (EPI_GROUPS - 1));
        // (image, tile row, tile column) of the CTA's tiles, stepped instead of divided out for every tile: the
        // eight or sixteen warps of this role walk every tile, and three divisions per tile and warp were a
        // good part of the instructions the SM issues per tile
        int n = (int)blockIdx.x / tiles_per_image;
        int ty = ((int)blockIdx.x - n * tiles_per_image) / args.tiles_x;
        int tx = (int)blockIdx.x - n * tiles_per_image - ty * args.tiles_x;
        const int step_n = (int)gridDim.x / tiles_per_image;
        const int step_rem = (int)gridDim.x - step_n * tiles_per_image;
        const int step_ty = step_rem / args.tiles_x, step_tx = step_rem - step_ty * args.tiles_x;
        bool first_pass = true;
        for (int tile = blockIdx.x; tile < args.num_tiles; tile += gridDim.x) {
            if (!first_pass) {
                tx += step_tx;
                if (tx >= args.tiles_x) { tx -= args.tiles_x; ++ty; }
                ty += step_ty;
                if (ty >= args.tiles_y) { ty -= args.tiles_y; ++n; }
                n += step_n;
            }
            first_pass = false;
            if (first_chunk < n_chunks) {  // else: no chunk of this tile falls to this group
            const bool got = bounded_wait(smem_u32(&bar_acc_full[acc]), acc_phase, abort_flag);
            if (!__all_sync(0xffffffffu, got)) {
                if (lane == 0 && !*abort_flag) {
                    *abort_flag = 1;
                    atomicOr(args.dev_status, DEV_STATUS_TIMEOUT_EPILOGUE);
                }
                break;
            }
            tc_fence_after();
            const int oy = ty * F_TH + quad * 2;
            const bool rows_live = oy < args.Ho;
            bool released = false;
            for (int ch = first_chunk; ch < n_chunks; ch += EPI_GROUPS) {
                uint32_t r[32];
                const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(acc * acc_cols + ch * EPI_COLS);
                tc_ld_32x32(taddr, r);
                tc_ld_wait();
                if (ch + EPI_GROUPS >= n_chunks) {
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&bar_acc_empty[acc]));
                    released = true;
                }
                if (!rows_live) continue;
                const int col0 = ch * EPI_COLS;
                if (lane == 0) tma_store_wait_read<0>();
                __syncwarp();
                const uint32_t row_addr = slab + (uint32_t)lane * 128u;
                const float* bias = (args.pw_bias != nullptr) ? args.pw_bias + col0 : nullptr;
                const int cols_left = args.Co - col0;
                if (NARROW) {  // 32 rows of 64 bytes in the 64-byte swizzle of the bfloat16 output map
                    if (args.pw_act == TFJSB_ACT_RELU6) stage_chunk_bf16<TFJSB_ACT_RELU6>(r, bias, cols_left, slab, lane);
                    else if (args.pw_act == TFJSB_ACT_RELU) stage_chunk_bf16<TFJSB_ACT_RELU>(r, bias, cols_left, slab, lane);
                    else stage_chunk_bf16<TFJSB_ACT_NONE>(r, bias, cols_left, slab, lane);
                } else if (args.pw_act == TFJSB_ACT_RELU6) stage_chunk<TFJSB_ACT_RELU6>(r, bias, cols_left, row_addr, lane);
                else if (args.pw_act == TFJSB_ACT_RELU) stage_chunk<TFJSB_ACT_RELU>(r, bias, cols_left, row_addr, lane);
                else stage_chunk<TFJSB_ACT_NONE>(r, bias, cols_left, row_addr, lane);
                fence_async_smem();
                __syncwarp();
                if (lane == 0) {
                    tma_store_4d(&map_y, slab, col0, tx * F_TW, oy, n);
                    tma_store_commit();
                }
            }
            if (!released) {
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&bar_acc_empty[acc]));
            }
            }
            first_chunk = (first_chunk + chunk_shift) & (EPI_GROUPS - 1);
            if (++acc == args.acc_stages) { acc = 0; acc_phase ^= 1u; }
        }
        if (lane == 0) tma_store_wait_all();
        __syncwarp();
    } else {
        if (CONV) {
            // ------------------------------------------------------------ im2col from the patch (warps 10..13)
            // Small-window convolution (fh*fw*Cin <= 32: one k-block): thread = pixel of the tile;
            // column k = (ky*fw + kx)*Cin + ci of a pixel's im2col row sits in the patch
            // at row r*sh + ky, float (c*sw)*Cin + kx*Cin + ci.
            const int p = threadIdx.x - CMP_WARP0 * 32;  // thread = pixel of the tile = row of A
            const int r = p >> 4, c = p & 15;
            static_assert(CMP_WARPS * 32 == BLOCK_M || !CONV, "one thread per A row");
            const int origin = (r * args.sh) * args.row_floats + (c * args.sw) * args.cin;
            int ps = 0, as = 0;
            uint32_t pphase = 0, aphase = 0;
            for (int tile = blockIdx.x; tile < args.num_tiles; tile += gridDim.x) {
                bool got = bounded_wait(smem_u32(&bar_patch_full[ps]), pphase, abort_flag);
                got = got && bounded_wait(smem_u32(&bar_a_empty[as]), aphase ^ 1u, abort_flag);
                if (!__all_sync(0xffffffffu, got)) {
                    if (lane == 0 && !*abort_flag) {
                        *abort_flag = 1;
                        atomicOr(args.dev_status, DEV_STATUS_TIMEOUT_DEPTHWISE);
                    }
                    break;
                }
                const float* patch = patch_ptr + (size_t)ps * (args.patch_stride / 4) + origin;
                const uint32_t row_addr = a_base + (uint32_t)as * A_STAGE_BYTES + (uint32_t)p * 128u;
                if (args.rows9) {
                    // 3 x 3 window on 3 channels: the nine values a filter row sees lie next to each other in the
                    // patch, 8-byte aligned, and in im2col order, so a row is four 8-byte loads and one 4-byte load
                    // (15 loads instead of 27, and a half-warp's 8-byte loads fall on 32 distinct banks)
                    float v[BLOCK_K];
#pragma unroll
                    for (int ky = 0; ky < 3; ++ky) {
                        const float* rowp = patch + ky * args.row_floats;
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const float2 t = *reinterpret_cast<const float2*>(rowp + 2 * j);
                            v[ky * 9 + 2 * j] = t.x;
                            v[ky * 9 + 2 * j + 1] = t.y;
                        }
                        v[ky * 9 + 8] = rowp[8];
                    }
#pragma unroll
                    for (int e = 27; e < BLOCK_K; ++e) v[e] = 0.0f;
#pragma unroll
                    for (int h = 0; h < BLOCK_K / 4; ++h) {
                        if (NARROW) {
#pragma unroll
                            for (int e = 0; e < 4; ++e) v[4 * h + e] = __bfloat162float(__float2bfloat16_rn(v[4 * h + e]));
                        }
                        const uint32_t dst = row_addr + (uint32_t)((h ^ (p & 7)) << 4);
                        asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "f"(v[4 * h]), "f"(v[4 * h + 1]),
                                     "f"(v[4 * h + 2]), "f"(v[4 * h + 3])
                                     : "memory");
                    }
                } else {
#pragma unroll
                for (int h = 0; h < BLOCK_K / 4; ++h) {
                    float v[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        v[e] = 4 * h + e < args.k_total ? patch[args.koff[4 * h + e]] : 0.0f;
                        if (NARROW) v[e] = __bfloat162float(__float2bfloat16_rn(v[e]));  // what is stored is a bfloat16
                    }
                    const uint32_t dst = row_addr + (uint32_t)((h ^ (p & 7)) << 4);
                    asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "f"(v[0]), "f"(v[1]), "f"(v[2]), "f"(v[3])
                                 : "memory");
                }
                }
                fence_async_smem();
                __syncwarp();
                if (lane == 0) {
                    mbar_arrive(smem_u32(&bar_a_full[as]));
                    mbar_arrive(smem_u32(&bar_patch_empty[ps]));
                }
                if (++ps == args.patch_stages) { ps = 0; pphase ^= 1u; }
                if (++as == args.a_stages) { as = 0; aphase ^= 1u; }
            }
        } else {
        // ---------------------------------------------------------------- depthwise (warps 10..25)
        // Two groups of eight warps take the k-blocks in turn.  Within a group, thread = (2 channels,
        // 2 tile columns, 4 tile rows): it walks the six patch rows its outputs need once, loading four
        // pixels per row; GEMM row of a pixel = row*16 + column.
        const int t = threadIdx.x - CMP_WARP0 * 32;
        const int group = t / (F_DW_GROUP_WARPS * 32);
        const int tg = t - group * (F_DW_GROUP_WARPS * 32);
        const int c2 = tg & 15;
        const int colg = (tg >> 4) & (F_TW / 2 - 1);
        const int rg = tg >> 7;
        constexpr int R = F_TH / 2;
        static_assert(F_DW_GROUP_WARPS * 32 == 16 * (F_TW / 2) * (F_TH / R), "one thread per 2 channels x 2 columns x R rows");
        int ps = 0, as = 0;
        uint32_t pphase = 0, aphase = 0;
        int turn = 0;  // which group's turn the next k-block is
        float2 w[9];
        float2 b = make_float2(0.f, 0.f);
        int loaded_kb = -1;
        bool ok = true;
        for (int tile = blockIdx.x; ok && tile < args.num_tiles; tile += gridDim.x) {
            for (int kb = 0; kb < num_k_blocks; ++kb) {
                if (turn == group) {
                    if (kb != loaded_kb) {
                        const int c = kb * BLOCK_K + c2 * 2;
#pragma unroll
                        for (int k = 0; k < 9; ++k) w[k] = __ldg(reinterpret_cast<const float2*>(args.dw_filter + (int64_t)k * args.C + c));
                        if (args.dw_bias) b = __ldg(reinterpret_cast<const float2*>(args.dw_bias + c));
                        loaded_kb = kb;
                    }
                    bool got = bounded_wait(smem_u32(&bar_patch_full[ps]), pphase, abort_flag);
                    got = got && bounded_wait(smem_u32(&bar_a_empty[as]), aphase ^ 1u, abort_flag);
                    if (!__all_sync(0xffffffffu, got)) {
                        if (lane == 0 && !*abort_flag) {
                            *abort_flag = 1;
                            atomicOr(args.dev_status, DEV_STATUS_TIMEOUT_DEPTHWISE);
                        }
                        ok = false;
                        break;
                    }
                    float2 acc[R][2];
#pragma unroll
                    for (int r = 0; r < R; ++r) acc[r][0] = acc[r][1] = make_float2(0.f, 0.f);
                    // element (two channels) index of this thread's first sample in the patch [10][18][32 channels]
                    const int origin = ((rg * R) * F_PW + colg * 2) * BLOCK_K + c2 * 2;
                    const float* patch = patch_ptr + (size_t)ps * (F_PATCH_STRIDE / 4) + origin;
                    const uint32_t* patch16 = reinterpret_cast<const uint32_t*>(reinterpret_cast<const uint8_t*>(patch_ptr) +
                                                                                (size_t)ps * args.patch_stride) + (origin >> 1);
#pragma unroll
                    for (int j = 0; j < R + 2; ++j) {
                        const float* row = patch + j * F_PW * BLOCK_K;
                        float2 v[4];
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            if (NARROW) {  // two bfloat16 channels in 32 bits: each is the upper half of its fp32
                                const uint32_t pair = patch16[(j * F_PW * BLOCK_K + q * BLOCK_K) >> 1];
                                v[q] = make_float2(__uint_as_float(pair << 16), __uint_as_float(pair & 0xffff0000u));
                            } else v[q] = *reinterpret_cast<const float2*>(row + q * BLOCK_K);
                        }
#pragma unroll
                        for (int ky = 0; ky < 3; ++ky) {
                            const int d = j - ky;
                            if (d >= 0 && d < R) {
#pragma unroll
                                for (int cc = 0; cc < 2; ++cc) {
                                    fma2(acc[d][cc], v[cc + 0], w[ky * 3 + 0]);
                                    fma2(acc[d][cc], v[cc + 1], w[ky * 3 + 1]);
                                    fma2(acc[d][cc], v[cc + 2], w[ky * 3 + 2]);
                                }
                            }
                        }
                    }
                    const uint32_t a_stage = a_base + (uint32_t)as * A_STAGE_BYTES;
                    if (args.dw_act == TFJSB_ACT_RELU6) store_depthwise_block<TFJSB_ACT_RELU6, NARROW>(acc, b, a_stage, rg, colg, c2);
                    else if (args.dw_act == TFJSB_ACT_RELU) store_depthwise_block<TFJSB_ACT_RELU, NARROW>(acc, b, a_stage, rg, colg, c2);
                    else store_depthwise_block<TFJSB_ACT_NONE, NARROW>(acc, b, a_stage, rg, colg, c2);
                    fence_async_smem();
                    __syncwarp();
                    if (lane == 0) {
                        mbar_arrive(smem_u32(&bar_a_full[as]));
                        mbar_arrive(smem_u32(&bar_patch_empty[ps]));
                    }
                }
                if (++turn == DW_GROUPS) turn = 0;
                if (++ps == args.patch_stages) { ps = 0; pphase ^= 1u; }
                if (++as == args.a_stages) { as = 0; aphase ^= 1u; }
            }
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

}  // namespace

bool dwpw_fused_supported(const ConvGeom& dw, int64_t Cout) {
    const int64_t tiles = dw.N * ((dw.Ho + F_TH - 1) / F_TH) * ((dw.Wo + F_TW - 1) / F_TW);
    return dw.fh == 3 && dw.fw == 3 && dw.sh == 1 && dw.sw == 1 && dw.dh == 1 && dw.dw == 1 && dw.mult == 1 &&
           dw.C >= BLOCK_K && dw.C % BLOCK_K == 0 && Cout >= 4 && Cout <= 512 && Cout % 4 == 0 && tiles >= 1 &&
           tiles < (1LL << 31) && dw.N < (1LL << 31);
}

tfjsb_status dwpw_fused_plan(tfjsb_ctx* ctx, const void* x, const float* bt, void* y, const ConvGeom& dw,
                             int64_t Cout, DwPwPlan* plan, bool narrow) {
    if (narrow && Cout % 8 != 0) return fail(ctx, TFJSB_ERR_UNSUPPORTED, "a bfloat16 output needs a channel count that is a multiple of 8");
    if (!dwpw_fused_supported(dw, Cout)) return fail(ctx, TFJSB_ERR_UNSUPPORTED, "shape not supported by the fused block kernel");
    if (!ctx->encode_tiled) return fail(ctx, TFJSB_ERR_CUDA, "cuTensorMapEncodeTiled is not available");
    plan->g = dw;
    plan->Co = (int)Cout;
    int bn = 32;
    while (bn < Cout && bn < 256) bn <<= 1;
    plan->block_n = bn;
    plan->n_sub = Cout > 256 ? 2 : 1;
    // tensor memory has 512 columns: two 256-wide halves leave room for one accumulator stage only
    plan->acc_stages = plan->n_sub == 2 ? 1 : (bn == 256 ? 2 : MAX_ACC_STAGES);
    plan->a_stages = plan->n_sub == 2 ? 2 : 3;
    plan->b_stages = plan->n_sub == 2 ? 3 : (bn == 256 ? 2 : 3);
    // all of Bt resident when its k-blocks fit the B ring's four barriers and leave room for three patches
    const int k_blocks = dw.C / BLOCK_K;
    // a bfloat16 patch is half the bytes (12 KiB keeps the stages 1024-aligned)
    const int patch_bytes = narrow ? F_PATCH_BYTES / 2 : F_PATCH_BYTES, patch_stride = narrow ? 12 * 1024 : F_PATCH_STRIDE;
    // one k-block per tile and a narrow output: the epilogue paces the kernel (see WIDE_EPI)
    plan->wide_epi = k_blocks == 1 && bn <= 128 && !getenv("TFJSB_NO_WIDE_EPI");
    const int epi_bytes = plan->wide_epi ? 2 * EPI_BYTES : EPI_BYTES;
    plan->b_resident = plan->n_sub == 1 && k_blocks <= 4 &&
                       epi_bytes + plan->a_stages * A_STAGE_BYTES + k_blocks * bn * BLOCK_K * 4 + 3 * patch_stride <= SMEM_LIMIT - 2048;
    if (plan->b_resident) plan->b_stages = k_blocks;
    const int fixed = epi_bytes + plan->a_stages * A_STAGE_BYTES + plan->b_stages * bn * BLOCK_K * 4;
    int ps = (SMEM_LIMIT - 2048 - fixed) / patch_stride;
    if (ps > 4) ps = 4;
    if (ps < 2) return fail(ctx, TFJSB_ERR_UNSUPPORTED, "no room for the input patch ring");
    plan->conv = false;
    plan->y_bf16 = narrow;
    plan->patch_stages = ps;
    plan->patch_bytes = patch_bytes;
    plan->patch_stride = patch_stride;
    plan->smem_bytes = (size_t)1024 + fixed + (size_t)ps * patch_stride;
    plan->tiles_x = (dw.Wo + F_TW - 1) / F_TW;
    plan->tiles_y = (dw.Ho + F_TH - 1) / F_TH;
    const int64_t tiles = dw.N * plan->tiles_x * plan->tiles_y;
    plan->num_tiles = (int)tiles;
    plan->grid = (int)(tiles < ctx->sm_count ? tiles : ctx->sm_count);

    auto encode = [&](CUtensorMap* map, const void* base, int rank, const cuuint64_t* dims, const cuuint64_t* strides,
                      const cuuint32_t* box, CUtensorMapSwizzle swz, const char* what, bool bf16 = false) -> tfjsb_status {
        cuuint32_t elem[4] = {1u, 1u, 1u, 1u};
        CUresult r = ctx->encode_tiled(map, bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32,
                                       (cuuint32_t)rank, const_cast<void*>(base), dims,
                                       strides, box, elem, CU_TENSOR_MAP_INTERLEAVE_NONE, swz,
                                       CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS)
            return fail(ctx, TFJSB_ERR_CUDA, std::string("cuTensorMapEncodeTiled failed for ") + what + " (CUresult " +
                                                 std::to_string((int)r) + ")");
        return TFJSB_OK;
    };
    tfjsb_status st;
    {
        cuuint64_t dims[4] = {(cuuint64_t)dw.C, (cuuint64_t)dw.W, (cuuint64_t)dw.H, (cuuint64_t)dw.N};
        const cuuint64_t eb = narrow ? 2u : 4u;  // bytes per stored value
        cuuint64_t strides[3] = {(cuuint64_t)dw.C * eb, (cuuint64_t)dw.W * dw.C * eb, (cuuint64_t)dw.H * dw.W * dw.C * eb};
        cuuint32_t box[4] = {(cuuint32_t)BLOCK_K, (cuuint32_t)F_PW, (cuuint32_t)F_PH, 1u};
        if ((st = encode(&plan->map_x, x, 4, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_NONE, "the block input", narrow)) != TFJSB_OK) return st;
    }
    {
        cuuint64_t dims[2] = {(cuuint64_t)dw.C, (cuuint64_t)Cout};
        cuuint64_t strides[1] = {(cuuint64_t)dw.C * 4u};
        cuuint32_t box[2] = {(cuuint32_t)BLOCK_K, (cuuint32_t)bn};
        if ((st = encode(&plan->map_b, bt, 2, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B, "the pointwise weights")) != TFJSB_OK) return st;
    }
    {
        cuuint64_t dims[4] = {(cuuint64_t)Cout, (cuuint64_t)dw.Wo, (cuuint64_t)dw.Ho, (cuuint64_t)dw.N};
        const cuuint64_t eb = narrow ? 2u : 4u;
        cuuint64_t strides[3] = {(cuuint64_t)Cout * eb, (cuuint64_t)dw.Wo * Cout * eb, (cuuint64_t)dw.Ho * dw.Wo * Cout * eb};
        cuuint32_t box[4] = {(cuuint32_t)EPI_COLS, (cuuint32_t)F_TW, 2u, 1u};
        if ((st = encode(&plan->map_y, y, 4, dims, strides, box, narrow ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B,
                         "the block output", narrow)) != TFJSB_OK) return st;
    }
    return TFJSB_OK;
}

// ---- small-window convolution on the same kernel ----------------------------------------------------
// conv2d whose whole im2col row fits one k-block (fh*fw*Cin <= 32, e.g. the 3x3x3 stem): the input
// patch of an 8 x 16 pixel tile comes in by one 3-D bulk tensor copy over x viewed as
// [N, H, W*Cin] and the compute warps only rearrange it into the A operand.
bool conv_patch_supported(const ConvGeom& g) {
    const int64_t k = (int64_t)g.fh * g.fw * g.C;
    const int64_t row_floats = (((int64_t)(F_TW - 1) * g.sw + g.fw) * g.C + 3) / 4 * 4;
    const int64_t rows = (int64_t)(F_TH - 1) * g.sh + g.fh;
    const int64_t tiles = g.N * ((g.Ho + F_TH - 1) / F_TH) * ((g.Wo + F_TW - 1) / F_TW);
    return k <= BLOCK_K && g.dh == 1 && g.dw == 1 && g.mult == 1 && g.Co >= 4 && g.Co <= 128 && g.Co % 4 == 0 &&
           row_floats <= 256 && rows <= 256 && ((int64_t)g.W * g.C) % 4 == 0 && (g.pl * g.C) % 4 == 0 &&
           ((int64_t)F_TW * g.sw * g.C) % 4 == 0 && rows * row_floats * 4 <= 15 * 1024 && tiles >= 1 && tiles < (1LL << 31) &&
           g.N < (1LL << 31);
}

tfjsb_status conv_patch_plan(tfjsb_ctx* ctx, const float* x, const float* bt, void* y, const ConvGeom& g, DwPwPlan* plan,
                             bool y_bf16) {
    if (y_bf16 && g.Co % 8 != 0) return fail(ctx, TFJSB_ERR_UNSUPPORTED, "a bfloat16 output needs a channel count that is a multiple of 8");
    plan->y_bf16 = y_bf16;
    if (!conv_patch_supported(g)) return fail(ctx, TFJSB_ERR_UNSUPPORTED, "shape not supported by the patch convolution kernel");
    if (!ctx->encode_tiled) return fail(ctx, TFJSB_ERR_CUDA, "cuTensorMapEncodeTiled is not available");
    plan->conv = true;
    plan->wide_epi = false;
    plan->g = g;
    plan->Co = g.Co;
    int bn = 32;
    while (bn < g.Co) bn <<= 1;
    plan->block_n = bn;
    plan->n_sub = 1;
    // two CTAs per SM: each takes half of tensor memory (256 columns) and half of shared memory
    plan->acc_stages = 256 / bn < F_MAX_ACC ? 256 / bn : F_MAX_ACC;
    plan->a_stages = 2;
    plan->b_stages = 1;  // the packed filter stays resident
    plan->b_resident = true;
    const int row_floats = (((F_TW - 1) * g.sw + g.fw) * g.C + 3) / 4 * 4;
    const int rows = (F_TH - 1) * g.sh + g.fh;
    plan->row_floats = row_floats;
    plan->patch_rows = rows;
    plan->patch_bytes = rows * row_floats * 4;
    plan->patch_stride = (plan->patch_bytes + 1023) / 1024 * 1024;
    const int fixed = EPI_BYTES + plan->a_stages * A_STAGE_BYTES + plan->b_stages * bn * BLOCK_K * 4;
    // small patches: a deep ring keeps enough input bytes in flight to cover the DRAM latency
    int ring = (F_CONV_SMEM - 1024 - fixed) / plan->patch_stride;
    if (ring > F_MAX_RING) ring = F_MAX_RING;
    if (ring < 2) return fail(ctx, TFJSB_ERR_UNSUPPORTED, "no room for the input patch ring");
    plan->patch_stages = ring;
    plan->smem_bytes = (size_t)1024 + fixed + (size_t)plan->patch_stages * plan->patch_stride;
    plan->tiles_x = (g.Wo + F_TW - 1) / F_TW;
    plan->tiles_y = (g.Ho + F_TH - 1) / F_TH;
    const int64_t tiles = g.N * plan->tiles_x * plan->tiles_y;
    plan->num_tiles = (int)tiles;
    plan->grid = (int)(tiles < 2 * ctx->sm_count ? tiles : 2 * ctx->sm_count);
    auto encode = [&](CUtensorMap* map, const void* base, int rank, const cuuint64_t* dims, const cuuint64_t* strides,
                      const cuuint32_t* box, CUtensorMapSwizzle swz, const char* what) -> tfjsb_status {
        cuuint32_t elem[4] = {1u, 1u, 1u, 1u};
        CUresult r = ctx->encode_tiled(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, (cuuint32_t)rank, const_cast<void*>(base), dims,
                                       strides, box, elem, CU_TENSOR_MAP_INTERLEAVE_NONE, swz,
                                       CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS)
            return fail(ctx, TFJSB_ERR_CUDA, std::string("cuTensorMapEncodeTiled failed for ") + what + " (CUresult " +
                                                 std::to_string((int)r) + ")");
        return TFJSB_OK;
    };
    tfjsb_status st;
    {
        cuuint64_t dims[3] = {(cuuint64_t)g.W * g.C, (cuuint64_t)g.H, (cuuint64_t)g.N};
        cuuint64_t strides[2] = {(cuuint64_t)g.W * g.C * 4u, (cuuint64_t)g.H * g.W * g.C * 4u};
        cuuint32_t box[3] = {(cuuint32_t)row_floats, (cuuint32_t)rows, 1u};
        if ((st = encode(&plan->map_x, x, 3, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_NONE, "the convolution input")) != TFJSB_OK) return st;
    }
    {
        const int64_t k_pad = BLOCK_K;
        cuuint64_t dims[2] = {(cuuint64_t)k_pad, (cuuint64_t)g.Co};
        cuuint64_t strides[1] = {(cuuint64_t)k_pad * 4u};
        cuuint32_t box[2] = {(cuuint32_t)BLOCK_K, (cuuint32_t)bn};
        if ((st = encode(&plan->map_b, bt, 2, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B, "the packed filter")) != TFJSB_OK) return st;
    }
    {
        cuuint64_t dims[4] = {(cuuint64_t)g.Co, (cuuint64_t)g.Wo, (cuuint64_t)g.Ho, (cuuint64_t)g.N};
        cuuint64_t strides[3] = {(cuuint64_t)g.Co * 4u, (cuuint64_t)g.Wo * g.Co * 4u, (cuuint64_t)g.Ho * g.Wo * g.Co * 4u};
        cuuint32_t box[4] = {(cuuint32_t)EPI_COLS, (cuuint32_t)F_TW, 2u, 1u};
        if (y_bf16) {
            for (cuuint64_t& v : strides) v /= 2;  // two bytes per value
            cuuint32_t elem[4] = {1u, 1u, 1u, 1u};
            CUresult r = ctx->encode_tiled(&plan->map_y, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, y, dims, strides, box, elem,
                                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B,
                                           CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
            if (r != CUDA_SUCCESS)
                return fail(ctx, TFJSB_ERR_CUDA, "cuTensorMapEncodeTiled failed for the bfloat16 convolution output (CUresult " +
                                                     std::to_string((int)r) + ")");
        } else if ((st = encode(&plan->map_y, y, 4, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B, "the convolution output")) != TFJSB_OK) return st;
    }
    return TFJSB_OK;
}

cudaError_t launch_dwpw_fused(const DwPwPlan& plan, const float* dw_filter, const float* dw_bias, int dw_act,
                              const float* pw_bias, int pw_act, unsigned int* dev_status, cudaStream_t s,
                              int64_t* launches) {
    {
        cudaError_t ae = cudaSuccess;
        if (ae == cudaSuccess) ae = smem_attr_once(reinterpret_cast<const void*>(&dwpw_fused_kernel<false>), SMEM_LIMIT - 2048);
        if (ae == cudaSuccess) ae = smem_attr_once(reinterpret_cast<const void*>(&dwpw_fused_kernel<true>), F_CONV_SMEM);
        if (ae == cudaSuccess) ae = smem_attr_once(reinterpret_cast<const void*>(&dwpw_fused_kernel<false, false, true>), SMEM_LIMIT - 2048);
        if (ae == cudaSuccess) ae = smem_attr_once(reinterpret_cast<const void*>(&dwpw_fused_kernel<false, false, false, true>), SMEM_LIMIT - 2048);
        if (ae == cudaSuccess) ae = smem_attr_once(reinterpret_cast<const void*>(&dwpw_fused_kernel<false, true>), SMEM_LIMIT - 2048);
        if (ae == cudaSuccess) ae = smem_attr_once(reinterpret_cast<const void*>(&dwpw_fused_kernel<false, true, true>), SMEM_LIMIT - 2048);
        if (ae == cudaSuccess) ae = smem_attr_once(reinterpret_cast<const void*>(&dwpw_fused_kernel<false, true, false, true>), SMEM_LIMIT - 2048);
        if (ae == cudaSuccess) ae = smem_attr_once(reinterpret_cast<const void*>(&dwpw_fused_kernel<true, true>), F_CONV_SMEM);
        if (ae != cudaSuccess) return ae;
    }
    FusedArgs a;
    a.C = plan.g.C; a.Co = plan.Co;
    a.Ho = plan.g.Ho; a.Wo = plan.g.Wo;
    a.pt = plan.g.pt; a.pl = plan.g.pl;
    a.tiles_x = plan.tiles_x; a.tiles_y = plan.tiles_y;
    a.num_tiles = plan.num_tiles;
    a.block_n = plan.block_n;
    a.n_sub = plan.n_sub;
    a.acc_stages = plan.acc_stages;
    a.patch_stages = plan.patch_stages; a.a_stages = plan.a_stages; a.b_stages = plan.b_stages;
    a.b_resident = plan.b_resident ? 1 : 0;
    a.patch_bytes = plan.patch_bytes; a.patch_stride = plan.patch_stride;
    a.cin = plan.g.C; a.fw_cin = plan.g.fw * plan.g.C; a.sh = plan.g.sh; a.sw = plan.g.sw;
    a.row_floats = plan.row_floats; a.k_total = plan.g.fh * plan.g.fw * plan.g.C;
    a.rows9 = plan.conv && plan.g.fh == 3 && a.fw_cin == 9 && (a.sw * a.cin) % 2 == 0 && plan.row_floats % 2 == 0;
    for (int k = 0; k < 32; ++k) {
        const int ky = a.fw_cin > 0 ? k / a.fw_cin : 0;
        a.koff[k] = (plan.conv && k < a.k_total) ? ky * plan.row_floats + (k - ky * a.fw_cin) : 0;
    }
    a.dw_filter = dw_filter; a.dw_bias = dw_bias; a.dw_act = dw_act;
    a.pw_bias = pw_bias; a.pw_act = pw_act;
    a.dev_status = dev_status;
    if (!plan.conv && plan.y_bf16) {
        cudaError_t en;
        if (plan.wide_epi && plan.b_resident)
            en = launch_k(dwpw_fused_kernel<false, true, false, true>, dim3(plan.grid), dim3(F_THREADS), plan.smem_bytes, s, plan.map_x,
                          plan.map_b, plan.map_y, a);
        else if (!plan.b_resident)
            en = launch_k(dwpw_fused_kernel<false, true, true>, dim3(plan.grid), dim3(F_THREADS), plan.smem_bytes, s, plan.map_x,
                          plan.map_b, plan.map_y, a);
        else
            en = launch_k(dwpw_fused_kernel<false, true>, dim3(plan.grid), dim3(F_THREADS), plan.smem_bytes, s, plan.map_x, plan.map_b,
                          plan.map_y, a);
        ++*launches;
        return en;
    }
    cudaError_t e = (plan.conv && plan.y_bf16)
                        ? launch_k(dwpw_fused_kernel<true, true>, dim3(plan.grid), dim3(F_CONV_THREADS), plan.smem_bytes, s,
                                   plan.map_x, plan.map_b, plan.map_y, a)
                    : (!plan.conv && plan.wide_epi && plan.b_resident)
                        ? launch_k(dwpw_fused_kernel<false, false, false, true>, dim3(plan.grid), dim3(F_THREADS), plan.smem_bytes, s,
                                   plan.map_x, plan.map_b, plan.map_y, a)
                    : (!plan.conv && !plan.b_resident)
                        ? launch_k(dwpw_fused_kernel<false, false, true>, dim3(plan.grid), dim3(F_THREADS), plan.smem_bytes, s,
                                   plan.map_x, plan.map_b, plan.map_y, a)
                    : plan.conv ? launch_k(dwpw_fused_kernel<true>, dim3(plan.grid), dim3(F_CONV_THREADS), plan.smem_bytes, s,
                                         plan.map_x, plan.map_b, plan.map_y, a)
                              : launch_k(dwpw_fused_kernel<false>, dim3(plan.grid), dim3(F_THREADS), plan.smem_bytes, s,
                                         plan.map_x, plan.map_b, plan.map_y, a);
    ++*launches;
    return e;
}

}  // namespace tfjsb

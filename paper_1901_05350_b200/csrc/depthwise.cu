// depthwiseConv2d (NHWC, filter [fh,fw,C,mult]) with the fused bias + activation epilogue.
//
// Not a dense contraction (9 multiply-adds per output for 8 bytes of traffic at stride 1), so it
// runs on CUDA cores and is bound by memory bandwidth.
//
// Fast path (3x3 window, multiplier 1, dilation 1, C % 4 == 0, stride 1 or 2 in both
// directions): each thread owns 4 consecutive channels (one float4) of one output column and a
// strip of ROWS output rows.  It walks the input rows that strip needs once, top to bottom,
// loading the three float4s (left, centre, right) of each row and feeding every output row the
// input row contributes to, so an input row is fetched once per strip rather than once per tap.
// Threads are laid out channel-fastest, then output column, so a warp's loads and stores are
// contiguous 512-byte runs; a block spans several output columns so the left/right neighbours a
// thread needs are lines its block has just brought into L1.
//
// Everything else (other windows, dilation, channel multipliers, odd channel counts) takes the
// scalar kernel: one thread per output element.
//
// Pipelined path (same shapes as the fast path, C >= 32, tensor maps available): the register
// kernel above is bound by load latency, not bandwidth (its loads sit in registers, ~80 per thread,
// so few warps fit and few bytes are in flight).  `depthwise3x3_tma_kernel` keeps the bytes in
// flight in shared memory instead: persistent CTAs walk tiles of TH x TW output pixels x 32
// channels; a producer warp issues the bulk tensor copy (TMA) of the next tiles' input patches
// ((TH-1)*S+3 rows x (TW-1)*S+3 columns x 128 bytes, zero-filled outside the image, which is the
// 'same' padding) into a ring of stages (full / empty mbarriers) while eight compute warps work
// on the landed tiles from shared memory with the same sliding-row scheme and store float4s
// straight to global memory.
#include <cuda_bf16.h>

#include <cstdlib>

#include "common.cuh"
#include "ptx_sm100.cuh"

namespace tfjsb {

namespace {

constexpr int DW_THREADS = 256;

__device__ __forceinline__ float4 ld4(const float* p) { return *reinterpret_cast<const float4*>(p); }
__device__ __forceinline__ void fma4(float4& acc, const float4& a, const float4& b) {
    acc.x = fmaf(a.x, b.x, acc.x); acc.y = fmaf(a.y, b.y, acc.y);
    acc.z = fmaf(a.z, b.z, acc.z); acc.w = fmaf(a.w, b.w, acc.w);
}

template <int S, int ROWS, int D = 1>
__global__ void __launch_bounds__(DW_THREADS)
depthwise3x3_kernel(const float* __restrict__ x, const float* __restrict__ f, const float* __restrict__ bias,
                    int act, float* __restrict__ y, ConvGeom g, int tc, int c4_tiles) {
    // block = tx_count output columns x tc channel quads
    const int C4 = g.C >> 2;
    const int tx_count = DW_THREADS / tc;
    const int c4 = (blockIdx.x % c4_tiles) * tc + (threadIdx.x % tc);
    const int ox = (blockIdx.x / c4_tiles) * tx_count + (threadIdx.x / tc);
    const int oy0 = blockIdx.y * ROWS;
    const int64_t n = blockIdx.z;
    if (c4 >= C4 || ox >= g.Wo) return;
    const int c = c4 * 4;

    float4 w[9];
#pragma unroll
    for (int t = 0; t < 9; ++t) w[t] = ld4(f + (int64_t)t * g.C + c);

    float4 acc[ROWS];
#pragma unroll
    for (int r = 0; r < ROWS; ++r) acc[r] = make_float4(0.f, 0.f, 0.f, 0.f);

    const int iy_base = oy0 * S - g.pt;
    const int ix_base = ox * S - g.pl;
    const bool in_x0 = ix_base >= 0 && ix_base < g.W;
    const bool in_x1 = ix_base + D >= 0 && ix_base + D < g.W;       // D: dilation (taps D pixels apart)
    const bool in_x2 = ix_base + 2 * D >= 0 && ix_base + 2 * D < g.W;
    const float* xn = x + n * (int64_t)g.H * g.W * g.C + c;
    const float4 zero = make_float4(0.f, 0.f, 0.f, 0.f);

    constexpr int IN_ROWS = (ROWS - 1) * S + 2 * D + 1;
#pragma unroll
    for (int j = 0; j < IN_ROWS; ++j) {
        const int iy = iy_base + j;
        float4 v0 = zero, v1 = zero, v2 = zero;
        if (iy >= 0 && iy < g.H) {
            const float* row = xn + ((int64_t)iy * g.W + ix_base) * g.C;
            if (in_x0) v0 = ld4(row);
            if (in_x1) v1 = ld4(row + D * g.C);
            if (in_x2) v2 = ld4(row + 2 * D * g.C);
        }
#pragma unroll
        for (int ky = 0; ky < 3; ++ky) {
            const int t = j - ky * D;
            if (t >= 0 && t % S == 0 && t / S < ROWS) {
                const int r = t / S;
                fma4(acc[r], v0, w[ky * 3 + 0]);
                fma4(acc[r], v1, w[ky * 3 + 1]);
                fma4(acc[r], v2, w[ky * 3 + 2]);
            }
        }
    }

    float4 b = zero;
    if (bias) b = ld4(bias + c);
#pragma unroll
    for (int r = 0; r < ROWS; ++r) {
        const int oy = oy0 + r;
        if (oy < g.Ho) {
            float4 v = acc[r];
            v.x = apply_act(v.x + b.x, act); v.y = apply_act(v.y + b.y, act);
            v.z = apply_act(v.z + b.z, act); v.w = apply_act(v.w + b.w, act);
            *reinterpret_cast<float4*>(y + ((n * g.Ho + oy) * (int64_t)g.Wo + ox) * g.Co + c) = v;
        }
    }
}

__global__ void depthwise_generic_kernel(const float* __restrict__ x, const float* __restrict__ f,
                                         const float* __restrict__ bias, int act, float* __restrict__ y,
                                         ConvGeom g, int64_t n_out) {
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_out; i += stride) {
        const int oc = (int)(i % g.Co);
        int64_t t = i / g.Co;
        const int ox = (int)(t % g.Wo); t /= g.Wo;
        const int oy = (int)(t % g.Ho);
        const int64_t n = t / g.Ho;
        const int c = oc / g.mult, q = oc % g.mult;
        float acc = 0.0f;
        for (int ky = 0; ky < g.fh; ++ky) {
            const int iy = oy * g.sh - g.pt + ky * g.dh;
            if (iy < 0 || iy >= g.H) continue;
            for (int kx = 0; kx < g.fw; ++kx) {
                const int ix = ox * g.sw - g.pl + kx * g.dw;
                if (ix < 0 || ix >= g.W) continue;
                acc = fmaf(x[((n * g.H + iy) * (int64_t)g.W + ix) * g.C + c],
                           f[((int64_t)(ky * g.fw + kx) * g.C + c) * g.mult + q], acc);
            }
        }
        if (bias) acc = acc + bias[oc];
        y[i] = apply_act(acc, act);
    }
}

// Bias, activation and store of one thread's R output rows (4 channels each) of the pipelined kernel;
// `idx` is the element index of the first row's first channel, OUT16 stores bfloat16 (rounded to nearest even).
template <int ACT, int R, bool OUT16>
__device__ __forceinline__ void store_rows(const float4 (&acc)[R], const float4 b, void* y, int64_t idx, int64_t row_pitch, int rows) {
#pragma unroll
    for (int r = 0; r < R; ++r) {
        if (r < rows) {
            float4 v = acc[r];
            v.x = apply_act_t<ACT>(v.x + b.x); v.y = apply_act_t<ACT>(v.y + b.y);
            v.z = apply_act_t<ACT>(v.z + b.z); v.w = apply_act_t<ACT>(v.w + b.w);
            if (OUT16) {
                const __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y), hi = __floats2bfloat162_rn(v.z, v.w);
                uint2 o;
                o.x = *reinterpret_cast<const uint32_t*>(&lo);
                o.y = *reinterpret_cast<const uint32_t*>(&hi);
                *reinterpret_cast<uint2*>(static_cast<__nv_bfloat16*>(y) + idx) = o;
            } else {
                *reinterpret_cast<float4*>(static_cast<float*>(y) + idx) = v;
            }
        }
        idx += row_pitch;
    }
}

template <int R, bool OUT16>
__device__ __forceinline__ void store_rows_act(int act, const float4 (&acc)[R], const float4 b, void* y, int64_t idx,
                                               int64_t row_pitch, int rows) {
    // the activation is chosen once per tile, not once per value: the kernel is close to issue bound
    if (act == TFJSB_ACT_RELU6) store_rows<TFJSB_ACT_RELU6, R, OUT16>(acc, b, y, idx, row_pitch, rows);
    else if (act == TFJSB_ACT_RELU) store_rows<TFJSB_ACT_RELU, R, OUT16>(acc, b, y, idx, row_pitch, rows);
    else store_rows<TFJSB_ACT_NONE, R, OUT16>(acc, b, y, idx, row_pitch, rows);
}

// Four consecutive channels of one patch sample as fp32: one 16-byte load, or one 8-byte load of four
// bfloat16 (each is the upper half of its fp32).
template <bool NARROW>
__device__ __forceinline__ float4 ld_quad(const uint8_t* p) {
    if (NARROW) {
        const uint2 raw = *reinterpret_cast<const uint2*>(p);
        return make_float4(__uint_as_float(raw.x << 16), __uint_as_float(raw.x & 0xffff0000u),
                           __uint_as_float(raw.y << 16), __uint_as_float(raw.y & 0xffff0000u));
    }
    return *reinterpret_cast<const float4*>(p);
}

// ---- pipelined kernel ---------------------------------------------------------------------------
constexpr int DW_CB = 32;          // channels per tile of the narrow instances: one 128-byte line per pixel
constexpr int DW_MAX_STAGES = 4;

struct DwTiling {
    int tiles_x, tiles_y, c_blocks, stages;
    long long num_tiles;
};

template <int S, int TW, int R, int D = 1, int CB = DW_CB, bool NARROW = false>
struct DwTile {
    static constexpr int QUADS = CB / 4;               // threads across a pixel's channels (4 channels each)
    static constexpr int RG = DW_THREADS / QUADS / TW; // row groups of threads: 256 = QUADS x TW x RG
    static constexpr int TH = RG * R;                  // output rows per tile
    static constexpr int TWIN = (TW - 1) * S + 2 * D + 1;  // input patch (D: dilation, taps D pixels apart)
    static constexpr int THIN = (TH - 1) * S + 2 * D + 1;
    static constexpr int EB = NARROW ? 2 : 4;                    // bytes per stored value (bfloat16 or fp32)
    static constexpr int STAGE_BYTES = THIN * TWIN * CB * EB;    // what one copy delivers
    static constexpr int STAGE_STRIDE = (STAGE_BYTES + 127) / 128 * 128;  // pitch of the ring
};

constexpr int DW_TMA_THREADS = DW_THREADS + 32;  // eight compute warps and the warp that issues the copies

// NARROW: the input is bfloat16 (the patch is copied as such and widened by the compute threads; filter and bias
// stay fp32, the sums are fp32 in the same order) and the output is bfloat16 or, with y_f32, fp32.
template <int S, int TW, int R, int D = 1, int CB = DW_CB, bool NARROW = false>
__global__ void __launch_bounds__(DW_TMA_THREADS, 2)
depthwise3x3_tma_kernel(const __grid_constant__ CUtensorMap map_x, const float* __restrict__ f,
                        const float* __restrict__ bias, int act, void* __restrict__ y, int y_f32, ConvGeom g, DwTiling t,
                        unsigned int* dev_status) {
    using T = DwTile<S, TW, R, D, CB, NARROW>;
    extern __shared__ uint8_t dw_smem_raw[];
    __shared__ __align__(8) uint64_t bar_full[DW_MAX_STAGES];   // copy landed (1 arrival + bytes)
    __shared__ __align__(8) uint64_t bar_empty[DW_MAX_STAGES];  // the eight compute warps are done with the stage
    __shared__ int4 tile_info[DW_MAX_STAGES];
    __shared__ int abort_flag_s;
    volatile int* abort_flag = &abort_flag_s;

    const uint32_t smem_base = (ptx::smem_u32(dw_smem_raw) + 127u) & ~127u;
    const uint8_t* smem_p = dw_smem_raw + (smem_base - ptx::smem_u32(dw_smem_raw));
    const int tid = threadIdx.x;
    const int warp = tid >> 5, lane = tid & 31;

    if (tid == 0) {
        for (int s = 0; s < t.stages; ++s) {
            ptx::mbar_init(ptx::smem_u32(&bar_full[s]), 1);
            ptx::mbar_init(ptx::smem_u32(&bar_empty[s]), DW_THREADS / 32);
        }
        abort_flag_s = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_x) : "memory");
    }
    __syncthreads();
    ptx::pdl_launch_dependents();
    ptx::pdl_wait();  // the input is the previous kernel's output

    const int num_tiles = (int)t.num_tiles;
    const int first = blockIdx.x, step = gridDim.x;
    const int my_tiles = first < num_tiles ? (num_tiles - first + step - 1) / step : 0;

    if (warp == DW_THREADS / 32) {
        // ------------------------------------------------------------ producer: one thread
        // tile index -> (channel block, tile column, tile row, image), channel block fastest.  Only this
        // thread pays for the divisions: it leaves the coordinates beside the stage for the compute
        // warps (written before its mbarrier arrive, read after their wait: release / acquire).
        if (lane == 0) {
            int slot = 0;
            uint32_t parity = 0;
            int i = 0;
            bool ok = true;
            for (; i < my_tiles; ++i) {
                if (!ptx::bounded_wait(ptx::smem_u32(&bar_empty[slot]), parity ^ 1u, abort_flag)) { ok = false; break; }
                const int tile = first + i * step;
                const int cb = tile % t.c_blocks;
                int q = tile / t.c_blocks;
                const int tx = q % t.tiles_x; q /= t.tiles_x;
                const int ty = q % t.tiles_y;
                const int n = q / t.tiles_y;
                tile_info[slot] = make_int4(cb, tx, ty, n);
                const uint32_t bar = ptx::smem_u32(&bar_full[slot]);
                ptx::mbar_arrive_expect_tx(bar, (uint32_t)T::STAGE_BYTES);
                ptx::tma_load_4d(smem_base + (uint32_t)slot * (uint32_t)T::STAGE_STRIDE, &map_x, bar, cb * CB,
                                 tx * TW * S - g.pl, ty * T::TH * S - g.pt, n);
                if (++slot == t.stages) { slot = 0; parity ^= 1u; }
            }
            if (!ok || *abort_flag) {
                if (!*abort_flag) *abort_flag = 1;
                atomicOr(dev_status, DEV_STATUS_TIMEOUT_DEPTHWISE);
                // wait (bounded) for the copies still in flight so nothing lands after the CTA has gone
                const int lo = i - t.stages > 0 ? i - t.stages : 0;
                for (int k = lo; k < i; ++k) {
                    const unsigned long long t0 = ptx::global_ns();
                    while (!ptx::mbar_try_wait(ptx::smem_u32(&bar_full[k % t.stages]), (uint32_t)((k / t.stages) & 1))) {
                        if (ptx::global_ns() - t0 > ptx::WAIT_LIMIT_NS) {
                            atomicOr(dev_status, DEV_STATUS_TIMEOUT_DRAIN);
                            break;
                        }
                    }
                }
            }
        }
        return;
    }

    // ---------------------------------------------------------------- compute warps
    // The warps never synchronise with each other: each waits for the stage, does its share of the
    // tile and reports the stage free, so a fast warp can run up to `stages` tiles ahead of a slow one.
    const int c4 = tid % T::QUADS;
    const int col = (tid / T::QUADS) % TW;
    const int rg = tid / (T::QUADS * TW);
    const int64_t row_pitch = (int64_t)g.Wo * g.Co;

    float4 w[9];
    float4 b = make_float4(0.f, 0.f, 0.f, 0.f);
    int loaded_cb = -1;
    int slot = 0;
    uint32_t parity = 0;
    for (int i = 0; i < my_tiles; ++i) {
        const bool got = ptx::bounded_wait(ptx::smem_u32(&bar_full[slot]), parity, abort_flag);
        if (!__all_sync(0xffffffffu, got)) {
            if (lane == 0) *abort_flag = 1;
            break;
        }
        const int4 info = tile_info[slot];
        const int cb = info.x, tx = info.y, ty = info.z;
        const int c = cb * CB + c4 * 4;
        const int ox = tx * TW + col;
        const int oy0 = ty * T::TH + rg * R;
        const bool live = c < g.C && ox < g.Wo && oy0 < g.Ho;

        if (live) {
            if (cb != loaded_cb) {
#pragma unroll
                for (int k = 0; k < 9; ++k) w[k] = __ldg(reinterpret_cast<const float4*>(f + (int64_t)k * g.C + c));
                if (bias) b = __ldg(reinterpret_cast<const float4*>(bias + c));
                loaded_cb = cb;
            }
            float4 acc[R];
#pragma unroll
            for (int r = 0; r < R; ++r) acc[r] = make_float4(0.f, 0.f, 0.f, 0.f);
            // byte offsets into the patch [THIN][TWIN][CB values]
            const uint8_t* patch = smem_p + (size_t)slot * T::STAGE_STRIDE +
                                   (size_t)((((rg * R * S) * T::TWIN + col * S) * CB + c4 * 4) * T::EB);
            constexpr int IN_ROWS = (R - 1) * S + 2 * D + 1;
#pragma unroll
            for (int j = 0; j < IN_ROWS; ++j) {
                const uint8_t* row = patch + j * T::TWIN * CB * T::EB;
                const float4 v0 = ld_quad<NARROW>(row), v1 = ld_quad<NARROW>(row + D * CB * T::EB),
                             v2 = ld_quad<NARROW>(row + 2 * D * CB * T::EB);
#pragma unroll
                for (int ky = 0; ky < 3; ++ky) {
                    const int d = j - ky * D;
                    if (d >= 0 && d % S == 0 && d / S < R) {
                        fma4_packed(acc[d / S], v0, w[ky * 3 + 0]);
                        fma4_packed(acc[d / S], v1, w[ky * 3 + 1]);
                        fma4_packed(acc[d / S], v2, w[ky * 3 + 2]);
                    }
                }
            }
            // the stage has been read: hand it back before the stores go out
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&bar_empty[slot]));
            const int64_t idx = (((int64_t)info.w * g.Ho + oy0) * g.Wo + ox) * g.Co + c;
            const int rows = g.Ho - oy0;
            if (NARROW && !y_f32) store_rows_act<R, true>(act, acc, b, y, idx, row_pitch, rows);
            else store_rows_act<R, false>(act, acc, b, y, idx, row_pitch, rows);
        } else {
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&bar_empty[slot]));
        }
        if (++slot == t.stages) { slot = 0; parity ^= 1u; }
    }
}

// the instances: {stride, tile width, tile height, bytes of a stage, pitch of the ring, channels per tile}
struct DwVariant {
    int S, TW, TH, stage_bytes, stage_stride, cb;
};
#define DW_VARIANT(S, TW, R, D, CB, NARROW)                                                       \
    {S, TW, DwTile<S, TW, R, D, CB, NARROW>::TH, DwTile<S, TW, R, D, CB, NARROW>::STAGE_BYTES,    \
     DwTile<S, TW, R, D, CB, NARROW>::STAGE_STRIDE, CB}
constexpr DwVariant kDwVariants[] = {
    // fp32, 32 channels per tile.  Seven rows per thread for every stride-1 image wider than 8 (seven divides the
    // heights of the usual networks, and against four rows per thread it measured [128,56,56,128] 84.0 -> 77.2 us,
    // [128,28,28,256] 41.5 -> 39.2 us, [128,112,112,32] no change)
    DW_VARIANT(1, 16, 7, 1, 32, false),   // 0: stride 1
    DW_VARIANT(1, 8, 2, 1, 32, false),    // 1: stride 1, images up to 8 wide
    DW_VARIANT(2, 16, 2, 1, 32, false),   // 2: stride 2
    DW_VARIANT(2, 8, 2, 1, 32, false),    // 3: stride 2, 8 outputs wide
    DW_VARIANT(1, 16, 4, 2, 32, false),   // 4: stride 1, dilation 2
    DW_VARIANT(1, 16, 4, 4, 32, false),   // 5: stride 1, dilation 4
    // fp32, 64 channels per tile (256-byte lines): half as many box rows for the copy unit per byte moved
    DW_VARIANT(1, 16, 7, 1, 64, false),   // 6: stride 1
    DW_VARIANT(1, 8, 4, 1, 64, false),    // 7: stride 1, images up to 8 wide (a whole 7 x 7 image per tile)
    DW_VARIANT(2, 8, 2, 1, 64, false),    // 8: stride 2, 8 outputs wide
    // bfloat16 storage: the same tiles on 2-byte values, 64 channels (one 128-byte line) then 32
    DW_VARIANT(1, 16, 7, 1, 64, true),    // 9
    DW_VARIANT(1, 8, 4, 1, 64, true),     // 10
    DW_VARIANT(2, 16, 2, 1, 64, true),    // 11
    DW_VARIANT(2, 8, 2, 1, 64, true),     // 12
    DW_VARIANT(1, 16, 7, 1, 32, true),    // 13
    DW_VARIANT(1, 8, 2, 1, 32, true),     // 14
    DW_VARIANT(2, 16, 2, 1, 32, true),    // 15
    DW_VARIANT(2, 8, 2, 1, 32, true),     // 16
};
#undef DW_VARIANT
constexpr int DW_FIRST_NARROW = 9;
constexpr int DW_SMEM_BUDGET = 113 * 1024;  // two CTAs per SM

template <int S, int TW, int R, int D = 1, int CB = DW_CB, bool NARROW = false>
cudaError_t launch_tma_instance(const DepthwisePlan& plan, const float* f, const float* bias, int act, void* y, bool y_f32,
                                const ConvGeom& g, unsigned int* dev_status, cudaStream_t s) {
    auto kernel = depthwise3x3_tma_kernel<S, TW, R, D, CB, NARROW>;
    cudaError_t ae = smem_attr_once(reinterpret_cast<const void*>(kernel), DW_SMEM_BUDGET);
    if (ae != cudaSuccess) return ae;
    DwTiling t{plan.tiles_x, plan.tiles_y, plan.c_blocks, plan.stages, (long long)plan.num_tiles};
    return launch_k(kernel, dim3(plan.grid), dim3(DW_TMA_THREADS), plan.smem_bytes, s, plan.map_x, f, bias, act, y,
                    y_f32 ? 1 : 0, g, t, dev_status);
}

cudaError_t launch_tma_variant(const DepthwisePlan& plan, const float* f, const float* bias, int act, void* y, bool y_f32,
                               const ConvGeom& g, unsigned int* dev_status, cudaStream_t s) {
#define DW_CASE(V, ...) case V: return launch_tma_instance<__VA_ARGS__>(plan, f, bias, act, y, y_f32, g, dev_status, s)
    switch (plan.variant) {
        DW_CASE(0, 1, 16, 7, 1, 32, false);
        DW_CASE(1, 1, 8, 2, 1, 32, false);
        DW_CASE(2, 2, 16, 2, 1, 32, false);
        DW_CASE(3, 2, 8, 2, 1, 32, false);
        DW_CASE(4, 1, 16, 4, 2, 32, false);
        DW_CASE(5, 1, 16, 4, 4, 32, false);
        DW_CASE(6, 1, 16, 7, 1, 64, false);
        DW_CASE(7, 1, 8, 4, 1, 64, false);
        DW_CASE(8, 2, 8, 2, 1, 64, false);
        DW_CASE(9, 1, 16, 7, 1, 64, true);
        DW_CASE(10, 1, 8, 4, 1, 64, true);
        DW_CASE(11, 2, 16, 2, 1, 64, true);
        DW_CASE(12, 2, 8, 2, 1, 64, true);
        DW_CASE(13, 1, 16, 7, 1, 32, true);
        DW_CASE(14, 1, 8, 2, 1, 32, true);
        DW_CASE(15, 2, 16, 2, 1, 32, true);
        DW_CASE(16, 2, 8, 2, 1, 32, true);
        default: return cudaErrorInvalidValue;
    }
#undef DW_CASE
}

int pow2_at_most(int v, int cap) {
    int p = 1;
    while (p < v && p < cap) p <<= 1;
    return p;
}

}  // namespace

tfjsb_status depthwise_plan(tfjsb_ctx* ctx, const void* x, const ConvGeom& g, DepthwisePlan* plan, bool narrow) {
    plan->variant = -1;
    plan->narrow = narrow;
    const bool dilated = g.dh == g.dw && (g.dh == 2 || g.dh == 4) && g.sh == 1;  // atrous layers
    const bool shape_ok = g.fh == 3 && g.fw == 3 && g.mult == 1 && ((g.dh == 1 && g.dw == 1) || dilated) && g.sh == g.sw &&
                          (g.sh == 1 || g.sh == 2) && (g.C % 4 == 0) && g.C >= DW_CB;
    if (!shape_ok || !ctx->encode_tiled) return TFJSB_OK;
    if (narrow && (dilated || g.C % 8 != 0)) return TFJSB_OK;  // 16-byte row pitches; no dilated instances in this format
    // the 8-wide stride-2 tile where it wastes fewer columns than the 16-wide one
    const bool wide8 = g.Wo <= 8 || (g.Wo + 7) / 8 * 8 < (g.Wo + 15) / 16 * 16;
    int v;
    if (dilated) v = g.dh == 2 ? 4 : 5;
    else if (narrow) v = DW_FIRST_NARROW + (g.C % 64 == 0 ? 0 : 4) + (g.sh == 1 ? (g.Wo <= 8 ? 1 : 0) : (wide8 ? 3 : 2));
    else {
        v = g.sh == 1 ? (g.Wo <= 8 ? 1 : 0) : (g.Wo <= 8 ? 3 : 2);
        // 64-channel tiles where the channel count allows.  Measured at batch 128: [112,112,64] stride 2
        // 90.1 -> 86.9 us, [7,7,1024] 19.5 -> 15.4 us, the 14 x 14 x 512 layers unchanged; the stride-2 form is
        // 8 outputs wide, so it is taken only where that wastes fewer columns than the 16-wide 32-channel one
        // ([28,28,256] stride 2 ran 27.3 -> 29.1 us with it).
        if (g.C % 64 == 0) {
            if (g.sh == 1) v = v == 0 ? 6 : 7;
            else if (wide8) v = 8;
        }
    }
    const DwVariant& d = kDwVariants[v];
    const cuuint64_t eb = narrow ? 2u : 4u;
    const int twin = (d.TW - 1) * d.S + 2 * g.dw + 1, thin = (d.TH - 1) * d.S + 2 * g.dh + 1;
    cuuint64_t dims[4] = {(cuuint64_t)g.C, (cuuint64_t)g.W, (cuuint64_t)g.H, (cuuint64_t)g.N};
    cuuint64_t strides[3] = {(cuuint64_t)g.C * eb, (cuuint64_t)g.W * g.C * eb, (cuuint64_t)g.H * g.W * g.C * eb};
    cuuint32_t box[4] = {(cuuint32_t)d.cb, (cuuint32_t)twin, (cuuint32_t)thin, 1u};
    cuuint32_t elem[4] = {1u, 1u, 1u, 1u};
    CUresult r = ctx->encode_tiled(&plan->map_x, narrow ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4,
                                   const_cast<void*>(x), dims, strides,
                                   box, elem, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                                   CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS)
        return fail(ctx, TFJSB_ERR_CUDA, "cuTensorMapEncodeTiled failed for the depthwise input (CUresult " +
                                             std::to_string((int)r) + ")");
    plan->tiles_x = (g.Wo + d.TW - 1) / d.TW;
    plan->tiles_y = (g.Ho + d.TH - 1) / d.TH;
    plan->c_blocks = (g.C + d.cb - 1) / d.cb;
    plan->num_tiles = (int64_t)plan->tiles_x * plan->tiles_y * plan->c_blocks * g.N;
    if (plan->num_tiles > 0x7fffffff) return TFJSB_OK;  // tile indices are 32-bit in the kernel
    int stages = (DW_SMEM_BUDGET - 256) / d.stage_stride;
    if (stages > DW_MAX_STAGES) stages = DW_MAX_STAGES;
    if (stages < 2) return TFJSB_OK;  // cannot happen with the instances above
    plan->stages = stages;
    plan->smem_bytes = (size_t)stages * d.stage_stride + 128;
    const int64_t max_grid = (int64_t)ctx->sm_count * 2;
    plan->grid = (int)(plan->num_tiles < max_grid ? plan->num_tiles : max_grid);
    // A CTA walks tiles first, first + grid, ...; the channel block is the fastest tile coordinate, so a grid
    // that is a multiple of the number of channel blocks keeps every CTA on ONE channel block: its nine filter
    // vectors and the bias are loaded once instead of once per tile (a dependent global load in front of a
    // tile's short burst of work), while the CTAs that run side by side still cover all channel blocks of the
    // same pixels, so whole pixel vectors are read from DRAM at about the same time.  Measured on
    // [128,14,14,512]: 22.7 -> 20.6 us; no change for the 7 x 7 and stride-2 layers.
    if (plan->grid > plan->c_blocks && plan->grid % plan->c_blocks != 0) {
        const int rounded = plan->grid / plan->c_blocks * plan->c_blocks;
        if (rounded * 8 >= plan->grid * 7) plan->grid = rounded;
    }
    plan->variant = v;
    return TFJSB_OK;
}

cudaError_t launch_depthwise(const DepthwisePlan& plan, const float* x, const float* f, const float* bias, int act,
                             float* y, const ConvGeom& g, unsigned int* dev_status, cudaStream_t s,
                             int64_t* launches) {
    const int64_t n_out = g.N * g.Ho * g.Wo * g.Co;
    if (n_out == 0) return cudaSuccess;
    if (plan.variant >= 0) {
        if (plan.narrow) return cudaErrorInvalidValue;  // a plan made for bfloat16 storage: launch_depthwise_tma_narrow
        cudaError_t e = launch_tma_variant(plan, f, bias, act, y, true, g, dev_status, s);
        ++*launches;
        return e;
    }
    // dilated windows (the atrous depthwise layers of output-stride-16 / -8 MobileNet variants): stride 1, dilation 2 or 4
    const bool dilated = g.dh == g.dw && (g.dh == 2 || g.dh == 4) && g.sh == 1;
    const bool fast = g.fh == 3 && g.fw == 3 && g.mult == 1 && ((g.dh == 1 && g.dw == 1) || dilated) && g.sh == g.sw &&
                      (g.sh == 1 || g.sh == 2) && (g.C % 4 == 0) && g.N <= 65535;
    if (fast) {
        constexpr int ROWS = 4;
        const int C4 = g.C / 4;
        const int tc = pow2_at_most(C4, 32);
        const int c4_tiles = (C4 + tc - 1) / tc;
        const int tx_count = DW_THREADS / tc;
        const int64_t gx = (int64_t)c4_tiles * ((g.Wo + tx_count - 1) / tx_count);
        const int gy = (g.Ho + ROWS - 1) / ROWS;
        if (gx <= 2147483647LL && gy <= 65535) {
            dim3 grid((unsigned)gx, (unsigned)gy, (unsigned)g.N);
            if (g.dh == 2)
                depthwise3x3_kernel<1, ROWS, 2><<<grid, DW_THREADS, 0, s>>>(x, f, bias, act, y, g, tc, c4_tiles);
            else if (g.dh == 4)
                depthwise3x3_kernel<1, ROWS, 4><<<grid, DW_THREADS, 0, s>>>(x, f, bias, act, y, g, tc, c4_tiles);
            else if (g.sh == 1)
                depthwise3x3_kernel<1, ROWS><<<grid, DW_THREADS, 0, s>>>(x, f, bias, act, y, g, tc, c4_tiles);
            else
                depthwise3x3_kernel<2, ROWS><<<grid, DW_THREADS, 0, s>>>(x, f, bias, act, y, g, tc, c4_tiles);
            ++*launches;
            return cudaGetLastError();
        }
    }
    int64_t blocks = (n_out + DW_THREADS - 1) / DW_THREADS;
    if (blocks > current_sm_count() * 32) blocks = current_sm_count() * 32;
    depthwise_generic_kernel<<<(unsigned)blocks, DW_THREADS, 0, s>>>(x, f, bias, act, y, g, n_out);
    ++*launches;
    return cudaGetLastError();
}

cudaError_t launch_depthwise_tma_narrow(const DepthwisePlan& plan, const float* f, const float* bias, int act, void* y,
                                        bool y_is_bf16, const ConvGeom& g, unsigned int* dev_status, cudaStream_t s,
                                        int64_t* launches) {
    if (g.N * g.Ho * g.Wo * g.Co == 0) return cudaSuccess;
    if (plan.variant < DW_FIRST_NARROW || !plan.narrow) return cudaErrorInvalidValue;
    cudaError_t e = launch_tma_variant(plan, f, bias, act, y, !y_is_bf16, g, dev_status, s);
    ++*launches;
    return e;
}

}  // namespace tfjsb

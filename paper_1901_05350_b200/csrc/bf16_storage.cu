// CUDA-core kernels of the narrow-storage mode: activations are bfloat16 in memory (the 16-bit
// analogue of the paper's half-float textures, Sec. 4.1.3), every sum is fp32, and a result is rounded
// once (to nearest even) when it is stored.  Filters arrive as fp32 arrays whose values are already
// bfloat16 (rounded when the model is built); biases are plain fp32.
//
//   conv_direct_narrow_kernel       conv2d, any window / stride / dilation; reads fp32 (the model input,
//                                   rounded to bfloat16 as it is read) or bfloat16
//   depthwise3x3_narrow_kernel      3x3 depthwise, stride 1 or 2, 8 channels x 2 output rows per thread
//   avg_pool_global_narrow_kernel   mean over H x W
//   convert kernels                 fp32 <-> bfloat16 (weights at set-up, debug read-back)
#include <cuda_bf16.h>

#include "common.cuh"
#include "ptx_sm100.cuh"

namespace tfjsb {

using namespace ptx;

namespace {

// ---- storage helpers ----------------------------------------------------------------------------
// A bfloat16 is the upper half of the fp32 with the same value.
__device__ __forceinline__ float bf16_lo(uint32_t pair) { return __uint_as_float(pair << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t pair) { return __uint_as_float(pair & 0xffff0000u); }
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    const __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&h);
}
__device__ __forceinline__ float round_bf16(float v) { return __bfloat162float(__float2bfloat16_rn(v)); }

__device__ __forceinline__ void unpack8(const uint4& q, float (&v)[8]) {
    v[0] = bf16_lo(q.x); v[1] = bf16_hi(q.x); v[2] = bf16_lo(q.y); v[3] = bf16_hi(q.y);
    v[4] = bf16_lo(q.z); v[5] = bf16_hi(q.z); v[6] = bf16_lo(q.w); v[7] = bf16_hi(q.w);
}

template <typename T>
__device__ __forceinline__ float load_stored(const T* p);
template <>
__device__ __forceinline__ float load_stored<float>(const float* p) { return round_bf16(__ldg(p)); }
template <>
__device__ __forceinline__ float load_stored<__nv_bfloat16>(const __nv_bfloat16* p) {
    return __uint_as_float((uint32_t)__ldg(reinterpret_cast<const unsigned short*>(p)) << 16);
}

// Eight consecutive results of one pixel: bias, activation, store (narrow: one 16-byte store).
template <bool OUT_NARROW>
__device__ __forceinline__ void store8(void* y, int64_t elem, float (&v)[8], const float* __restrict__ bias, int act) {
#pragma unroll
    for (int e = 0; e < 8; ++e) v[e] = apply_act(bias ? v[e] + __ldg(bias + e) : v[e], act);
    if (OUT_NARROW) {
        uint4 q;
        q.x = pack_bf16(v[0], v[1]); q.y = pack_bf16(v[2], v[3]); q.z = pack_bf16(v[4], v[5]); q.w = pack_bf16(v[6], v[7]);
        *reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(y) + elem) = q;
    } else {
        float4* dst = reinterpret_cast<float4*>(static_cast<float*>(y) + elem);
        dst[0] = make_float4(v[0], v[1], v[2], v[3]);
        dst[1] = make_float4(v[4], v[5], v[6], v[7]);
    }
}

// ---- conv2d -------------------------------------------------------------------------------------
// One thread: one output pixel, eight consecutive output channels (fewer at a ragged end).  The
// threads of a pixel sit next to each other, so the input samples they share come from L1, and a
// warp's filter loads are a handful of distinct 32-byte pieces.
template <typename IN_T, bool OUT_NARROW>
__global__ void __launch_bounds__(256)
conv_direct_narrow_kernel(const IN_T* __restrict__ x, const float* __restrict__ f, const float* __restrict__ bias, int act,
                          void* __restrict__ y, const ConvGeom g, int groups, int64_t total) {
    pdl_launch_dependents();
    pdl_wait();
    const bool vec = (g.Co & 7) == 0;
    for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < total; t += (int64_t)gridDim.x * blockDim.x) {
        const int cg = (int)(t % groups);
        const int64_t p = t / groups;
        const int ox = (int)(p % g.Wo);
        const int oy = (int)((p / g.Wo) % g.Ho);
        const int64_t n = p / ((int64_t)g.Wo * g.Ho);
        const int c0 = cg * 8;
        float acc[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[e] = 0.0f;
        const IN_T* xn = x + n * (int64_t)g.H * g.W * g.C;
        for (int ky = 0; ky < g.fh; ++ky) {
            const int iy = oy * g.sh - g.pt + ky * g.dh;
            if (iy < 0 || iy >= g.H) continue;
            for (int kx = 0; kx < g.fw; ++kx) {
                const int ix = ox * g.sw - g.pl + kx * g.dw;
                if (ix < 0 || ix >= g.W) continue;
                const IN_T* xp = xn + ((int64_t)iy * g.W + ix) * g.C;
                const float* fp = f + ((int64_t)(ky * g.fw + kx) * g.C) * g.Co + c0;
                for (int ci = 0; ci < g.C; ++ci, fp += g.Co) {
                    const float xv = load_stored(xp + ci);
                    if (vec) {
                        const float4 w0 = __ldg(reinterpret_cast<const float4*>(fp));
                        const float4 w1 = __ldg(reinterpret_cast<const float4*>(fp + 4));
                        acc[0] = fmaf(xv, w0.x, acc[0]); acc[1] = fmaf(xv, w0.y, acc[1]);
                        acc[2] = fmaf(xv, w0.z, acc[2]); acc[3] = fmaf(xv, w0.w, acc[3]);
                        acc[4] = fmaf(xv, w1.x, acc[4]); acc[5] = fmaf(xv, w1.y, acc[5]);
                        acc[6] = fmaf(xv, w1.z, acc[6]); acc[7] = fmaf(xv, w1.w, acc[7]);
                    } else {
#pragma unroll
                        for (int e = 0; e < 8; ++e)
                            if (c0 + e < g.Co) acc[e] = fmaf(xv, __ldg(fp + e), acc[e]);
                    }
                }
            }
        }
        const int64_t elem = p * g.Co + c0;
        if (vec) {
            store8<OUT_NARROW>(y, elem, acc, bias ? bias + c0 : nullptr, act);
        } else {
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                if (c0 + e >= g.Co) continue;
                const float v = apply_act(bias ? acc[e] + __ldg(bias + c0 + e) : acc[e], act);
                if (OUT_NARROW) static_cast<__nv_bfloat16*>(y)[elem + e] = __float2bfloat16_rn(v);
                else static_cast<float*>(y)[elem + e] = v;
            }
        }
    }
}

// ---- 3x3 conv2d over a 3-channel fp32 image (the usual first layer) ---------------------------------
// One thread: one output pixel, all COUT (<= 32) output channels.  The 27 input samples are requested
// up front and rounded to bfloat16; the filter sits in shared memory as [27][COUT] and is read as
// 16-byte broadcasts; the 27 x COUT multiply-adds are issued two per instruction.
template <int COUT, bool OUT_NARROW>
__global__ void __launch_bounds__(128)
conv3x3_rgb_narrow_kernel(const float* __restrict__ x, const float* __restrict__ f, const float* __restrict__ bias, int act,
                          void* __restrict__ y, const ConvGeom g, int64_t total) {
    __shared__ __align__(16) float w_s[27 * COUT];
    __shared__ __align__(16) float b_s[COUT];
    for (int i = threadIdx.x; i < 27 * COUT; i += blockDim.x) w_s[i] = __ldg(f + i);  // set-up data, not the predecessor's
    for (int i = threadIdx.x; i < COUT; i += blockDim.x) b_s[i] = bias ? __ldg(bias + i) : 0.0f;
    __syncthreads();
    pdl_launch_dependents();
    pdl_wait();
    for (int64_t p = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; p < total; p += (int64_t)gridDim.x * blockDim.x) {
        const int ox = (int)(p % g.Wo);
        const int oy = (int)((p / g.Wo) % g.Ho);
        const int64_t n = p / ((int64_t)g.Wo * g.Ho);
        const float* xn = x + n * (int64_t)g.H * g.W * 3;
        const int iy0 = oy * g.sh - g.pt, ix0 = ox * g.sw - g.pl;
        float xv[27];
#pragma unroll
        for (int ky = 0; ky < 3; ++ky) {
            const int iy = iy0 + ky;
            const bool row_ok = iy >= 0 && iy < g.H;
#pragma unroll
            for (int kx = 0; kx < 3; ++kx) {
                const int ix = ix0 + kx;
                const bool ok = row_ok && ix >= 0 && ix < g.W;
                const float* xp = xn + ((int64_t)iy * g.W + ix) * 3;
#pragma unroll
                for (int ci = 0; ci < 3; ++ci) xv[(ky * 3 + kx) * 3 + ci] = ok ? __ldg(xp + ci) : 0.0f;
            }
        }
        float2 acc[COUT / 2];
#pragma unroll
        for (int c = 0; c < COUT / 2; ++c) acc[c] = make_float2(0.0f, 0.0f);
#pragma unroll
        for (int k = 0; k < 27; ++k) {
            const float v = round_bf16(xv[k]);
            const float2 vv = make_float2(v, v);
#pragma unroll
            for (int c = 0; c < COUT / 4; ++c) {
                const float4 w = *reinterpret_cast<const float4*>(&w_s[k * COUT + 4 * c]);
                fma2(acc[2 * c], vv, make_float2(w.x, w.y));
                fma2(acc[2 * c + 1], vv, make_float2(w.z, w.w));
            }
        }
#pragma unroll
        for (int c8 = 0; c8 < COUT / 8; ++c8) {
            float v[8];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                v[2 * e] = acc[c8 * 4 + e].x + b_s[c8 * 8 + 2 * e];
                v[2 * e + 1] = acc[c8 * 4 + e].y + b_s[c8 * 8 + 2 * e + 1];
            }
            store8<OUT_NARROW>(y, p * COUT + c8 * 8, v, nullptr, act);
        }
    }
}

// ---- depthwise 3x3 ------------------------------------------------------------------------------
// One thread: eight channels (one 16-byte load per input sample) of DW_ROWS consecutive output rows at
// one output column.  All of the thread's input samples are requested before the first is used: a
// thread is one round trip to memory long, not one per input row, and with a dozen 16-byte loads in
// flight per thread a dozen warps per SM keep enough bytes in flight to cover the memory latency.
// Each input row contributes to the (up to three) output rows whose windows contain it; the taps come
// from L1 (every thread of a channel group reads the same 72 values).
constexpr int DW_ROWS = 2;

template <int S, bool OUT_NARROW>
__global__ void __launch_bounds__(128)
depthwise3x3_narrow_kernel(const __nv_bfloat16* __restrict__ x, const float* __restrict__ f, const float* __restrict__ bias,
                           int act, void* __restrict__ y, const ConvGeom g, int row_blocks, int64_t total) {
    pdl_launch_dependents();
    pdl_wait();
    const int c8n = g.C >> 3;
    constexpr int IN_ROWS = (DW_ROWS - 1) * S + 3;
    for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < total; t += (int64_t)gridDim.x * blockDim.x) {
        const int c0 = (int)(t % c8n) * 8;
        int64_t r = t / c8n;
        const int ox = (int)(r % g.Wo);
        r /= g.Wo;
        const int oy0 = (int)(r % row_blocks) * DW_ROWS;
        const int64_t n = r / row_blocks;

        const __nv_bfloat16* xn = x + n * (int64_t)g.H * g.W * g.C + c0;
        const int iy_first = oy0 * S - g.pt;
        const int ix0 = ox * S - g.pl;
        uint4 raw[IN_ROWS][3];
#pragma unroll
        for (int ir = 0; ir < IN_ROWS; ++ir) {
            const int iy = iy_first + ir;
            const bool row_ok = iy >= 0 && iy < g.H;
#pragma unroll
            for (int kx = 0; kx < 3; ++kx) {
                const int ix = ix0 + kx;
                raw[ir][kx] = make_uint4(0u, 0u, 0u, 0u);
                if (row_ok && ix >= 0 && ix < g.W)
                    raw[ir][kx] = __ldg(reinterpret_cast<const uint4*>(xn + ((int64_t)iy * g.W + ix) * g.C));
            }
        }
        float acc[DW_ROWS][8];
#pragma unroll
        for (int o = 0; o < DW_ROWS; ++o)
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[o][e] = 0.0f;
#pragma unroll
        for (int kx = 0; kx < 3; ++kx) {
#pragma unroll
            for (int ky = 0; ky < 3; ++ky) {
                float w[8];
                const float4 wa = __ldg(reinterpret_cast<const float4*>(f + (int64_t)(ky * 3 + kx) * g.C + c0));
                const float4 wb = __ldg(reinterpret_cast<const float4*>(f + (int64_t)(ky * 3 + kx) * g.C + c0 + 4));
                w[0] = wa.x; w[1] = wa.y; w[2] = wa.z; w[3] = wa.w; w[4] = wb.x; w[5] = wb.y; w[6] = wb.z; w[7] = wb.w;
#pragma unroll
                for (int o = 0; o < DW_ROWS; ++o) {
                    float v[8];
                    unpack8(raw[o * S + ky][kx], v);
#pragma unroll
                    for (int e = 0; e < 8; ++e) acc[o][e] = fmaf(v[e], w[e], acc[o][e]);
                }
            }
        }
#pragma unroll
        for (int o = 0; o < DW_ROWS; ++o) {
            const int oy = oy0 + o;
            if (oy >= g.Ho) break;
            const int64_t elem = ((n * g.Ho + oy) * (int64_t)g.Wo + ox) * g.C + c0;
            store8<OUT_NARROW>(y, elem, acc[o], bias ? bias + c0 : nullptr, act);
        }
    }
}

// ---- global average pool ------------------------------------------------------------------------
// One thread: eight channels of one image; the positions are summed in order in fp32 and divided by
// their number.
template <bool OUT_NARROW>
__global__ void __launch_bounds__(128)
avg_pool_global_narrow_kernel(const __nv_bfloat16* __restrict__ x, void* __restrict__ y, int64_t images, int positions, int C) {
    pdl_launch_dependents();
    pdl_wait();
    const int c8n = C >> 3;
    const int64_t total = images * c8n;
    for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < total; t += (int64_t)gridDim.x * blockDim.x) {
        const int c0 = (int)(t % c8n) * 8;
        const int64_t n = t / c8n;
        const __nv_bfloat16* xp = x + n * (int64_t)positions * C + c0;
        float acc[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[e] = 0.0f;
        for (int p = 0; p < positions; ++p) {
            float v[8];
            unpack8(__ldg(reinterpret_cast<const uint4*>(xp + (int64_t)p * C)), v);
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[e] += v[e];
        }
        const float count = (float)positions;
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[e] = __fdiv_rn(acc[e], count);
        store8<OUT_NARROW>(y, n * C + c0, acc, nullptr, TFJSB_ACT_NONE);
    }
}

// ---- conversions ---------------------------------------------------------------------------------
__global__ void f32_to_bf16_kernel(const float* __restrict__ in, __nv_bfloat16* __restrict__ out, int64_t n) {
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x)
        out[i] = __float2bfloat16_rn(in[i]);
}
__global__ void bf16_to_f32_kernel(const __nv_bfloat16* __restrict__ in, float* __restrict__ out, int64_t n) {
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x)
        out[i] = __bfloat162float(in[i]);
}
__global__ void round_to_bf16_in_place_kernel(float* __restrict__ v, int64_t n) {
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x)
        v[i] = round_bf16(v[i]);
}

// out [r*N, r*K]: r copies of km [N, K] down the diagonal, zeros elsewhere
__global__ void block_diagonal_kernel(const float* __restrict__ km, float* __restrict__ out, int64_t N, int64_t K, int r) {
    const int64_t cols = (int64_t)r * K, total = (int64_t)r * N * cols;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t row = i / cols, col = i - row * cols;
        const int64_t j = row / N, n = row - j * N;
        out[i] = (col / K == j) ? km[n * K + (col - j * K)] : 0.0f;
    }
}

int grid_for(int64_t threads, int block) {
    const int64_t blocks = (threads + block - 1) / block;
    const int64_t cap = 148LL * 64;
    return (int)(blocks < 1 ? 1 : (blocks > cap ? cap : blocks));
}

template <int COUT>
cudaError_t launch_rgb(const float* x, const float* f, const float* bias, int act, void* y, bool y_is_bf16, const ConvGeom& g,
                       cudaStream_t s) {
    const int64_t total = g.N * g.Ho * g.Wo;
    const dim3 grid(grid_for(total, 128)), block(128);
    return y_is_bf16 ? launch_k(conv3x3_rgb_narrow_kernel<COUT, true>, grid, block, 0, s, x, f, bias, act, y, g, total)
                     : launch_k(conv3x3_rgb_narrow_kernel<COUT, false>, grid, block, 0, s, x, f, bias, act, y, g, total);
}

}  // namespace

cudaError_t launch_conv_narrow(const void* x, bool x_is_f32, const float* f, const float* bias, int act, void* y,
                               bool y_is_bf16, const ConvGeom& g, cudaStream_t s, int64_t* launches) {
    if (x_is_f32 && g.fh == 3 && g.fw == 3 && g.C == 3 && g.dh == 1 && g.dw == 1 && g.Co <= 32 && (g.Co % 8) == 0) {
        const float* xf = static_cast<const float*>(x);
        cudaError_t e = g.Co == 32 ? launch_rgb<32>(xf, f, bias, act, y, y_is_bf16, g, s)
                        : g.Co == 24 ? launch_rgb<24>(xf, f, bias, act, y, y_is_bf16, g, s)
                        : g.Co == 16 ? launch_rgb<16>(xf, f, bias, act, y, y_is_bf16, g, s)
                                     : launch_rgb<8>(xf, f, bias, act, y, y_is_bf16, g, s);
        ++*launches;
        return e;
    }
    const int groups = (g.Co + 7) / 8;
    const int64_t total = g.N * g.Ho * g.Wo * groups;
    const dim3 grid(grid_for(total, 256)), block(256);
    cudaError_t e;
    if (x_is_f32) {
        const float* xf = static_cast<const float*>(x);
        e = y_is_bf16 ? launch_k(conv_direct_narrow_kernel<float, true>, grid, block, 0, s, xf, f, bias, act, y, g, groups, total)
                      : launch_k(conv_direct_narrow_kernel<float, false>, grid, block, 0, s, xf, f, bias, act, y, g, groups, total);
    } else {
        const __nv_bfloat16* xh = static_cast<const __nv_bfloat16*>(x);
        e = y_is_bf16 ? launch_k(conv_direct_narrow_kernel<__nv_bfloat16, true>, grid, block, 0, s, xh, f, bias, act, y, g, groups, total)
                      : launch_k(conv_direct_narrow_kernel<__nv_bfloat16, false>, grid, block, 0, s, xh, f, bias, act, y, g, groups, total);
    }
    ++*launches;
    return e;
}

bool depthwise_narrow_supported(const ConvGeom& g) {
    return g.fh == 3 && g.fw == 3 && g.mult == 1 && g.dh == 1 && g.dw == 1 && g.sh == g.sw && (g.sh == 1 || g.sh == 2) &&
           (g.C % 8) == 0;
}

cudaError_t launch_depthwise_narrow(const void* x, const float* f, const float* bias, int act, void* y, bool y_is_bf16,
                                    const ConvGeom& g, cudaStream_t s, int64_t* launches) {
    const int row_blocks = (g.Ho + DW_ROWS - 1) / DW_ROWS;
    const int64_t total = g.N * row_blocks * g.Wo * (g.C / 8);
    const dim3 grid(grid_for(total, 128)), block(128);
    const __nv_bfloat16* xh = static_cast<const __nv_bfloat16*>(x);
    cudaError_t e;
    if (g.sh == 1)
        e = y_is_bf16 ? launch_k(depthwise3x3_narrow_kernel<1, true>, grid, block, 0, s, xh, f, bias, act, y, g, row_blocks, total)
                      : launch_k(depthwise3x3_narrow_kernel<1, false>, grid, block, 0, s, xh, f, bias, act, y, g, row_blocks, total);
    else
        e = y_is_bf16 ? launch_k(depthwise3x3_narrow_kernel<2, true>, grid, block, 0, s, xh, f, bias, act, y, g, row_blocks, total)
                      : launch_k(depthwise3x3_narrow_kernel<2, false>, grid, block, 0, s, xh, f, bias, act, y, g, row_blocks, total);
    ++*launches;
    return e;
}

cudaError_t launch_avg_pool_global_narrow(const void* x, void* y, bool y_is_bf16, int64_t images, int positions, int C,
                                          cudaStream_t s, int64_t* launches) {
    const int64_t total = images * (C / 8);
    const dim3 grid(grid_for(total, 128)), block(128);
    const __nv_bfloat16* xh = static_cast<const __nv_bfloat16*>(x);
    cudaError_t e = y_is_bf16 ? launch_k(avg_pool_global_narrow_kernel<true>, grid, block, 0, s, xh, y, images, positions, C)
                              : launch_k(avg_pool_global_narrow_kernel<false>, grid, block, 0, s, xh, y, images, positions, C);
    ++*launches;
    return e;
}

cudaError_t launch_f32_to_bf16(const float* in, void* out, int64_t n, cudaStream_t s, int64_t* launches) {
    f32_to_bf16_kernel<<<grid_for(n, 256), 256, 0, s>>>(in, static_cast<__nv_bfloat16*>(out), n);
    ++*launches;
    return cudaGetLastError();
}
cudaError_t launch_bf16_to_f32(const void* in, float* out, int64_t n, cudaStream_t s, int64_t* launches) {
    bf16_to_f32_kernel<<<grid_for(n, 256), 256, 0, s>>>(static_cast<const __nv_bfloat16*>(in), out, n);
    ++*launches;
    return cudaGetLastError();
}
cudaError_t launch_block_diagonal(const float* km, float* out, int64_t N, int64_t K, int r, cudaStream_t s, int64_t* launches) {
    block_diagonal_kernel<<<grid_for((int64_t)r * N * r * K, 256), 256, 0, s>>>(km, out, N, K, r);
    ++*launches;
    return cudaGetLastError();
}
cudaError_t launch_round_to_bf16_in_place(float* v, int64_t n, cudaStream_t s, int64_t* launches) {
    round_to_bf16_in_place_kernel<<<grid_for(n, 256), 256, 0, s>>>(v, n);
    ++*launches;
    return cudaGetLastError();
}

}  // namespace tfjsb

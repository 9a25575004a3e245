// CUDA-core kernels of the narrow-storage mode: activations are bfloat16 in memory (the 16-bit
// analogue of the paper's half-float textures, Sec. 4.1.3), every sum is fp32, and a result is rounded
// once (to nearest even) when it is stored.  Filters arrive as fp32 arrays whose values are already
// bfloat16 (rounded when the model is built); biases are plain fp32.
//
//   conv_direct_narrow_kernel       conv2d, any window / stride / dilation; reads fp32 (the model input,
//                                   rounded to bfloat16 as it is read) or bfloat16
//   depthwise3x3_narrow_kernel      3x3 depthwise, stride 1 or 2, 8 channels x a 2x2 / 1x2 block of pixels per thread
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
// One thread: two output pixels (128 pixels apart, so that a warp's loads and stores stay dense), all
// COUT (<= 32) output channels of each.  The kernel is bound by the L1 / shared-memory pipe, so it
// spends as few of that pipe's cycles as it can: the filter sits in shared memory as [27][COUT] and
// each 16-byte broadcast read of it feeds both pixels; the 27 input samples of a pixel (three runs of
// nine consecutive floats) are fetched row by row, as 8-byte loads where the run is aligned and inside
// the image.
// Samples are rounded to bfloat16 as they are used; multiply-adds go two per instruction.
// Where one output pixel's 3 x 3 window starts, and how its rows may be fetched.
struct RgbWindow {
    const float* origin;  // sample (iy0, ix0, channel 0) of the pixel's image; may lie outside the image
    int iy0, ix0;
    bool live, fast;
};
__device__ __forceinline__ RgbWindow rgb_window(const float* __restrict__ x, const ConvGeom& g, int64_t p, bool live) {
    RgbWindow w;
    w.live = live;
    const int64_t q = live ? p : 0;
    const int ox = (int)(q % g.Wo);
    const int oy = (int)((q / g.Wo) % g.Ho);
    const int64_t n = q / ((int64_t)g.Wo * g.Ho);
    w.iy0 = oy * g.sh - g.pt;
    w.ix0 = ox * g.sw - g.pl;
    w.origin = x + (n * (int64_t)g.H * g.W + (int64_t)w.iy0 * g.W + w.ix0) * 3;
    // a row's nine floats start on an 8-byte boundary when (iy * W + ix0) * 3 is even
    w.fast = w.ix0 >= 0 && w.ix0 + 2 < g.W && (g.W & 1) == 0 && (w.ix0 & 1) == 0;
    return w;
}
// The nine samples (three pixels x three channels) of window row ky; zeros outside the image.
__device__ __forceinline__ void load_rgb_row(const RgbWindow& w, const ConvGeom& g, int ky, float (&v)[9]) {
#pragma unroll
    for (int k = 0; k < 9; ++k) v[k] = 0.0f;
    const int iy = w.iy0 + ky;
    if (!w.live || iy < 0 || iy >= g.H) return;
    const float* rp = w.origin + (int64_t)ky * g.W * 3;
    if (w.fast) {
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const float2 t = __ldg(reinterpret_cast<const float2*>(rp) + q);
            v[2 * q] = t.x;
            v[2 * q + 1] = t.y;
        }
        v[8] = __ldg(rp + 8);
    } else {
#pragma unroll
        for (int kx = 0; kx < 3; ++kx) {
            const int ix = w.ix0 + kx;
            if (ix < 0 || ix >= g.W) continue;
#pragma unroll
            for (int ci = 0; ci < 3; ++ci) v[kx * 3 + ci] = __ldg(rp + kx * 3 + ci);
        }
    }
}

template <int COUT, int ACT, bool OUT_NARROW>
__global__ void __launch_bounds__(128, 4)
conv3x3_rgb_narrow_kernel(const float* __restrict__ x, const float* __restrict__ f, const float* __restrict__ bias,
                          void* __restrict__ y, const ConvGeom g, int64_t total) {
    __shared__ __align__(16) float w_s[27 * COUT];
    __shared__ __align__(16) float b_s[COUT];
    for (int i = threadIdx.x; i < 27 * COUT; i += blockDim.x) w_s[i] = __ldg(f + i);  // set-up data, not the predecessor's
    for (int i = threadIdx.x; i < COUT; i += blockDim.x) b_s[i] = bias ? __ldg(bias + i) : 0.0f;
    __syncthreads();
    pdl_launch_dependents();
    pdl_wait();
    for (int64_t base = (int64_t)blockIdx.x * 256; base < total; base += (int64_t)gridDim.x * 256) {
        const int64_t p0 = base + threadIdx.x, p1 = p0 + 128;
        const RgbWindow wa = rgb_window(x, g, p0, p0 < total), wb = rgb_window(x, g, p1, p1 < total);
        float2 acc0[COUT / 2], acc1[COUT / 2];
#pragma unroll
        for (int c = 0; c < COUT / 2; ++c) acc0[c] = acc1[c] = make_float2(0.0f, 0.0f);
        // one window row at a time: eighteen samples in flight per thread, few enough registers for
        // four blocks per SM
#pragma unroll
        for (int ky = 0; ky < 3; ++ky) {
            float xa[9], xb[9];
            load_rgb_row(wa, g, ky, xa);
            load_rgb_row(wb, g, ky, xb);
#pragma unroll
            for (int k = 0; k < 9; ++k) {
                const float va = round_bf16(xa[k]), vb = round_bf16(xb[k]);
                const float2 a2 = make_float2(va, va), b2 = make_float2(vb, vb);
#pragma unroll
                for (int c = 0; c < COUT / 4; ++c) {
                    const float4 w = *reinterpret_cast<const float4*>(&w_s[(ky * 9 + k) * COUT + 4 * c]);
                    const float2 wl = make_float2(w.x, w.y), wh = make_float2(w.z, w.w);
                    fma2(acc0[2 * c], a2, wl);
                    fma2(acc0[2 * c + 1], a2, wh);
                    fma2(acc1[2 * c], b2, wl);
                    fma2(acc1[2 * c + 1], b2, wh);
                }
            }
        }
#pragma unroll
        for (int c8 = 0; c8 < COUT / 8; ++c8) {
            const float4 ba = *reinterpret_cast<const float4*>(&b_s[c8 * 8]);
            const float4 bb = *reinterpret_cast<const float4*>(&b_s[c8 * 8 + 4]);
            const float b8[8] = {ba.x, ba.y, ba.z, ba.w, bb.x, bb.y, bb.z, bb.w};
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                const int64_t p = half ? p1 : p0;
                if (p >= total) continue;
                float v[8];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float2 a = half ? acc1[c8 * 4 + e] : acc0[c8 * 4 + e];
                    v[2 * e] = apply_act_t<ACT>(a.x + b8[2 * e]);
                    v[2 * e + 1] = apply_act_t<ACT>(a.y + b8[2 * e + 1]);
                }
                const int64_t elem = p * COUT + c8 * 8;
                if (OUT_NARROW) {
                    uint4 o;
                    o.x = pack_bf16(v[0], v[1]); o.y = pack_bf16(v[2], v[3]); o.z = pack_bf16(v[4], v[5]); o.w = pack_bf16(v[6], v[7]);
                    *reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(y) + elem) = o;
                } else {
                    float4* dst = reinterpret_cast<float4*>(static_cast<float*>(y) + elem);
                    dst[0] = make_float4(v[0], v[1], v[2], v[3]);
                    dst[1] = make_float4(v[4], v[5], v[6], v[7]);
                }
            }
        }
    }
}

// ---- depthwise 3x3 ------------------------------------------------------------------------------
// One thread: eight channels (one 16-byte load per input sample) of a TR x TC block of output pixels.
// The kernel is bound by instruction issue, not by memory, so the design minimises instructions per
// output: the block's input samples ((TR-1)S+3 rows x (TC-1)S+3 columns) are each loaded and widened to
// fp32 once and used by every output whose window contains them; multiply-adds go two per instruction;
// indices are 32-bit.  All loads are requested before the first is used, so a thread is one round
// trip to memory long.  Taps come from L1 (every thread of a channel group reads the same 72 values).
template <int S, int TR, int TC, int ACT, bool OUT_NARROW>
__global__ void __launch_bounds__(128)
depthwise3x3_narrow_kernel(const __nv_bfloat16* __restrict__ x, const float* __restrict__ f, const float* __restrict__ bias,
                           void* __restrict__ y, const ConvGeom g, int row_blocks, int col_blocks, uint32_t total) {
    pdl_launch_dependents();
    pdl_wait();
    const uint32_t c8n = (uint32_t)g.C >> 3;  // 16-byte pieces per pixel
    constexpr int IN_ROWS = (TR - 1) * S + 3, IN_COLS = (TC - 1) * S + 3;
    for (uint32_t t = blockIdx.x * blockDim.x + threadIdx.x; t < total; t += gridDim.x * blockDim.x) {
        uint32_t r = t / c8n;
        const uint32_t cg = t - r * c8n;
        uint32_t q = r / (uint32_t)col_blocks;
        const int ox0 = (int)(r - q * (uint32_t)col_blocks) * TC;
        const uint32_t n = q / (uint32_t)row_blocks;
        const int oy0 = (int)(q - n * (uint32_t)row_blocks) * TR;

        // 16-byte pieces of this image, this channel group: piece (iy * W + ix) * c8n
        const uint4* xn = reinterpret_cast<const uint4*>(x) + ((int64_t)n * g.H * g.W * c8n + cg);
        const int iy_first = oy0 * S - g.pt;
        const int ix_first = ox0 * S - g.pl;
        uint4 raw[IN_ROWS][IN_COLS];
        if (iy_first >= 0 && iy_first + IN_ROWS <= g.H && ix_first >= 0 && ix_first + IN_COLS <= g.W) {
            // the whole window lies inside the image (most blocks): one base address, constant strides
            const uint4* x0 = xn + (iy_first * g.W + ix_first) * (int)c8n;
            const int row_pitch = g.W * (int)c8n;
#pragma unroll
            for (int ir = 0; ir < IN_ROWS; ++ir)
#pragma unroll
                for (int ic = 0; ic < IN_COLS; ++ic) raw[ir][ic] = __ldg(x0 + ir * row_pitch + ic * (int)c8n);
        } else {
            int col_off[IN_COLS];
            bool col_ok[IN_COLS];
#pragma unroll
            for (int ic = 0; ic < IN_COLS; ++ic) {
                const int ix = ix_first + ic;
                col_ok[ic] = ix >= 0 && ix < g.W;
                col_off[ic] = ix * (int)c8n;
            }
#pragma unroll
            for (int ir = 0; ir < IN_ROWS; ++ir) {
                const int iy = iy_first + ir;
                const bool row_ok = iy >= 0 && iy < g.H;
                const uint4* xr = xn + iy * g.W * (int)c8n;
#pragma unroll
                for (int ic = 0; ic < IN_COLS; ++ic) {
                    raw[ir][ic] = make_uint4(0u, 0u, 0u, 0u);
                    if (row_ok && col_ok[ic]) raw[ir][ic] = __ldg(xr + col_off[ic]);
                }
            }
        }
        const float4* fq = reinterpret_cast<const float4*>(f) + 2 * cg;  // tap k: pieces k * (C / 4) + {0, 1}
        float2 w[9][4];
#pragma unroll
        for (int k = 0; k < 9; ++k) {
            const float4 wa = __ldg(fq + k * 2 * (int)c8n);
            const float4 wb = __ldg(fq + k * 2 * (int)c8n + 1);
            w[k][0] = make_float2(wa.x, wa.y); w[k][1] = make_float2(wa.z, wa.w);
            w[k][2] = make_float2(wb.x, wb.y); w[k][3] = make_float2(wb.z, wb.w);
        }
        // the accumulators start from the bias
        float2 b2[4];
        if (bias != nullptr) {
            const float4 ba = __ldg(reinterpret_cast<const float4*>(bias) + 2 * cg);
            const float4 bb = __ldg(reinterpret_cast<const float4*>(bias) + 2 * cg + 1);
            b2[0] = make_float2(ba.x, ba.y); b2[1] = make_float2(ba.z, ba.w);
            b2[2] = make_float2(bb.x, bb.y); b2[3] = make_float2(bb.z, bb.w);
        } else {
#pragma unroll
            for (int e = 0; e < 4; ++e) b2[e] = make_float2(0.0f, 0.0f);
        }
        float2 acc[TR][TC][4];
#pragma unroll
        for (int a = 0; a < TR; ++a)
#pragma unroll
            for (int b = 0; b < TC; ++b)
#pragma unroll
                for (int e = 0; e < 4; ++e) acc[a][b][e] = make_float2(0.0f, 0.0f);
#pragma unroll
        for (int ir = 0; ir < IN_ROWS; ++ir) {
#pragma unroll
            for (int ic = 0; ic < IN_COLS; ++ic) {
                float2 v[4];
                v[0] = make_float2(bf16_lo(raw[ir][ic].x), bf16_hi(raw[ir][ic].x));
                v[1] = make_float2(bf16_lo(raw[ir][ic].y), bf16_hi(raw[ir][ic].y));
                v[2] = make_float2(bf16_lo(raw[ir][ic].z), bf16_hi(raw[ir][ic].z));
                v[3] = make_float2(bf16_lo(raw[ir][ic].w), bf16_hi(raw[ir][ic].w));
#pragma unroll
                for (int a = 0; a < TR; ++a) {
                    const int ky = ir - a * S;  // all compile-time after unrolling
                    if (ky < 0 || ky > 2) continue;
#pragma unroll
                    for (int b = 0; b < TC; ++b) {
                        const int kx = ic - b * S;
                        if (kx < 0 || kx > 2) continue;
#pragma unroll
                        for (int e = 0; e < 4; ++e) fma2(acc[a][b][e], v[e], w[ky * 3 + kx][e]);
                    }
                }
            }
        }
#pragma unroll
        for (int a = 0; a < TR; ++a) {
            const int oy = oy0 + a;
            if (oy >= g.Ho) break;
#pragma unroll
            for (int b = 0; b < TC; ++b) {
                const int ox = ox0 + b;
                if (ox >= g.Wo) break;
                float v[8];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    // the sum of the products first, then one addition of the bias, as everywhere
                    v[2 * e] = apply_act_t<ACT>(acc[a][b][e].x + b2[e].x);
                    v[2 * e + 1] = apply_act_t<ACT>(acc[a][b][e].y + b2[e].y);
                }
                const int64_t piece = (((int64_t)n * g.Ho + oy) * g.Wo + ox) * c8n + cg;
                if (OUT_NARROW) {
                    uint4 o;
                    o.x = pack_bf16(v[0], v[1]); o.y = pack_bf16(v[2], v[3]); o.z = pack_bf16(v[4], v[5]); o.w = pack_bf16(v[6], v[7]);
                    static_cast<uint4*>(y)[piece] = o;
                } else {
                    float4* dst = static_cast<float4*>(y) + 2 * piece;
                    dst[0] = make_float4(v[0], v[1], v[2], v[3]);
                    dst[1] = make_float4(v[4], v[5], v[6], v[7]);
                }
            }
        }
    }
}

// ---- global average pool ------------------------------------------------------------------------
// Eight lanes share eight channels of one image: lane j sums positions j, j + 8, ... in fp32, the
// partial sums meet in a butterfly over the eight lanes, and lane 0 divides by the number of positions
// and stores.  (One thread per channel group left most of the chip idle: 128 images x 128 groups.)
template <bool OUT_NARROW>
__global__ void __launch_bounds__(256)
avg_pool_global_narrow_kernel(const __nv_bfloat16* __restrict__ x, void* __restrict__ y, int64_t images, int positions, int C) {
    pdl_launch_dependents();
    pdl_wait();
    const int c8n = C >> 3;
    const int64_t total = images * c8n * 8;  // a multiple of 8: the eight lanes of a group stay together
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    const int lane = threadIdx.x & 31;
    // whole warps enter the loop body together (the butterfly needs all 32 lanes); lanes past the end idle
    for (int64_t base = (int64_t)blockIdx.x * blockDim.x + (threadIdx.x - lane); base < total; base += stride) {
        const int64_t t = base + lane;
        const bool live = t < total;
        const int part = (int)(t & 7);
        const int64_t grp = live ? (t >> 3) : 0;
        const int c0 = (int)(grp % c8n) * 8;
        const int64_t n = grp / c8n;
        const __nv_bfloat16* xp = x + n * (int64_t)positions * C + c0;
        float acc[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[e] = 0.0f;
        for (int p = part; live && p < positions; p += 8) {
            float v[8];
            unpack8(__ldg(reinterpret_cast<const uint4*>(xp + (int64_t)p * C)), v);
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[e] += v[e];
        }
#pragma unroll
        for (int m = 1; m < 8; m <<= 1)
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[e] += __shfl_xor_sync(0xffffffffu, acc[e], m);
        if (live && part == 0) {
            const float count = (float)positions;
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[e] = __fdiv_rn(acc[e], count);
            store8<OUT_NARROW>(y, n * C + c0, acc, nullptr, TFJSB_ACT_NONE);
        }
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
    const int64_t cap = (int64_t)current_sm_count() * 64;
    return (int)(blocks < 1 ? 1 : (blocks > cap ? cap : blocks));
}

template <int COUT, int ACT>
cudaError_t launch_rgb_act(const float* x, const float* f, const float* bias, void* y, bool y_is_bf16, const ConvGeom& g,
                           cudaStream_t s) {
    const int64_t total = g.N * g.Ho * g.Wo;
    const dim3 grid(grid_for(total, 256)), block(128);  // 256 pixels per block and pass
    return y_is_bf16 ? launch_k_serial(conv3x3_rgb_narrow_kernel<COUT, ACT, true>, grid, block, 0, s, x, f, bias, y, g, total)
                     : launch_k_serial(conv3x3_rgb_narrow_kernel<COUT, ACT, false>, grid, block, 0, s, x, f, bias, y, g, total);
}
template <int COUT>
cudaError_t launch_rgb(const float* x, const float* f, const float* bias, int act, void* y, bool y_is_bf16, const ConvGeom& g,
                       cudaStream_t s) {
    if (act == TFJSB_ACT_RELU6) return launch_rgb_act<COUT, TFJSB_ACT_RELU6>(x, f, bias, y, y_is_bf16, g, s);
    if (act == TFJSB_ACT_RELU) return launch_rgb_act<COUT, TFJSB_ACT_RELU>(x, f, bias, y, y_is_bf16, g, s);
    return launch_rgb_act<COUT, TFJSB_ACT_NONE>(x, f, bias, y, y_is_bf16, g, s);
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
        e = y_is_bf16 ? launch_k_serial(conv_direct_narrow_kernel<float, true>, grid, block, 0, s, xf, f, bias, act, y, g, groups, total)
                      : launch_k_serial(conv_direct_narrow_kernel<float, false>, grid, block, 0, s, xf, f, bias, act, y, g, groups, total);
    } else {
        const __nv_bfloat16* xh = static_cast<const __nv_bfloat16*>(x);
        e = y_is_bf16 ? launch_k_serial(conv_direct_narrow_kernel<__nv_bfloat16, true>, grid, block, 0, s, xh, f, bias, act, y, g, groups, total)
                      : launch_k_serial(conv_direct_narrow_kernel<__nv_bfloat16, false>, grid, block, 0, s, xh, f, bias, act, y, g, groups, total);
    }
    ++*launches;
    return e;
}

bool depthwise_narrow_supported(const ConvGeom& g) {
    return g.fh == 3 && g.fw == 3 && g.mult == 1 && g.dh == 1 && g.dw == 1 && g.sh == g.sw && (g.sh == 1 || g.sh == 2) &&
           (g.C % 8) == 0 && g.N * g.Ho * g.Wo * (g.C / 8) < (1LL << 31) && (int64_t)g.H * g.W * g.C < (1LL << 31);
}

namespace {
template <int S, int TR, int TC, int ACT>
cudaError_t launch_dw_act(const __nv_bfloat16* x, const float* f, const float* bias, void* y, bool y_is_bf16,
                          const ConvGeom& g, cudaStream_t s) {
    const int row_blocks = (g.Ho + TR - 1) / TR, col_blocks = (g.Wo + TC - 1) / TC;
    const uint32_t total = (uint32_t)(g.N * row_blocks * col_blocks * (g.C / 8));
    const dim3 grid(grid_for(total, 128)), block(128);
    return y_is_bf16 ? launch_k_serial(depthwise3x3_narrow_kernel<S, TR, TC, ACT, true>, grid, block, 0, s, x, f, bias, y, g,
                                row_blocks, col_blocks, total)
                     : launch_k_serial(depthwise3x3_narrow_kernel<S, TR, TC, ACT, false>, grid, block, 0, s, x, f, bias, y, g,
                                row_blocks, col_blocks, total);
}
template <int S, int TR, int TC>
cudaError_t launch_dw(const __nv_bfloat16* x, const float* f, const float* bias, int act, void* y, bool y_is_bf16,
                      const ConvGeom& g, cudaStream_t s) {
    if (act == TFJSB_ACT_RELU6) return launch_dw_act<S, TR, TC, TFJSB_ACT_RELU6>(x, f, bias, y, y_is_bf16, g, s);
    if (act == TFJSB_ACT_RELU) return launch_dw_act<S, TR, TC, TFJSB_ACT_RELU>(x, f, bias, y, y_is_bf16, g, s);
    return launch_dw_act<S, TR, TC, TFJSB_ACT_NONE>(x, f, bias, y, y_is_bf16, g, s);
}
}  // namespace

cudaError_t launch_depthwise_narrow(const void* x, const float* f, const float* bias, int act, void* y, bool y_is_bf16,
                                    const ConvGeom& g, cudaStream_t s, int64_t* launches) {
    const __nv_bfloat16* xh = static_cast<const __nv_bfloat16*>(x);
    // stride 1: 2 x 2 outputs from 4 x 4 samples; stride 2: 1 x 2 outputs from 3 x 5 samples
    cudaError_t e = g.sh == 1 ? launch_dw<1, 2, 2>(xh, f, bias, act, y, y_is_bf16, g, s)
                              : launch_dw<2, 1, 2>(xh, f, bias, act, y, y_is_bf16, g, s);
    ++*launches;
    return e;
}

cudaError_t launch_avg_pool_global_narrow(const void* x, void* y, bool y_is_bf16, int64_t images, int positions, int C,
                                          cudaStream_t s, int64_t* launches) {
    const int64_t total = images * (C / 8) * 8;
    const dim3 grid(grid_for(total, 256)), block(256);
    const __nv_bfloat16* xh = static_cast<const __nv_bfloat16*>(x);
    cudaError_t e = y_is_bf16 ? launch_k_serial(avg_pool_global_narrow_kernel<true>, grid, block, 0, s, xh, y, images, positions, C)
                              : launch_k_serial(avg_pool_global_narrow_kernel<false>, grid, block, 0, s, xh, y, images, positions, C);
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

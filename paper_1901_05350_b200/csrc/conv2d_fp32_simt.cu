// Direct NHWC convolution on CUDA cores with the fused bias + activation epilogue.
//
// Serves every conv2d that is not a 1x1/stride-1 GEMM: any window, stride, dilation, channel
// count (the 3-channel stem of the MobileNet configs in particular, whose 12-byte pixel pitch
// no bulk tensor copy can address).  Plain FFMA, fp32 accumulation in (ky, kx, ci) order.
//
// A 128-thread block owns 128 consecutive output pixels (flattened n, oy, ox) and a chunk of
// 32 output channels.  The filter is walked in slices of 64 rows of the implicit
// [fh*fw*Cin, Cout] matrix, each slice staged in shared memory and read back as broadcast
// float4s; every thread keeps its pixel's 32 accumulators in registers.  Results go through a
// padded shared-memory tile so the global store is coalesced along the channel dimension.
#include "common.cuh"

namespace tfjsb {

namespace {

constexpr int PIX = 128;  // output pixels per block = threads per block
constexpr int CO_T = 32;  // output channels per block
constexpr int KC = 64;    // filter rows per shared-memory slice

__global__ void __launch_bounds__(PIX)
conv2d_fp32_kernel(const float* __restrict__ x, const float* __restrict__ f, const float* __restrict__ bias, int act,
                   float* __restrict__ y, ConvGeom g, int64_t total_pix) {
    __shared__ __align__(16) float fs[KC][CO_T];
    __shared__ float ys[PIX][CO_T + 1];

    const int tid = threadIdx.x;
    const int64_t pix0 = (int64_t)blockIdx.x * PIX;
    const int co0 = blockIdx.y * CO_T;
    const int64_t p = pix0 + tid;
    const bool live = p < total_pix;

    int oy = 0, ox = 0;
    int64_t n = 0;
    if (live) {
        ox = (int)(p % g.Wo);
        const int64_t t = p / g.Wo;
        oy = (int)(t % g.Ho);
        n = t / g.Ho;
    }
    const int iy0 = oy * g.sh - g.pt, ix0 = ox * g.sw - g.pl;
    const float* xn = x + n * (int64_t)g.H * g.W * g.C;

    float acc[CO_T];
#pragma unroll
    for (int j = 0; j < CO_T; ++j) acc[j] = 0.0f;

    const int k_total = g.fh * g.fw * g.C;
    // (ky, kx, ci) of filter row k, advanced incrementally
    int ky = 0, kx = 0, ci = 0;
    for (int k0 = 0; k0 < k_total; k0 += KC) {
        for (int idx = tid; idx < KC * CO_T; idx += PIX) {
            const int kk = idx / CO_T, co = idx % CO_T;
            const int k = k0 + kk;
            fs[kk][co] = (k < k_total && co0 + co < g.Co) ? f[(int64_t)k * g.Co + co0 + co] : 0.0f;
        }
        __syncthreads();
        const int k_end = (k_total - k0 < KC) ? (k_total - k0) : KC;
        for (int kk = 0; kk < k_end; ++kk) {
            const int iy = iy0 + ky * g.dh, ix = ix0 + kx * g.dw;
            float xv = 0.0f;
            if (live && iy >= 0 && iy < g.H && ix >= 0 && ix < g.W) xv = xn[((int64_t)iy * g.W + ix) * g.C + ci];
#pragma unroll
            for (int j = 0; j < CO_T; j += 4) {
                const float4 w = *reinterpret_cast<const float4*>(&fs[kk][j]);
                acc[j + 0] = fmaf(xv, w.x, acc[j + 0]);
                acc[j + 1] = fmaf(xv, w.y, acc[j + 1]);
                acc[j + 2] = fmaf(xv, w.z, acc[j + 2]);
                acc[j + 3] = fmaf(xv, w.w, acc[j + 3]);
            }
            if (++ci == g.C) {
                ci = 0;
                if (++kx == g.fw) { kx = 0; ++ky; }
            }
        }
        __syncthreads();
    }

#pragma unroll
    for (int j = 0; j < CO_T; ++j) {
        float v = acc[j];
        if (bias && co0 + j < g.Co) v = v + bias[co0 + j];
        ys[tid][j] = apply_act(v, act);
    }
    __syncthreads();
    for (int idx = tid; idx < PIX * CO_T; idx += PIX) {
        const int pp = idx / CO_T, co = idx % CO_T;
        if (pix0 + pp < total_pix && co0 + co < g.Co) y[(pix0 + pp) * g.Co + co0 + co] = ys[pp][co];
    }
}

}  // namespace

cudaError_t launch_conv2d_fp32(const float* x, const float* f, const float* bias, int act, float* y,
                               const ConvGeom& g, cudaStream_t s, int64_t* launches) {
    const int64_t total_pix = g.N * g.Ho * g.Wo;
    if (total_pix == 0 || g.Co == 0) return cudaSuccess;
    const int64_t gx = (total_pix + PIX - 1) / PIX;
    const int gy = (g.Co + CO_T - 1) / CO_T;
    if (gx > 2147483647LL || gy > 65535) return cudaErrorInvalidConfiguration;
    conv2d_fp32_kernel<<<dim3((unsigned)gx, (unsigned)gy), PIX, 0, s>>>(x, f, bias, act, y, g, total_pix);
    ++*launches;
    return cudaGetLastError();
}

}  // namespace tfjsb

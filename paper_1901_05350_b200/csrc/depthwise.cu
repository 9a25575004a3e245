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
#include "common.cuh"

namespace tfjsb {

namespace {

constexpr int DW_THREADS = 256;

__device__ __forceinline__ float4 ld4(const float* p) { return *reinterpret_cast<const float4*>(p); }
__device__ __forceinline__ void fma4(float4& acc, const float4& a, const float4& b) {
    acc.x = fmaf(a.x, b.x, acc.x); acc.y = fmaf(a.y, b.y, acc.y);
    acc.z = fmaf(a.z, b.z, acc.z); acc.w = fmaf(a.w, b.w, acc.w);
}

template <int S, int ROWS>
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
    const bool in_x1 = ix_base + 1 >= 0 && ix_base + 1 < g.W;
    const bool in_x2 = ix_base + 2 >= 0 && ix_base + 2 < g.W;
    const float* xn = x + n * (int64_t)g.H * g.W * g.C + c;
    const float4 zero = make_float4(0.f, 0.f, 0.f, 0.f);

    constexpr int IN_ROWS = (ROWS - 1) * S + 3;
#pragma unroll
    for (int j = 0; j < IN_ROWS; ++j) {
        const int iy = iy_base + j;
        float4 v0 = zero, v1 = zero, v2 = zero;
        if (iy >= 0 && iy < g.H) {
            const float* row = xn + ((int64_t)iy * g.W + ix_base) * g.C;
            if (in_x0) v0 = ld4(row);
            if (in_x1) v1 = ld4(row + g.C);
            if (in_x2) v2 = ld4(row + 2 * g.C);
        }
#pragma unroll
        for (int ky = 0; ky < 3; ++ky) {
            const int t = j - ky;
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

int pow2_at_most(int v, int cap) {
    int p = 1;
    while (p < v && p < cap) p <<= 1;
    return p;
}

}  // namespace

cudaError_t launch_depthwise(const float* x, const float* f, const float* bias, int act, float* y,
                             const ConvGeom& g, cudaStream_t s, int64_t* launches) {
    const int64_t n_out = g.N * g.Ho * g.Wo * g.Co;
    if (n_out == 0) return cudaSuccess;
    const bool fast = g.fh == 3 && g.fw == 3 && g.mult == 1 && g.dh == 1 && g.dw == 1 && g.sh == g.sw &&
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
            if (g.sh == 1)
                depthwise3x3_kernel<1, ROWS><<<grid, DW_THREADS, 0, s>>>(x, f, bias, act, y, g, tc, c4_tiles);
            else
                depthwise3x3_kernel<2, ROWS><<<grid, DW_THREADS, 0, s>>>(x, f, bias, act, y, g, tc, c4_tiles);
            ++*launches;
            return cudaGetLastError();
        }
    }
    int64_t blocks = (n_out + DW_THREADS - 1) / DW_THREADS;
    if (blocks > 148 * 32) blocks = 148 * 32;
    depthwise_generic_kernel<<<(unsigned)blocks, DW_THREADS, 0, s>>>(x, f, bias, act, y, g, n_out);
    ++*launches;
    return cudaGetLastError();
}

}  // namespace tfjsb

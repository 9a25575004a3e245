// Gradient kernels of conv2d, depthwiseConv2d and the bias + activation epilogue (the per-kernel
// gradient functions that eager differentiation calls, Sec. 3.5 of the paper): CUDA-core kernels for
// any window, stride and dilation.  The pointwise (1x1, stride 1) convolution, whose two gradients are
// plain matrix products, runs on the tensor-core GEMMs instead (see the entry points in api.cu).
//
//   dx[n,iy,ix,ci]   = sum over the (output pixel, tap) pairs that read (iy,ix) in the forward pass, and co,
//                      of dy[n,oy,ox,co] * f[ky,kx,ci,co]
//   df[ky,kx,ci,co]  = sum over n,oy,ox of x[n, oy*sh - pt + ky*dh, ox*sw - pl + kx*dw, ci] * dy[n,oy,ox,co]
// and the depthwise forms with co = c*mult + q.  Sums over pixels (filter and bias gradients) are taken
// in two steps, partial sums per slice of the pixels into scratch and then a sum over the slices in slice
// order, so that the result does not depend on scheduling.
#include "common.cuh"

namespace tfjsb {

namespace {

constexpr int BP_THREADS = 256;

// Output row / column that tap k of a forward window maps input coordinate i to, or -1 when none does:
// o*s - p + k*d = i.
__device__ __forceinline__ int source_of(int i, int p, int k, int d, int s, int limit) {
    const int t = i + p - k * d;
    if (t < 0) return -1;
    const int o = t / s;
    return (o * s == t && o < limit) ? o : -1;
}

// ---- conv2d, gradient with respect to the input ---------------------------------------------------
// thread = one input sample (n, iy, ix, ci), ci fastest; the dy row of a source pixel is the same address
// for the threads of a pixel (a broadcast), the filter row f[tap, ci, :] is contiguous per thread.
__global__ void __launch_bounds__(BP_THREADS)
conv2d_backprop_input_kernel(const float* __restrict__ dy, const float* __restrict__ f, float* __restrict__ dx, ConvGeom g,
                             int64_t total) {
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += stride) {
        const int ci = (int)(e % g.C);
        int64_t p = e / g.C;
        const int ix = (int)(p % g.W);
        p /= g.W;
        const int iy = (int)(p % g.H);
        const int64_t n = p / g.H;
        float acc = 0.f;
        for (int ky = 0; ky < g.fh; ++ky) {
            const int oy = source_of(iy, g.pt, ky, g.dh, g.sh, g.Ho);
            if (oy < 0) continue;
            for (int kx = 0; kx < g.fw; ++kx) {
                const int ox = source_of(ix, g.pl, kx, g.dw, g.sw, g.Wo);
                if (ox < 0) continue;
                const float* gp = dy + ((n * g.Ho + oy) * (int64_t)g.Wo + ox) * g.Co;
                const float* fp = f + ((int64_t)(ky * g.fw + kx) * g.C + ci) * g.Co;
                for (int co = 0; co < g.Co; ++co) acc = fmaf(__ldg(gp + co), __ldg(fp + co), acc);
            }
        }
        dx[e] = acc;
    }
}

// ---- conv2d, gradient with respect to the filter: partial sums ---------------------------------------
// Block = a 32 x 32 tile of (ci, co) for one tap and one slice of the output pixels; 32 pixels at a time go
// through shared memory (x samples [32 pixels][32 ci], dy [32 pixels][32 co]); thread (tx = co, ty = ci).
__global__ void __launch_bounds__(1024)
conv2d_backprop_filter_partial_kernel(const float* __restrict__ x, const float* __restrict__ dy, float* __restrict__ partial,
                                      ConvGeom g, int64_t pixels, int64_t pixels_per_slice, int ci_tiles, int co_tiles) {
    __shared__ float xs[32][33];
    __shared__ float gs[32][33];
    int b = blockIdx.x;
    const int co0 = (b % co_tiles) * 32;
    b /= co_tiles;
    const int ci0 = (b % ci_tiles) * 32;
    const int tap = b / ci_tiles;
    const int ky = tap / g.fw, kx = tap - ky * g.fw;
    const int slice = blockIdx.y;
    const int64_t p_begin = (int64_t)slice * pixels_per_slice;
    const int64_t p_end = min(pixels, p_begin + pixels_per_slice);
    const int tx = threadIdx.x, ty = threadIdx.y;
    float acc = 0.f;
    for (int64_t p0 = p_begin; p0 < p_end; p0 += 32) {
        // row ty of both tiles is output pixel p0 + ty; column tx is channel ci0 + tx (resp. co0 + tx)
        const int64_t p = p0 + ty;
        float xv = 0.f, gv = 0.f;
        if (p < p_end) {
            const int ox = (int)(p % g.Wo);
            const int64_t r = p / g.Wo;
            const int oy = (int)(r % g.Ho);
            const int64_t n = r / g.Ho;
            const int iy = oy * g.sh - g.pt + ky * g.dh, ix = ox * g.sw - g.pl + kx * g.dw;
            if (iy >= 0 && iy < g.H && ix >= 0 && ix < g.W && ci0 + tx < g.C)
                xv = __ldg(x + ((n * g.H + iy) * (int64_t)g.W + ix) * g.C + ci0 + tx);
            if (co0 + tx < g.Co) gv = __ldg(dy + p * g.Co + co0 + tx);
        }
        xs[ty][tx] = xv;
        gs[ty][tx] = gv;
        __syncthreads();
#pragma unroll
        for (int k = 0; k < 32; ++k) acc = fmaf(xs[k][ty], gs[k][tx], acc);
        __syncthreads();
    }
    if (ci0 + ty < g.C && co0 + tx < g.Co)
        partial[((int64_t)slice * g.fh * g.fw + tap) * g.C * g.Co + (int64_t)(ci0 + ty) * g.Co + co0 + tx] = acc;
}

// out[c] = sum over r < rows (in order) of in[r, c]
__global__ void __launch_bounds__(BP_THREADS)
sum_rows_kernel(const float* __restrict__ in, float* __restrict__ out, int64_t rows, int64_t C) {
    const int64_t c = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= C) return;
    float acc = 0.f;
    for (int64_t r = 0; r < rows; ++r) acc += in[r * C + c];
    out[c] = acc;
}

// partial[slice, c] = sum over the rows of the slice of in[r, c]; block = 32 columns x 8 row lanes
__global__ void __launch_bounds__(BP_THREADS)
sum_rows_partial_kernel(const float* __restrict__ in, float* __restrict__ partial, int64_t rows, int64_t C,
                        int64_t rows_per_slice) {
    __shared__ float red[8][32];
    const int64_t c = (int64_t)blockIdx.x * 32 + threadIdx.x;
    const int64_t r_begin = (int64_t)blockIdx.y * rows_per_slice;
    const int64_t r_end = min(rows, r_begin + rows_per_slice);
    float acc = 0.f;
    if (c < C)
        for (int64_t r = r_begin + threadIdx.y; r < r_end; r += 8) acc += __ldg(in + r * C + c);
    red[threadIdx.y][threadIdx.x] = acc;
    __syncthreads();
    if (threadIdx.y == 0 && c < C) {
        float v = red[0][threadIdx.x];
#pragma unroll
        for (int k = 1; k < 8; ++k) v += red[k][threadIdx.x];
        partial[(int64_t)blockIdx.y * C + c] = v;
    }
}

// ---- depthwise, gradient with respect to the input ---------------------------------------------------
__global__ void __launch_bounds__(BP_THREADS)
depthwise_backprop_input_kernel(const float* __restrict__ dy, const float* __restrict__ f, float* __restrict__ dx, ConvGeom g,
                                int64_t total) {
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += stride) {
        const int c = (int)(e % g.C);
        int64_t p = e / g.C;
        const int ix = (int)(p % g.W);
        p /= g.W;
        const int iy = (int)(p % g.H);
        const int64_t n = p / g.H;
        float acc = 0.f;
        for (int ky = 0; ky < g.fh; ++ky) {
            const int oy = source_of(iy, g.pt, ky, g.dh, g.sh, g.Ho);
            if (oy < 0) continue;
            for (int kx = 0; kx < g.fw; ++kx) {
                const int ox = source_of(ix, g.pl, kx, g.dw, g.sw, g.Wo);
                if (ox < 0) continue;
                const float* gp = dy + ((n * g.Ho + oy) * (int64_t)g.Wo + ox) * g.Co + (int64_t)c * g.mult;
                const float* fp = f + ((int64_t)(ky * g.fw + kx) * g.C + c) * g.mult;
                for (int q = 0; q < g.mult; ++q) acc = fmaf(__ldg(gp + q), __ldg(fp + q), acc);
            }
        }
        dx[e] = acc;
    }
}

// ---- depthwise, gradient with respect to the filter: partial sums ------------------------------------
// Block = 32 output channels (tx) x 8 pixel lanes (ty) for one tap (blockIdx.z) and one slice of the
// output pixels (blockIdx.y).
__global__ void __launch_bounds__(BP_THREADS)
depthwise_backprop_filter_partial_kernel(const float* __restrict__ x, const float* __restrict__ dy, float* __restrict__ partial,
                                         ConvGeom g, int64_t pixels, int64_t pixels_per_slice) {
    __shared__ float red[8][32];
    const int oc = blockIdx.x * 32 + threadIdx.x;
    const int tap = blockIdx.z;
    const int ky = tap / g.fw, kx = tap - ky * g.fw;
    const int64_t p_begin = (int64_t)blockIdx.y * pixels_per_slice;
    const int64_t p_end = min(pixels, p_begin + pixels_per_slice);
    float acc = 0.f;
    if (oc < g.Co) {
        const int c = oc / g.mult;
        for (int64_t p = p_begin + threadIdx.y; p < p_end; p += 8) {
            const int ox = (int)(p % g.Wo);
            const int64_t r = p / g.Wo;
            const int oy = (int)(r % g.Ho);
            const int64_t n = r / g.Ho;
            const int iy = oy * g.sh - g.pt + ky * g.dh, ix = ox * g.sw - g.pl + kx * g.dw;
            if (iy >= 0 && iy < g.H && ix >= 0 && ix < g.W)
                acc = fmaf(__ldg(x + ((n * g.H + iy) * (int64_t)g.W + ix) * g.C + c), __ldg(dy + p * g.Co + oc), acc);
        }
    }
    red[threadIdx.y][threadIdx.x] = acc;
    __syncthreads();
    if (threadIdx.y == 0 && oc < g.Co) {
        float v = red[0][threadIdx.x];
#pragma unroll
        for (int k = 1; k < 8; ++k) v += red[k][threadIdx.x];
        partial[((int64_t)blockIdx.y * g.fh * g.fw + tap) * g.Co + oc] = v;
    }
}

// ---- epilogue ---------------------------------------------------------------------------------------
// dz = dy where the activation passed its input through (judged by the forward output y), +0 elsewhere
__global__ void __launch_bounds__(BP_THREADS)
act_backprop_kernel(const float* __restrict__ y, const float* __restrict__ dy, float* __restrict__ dz, int64_t n, int act) {
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) {
        const float v = y[i];
        const bool pass = act == TFJSB_ACT_NONE || (v > 0.f && (act == TFJSB_ACT_RELU || v < 6.f));
        dz[i] = pass ? dy[i] : 0.f;
    }
}

// out[b, c, r] = in[b, r, c] for B matrices of shape [rows, cols] stored one after the other
__global__ void transpose_batched_kernel(const float* __restrict__ in, float* __restrict__ out, int64_t rows, int64_t cols) {
    __shared__ float tile[32][33];
    in += (int64_t)blockIdx.z * rows * cols;
    out += (int64_t)blockIdx.z * rows * cols;
    const int64_t c0 = (int64_t)blockIdx.x * 32, r0 = (int64_t)blockIdx.y * 32;
    for (int j = threadIdx.y; j < 32; j += 8) {
        const int64_t r = r0 + j, c = c0 + threadIdx.x;
        if (r < rows && c < cols) tile[j][threadIdx.x] = in[r * cols + c];
    }
    __syncthreads();
    for (int j = threadIdx.y; j < 32; j += 8) {
        const int64_t c = c0 + j, r = r0 + threadIdx.x;
        if (r < rows && c < cols) out[c * rows + r] = tile[threadIdx.x][j];
    }
}

int blocks_for(int64_t items, int sm_count) {
    int64_t b = (items + BP_THREADS - 1) / BP_THREADS;
    const int64_t cap = (int64_t)sm_count * 16;
    return (int)(b < 1 ? 1 : (b > cap ? cap : b));
}

}  // namespace

int backprop_slices(int64_t rows, int sm_count) {
    // enough slices for a few blocks per SM, at least 256 rows each
    int64_t s = rows / 256;
    if (s > 4 * (int64_t)sm_count) s = 4 * (int64_t)sm_count;
    return (int)(s < 1 ? 1 : s);
}

cudaError_t launch_conv2d_backprop_input(const float* dy, const float* f, float* dx, const ConvGeom& g, int sm_count,
                                         cudaStream_t s, int64_t* launches) {
    const int64_t total = g.N * g.H * g.W * g.C;
    conv2d_backprop_input_kernel<<<blocks_for(total, sm_count), BP_THREADS, 0, s>>>(dy, f, dx, g, total);
    ++*launches;
    return cudaGetLastError();
}

cudaError_t launch_sum_rows(const float* in, float* out, float* partial, int64_t rows, int64_t C, int slices, cudaStream_t s,
                            int64_t* launches) {
    if (slices <= 1) {
        sum_rows_kernel<<<(unsigned)((C + BP_THREADS - 1) / BP_THREADS), BP_THREADS, 0, s>>>(in, out, rows, C);
        ++*launches;
        return cudaGetLastError();
    }
    const int64_t per = (rows + slices - 1) / slices;
    sum_rows_partial_kernel<<<dim3((unsigned)((C + 31) / 32), (unsigned)slices), dim3(32, 8), 0, s>>>(in, partial, rows, C, per);
    sum_rows_kernel<<<(unsigned)((C + BP_THREADS - 1) / BP_THREADS), BP_THREADS, 0, s>>>(partial, out, slices, C);
    *launches += 2;
    return cudaGetLastError();
}

cudaError_t launch_conv2d_backprop_filter(const float* x, const float* dy, float* df, float* partial, int slices,
                                          const ConvGeom& g, cudaStream_t s, int64_t* launches) {
    const int64_t pixels = g.N * g.Ho * g.Wo;
    const int64_t per = ((pixels + slices - 1) / slices + 31) / 32 * 32;
    const int ci_tiles = (g.C + 31) / 32, co_tiles = (g.Co + 31) / 32;
    const int64_t blocks = (int64_t)g.fh * g.fw * ci_tiles * co_tiles;
    if (blocks >= (1LL << 31)) return cudaErrorInvalidConfiguration;
    const int64_t elems = (int64_t)g.fh * g.fw * g.C * g.Co;
    conv2d_backprop_filter_partial_kernel<<<dim3((unsigned)blocks, (unsigned)slices), dim3(32, 32), 0, s>>>(
        x, dy, slices > 1 ? partial : df, g, pixels, per, ci_tiles, co_tiles);
    ++*launches;
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess || slices <= 1) return e;
    return launch_sum_rows(partial, df, nullptr, slices, elems, 1, s, launches);
}

cudaError_t launch_depthwise_backprop_input(const float* dy, const float* f, float* dx, const ConvGeom& g, int sm_count,
                                            cudaStream_t s, int64_t* launches) {
    const int64_t total = g.N * g.H * g.W * g.C;
    depthwise_backprop_input_kernel<<<blocks_for(total, sm_count), BP_THREADS, 0, s>>>(dy, f, dx, g, total);
    ++*launches;
    return cudaGetLastError();
}

cudaError_t launch_depthwise_backprop_filter(const float* x, const float* dy, float* df, float* partial, int slices,
                                             const ConvGeom& g, cudaStream_t s, int64_t* launches) {
    const int64_t pixels = g.N * g.Ho * g.Wo;
    const int64_t per = (pixels + slices - 1) / slices;
    const int taps = g.fh * g.fw;
    if (taps > 65535 || slices > 65535) return cudaErrorInvalidConfiguration;
    depthwise_backprop_filter_partial_kernel<<<dim3((unsigned)((g.Co + 31) / 32), (unsigned)slices, (unsigned)taps), dim3(32, 8), 0,
                                               s>>>(x, dy, slices > 1 ? partial : df, g, pixels, per);
    ++*launches;
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess || slices <= 1) return e;
    return launch_sum_rows(partial, df, nullptr, slices, (int64_t)taps * g.Co, 1, s, launches);
}

cudaError_t launch_act_backprop(const float* y, const float* dy, float* dz, int64_t n, int act, int sm_count, cudaStream_t s,
                                int64_t* launches) {
    act_backprop_kernel<<<blocks_for(n, sm_count), BP_THREADS, 0, s>>>(y, dy, dz, n, act);
    ++*launches;
    return cudaGetLastError();
}

cudaError_t launch_transpose_batched(const float* in, float* out, int64_t batches, int64_t rows, int64_t cols, cudaStream_t s,
                                     int64_t* launches) {
    if (rows == 0 || cols == 0 || batches == 0) return cudaSuccess;
    dim3 grid((unsigned)((cols + 31) / 32), (unsigned)((rows + 31) / 32), (unsigned)batches);
    if ((rows + 31) / 32 > 65535 || batches > 65535) return cudaErrorInvalidConfiguration;
    transpose_batched_kernel<<<grid, dim3(32, 8), 0, s>>>(in, out, rows, cols);
    ++*launches;
    return cudaGetLastError();
}

}  // namespace tfjsb

// Bandwidth-bound helpers: the standalone bias+activation op, avgPool, softmax, and the
// 2-D transpose used to make matMul operands K-contiguous.
#include "common.cuh"
#include "ptx_sm100.cuh"

namespace tfjsb {

namespace {

constexpr int kThreads = 256;

inline int grid_for(int64_t work_items, int threads, int max_blocks) {
    int64_t b = (work_items + threads - 1) / threads;
    if (b < 1) b = 1;
    if (b > max_blocks) b = max_blocks;
    return (int)b;
}

// ---- bias + activation ----------------------------------------------------------------------
// out[r, c] = act(x[r, c] + bias[c]).  float4 path: C % 4 == 0, so a float4 never straddles rows.
__global__ void bias_act_vec4_kernel(const float4* __restrict__ x, const float* __restrict__ bias,
                                     float4* __restrict__ y, int64_t n_vec, int C4, int act) {
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_vec; i += stride) {
        float4 v = x[i];
        if (bias) {
            const int c = (int)(i % C4) * 4;
            const float4 b = *reinterpret_cast<const float4*>(bias + c);
            v.x = v.x + b.x; v.y = v.y + b.y; v.z = v.z + b.z; v.w = v.w + b.w;
        }
        v.x = apply_act(v.x, act); v.y = apply_act(v.y, act);
        v.z = apply_act(v.z, act); v.w = apply_act(v.w, act);
        y[i] = v;
    }
}

__global__ void bias_act_scalar_kernel(const float* __restrict__ x, const float* __restrict__ bias,
                                       float* __restrict__ y, int64_t n, int64_t C, int act) {
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) {
        float v = x[i];
        if (bias) v = v + bias[i % C];
        y[i] = apply_act(v, act);
    }
}

// ---- avgPool ----------------------------------------------------------------------------------
// One thread per output element, channel fastest (coalesced).  Padding never counts.
__global__ void avg_pool_window_kernel(const float* __restrict__ x, float* __restrict__ y, ConvGeom g,
                                       int64_t n_out) {
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_out; i += stride) {
        const int c = (int)(i % g.C);
        int64_t t = i / g.C;
        const int ox = (int)(t % g.Wo); t /= g.Wo;
        const int oy = (int)(t % g.Ho);
        const int64_t n = t / g.Ho;
        float acc = 0.0f;
        int count = 0;
        for (int ky = 0; ky < g.fh; ++ky) {
            const int iy = oy * g.sh - g.pt + ky;
            if (iy < 0 || iy >= g.H) continue;
            for (int kx = 0; kx < g.fw; ++kx) {
                const int ix = ox * g.sw - g.pl + kx;
                if (ix < 0 || ix >= g.W) continue;
                acc += x[((n * g.H + iy) * (int64_t)g.W + ix) * g.C + c];
                ++count;
            }
        }
        y[i] = acc / (float)count;
    }
}

// ---- maxPool ----------------------------------------------------------------------------------
// One thread per output element, channel fastest (coalesced).  Padding never takes part; max.NaN keeps
// a NaN that is in the window.
__global__ void max_pool_window_kernel(const float* __restrict__ x, float* __restrict__ y, ConvGeom g,
                                       int64_t n_out) {
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_out; i += stride) {
        const int c = (int)(i % g.C);
        int64_t t = i / g.C;
        const int ox = (int)(t % g.Wo); t /= g.Wo;
        const int oy = (int)(t % g.Ho);
        const int64_t n = t / g.Ho;
        float m = __int_as_float(0xff800000);  // -inf
        for (int ky = 0; ky < g.fh; ++ky) {
            const int iy = oy * g.sh - g.pt + ky;
            if (iy < 0 || iy >= g.H) continue;
            for (int kx = 0; kx < g.fw; ++kx) {
                const int ix = ox * g.sw - g.pl + kx;
                if (ix < 0 || ix >= g.W) continue;
                const float v = x[((n * g.H + iy) * (int64_t)g.W + ix) * g.C + c];
                asm("max.NaN.f32 %0, %0, %1;" : "+f"(m) : "f"(v));
            }
        }
        y[i] = m;
    }
}

// The same with four channels per thread (C % 4 == 0): one 16-byte load per window element, a warp
// reads 512 contiguous bytes per tap; neighbouring outputs' windows overlap in L1/L2.
__device__ __forceinline__ void max4_nan(float4& m, const float4& v) {
    asm("max.NaN.f32 %0, %0, %1;" : "+f"(m.x) : "f"(v.x));
    asm("max.NaN.f32 %0, %0, %1;" : "+f"(m.y) : "f"(v.y));
    asm("max.NaN.f32 %0, %0, %1;" : "+f"(m.z) : "f"(v.z));
    asm("max.NaN.f32 %0, %0, %1;" : "+f"(m.w) : "f"(v.w));
}
__global__ void max_pool_vec4_kernel(const float* __restrict__ x, float* __restrict__ y, ConvGeom g, int64_t n_out4) {
    const int C4 = g.C >> 2;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_out4; i += stride) {
        const int c = (int)(i % C4) * 4;
        int64_t t = i / C4;
        const int ox = (int)(t % g.Wo); t /= g.Wo;
        const int oy = (int)(t % g.Ho);
        const int64_t n = t / g.Ho;
        const float ninf = __int_as_float(0xff800000);
        float4 m = make_float4(ninf, ninf, ninf, ninf);
        const int iy0 = oy * g.sh - g.pt, ix0 = ox * g.sw - g.pl;
        const int ky0 = iy0 < 0 ? -iy0 : 0, ky1 = min(g.fh, g.H - iy0);
        const int kx0 = ix0 < 0 ? -ix0 : 0, kx1 = min(g.fw, g.W - ix0);
        for (int ky = ky0; ky < ky1; ++ky) {
            const float* row = x + ((n * g.H + iy0 + ky) * (int64_t)g.W + ix0) * g.C + c;
            for (int kx = kx0; kx < kx1; ++kx) max4_nan(m, __ldg(reinterpret_cast<const float4*>(row + (int64_t)kx * g.C)));
        }
        *reinterpret_cast<float4*>(y + i * 4) = m;
    }
}

// ---- elementwise binary ops (the addition shader of the paper's Fig. 3: one output value per thread) ----
// out[i] = a[i] op b[i % b_len]; OP 0 add, 1 subtract, 2 multiply: one fp32 operation, so bit-exact.
template <int OP>
__device__ __forceinline__ float binary_op(float u, float v) {
    return OP == 0 ? __fadd_rn(u, v) : (OP == 1 ? __fsub_rn(u, v) : __fmul_rn(u, v));
}
// float4 path: n and b_len multiples of 4 (a float4 never straddles a period of b)
template <int OP>
__global__ void binary_vec4_kernel(const float4* __restrict__ a, const float4* __restrict__ b, float4* __restrict__ out,
                                   int64_t n4, int64_t b_len4) {
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += stride) {
        const float4 u = a[i];
        const float4 v = b_len4 == n4 ? b[i] : __ldg(b + i % b_len4);
        out[i] = make_float4(binary_op<OP>(u.x, v.x), binary_op<OP>(u.y, v.y), binary_op<OP>(u.z, v.z), binary_op<OP>(u.w, v.w));
    }
}
template <int OP>
__global__ void binary_scalar_kernel(const float* __restrict__ a, const float* __restrict__ b, float* __restrict__ out,
                                     int64_t n, int64_t b_len) {
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride)
        out[i] = binary_op<OP>(a[i], b[i % b_len]);
}

// Global pool: a block owns (image n, 128 consecutive channels).  Lane = 4 channels (one float4, so a
// warp reads 512 contiguous bytes per position), the 8 warps stride over the H*W positions, partial
// sums meet in shared memory.  C % 4 == 0.
__global__ void avg_pool_global_vec4_kernel(const float* __restrict__ x, float* __restrict__ y, int HW, int C) {
    __shared__ float4 partial[8][32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int c = (blockIdx.x * 32 + lane) * 4;
    const int64_t n = blockIdx.y;
    ptx::pdl_launch_dependents();
    ptx::pdl_wait();
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    if (c < C) {
        const float* base = x + n * (int64_t)HW * C + c;
        // four loads in flight per thread (the sum order stays p ascending)
        int p = warp;
        for (; p + 24 < HW; p += 32) {
            float4 v[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) v[u] = *reinterpret_cast<const float4*>(base + (int64_t)(p + 8 * u) * C);
#pragma unroll
            for (int u = 0; u < 4; ++u) { acc.x += v[u].x; acc.y += v[u].y; acc.z += v[u].z; acc.w += v[u].w; }
        }
        for (; p < HW; p += 8) {
            const float4 v = *reinterpret_cast<const float4*>(base + (int64_t)p * C);
            acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
        }
    }
    partial[warp][lane] = acc;
    __syncthreads();
    if (warp == 0 && c < C) {
        float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int w = 0; w < 8; ++w) {
            const float4 v = partial[w][lane];
            s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
        }
        const float inv = (float)HW;
        *reinterpret_cast<float4*>(y + n * C + c) = make_float4(s.x / inv, s.y / inv, s.z / inv, s.w / inv);
    }
}

// The same with one channel per lane, for channel counts that are not multiples of 4.
__global__ void avg_pool_global_kernel(const float* __restrict__ x, float* __restrict__ y, int HW, int C) {
    __shared__ float partial[8][32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int c = blockIdx.x * 32 + lane;
    const int64_t n = blockIdx.y;
    ptx::pdl_launch_dependents();
    ptx::pdl_wait();
    float acc = 0.0f;
    if (c < C) {
        const float* base = x + n * (int64_t)HW * C + c;
        for (int p = warp; p < HW; p += 8) acc += base[(int64_t)p * C];
    }
    partial[warp][lane] = acc;
    __syncthreads();
    if (warp == 0 && c < C) {
        float s = 0.0f;
#pragma unroll
        for (int w = 0; w < 8; ++w) s += partial[w][lane];
        y[n * C + c] = s / (float)HW;
    }
}

// ---- softmax ----------------------------------------------------------------------------------
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// One block (kThreads) per row: max, then sum of exp(x - max), then the quotient.
__global__ void softmax_rows_kernel(const float* __restrict__ x, float* __restrict__ y, int64_t cols) {
    __shared__ float red[kThreads / 32];
    __shared__ float bcast;
    const float* xr = x + (int64_t)blockIdx.x * cols;
    float* yr = y + (int64_t)blockIdx.x * cols;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    ptx::pdl_launch_dependents();
    ptx::pdl_wait();

    float m = -INFINITY;
    for (int64_t j = threadIdx.x; j < cols; j += kThreads) m = fmaxf(m, xr[j]);
    m = warp_max(m);
    if (lane == 0) red[warp] = m;
    __syncthreads();
    if (warp == 0) {
        float v = lane < kThreads / 32 ? red[lane] : -INFINITY;
        v = warp_max(v);
        if (lane == 0) bcast = v;
    }
    __syncthreads();
    m = bcast;

    float sum = 0.0f;
    for (int64_t j = threadIdx.x; j < cols; j += kThreads) sum += expf(xr[j] - m);
    sum = warp_sum(sum);
    __syncthreads();  // red[] and bcast are reused
    if (lane == 0) red[warp] = sum;
    __syncthreads();
    if (warp == 0) {
        float v = lane < kThreads / 32 ? red[lane] : 0.0f;
        v = warp_sum(v);
        if (lane == 0) bcast = v;
    }
    __syncthreads();
    sum = bcast;

    for (int64_t j = threadIdx.x; j < cols; j += kThreads) yr[j] = expf(xr[j] - m) / sum;
}

// ---- transpose --------------------------------------------------------------------------------
__global__ void transpose_kernel(const float* __restrict__ in, float* __restrict__ out, int64_t rows,
                                 int64_t cols) {
    __shared__ float tile[32][33];
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

// ---- filter packing for the implicit-GEMM convolution ------------------------------------------------
__global__ void pack_filter_kernel(const float* __restrict__ f, float* __restrict__ out, int64_t K, int64_t N,
                                   int64_t k_pad) {
    const int64_t total = N * k_pad;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += stride) {
        const int64_t n = i / k_pad, k = i - n * k_pad;
        out[i] = k < K ? f[k * N + n] : 0.0f;
    }
}

}  // namespace

cudaError_t launch_pack_filter(const float* f, float* out, int64_t K, int64_t N, int64_t k_pad, cudaStream_t s,
                               int64_t* launches) {
    const int64_t total = N * k_pad;
    if (total == 0) return cudaSuccess;
    pack_filter_kernel<<<grid_for(total, kThreads, current_sm_count() * 8), kThreads, 0, s>>>(f, out, K, N, k_pad);
    ++*launches;
    return cudaGetLastError();
}

cudaError_t launch_bias_act(const float* x, const float* bias, float* y, int64_t rows, int64_t C, int act,
                            cudaStream_t s, int64_t* launches) {
    const int64_t n = rows * C;
    if (n == 0) return cudaSuccess;
    if (C % 4 == 0) {
        const int64_t n_vec = n / 4;
        bias_act_vec4_kernel<<<grid_for(n_vec, kThreads, current_sm_count() * 16), kThreads, 0, s>>>(
            reinterpret_cast<const float4*>(x), bias, reinterpret_cast<float4*>(y), n_vec, (int)(C / 4), act);
    } else {
        bias_act_scalar_kernel<<<grid_for(n, kThreads, current_sm_count() * 16), kThreads, 0, s>>>(x, bias, y, n, C, act);
    }
    ++*launches;
    return cudaGetLastError();
}

cudaError_t launch_avg_pool(const float* x, float* y, const ConvGeom& g, cudaStream_t s, int64_t* launches) {
    const int64_t n_out = g.N * g.Ho * g.Wo * g.C;
    if (n_out == 0) return cudaSuccess;
    const bool global = g.Ho == 1 && g.Wo == 1 && g.fh == g.H && g.fw == g.W && g.pt == 0 && g.pl == 0 &&
                        g.N <= 65535;
    if (global) {
        cudaError_t e;
        if (g.C % 4 == 0) {
            dim3 grid((g.C / 4 + 31) / 32, (unsigned)g.N);
            e = launch_k(avg_pool_global_vec4_kernel, grid, dim3(256), 0, s, x, y, g.H * g.W, g.C);
        } else {
            dim3 grid((g.C + 31) / 32, (unsigned)g.N);
            e = launch_k(avg_pool_global_kernel, grid, dim3(256), 0, s, x, y, g.H * g.W, g.C);
        }
        ++*launches;
        return e;
    } else {
        avg_pool_window_kernel<<<grid_for(n_out, kThreads, current_sm_count() * 16), kThreads, 0, s>>>(x, y, g, n_out);
    }
    ++*launches;
    return cudaGetLastError();
}

cudaError_t launch_max_pool(const float* x, float* y, const ConvGeom& g, cudaStream_t s, int64_t* launches) {
    const int64_t n_out = g.N * g.Ho * g.Wo * g.C;
    if (n_out == 0) return cudaSuccess;
    if (g.C % 4 == 0)
        max_pool_vec4_kernel<<<grid_for(n_out / 4, kThreads, current_sm_count() * 32), kThreads, 0, s>>>(x, y, g, n_out / 4);
    else
        max_pool_window_kernel<<<grid_for(n_out, kThreads, current_sm_count() * 16), kThreads, 0, s>>>(x, y, g, n_out);
    ++*launches;
    return cudaGetLastError();
}

template <int OP>
static cudaError_t launch_binary_op(const float* a, const float* b, float* out, int64_t n, int64_t b_len, cudaStream_t s) {
    if (n % 4 == 0 && b_len % 4 == 0)
        binary_vec4_kernel<OP><<<grid_for(n / 4, kThreads, current_sm_count() * 16), kThreads, 0, s>>>(
            reinterpret_cast<const float4*>(a), reinterpret_cast<const float4*>(b), reinterpret_cast<float4*>(out), n / 4, b_len / 4);
    else
        binary_scalar_kernel<OP><<<grid_for(n, kThreads, current_sm_count() * 16), kThreads, 0, s>>>(a, b, out, n, b_len);
    return cudaGetLastError();
}

cudaError_t launch_binary(int op, const float* a, const float* b, float* out, int64_t n, int64_t b_len, cudaStream_t s,
                          int64_t* launches) {
    if (n == 0) return cudaSuccess;
    ++*launches;
    if (op == TFJSB_BINARY_ADD) return launch_binary_op<0>(a, b, out, n, b_len, s);
    if (op == TFJSB_BINARY_SUB) return launch_binary_op<1>(a, b, out, n, b_len, s);
    return launch_binary_op<2>(a, b, out, n, b_len, s);
}

cudaError_t launch_softmax(const float* x, float* y, int64_t rows, int64_t cols, cudaStream_t s,
                           int64_t* launches) {
    if (rows == 0) return cudaSuccess;
    // gridDim.x is 2^31-1: enough for any tensor that fits in memory
    cudaError_t e = launch_k(softmax_rows_kernel, dim3((unsigned)rows), dim3(kThreads), 0, s, x, y, cols);
    ++*launches;
    return e;
}

cudaError_t launch_transpose(const float* in, float* out, int64_t rows, int64_t cols, cudaStream_t s,
                             int64_t* launches) {
    if (rows == 0 || cols == 0) return cudaSuccess;
    dim3 grid((unsigned)((cols + 31) / 32), (unsigned)((rows + 31) / 32));
    if (grid.y > 65535) return cudaErrorInvalidConfiguration;
    transpose_kernel<<<grid, dim3(32, 8), 0, s>>>(in, out, rows, cols);
    ++*launches;
    return cudaGetLastError();
}

}  // namespace tfjsb

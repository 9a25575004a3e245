// CUDA-core fp32 GEMM with the fused bias + activation epilogue.
//
// The exactness variant of matMul / 1x1 conv / dense: plain FFMA, fp32 accumulation in k
// order, no reduced-precision operands.  It also serves every shape the tensor-core kernel
// cannot take (row pitches that are not multiples of 16 bytes).  Operands are addressed
// through (row stride, column stride) pairs so all four transpose combinations share one kernel.
//
// Tiling: a 128x128 output tile per 256-thread block, 16-deep k slices staged in shared
// memory (k-major, so the inner product reads contiguous float4s), an 8x8 register tile per
// thread split into two 4-wide halves 64 apart to keep shared-memory reads conflict-free.
#include "common.cuh"

namespace tfjsb {

namespace {

constexpr int BM = 128, BN = 128, BK = 16, THREADS = 256;

__global__ void __launch_bounds__(THREADS)
gemm_fp32_kernel(const float* __restrict__ a, int64_t a_rs, int64_t a_cs, const float* __restrict__ b,
                 int64_t b_rs, int64_t b_cs, const float* __restrict__ bias, int act, float* __restrict__ c,
                 int64_t ldc, int64_t M, int64_t N, int64_t K) {
    __shared__ __align__(16) float As[BK][BM];
    __shared__ __align__(16) float Bs[BK][BN];

    const int tid = threadIdx.x;
    const int tx = tid & 15, ty = tid >> 4;  // 16 x 16 threads
    const int64_t m0 = (int64_t)blockIdx.y * BM, n0 = (int64_t)blockIdx.x * BN;

    float acc[8][8];
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[i][j] = 0.0f;

    // Loader mapping: make the unit-stride index the fastest-varying one across threads.
    const bool a_k_fast = (a_cs == 1);
    const bool b_k_fast = (b_rs == 1);

    for (int64_t k0 = 0; k0 < K; k0 += BK) {
#pragma unroll
        for (int it = 0; it < (BM * BK) / THREADS; ++it) {
            const int idx = it * THREADS + tid;
            const int i = a_k_fast ? idx / BK : idx % BM;
            const int k = a_k_fast ? idx % BK : idx / BM;
            const int64_t gi = m0 + i, gk = k0 + k;
            As[k][i] = (gi < M && gk < K) ? a[gi * a_rs + gk * a_cs] : 0.0f;
        }
#pragma unroll
        for (int it = 0; it < (BN * BK) / THREADS; ++it) {
            const int idx = it * THREADS + tid;
            const int j = b_k_fast ? idx / BK : idx % BN;
            const int k = b_k_fast ? idx % BK : idx / BN;
            const int64_t gj = n0 + j, gk = k0 + k;
            Bs[k][j] = (gj < N && gk < K) ? b[gk * b_rs + gj * b_cs] : 0.0f;
        }
        __syncthreads();
#pragma unroll
        for (int k = 0; k < BK; ++k) {
            float av[8], bv[8];
            *reinterpret_cast<float4*>(&av[0]) = *reinterpret_cast<const float4*>(&As[k][ty * 4]);
            *reinterpret_cast<float4*>(&av[4]) = *reinterpret_cast<const float4*>(&As[k][64 + ty * 4]);
            *reinterpret_cast<float4*>(&bv[0]) = *reinterpret_cast<const float4*>(&Bs[k][tx * 4]);
            *reinterpret_cast<float4*>(&bv[4]) = *reinterpret_cast<const float4*>(&Bs[k][64 + tx * 4]);
#pragma unroll
            for (int i = 0; i < 8; ++i)
#pragma unroll
                for (int j = 0; j < 8; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
        }
        __syncthreads();
    }

#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int64_t gi = m0 + (i < 4 ? ty * 4 + i : 64 + ty * 4 + (i - 4));
        if (gi >= M) continue;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int64_t gj = n0 + (j < 4 ? tx * 4 + j : 64 + tx * 4 + (j - 4));
            if (gj >= N) continue;
            float v = acc[i][j];
            if (bias) v = v + bias[gj];
            c[gi * ldc + gj] = apply_act(v, act);
        }
    }
}

}  // namespace

cudaError_t launch_gemm_fp32(const float* a, int64_t a_rs, int64_t a_cs, const float* b, int64_t b_rs, int64_t b_cs,
                             const float* bias, int act, float* c, int64_t ldc, int64_t M, int64_t N, int64_t K,
                             cudaStream_t s, int64_t* launches) {
    if (M == 0 || N == 0) return cudaSuccess;
    const int64_t gy = (M + BM - 1) / BM, gx = (N + BN - 1) / BN;
    if (gy > 65535) {
        // Rows beyond the grid.y limit: split the row range into chunks.
        const int64_t rows_per = (int64_t)65535 * BM;
        for (int64_t r = 0; r < M; r += rows_per) {
            const int64_t m = (M - r < rows_per) ? (M - r) : rows_per;
            cudaError_t e = launch_gemm_fp32(a + r * a_rs, a_rs, a_cs, b, b_rs, b_cs, bias, act, c + r * ldc, ldc, m,
                                             N, K, s, launches);
            if (e != cudaSuccess) return e;
        }
        return cudaSuccess;
    }
    dim3 grid((unsigned)gx, (unsigned)gy);
    gemm_fp32_kernel<<<grid, THREADS, 0, s>>>(a, a_rs, a_cs, b, b_rs, b_cs, bias, act, c, ldc, M, N, K);
    ++*launches;
    return cudaGetLastError();
}

}  // namespace tfjsb

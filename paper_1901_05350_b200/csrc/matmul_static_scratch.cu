// tfjsb_matmul_static_scratch: tfjsb_matmul for callers that must not allocate device memory.
//
// The tensor-core matMul needs both operands K-contiguous, so an operand that is stored the
// other way round is first transposed into scratch memory.  tfjsb_matmul takes that scratch
// from cudaMalloc (growing it on demand).  Some callers cannot do that where they call the
// library: a real-time loop that may not take the allocator's lock or the device
// synchronisation an allocation can imply, a service whose device-memory budget was fixed at
// start-up, any code that runs at a point where cudaMalloc is not permitted.  For them the
// scratch of this entry point is a fixed array in the library's device image: it exists on
// every GPU that loads the library, from load until the process exits, and no call allocates
// or frees anything.
//
// Consequences of the fixed array
//   * Size limit: the operands that need transposing (a when transpose_a, b when not
//     transpose_b), each rounded up to 64 floats, must fit in STATIC_SCRATCH_FLOATS together.
//     Larger problems are rejected with TFJSB_ERR_UNSUPPORTED before anything is launched.
//   * One array per GPU, shared by every call and every context: two calls whose kernels can
//     overlap on the GPU (different streams, no dependency between them) race on it.  Issue
//     calls on one stream, or order them with events.
//   * The array keeps whatever the previous call left there.  Nothing needs clearing: the
//     transpose kernels overwrite every element the GEMM reads before it reads it.
//   * The device address of the array is looked up once per GPU, by the first call made on
//     that GPU (cudaGetSymbolAddress with that device current).  Make that first call before
//     any stream capture begins.
#include <mutex>

#include "common.cuh"

using namespace tfjsb;

namespace {

constexpr size_t STATIC_SCRATCH_FLOATS = (size_t)4 << 20;  // 4 Mi floats = 16 MiB per GPU
constexpr int MAX_DEVICES = 64;

// In host code this name is only a handle for the runtime's symbol table, never a device address.
static __device__ __align__(256) float g_static_scratch[STATIC_SCRATCH_FLOATS];

std::mutex g_setup_mutex;
float* g_scratch_address[MAX_DEVICES] = {nullptr};

// Device address of the array on the current device, resolved once per device.
tfjsb_status static_scratch_address(tfjsb_ctx* ctx, float** out) {
    int device = -1;
    cudaError_t e = cudaGetDevice(&device);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "cudaGetDevice");
    if (device < 0 || device >= MAX_DEVICES) return fail(ctx, TFJSB_ERR_UNSUPPORTED, "device ordinal above 63");
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_scratch_address[device]) {
        float* ptr = nullptr;
        e = cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_static_scratch);
        if (e != cudaSuccess) return cuda_fail(ctx, e, "cudaGetSymbolAddress(static scratch)");
        if (!ptr) return fail(ctx, TFJSB_ERR_CUDA, "cudaGetSymbolAddress returned a null address");
        g_scratch_address[device] = ptr;
    }
    *out = g_scratch_address[device];
    return TFJSB_OK;
}

bool misaligned_or_null(const tfjsb_tensor* t) {
    return !t || t->rank != 2 || t->dims[0] < 0 || t->dims[1] < 0 ||
           (t->dims[0] * t->dims[1] > 0 && (!t->data || (reinterpret_cast<uintptr_t>(t->data) & 15u)));
}

size_t round_up_64(size_t v) { return (v + 63) / 64 * 64; }

}  // namespace

extern "C" tfjsb_status tfjsb_matmul_static_scratch(tfjsb_ctx* ctx, const tfjsb_tensor* a, const tfjsb_tensor* b,
                                                    int transpose_a, int transpose_b, tfjsb_tensor* out,
                                                    void* stream) {
    if (!ctx) return TFJSB_ERR_INVALID_ARG;
    if (misaligned_or_null(a) || misaligned_or_null(b) || misaligned_or_null(out))
        return fail(ctx, TFJSB_ERR_INVALID_ARG, "a, b and out must be rank-2 tensors with 16-byte aligned device data");
    const int64_t M = transpose_a ? a->dims[1] : a->dims[0];
    const int64_t K = transpose_a ? a->dims[0] : a->dims[1];
    const int64_t Kb = transpose_b ? b->dims[1] : b->dims[0];
    const int64_t N = transpose_b ? b->dims[0] : b->dims[1];
    if (K != Kb)
        return fail(ctx, TFJSB_ERR_SHAPE, "inner dimensions differ: " + std::to_string(K) + " vs " + std::to_string(Kb));
    if (out->dims[0] != M || out->dims[1] != N)
        return fail(ctx, TFJSB_ERR_SHAPE, "out must be [" + std::to_string(M) + "," + std::to_string(N) + "]");
    if (out->data == a->data || out->data == b->data) return fail(ctx, TFJSB_ERR_INVALID_ARG, "out aliases an input");
    if (M == 0 || N == 0) return TFJSB_OK;

    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const float* pa = static_cast<const float*>(a->data);
    const float* pb = static_cast<const float*>(b->data);
    float* pc = static_cast<float*>(out->data);
    cudaError_t e;

    if (ctx->math == TFJSB_MATH_TF32 && gemm_tf32_supported(M, N, K) && ctx->encode_tiled) {
        const size_t need_a = transpose_a ? round_up_64((size_t)M * K) : 0;
        const size_t need_b = !transpose_b ? round_up_64((size_t)N * K) : 0;
        if (need_a + need_b > STATIC_SCRATCH_FLOATS)
            return fail(ctx, TFJSB_ERR_UNSUPPORTED,
                        "operands to transpose need " + std::to_string(need_a + need_b) +
                            " floats of scratch; the static scratch array holds " +
                            std::to_string(STATIC_SCRATCH_FLOATS) + " (use tfjsb_matmul for larger problems)");
        const float* a_km = pa;
        const float* b_km = pb;
        if (need_a + need_b > 0) {
            float* scratch = nullptr;
            tfjsb_status st = static_scratch_address(ctx, &scratch);
            if (st != TFJSB_OK) return st;
            if (transpose_a) {
                if ((e = launch_transpose(pa, scratch, K, M, s, &ctx->launches)) != cudaSuccess)
                    return cuda_fail(ctx, e, "transpose(a)");
                a_km = scratch;
            }
            if (!transpose_b) {
                if ((e = launch_transpose(pb, scratch + need_a, K, N, s, &ctx->launches)) != cudaSuccess)
                    return cuda_fail(ctx, e, "transpose(b)");
                b_km = scratch + need_a;
            }
        }
        GemmTf32Plan plan;
        tfjsb_status st = gemm_tf32_plan(ctx, a_km, b_km, pc, M, N, K, &plan);
        if (st != TFJSB_OK) return st;
        if ((e = launch_gemm_tf32(plan, nullptr, TFJSB_ACT_NONE, ctx->dev_status, s, &ctx->launches)) != cudaSuccess)
            return cuda_fail(ctx, e, "tf32 gemm launch");
        return TFJSB_OK;
    }
    // CUDA-core path: strided operand access, no scratch at all
    const int64_t a_rs = transpose_a ? 1 : K, a_cs = transpose_a ? M : 1;
    const int64_t b_rs = transpose_b ? 1 : N, b_cs = transpose_b ? K : 1;
    if ((e = launch_gemm_fp32(pa, a_rs, a_cs, pb, b_rs, b_cs, nullptr, TFJSB_ACT_NONE, pc, N, M, N, K, s,
                              &ctx->launches)) != cudaSuccess)
        return cuda_fail(ctx, e, "fp32 gemm launch");
    return TFJSB_OK;
}

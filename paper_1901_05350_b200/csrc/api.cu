// C ABI of libtfjsb.so: context, shape inference, argument checks and dispatch of the op calls.
// All validation happens here, on the host, before anything is launched.
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <map>
#include <mutex>
#include <utility>

#include "common.cuh"

using namespace tfjsb;

namespace tfjsb {

thread_local bool g_launch_pdl = false;

tfjsb_status fail(tfjsb_ctx* ctx, tfjsb_status st, const std::string& msg) {
    if (ctx) ctx->last_error = msg;
    return st;
}

tfjsb_status cuda_fail(tfjsb_ctx* ctx, cudaError_t err, const char* what) {
    return fail(ctx, err == cudaErrorMemoryAllocation ? TFJSB_ERR_OOM : TFJSB_ERR_CUDA,
                std::string(what) + ": " + cudaGetErrorString(err));
}

tfjsb_status ensure_scratch(tfjsb_ctx* ctx, Scratch* s, size_t bytes) {
    if (s->bytes >= bytes) return TFJSB_OK;
    if (s->ptr) {
        // earlier launches may still be reading the old block: keep it until the device is known to be idle
        ctx->retired.push_back(s->ptr);
        s->ptr = nullptr;
        if (bytes < 2 * s->bytes) bytes = 2 * s->bytes;
        s->bytes = 0;
    }
    bytes = (bytes + 255) / 256 * 256;
    cudaError_t e = cudaMalloc(&s->ptr, bytes);
    if (e != cudaSuccess) {
        (void)cudaGetLastError();
        s->ptr = nullptr;
        return fail(ctx, TFJSB_ERR_OOM, "could not allocate " + std::to_string(bytes) + " bytes of scratch");
    }
    s->bytes = bytes;
    return TFJSB_OK;
}

cudaError_t smem_attr_once(const void* kernel, int bytes) {
    static std::mutex mu;
    static std::map<std::pair<const void*, int>, int> done;  // (kernel, device) -> bytes set
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    std::lock_guard<std::mutex> lock(mu);
    auto it = done.find({kernel, dev});
    if (it != done.end() && it->second >= bytes) return cudaSuccess;
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e == cudaSuccess) done[{kernel, dev}] = bytes;
    return e;
}

int current_sm_count() {
    static std::mutex mu;
    static std::map<int, int> count;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 148;
    std::lock_guard<std::mutex> lock(mu);
    auto it = count.find(dev);
    if (it != count.end()) return it->second;
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) n = 148;
    count[dev] = n;
    return n;
}

}  // namespace tfjsb

namespace {

bool window_geometry(int64_t in, int k, int s, int d, int pad, int64_t* out, int* before, int* after) {
    if (in < 1 || k < 1 || s < 1 || d < 1) return false;
    const int64_t ek = (int64_t)(k - 1) * d + 1;
    if (pad == TFJSB_PAD_VALID) {
        if (in < ek) return false;
        *out = (in - ek) / s + 1;
        *before = *after = 0;
        return true;
    }
    if (pad == TFJSB_PAD_SAME) {
        *out = (in + s - 1) / s;
        int64_t total = (*out - 1) * s + ek - in;
        if (total < 0) total = 0;
        *before = (int)(total / 2);
        *after = (int)(total - total / 2);
        return true;
    }
    return false;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int64_t numel(const tfjsb_tensor* t) {
    int64_t n = 1;
    for (int i = 0; i < t->rank; ++i) n *= t->dims[i];
    return n;
}

tfjsb_status check_tensor(tfjsb_ctx* ctx, const tfjsb_tensor* t, const char* name, int min_rank, int max_rank) {
    if (!t) return fail(ctx, TFJSB_ERR_INVALID_ARG, std::string(name) + " is null");
    if (t->rank < min_rank || t->rank > max_rank)
        return fail(ctx, TFJSB_ERR_INVALID_ARG,
                    std::string(name) + " has rank " + std::to_string(t->rank) + ", expected " +
                        (min_rank == max_rank ? std::to_string(min_rank)
                                              : std::to_string(min_rank) + ".." + std::to_string(max_rank)));
    for (int i = 0; i < t->rank; ++i)
        if (t->dims[i] < 0) return fail(ctx, TFJSB_ERR_SHAPE, std::string(name) + " has a negative dimension");
    if (numel(t) > 0) {
        if (!t->data) return fail(ctx, TFJSB_ERR_INVALID_ARG, std::string(name) + ".data is null");
        if (!aligned16(t->data)) return fail(ctx, TFJSB_ERR_INVALID_ARG, std::string(name) + ".data is not 16-byte aligned");
    }
    return TFJSB_OK;
}

bool overlaps(const tfjsb_tensor* a, const tfjsb_tensor* b) {
    if (!a || !b || !a->data || !b->data) return false;
    const char* a0 = static_cast<const char*>(a->data);
    const char* b0 = static_cast<const char*>(b->data);
    const char* a1 = a0 + numel(a) * 4;
    const char* b1 = b0 + numel(b) * 4;
    return a0 < b1 && b0 < a1;
}

// Shared checks of conv2d / depthwise / avgPool: fills `g`, verifies `out`.
tfjsb_status conv_geometry(tfjsb_ctx* ctx, const tfjsb_tensor* x, int fh, int fw, const int strides[2], int pad,
                           const int dilations[2], int64_t out_channels, const tfjsb_tensor* out, ConvGeom* g) {
    if (!strides || !dilations) return fail(ctx, TFJSB_ERR_INVALID_ARG, "strides / dilations are null");
    if (pad != TFJSB_PAD_VALID && pad != TFJSB_PAD_SAME) return fail(ctx, TFJSB_ERR_INVALID_ARG, "unknown padding mode");
    if (strides[0] < 1 || strides[1] < 1) return fail(ctx, TFJSB_ERR_INVALID_ARG, "strides must be >= 1");
    if (dilations[0] < 1 || dilations[1] < 1) return fail(ctx, TFJSB_ERR_INVALID_ARG, "dilations must be >= 1");
    if ((strides[0] > 1 || strides[1] > 1) && (dilations[0] > 1 || dilations[1] > 1))
        return fail(ctx, TFJSB_ERR_UNSUPPORTED, "a stride > 1 together with a dilation > 1 is not supported");
    if (fh < 1 || fw < 1) return fail(ctx, TFJSB_ERR_SHAPE, "filter window must be at least 1x1");
    if (x->dims[1] > 0x3fffffff || x->dims[2] > 0x3fffffff || x->dims[3] > 0x3fffffff || out_channels > 0x3fffffff)
        return fail(ctx, TFJSB_ERR_UNSUPPORTED, "spatial / channel extents above 2^30 are not supported");
    g->N = x->dims[0];
    g->H = (int)x->dims[1]; g->W = (int)x->dims[2]; g->C = (int)x->dims[3];
    g->fh = fh; g->fw = fw;
    g->Co = (int)out_channels;
    g->mult = 1;
    g->sh = strides[0]; g->sw = strides[1];
    g->dh = dilations[0]; g->dw = dilations[1];
    int64_t ho, wo;
    int pb, pr;
    if (!window_geometry(g->H, fh, g->sh, g->dh, pad, &ho, &g->pt, &pb) ||
        !window_geometry(g->W, fw, g->sw, g->dw, pad, &wo, &g->pl, &pr))
        return fail(ctx, TFJSB_ERR_SHAPE, "the filter window does not fit the input under 'valid' padding");
    g->Ho = (int)ho; g->Wo = (int)wo;
    if (out->rank != 4 || out->dims[0] != g->N || out->dims[1] != g->Ho || out->dims[2] != g->Wo ||
        out->dims[3] != out_channels) {
        char buf[200];
        snprintf(buf, sizeof buf, "out must be [%lld,%d,%d,%lld]", (long long)g->N, g->Ho, g->Wo, (long long)out_channels);
        return fail(ctx, TFJSB_ERR_SHAPE, buf);
    }
    return TFJSB_OK;
}

tfjsb_status check_bias(tfjsb_ctx* ctx, const tfjsb_tensor* bias, int64_t channels, int act) {
    if (act != TFJSB_ACT_NONE && act != TFJSB_ACT_RELU && act != TFJSB_ACT_RELU6)
        return fail(ctx, TFJSB_ERR_INVALID_ARG, "unknown activation");
    if (!bias) return TFJSB_OK;
    tfjsb_status st = check_tensor(ctx, bias, "bias", 1, 1);
    if (st != TFJSB_OK) return st;
    if (bias->dims[0] != channels)
        return fail(ctx, TFJSB_ERR_SHAPE, "bias length " + std::to_string(bias->dims[0]) + " != output channels " +
                                              std::to_string(channels));
    return TFJSB_OK;
}

#define TFJSB_REQUIRE_CTX(ctx) \
    if (!(ctx)) return TFJSB_ERR_INVALID_ARG

}  // namespace

extern "C" {

tfjsb_status tfjsb_init(int device, tfjsb_ctx** out) {
    if (!out) return TFJSB_ERR_INVALID_ARG;
    *out = nullptr;
    int count = 0;
    cudaError_t e = cudaGetDeviceCount(&count);
    if (e != cudaSuccess || device < 0 || device >= count) {
        (void)cudaGetLastError();
        return TFJSB_ERR_CUDA;
    }
    if ((e = cudaSetDevice(device)) != cudaSuccess) return TFJSB_ERR_CUDA;
    cudaDeviceProp prop;
    if ((e = cudaGetDeviceProperties(&prop, device)) != cudaSuccess) return TFJSB_ERR_CUDA;
    if (prop.major != 10) return TFJSB_ERR_CUDA;  // the kernels are built for sm_100a only
    tfjsb_ctx* ctx = new tfjsb_ctx();
    ctx->device = device;
    ctx->sm_count = prop.multiProcessorCount;
    if ((e = cudaMalloc(&ctx->dev_status, sizeof(unsigned int))) != cudaSuccess ||
        (e = cudaMemset(ctx->dev_status, 0, sizeof(unsigned int))) != cudaSuccess) {
        delete ctx;
        return TFJSB_ERR_CUDA;
    }
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
    if (e == cudaSuccess && qres == cudaDriverEntryPointSuccess) ctx->encode_tiled = reinterpret_cast<EncodeTiledFn>(fn);
    else (void)cudaGetLastError();
    *out = ctx;
    return TFJSB_OK;
}

tfjsb_status tfjsb_shutdown(tfjsb_ctx* ctx) {
    TFJSB_REQUIRE_CTX(ctx);
    if (ctx->live_models > 0) return fail(ctx, TFJSB_ERR_INVALID_ARG, "destroy the context's models first");
    cudaSetDevice(ctx->device);
    cudaDeviceSynchronize();
    if (ctx->dev_status) cudaFree(ctx->dev_status);
    if (ctx->scratch_a.ptr) cudaFree(ctx->scratch_a.ptr);
    if (ctx->scratch_b.ptr) cudaFree(ctx->scratch_b.ptr);
    if (ctx->scratch_c.ptr) cudaFree(ctx->scratch_c.ptr);
    for (void* p : ctx->retired) cudaFree(p);
    delete ctx;
    return TFJSB_OK;
}

tfjsb_status tfjsb_set_math(tfjsb_ctx* ctx, tfjsb_math mode) {
    TFJSB_REQUIRE_CTX(ctx);
    if (mode != TFJSB_MATH_TF32 && mode != TFJSB_MATH_FP32 && mode != TFJSB_MATH_BF16) return fail(ctx, TFJSB_ERR_INVALID_ARG, "unknown math mode");
    ctx->math = mode;
    return TFJSB_OK;
}

const char* tfjsb_last_error(tfjsb_ctx* ctx) { return ctx ? ctx->last_error.c_str() : "null context"; }

tfjsb_status tfjsb_check_device_status(tfjsb_ctx* ctx, void* stream) {
    TFJSB_REQUIRE_CTX(ctx);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    cudaError_t e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "cudaStreamSynchronize");
    unsigned int word = 0;
    e = cudaMemcpy(&word, ctx->dev_status, sizeof word, cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "reading the device status word");
    if (word != DEV_STATUS_OK) {
        cudaMemset(ctx->dev_status, 0, sizeof word);
        char buf[96];
        snprintf(buf, sizeof buf, "a bounded device-side wait gave up (status bits 0x%x)", word);
        return fail(ctx, TFJSB_ERR_TIMEOUT, buf);
    }
    return TFJSB_OK;
}

int64_t tfjsb_launch_count(tfjsb_ctx* ctx) { return ctx ? ctx->launches : -1; }

tfjsb_status tfjsb_window_out_shape(int64_t in, int k, int stride, int dilation, tfjsb_pad pad, int64_t* out,
                                    int* pad_before, int* pad_after) {
    if (in < 1 || k < 1 || stride < 1 || dilation < 1) return TFJSB_ERR_INVALID_ARG;
    if (pad != TFJSB_PAD_VALID && pad != TFJSB_PAD_SAME) return TFJSB_ERR_INVALID_ARG;
    int64_t o;
    int b, a;
    if (!window_geometry(in, k, stride, dilation, pad, &o, &b, &a)) return TFJSB_ERR_SHAPE;
    if (out) *out = o;
    if (pad_before) *pad_before = b;
    if (pad_after) *pad_after = a;
    return TFJSB_OK;
}

// One rank-2 product C[M,N] = op(A) op(B) on device pointers (arguments already validated): the tensor
// cores when the math mode, the shape and the alignment of the pointers allow, else the CUDA-core kernel.
static tfjsb_status matmul_2d(tfjsb_ctx* ctx, const float* pa, const float* pb, float* pc, int64_t M, int64_t K, int64_t N,
                              int transpose_a, int transpose_b, cudaStream_t s) {
    tfjsb_status st;
    cudaError_t e;

    if (ctx->math == TFJSB_MATH_TF32 && gemm_tf32_supported(M, N, K) && ctx->encode_tiled && aligned16(pa) && aligned16(pb) &&
        aligned16(pc)) {
        // make both operands K-contiguous: A as [M,K], B as [N,K]
        const float* a_km = pa;
        const float* b_km = pb;
        if (transpose_a) {  // stored [K,M]
            if ((st = ensure_scratch(ctx, &ctx->scratch_a, (size_t)M * K * 4)) != TFJSB_OK) return st;
            if ((e = launch_transpose(pa, ctx->scratch_a.ptr, K, M, s, &ctx->launches)) != cudaSuccess)
                return cuda_fail(ctx, e, "transpose(a)");
            a_km = ctx->scratch_a.ptr;
        }
        if (!transpose_b) {  // stored [K,N]
            if ((st = ensure_scratch(ctx, &ctx->scratch_b, (size_t)N * K * 4)) != TFJSB_OK) return st;
            if ((e = launch_transpose(pb, ctx->scratch_b.ptr, K, N, s, &ctx->launches)) != cudaSuccess)
                return cuda_fail(ctx, e, "transpose(b)");
            b_km = ctx->scratch_b.ptr;
        }
        GemmTf32Plan plan;
        if ((st = gemm_tf32_plan(ctx, a_km, b_km, pc, M, N, K, &plan)) != TFJSB_OK) return st;
        if ((e = launch_gemm_tf32(plan, nullptr, TFJSB_ACT_NONE, ctx->dev_status, s, &ctx->launches)) != cudaSuccess)
            return cuda_fail(ctx, e, "tf32 gemm launch");
        return TFJSB_OK;
    }
    const int64_t a_rs = transpose_a ? 1 : K, a_cs = transpose_a ? M : 1;
    const int64_t b_rs = transpose_b ? 1 : N, b_cs = transpose_b ? K : 1;
    if ((e = launch_gemm_fp32(pa, a_rs, a_cs, pb, b_rs, b_cs, nullptr, TFJSB_ACT_NONE, pc, N, M, N, K, s,
                              &ctx->launches)) != cudaSuccess)
        return cuda_fail(ctx, e, "fp32 gemm launch");
    return TFJSB_OK;
}


tfjsb_status tfjsb_matmul(tfjsb_ctx* ctx, const tfjsb_tensor* a, const tfjsb_tensor* b, int transpose_a,
                          int transpose_b, tfjsb_tensor* out, void* stream) {
    TFJSB_REQUIRE_CTX(ctx);
    tfjsb_status st;
    if ((st = check_tensor(ctx, a, "a", 2, 2)) != TFJSB_OK) return st;
    if ((st = check_tensor(ctx, b, "b", 2, 2)) != TFJSB_OK) return st;
    if ((st = check_tensor(ctx, out, "out", 2, 2)) != TFJSB_OK) return st;
    const int64_t M = transpose_a ? a->dims[1] : a->dims[0];
    const int64_t K = transpose_a ? a->dims[0] : a->dims[1];
    const int64_t Kb = transpose_b ? b->dims[1] : b->dims[0];
    const int64_t N = transpose_b ? b->dims[0] : b->dims[1];
    if (K != Kb)
        return fail(ctx, TFJSB_ERR_SHAPE, "inner dimensions differ: " + std::to_string(K) + " vs " + std::to_string(Kb));
    if (out->dims[0] != M || out->dims[1] != N)
        return fail(ctx, TFJSB_ERR_SHAPE, "out must be [" + std::to_string(M) + "," + std::to_string(N) + "]");
    if (overlaps(out, a) || overlaps(out, b)) return fail(ctx, TFJSB_ERR_INVALID_ARG, "out aliases an input");
    if (M == 0 || N == 0) return TFJSB_OK;
    return matmul_2d(ctx, static_cast<const float*>(a->data), static_cast<const float*>(b->data),
                     static_cast<float*>(out->data), M, K, N, transpose_a, transpose_b, static_cast<cudaStream_t>(stream));
}

tfjsb_status tfjsb_matmul_bf16(tfjsb_ctx* ctx, const void* a, const void* bt, const float* bias, tfjsb_act act, void* out,
                               int out_is_bf16, int64_t M, int64_t N, int64_t K, void* stream) {
    TFJSB_REQUIRE_CTX(ctx);
    if (act != TFJSB_ACT_NONE && act != TFJSB_ACT_RELU && act != TFJSB_ACT_RELU6)
        return fail(ctx, TFJSB_ERR_INVALID_ARG, "unknown activation");
    if (M < 0 || N < 0 || K < 0) return fail(ctx, TFJSB_ERR_SHAPE, "negative size");
    if (M == 0 || N == 0) return TFJSB_OK;  // nothing to compute (empty tensors may have null pointers)
    if (!a || !bt || !out) return fail(ctx, TFJSB_ERR_INVALID_ARG, "a / bt / out is null");
    if (!aligned16(a) || !aligned16(bt) || !aligned16(out) || (bias && !aligned16(bias)))
        return fail(ctx, TFJSB_ERR_UNSUPPORTED, "pointers must be 16-byte aligned");
    if (a == out || bt == out) return fail(ctx, TFJSB_ERR_INVALID_ARG, "out aliases an input");
    GemmBf16Plan plan;
    tfjsb_status st = gemm_bf16_plan(ctx, a, bt, out, out_is_bf16 != 0, M, N, K, &plan);
    if (st != TFJSB_OK) return st;
    cudaError_t e = launch_gemm_bf16(plan, bias, act, ctx->dev_status, static_cast<cudaStream_t>(stream), &ctx->launches);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "bf16 gemm launch");
    return TFJSB_OK;
}

tfjsb_status tfjsb_batch_matmul(tfjsb_ctx* ctx, const tfjsb_tensor* a, const tfjsb_tensor* b, int transpose_a,
                                int transpose_b, tfjsb_tensor* out, void* stream) {
    TFJSB_REQUIRE_CTX(ctx);
    tfjsb_status st;
    if ((st = check_tensor(ctx, a, "a", 3, 3)) != TFJSB_OK) return st;
    if ((st = check_tensor(ctx, b, "b", 3, 3)) != TFJSB_OK) return st;
    if ((st = check_tensor(ctx, out, "out", 3, 3)) != TFJSB_OK) return st;
    const int64_t B = a->dims[0];
    if (b->dims[0] != B || out->dims[0] != B) return fail(ctx, TFJSB_ERR_SHAPE, "leading dimensions differ");
    const int64_t M = transpose_a ? a->dims[2] : a->dims[1];
    const int64_t K = transpose_a ? a->dims[1] : a->dims[2];
    const int64_t Kb = transpose_b ? b->dims[2] : b->dims[1];
    const int64_t N = transpose_b ? b->dims[1] : b->dims[2];
    if (K != Kb)
        return fail(ctx, TFJSB_ERR_SHAPE, "inner dimensions differ: " + std::to_string(K) + " vs " + std::to_string(Kb));
    if (out->dims[1] != M || out->dims[2] != N)
        return fail(ctx, TFJSB_ERR_SHAPE, "out must be [B," + std::to_string(M) + "," + std::to_string(N) + "]");
    if (overlaps(out, a) || overlaps(out, b)) return fail(ctx, TFJSB_ERR_INVALID_ARG, "out aliases an input");
    if (B == 0 || M == 0 || N == 0) return TFJSB_OK;
    const float* pa = static_cast<const float*>(a->data);
    const float* pb = static_cast<const float*>(b->data);
    float* pc = static_cast<float*>(out->data);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (B > 1 && ctx->math == TFJSB_MATH_TF32 && gemm_tf32_supported(M, N, K) && ctx->encode_tiled) {
        // All products in one launch of the tensor-core kernel: their tiles share the SMs.  Operands
        // that are not K-contiguous are transposed into scratch first, one product at a time.
        cudaError_t e;
        const float* a_km = pa;
        const float* b_km = pb;
        if (transpose_a) {
            if ((st = ensure_scratch(ctx, &ctx->scratch_a, (size_t)B * M * K * 4)) != TFJSB_OK) return st;
            for (int64_t i = 0; i < B; ++i)
                if ((e = launch_transpose(pa + i * M * K, ctx->scratch_a.ptr + i * M * K, K, M, s, &ctx->launches)) != cudaSuccess)
                    return cuda_fail(ctx, e, "transpose(a)");
            a_km = ctx->scratch_a.ptr;
        }
        if (!transpose_b) {
            if ((st = ensure_scratch(ctx, &ctx->scratch_b, (size_t)B * N * K * 4)) != TFJSB_OK) return st;
            for (int64_t i = 0; i < B; ++i)
                if ((e = launch_transpose(pb + i * N * K, ctx->scratch_b.ptr + i * N * K, K, N, s, &ctx->launches)) != cudaSuccess)
                    return cuda_fail(ctx, e, "transpose(b)");
            b_km = ctx->scratch_b.ptr;
        }
        GemmTf32Plan plan;
        if ((st = gemm_tf32_plan(ctx, a_km, b_km, pc, M, N, K, &plan, B)) != TFJSB_OK) return st;
        if ((e = launch_gemm_tf32(plan, nullptr, TFJSB_ACT_NONE, ctx->dev_status, s, &ctx->launches)) != cudaSuccess)
            return cuda_fail(ctx, e, "batched tf32 gemm launch");
        return TFJSB_OK;
    }
    for (int64_t i = 0; i < B; ++i) {
        st = matmul_2d(ctx, pa + i * M * K, pb + i * K * N, pc + i * M * N, M, K, N, transpose_a, transpose_b,
                       static_cast<cudaStream_t>(stream));
        if (st != TFJSB_OK) return st;
    }
    return TFJSB_OK;
}

tfjsb_status tfjsb_conv2d(tfjsb_ctx* ctx, const tfjsb_tensor* x, const tfjsb_tensor* filter, const int strides[2],
                          tfjsb_pad pad, const int dilations[2], const tfjsb_tensor* bias, tfjsb_act act,
                          tfjsb_tensor* out, void* stream) {
    TFJSB_REQUIRE_CTX(ctx);
    tfjsb_status st;
    if ((st = check_tensor(ctx, x, "x", 4, 4)) != TFJSB_OK) return st;
    if ((st = check_tensor(ctx, filter, "filter", 4, 4)) != TFJSB_OK) return st;
    if ((st = check_tensor(ctx, out, "out", 4, 4)) != TFJSB_OK) return st;
    if (filter->dims[2] != x->dims[3])
        return fail(ctx, TFJSB_ERR_SHAPE, "filter has " + std::to_string(filter->dims[2]) + " input channels, x has " +
                                              std::to_string(x->dims[3]));
    if (filter->dims[0] > 0x7fff || filter->dims[1] > 0x7fff) return fail(ctx, TFJSB_ERR_UNSUPPORTED, "filter window too large");
    const int64_t Cout = filter->dims[3];
    if ((st = check_bias(ctx, bias, Cout, act)) != TFJSB_OK) return st;
    ConvGeom g;
    if ((st = conv_geometry(ctx, x, (int)filter->dims[0], (int)filter->dims[1], strides, pad, dilations, Cout, out, &g)) !=
        TFJSB_OK)
        return st;
    if (overlaps(out, x) || overlaps(out, filter) || overlaps(out, bias)) return fail(ctx, TFJSB_ERR_INVALID_ARG, "out aliases an input");
    if (numel(out) == 0) return TFJSB_OK;
    if (g.C == 0) return fail(ctx, TFJSB_ERR_SHAPE, "x has no channels");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const float* px = static_cast<const float*>(x->data);
    const float* pf = static_cast<const float*>(filter->data);
    const float* pbias = bias ? static_cast<const float*>(bias->data) : nullptr;
    float* py = static_cast<float*>(out->data);
    cudaError_t e;

    const bool pointwise = g.fh == 1 && g.fw == 1 && g.sh == 1 && g.sw == 1;
    if (pointwise) {
        // x viewed as [N*H*W, Cin] (a free reshape), filter as [Cin, Cout]
        const int64_t M = g.N * g.H * g.W, K = g.C, N = Cout;
        if (ctx->math == TFJSB_MATH_TF32 && gemm_tf32_supported(M, N, K) && ctx->encode_tiled) {
            if ((st = ensure_scratch(ctx, &ctx->scratch_b, (size_t)N * K * 4)) != TFJSB_OK) return st;
            if ((e = launch_transpose(pf, ctx->scratch_b.ptr, K, N, s, &ctx->launches)) != cudaSuccess)
                return cuda_fail(ctx, e, "transpose(filter)");
            GemmTf32Plan plan;
            if ((st = gemm_tf32_plan(ctx, px, ctx->scratch_b.ptr, py, M, N, K, &plan)) != TFJSB_OK) return st;
            if ((e = launch_gemm_tf32(plan, pbias, act, ctx->dev_status, s, &ctx->launches)) != cudaSuccess)
                return cuda_fail(ctx, e, "tf32 gemm launch");
            return TFJSB_OK;
        }
        if ((e = launch_gemm_fp32(px, K, 1, pf, N, 1, pbias, act, py, N, M, N, K, s, &ctx->launches)) != cudaSuccess)
            return cuda_fail(ctx, e, "fp32 gemm launch");
        return TFJSB_OK;
    }
    if (ctx->math == TFJSB_MATH_TF32 && conv_igemm_supported(g) && ctx->encode_tiled) {
        // implicit GEMM on the tensor cores: the filter is packed [Cout, k_pad] into scratch first
        const int64_t k_pad = conv_igemm_k_pad(g);
        if ((st = ensure_scratch(ctx, &ctx->scratch_b, (size_t)Cout * k_pad * 4)) != TFJSB_OK) return st;
        if ((e = launch_pack_filter(pf, ctx->scratch_b.ptr, (int64_t)g.fh * g.fw * g.C, Cout, k_pad, s, &ctx->launches)) !=
            cudaSuccess)
            return cuda_fail(ctx, e, "filter packing");
        if (conv_patch_supported(g) && !getenv("TFJSB_NO_PATCH_CONV")) {
            DwPwPlan pplan;
            if ((st = conv_patch_plan(ctx, px, ctx->scratch_b.ptr, py, g, &pplan)) != TFJSB_OK) return st;
            if ((e = launch_dwpw_fused(pplan, nullptr, nullptr, TFJSB_ACT_NONE, pbias, act, ctx->dev_status, s,
                                       &ctx->launches)) != cudaSuccess)
                return cuda_fail(ctx, e, "patch conv2d launch");
            return TFJSB_OK;
        }
        GemmTf32Plan plan;
        if ((st = conv_igemm_plan(ctx, px, ctx->scratch_b.ptr, py, g, &plan)) != TFJSB_OK) return st;
        if ((e = launch_gemm_tf32(plan, pbias, act, ctx->dev_status, s, &ctx->launches)) != cudaSuccess)
            return cuda_fail(ctx, e, "implicit-GEMM conv2d launch");
        return TFJSB_OK;
    }
    if ((e = launch_conv2d_fp32(px, pf, pbias, act, py, g, s, &ctx->launches)) != cudaSuccess)
        return cuda_fail(ctx, e, "conv2d launch");
    return TFJSB_OK;
}

tfjsb_status tfjsb_depthwise_conv2d(tfjsb_ctx* ctx, const tfjsb_tensor* x, const tfjsb_tensor* filter,
                                    const int strides[2], tfjsb_pad pad, const int dilations[2],
                                    const tfjsb_tensor* bias, tfjsb_act act, tfjsb_tensor* out, void* stream) {
    TFJSB_REQUIRE_CTX(ctx);
    tfjsb_status st;
    if ((st = check_tensor(ctx, x, "x", 4, 4)) != TFJSB_OK) return st;
    if ((st = check_tensor(ctx, filter, "filter", 4, 4)) != TFJSB_OK) return st;
    if ((st = check_tensor(ctx, out, "out", 4, 4)) != TFJSB_OK) return st;
    if (filter->dims[2] != x->dims[3])
        return fail(ctx, TFJSB_ERR_SHAPE, "filter has " + std::to_string(filter->dims[2]) + " channels, x has " +
                                              std::to_string(x->dims[3]));
    if (filter->dims[3] < 1) return fail(ctx, TFJSB_ERR_SHAPE, "channel multiplier must be >= 1");
    if (filter->dims[0] > 0x7fff || filter->dims[1] > 0x7fff) return fail(ctx, TFJSB_ERR_UNSUPPORTED, "filter window too large");
    const int64_t Co = x->dims[3] * filter->dims[3];
    if ((st = check_bias(ctx, bias, Co, act)) != TFJSB_OK) return st;
    ConvGeom g;
    if ((st = conv_geometry(ctx, x, (int)filter->dims[0], (int)filter->dims[1], strides, pad, dilations, Co, out, &g)) !=
        TFJSB_OK)
        return st;
    g.mult = (int)filter->dims[3];
    if (overlaps(out, x) || overlaps(out, filter) || overlaps(out, bias)) return fail(ctx, TFJSB_ERR_INVALID_ARG, "out aliases an input");
    if (numel(out) == 0) return TFJSB_OK;
    DepthwisePlan plan;
    if ((st = depthwise_plan(ctx, static_cast<const float*>(x->data), g, &plan)) != TFJSB_OK) return st;
    cudaError_t e = launch_depthwise(plan, static_cast<const float*>(x->data), static_cast<const float*>(filter->data),
                                     bias ? static_cast<const float*>(bias->data) : nullptr, act,
                                     static_cast<float*>(out->data), g, ctx->dev_status,
                                     static_cast<cudaStream_t>(stream), &ctx->launches);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "depthwise launch");
    return TFJSB_OK;
}

tfjsb_status tfjsb_avg_pool(tfjsb_ctx* ctx, const tfjsb_tensor* x, const int filter_size[2], const int strides[2],
                            tfjsb_pad pad, tfjsb_tensor* out, void* stream) {
    TFJSB_REQUIRE_CTX(ctx);
    tfjsb_status st;
    if ((st = check_tensor(ctx, x, "x", 4, 4)) != TFJSB_OK) return st;
    if ((st = check_tensor(ctx, out, "out", 4, 4)) != TFJSB_OK) return st;
    if (!filter_size) return fail(ctx, TFJSB_ERR_INVALID_ARG, "filter_size is null");
    const int ones[2] = {1, 1};
    ConvGeom g;
    if ((st = conv_geometry(ctx, x, filter_size[0], filter_size[1], strides, pad, ones, x->dims[3], out, &g)) != TFJSB_OK)
        return st;
    if (overlaps(out, x)) return fail(ctx, TFJSB_ERR_INVALID_ARG, "out aliases an input");
    if (numel(out) == 0) return TFJSB_OK;
    cudaError_t e = launch_avg_pool(static_cast<const float*>(x->data), static_cast<float*>(out->data), g,
                                    static_cast<cudaStream_t>(stream), &ctx->launches);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "avg_pool launch");
    return TFJSB_OK;
}

tfjsb_status tfjsb_max_pool(tfjsb_ctx* ctx, const tfjsb_tensor* x, const int filter_size[2], const int strides[2],
                            tfjsb_pad pad, tfjsb_tensor* out, void* stream) {
    TFJSB_REQUIRE_CTX(ctx);
    tfjsb_status st;
    if ((st = check_tensor(ctx, x, "x", 4, 4)) != TFJSB_OK) return st;
    if ((st = check_tensor(ctx, out, "out", 4, 4)) != TFJSB_OK) return st;
    if (!filter_size) return fail(ctx, TFJSB_ERR_INVALID_ARG, "filter_size is null");
    const int ones[2] = {1, 1};
    ConvGeom g;
    if ((st = conv_geometry(ctx, x, filter_size[0], filter_size[1], strides, pad, ones, x->dims[3], out, &g)) != TFJSB_OK)
        return st;
    if (overlaps(out, x)) return fail(ctx, TFJSB_ERR_INVALID_ARG, "out aliases an input");
    if (numel(out) == 0) return TFJSB_OK;
    cudaError_t e = launch_max_pool(static_cast<const float*>(x->data), static_cast<float*>(out->data), g,
                                    static_cast<cudaStream_t>(stream), &ctx->launches);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "max_pool launch");
    return TFJSB_OK;
}

tfjsb_status tfjsb_binary(tfjsb_ctx* ctx, tfjsb_binary_op op, const tfjsb_tensor* a, const tfjsb_tensor* b,
                          tfjsb_tensor* out, void* stream) {
    TFJSB_REQUIRE_CTX(ctx);
    tfjsb_status st;
    if (op != TFJSB_BINARY_ADD && op != TFJSB_BINARY_SUB && op != TFJSB_BINARY_MUL)
        return fail(ctx, TFJSB_ERR_INVALID_ARG, "unknown binary op");
    if ((st = check_tensor(ctx, a, "a", 1, 4)) != TFJSB_OK) return st;
    if ((st = check_tensor(ctx, b, "b", 1, 4)) != TFJSB_OK) return st;
    if ((st = check_tensor(ctx, out, "out", 1, 4)) != TFJSB_OK) return st;
    bool out_ok = out->rank == a->rank;
    for (int i = 0; out_ok && i < a->rank; ++i) out_ok = out->dims[i] == a->dims[i];
    if (!out_ok) return fail(ctx, TFJSB_ERR_SHAPE, "out must have the shape of a");
    bool same = b->rank == a->rank;
    for (int i = 0; same && i < a->rank; ++i) same = b->dims[i] == a->dims[i];
    const bool vector = b->rank == 1 && b->dims[0] == a->dims[a->rank - 1];
    if (!same && !vector) return fail(ctx, TFJSB_ERR_SHAPE, "b must have a's shape or be a vector of a's last dimension");
    if (overlaps(out, a) || overlaps(out, b)) return fail(ctx, TFJSB_ERR_INVALID_ARG, "out aliases an input");
    if (numel(a) == 0) return TFJSB_OK;
    cudaError_t e = launch_binary(op, static_cast<const float*>(a->data), static_cast<const float*>(b->data),
                                  static_cast<float*>(out->data), numel(a), numel(b), static_cast<cudaStream_t>(stream),
                                  &ctx->launches);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "binary op launch");
    return TFJSB_OK;
}

tfjsb_status tfjsb_softmax(tfjsb_ctx* ctx, const tfjsb_tensor* logits, tfjsb_tensor* out, void* stream) {
    TFJSB_REQUIRE_CTX(ctx);
    tfjsb_status st;
    if ((st = check_tensor(ctx, logits, "logits", 1, 4)) != TFJSB_OK) return st;
    if ((st = check_tensor(ctx, out, "out", 1, 4)) != TFJSB_OK) return st;
    if (out->rank != logits->rank) return fail(ctx, TFJSB_ERR_SHAPE, "out must have the shape of logits");
    for (int i = 0; i < logits->rank; ++i)
        if (out->dims[i] != logits->dims[i]) return fail(ctx, TFJSB_ERR_SHAPE, "out must have the shape of logits");
    if (overlaps(out, logits)) return fail(ctx, TFJSB_ERR_INVALID_ARG, "out aliases an input");
    const int64_t cols = logits->dims[logits->rank - 1];
    if (cols < 1) return fail(ctx, TFJSB_ERR_SHAPE, "softmax needs at least one element in the last dimension");
    const int64_t rows = numel(logits) / cols;
    if (rows == 0) return TFJSB_OK;
    if (rows > 2147483647LL) return fail(ctx, TFJSB_ERR_UNSUPPORTED, "too many rows");
    cudaError_t e = launch_softmax(static_cast<const float*>(logits->data), static_cast<float*>(out->data), rows, cols,
                                   static_cast<cudaStream_t>(stream), &ctx->launches);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "softmax launch");
    return TFJSB_OK;
}

tfjsb_status tfjsb_bias_act(tfjsb_ctx* ctx, const tfjsb_tensor* x, const tfjsb_tensor* bias, tfjsb_act act,
                            tfjsb_tensor* out, void* stream) {
    TFJSB_REQUIRE_CTX(ctx);
    tfjsb_status st;
    if ((st = check_tensor(ctx, x, "x", 1, 4)) != TFJSB_OK) return st;
    if ((st = check_tensor(ctx, out, "out", 1, 4)) != TFJSB_OK) return st;
    if (out->rank != x->rank) return fail(ctx, TFJSB_ERR_SHAPE, "out must have the shape of x");
    for (int i = 0; i < x->rank; ++i)
        if (out->dims[i] != x->dims[i]) return fail(ctx, TFJSB_ERR_SHAPE, "out must have the shape of x");
    const int64_t C = x->dims[x->rank - 1];
    if ((st = check_bias(ctx, bias, C, act)) != TFJSB_OK) return st;
    if (overlaps(out, x) || overlaps(out, bias)) return fail(ctx, TFJSB_ERR_INVALID_ARG, "out aliases an input");
    if (numel(x) == 0) return TFJSB_OK;
    cudaError_t e = launch_bias_act(static_cast<const float*>(x->data), bias ? static_cast<const float*>(bias->data) : nullptr,
                                    static_cast<float*>(out->data), numel(x) / C, C, act,
                                    static_cast<cudaStream_t>(stream), &ctx->launches);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "bias_act launch");
    return TFJSB_OK;
}

tfjsb_status tfjsb_reserve_scratch(tfjsb_ctx* ctx, int64_t bytes) {
    TFJSB_REQUIRE_CTX(ctx);
    if (bytes < 0) return fail(ctx, TFJSB_ERR_INVALID_ARG, "negative size");
    tfjsb_status st;
    if ((st = ensure_scratch(ctx, &ctx->scratch_a, (size_t)bytes)) != TFJSB_OK) return st;
    if ((st = ensure_scratch(ctx, &ctx->scratch_b, (size_t)bytes)) != TFJSB_OK) return st;
    return ensure_scratch(ctx, &ctx->scratch_c, (size_t)bytes);
}

// ---- gradients --------------------------------------------------------------------------------------

namespace {

// Checks shared by the four convolution gradients: `xs` has the forward input's shape, `fs` the filter's,
// `dy` the forward output's; fills the forward geometry.
tfjsb_status grad_geometry(tfjsb_ctx* ctx, const tfjsb_tensor* xs, const tfjsb_tensor* fs, const tfjsb_tensor* dy,
                           const int strides[2], int pad, const int dilations[2], bool depthwise, ConvGeom* g) {
    if (fs->dims[2] != xs->dims[3])
        return fail(ctx, TFJSB_ERR_SHAPE, "filter has " + std::to_string(fs->dims[2]) + " input channels, x has " +
                                              std::to_string(xs->dims[3]));
    if (fs->dims[0] > 0x7fff || fs->dims[1] > 0x7fff) return fail(ctx, TFJSB_ERR_UNSUPPORTED, "filter window too large");
    if (depthwise && fs->dims[3] < 1) return fail(ctx, TFJSB_ERR_SHAPE, "channel multiplier must be >= 1");
    const int64_t co = depthwise ? xs->dims[3] * fs->dims[3] : fs->dims[3];
    tfjsb_status st = conv_geometry(ctx, xs, (int)fs->dims[0], (int)fs->dims[1], strides, pad, dilations, co, dy, g);
    if (st != TFJSB_OK) return st;
    if (depthwise) g->mult = (int)fs->dims[3];
    return TFJSB_OK;
}

}  // namespace

tfjsb_status tfjsb_conv2d_backprop_input(tfjsb_ctx* ctx, const tfjsb_tensor* dy, const tfjsb_tensor* filter, const int strides[2],
                                         tfjsb_pad pad, const int dilations[2], tfjsb_tensor* dx, void* stream) {
    TFJSB_REQUIRE_CTX(ctx);
    tfjsb_status st;
    if ((st = check_tensor(ctx, dy, "dy", 4, 4)) != TFJSB_OK) return st;
    if ((st = check_tensor(ctx, filter, "filter", 4, 4)) != TFJSB_OK) return st;
    if ((st = check_tensor(ctx, dx, "dx", 4, 4)) != TFJSB_OK) return st;
    ConvGeom g;
    if ((st = grad_geometry(ctx, dx, filter, dy, strides, pad, dilations, false, &g)) != TFJSB_OK) return st;
    if (overlaps(dx, dy) || overlaps(dx, filter)) return fail(ctx, TFJSB_ERR_INVALID_ARG, "dx aliases an input");
    if (numel(dx) == 0) return TFJSB_OK;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const float* pg = static_cast<const float*>(dy->data);
    const float* pf = static_cast<const float*>(filter->data);
    float* pdx = static_cast<float*>(dx->data);
    if (numel(dy) == 0 || g.Co == 0) {
        cudaError_t e = cudaMemsetAsync(pdx, 0, (size_t)numel(dx) * 4, s);
        return e == cudaSuccess ? TFJSB_OK : cuda_fail(ctx, e, "cudaMemsetAsync");
    }
    if (g.fh == 1 && g.fw == 1 && g.sh == 1 && g.sw == 1)
        // dx [M, Cin] = dy [M, Cout] . f [Cin, Cout]^T: both operands already have the summed index contiguous
        return matmul_2d(ctx, pg, pf, pdx, g.N * g.H * g.W, g.Co, g.C, 0, 1, s);
    cudaError_t e = launch_conv2d_backprop_input(pg, pf, pdx, g, ctx->sm_count, s, &ctx->launches);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "conv2d_backprop_input launch");
    return TFJSB_OK;
}

tfjsb_status tfjsb_conv2d_backprop_filter(tfjsb_ctx* ctx, const tfjsb_tensor* x, const tfjsb_tensor* dy, const int strides[2],
                                          tfjsb_pad pad, const int dilations[2], tfjsb_tensor* dfilter, void* stream) {
    TFJSB_REQUIRE_CTX(ctx);
    tfjsb_status st;
    if ((st = check_tensor(ctx, x, "x", 4, 4)) != TFJSB_OK) return st;
    if ((st = check_tensor(ctx, dy, "dy", 4, 4)) != TFJSB_OK) return st;
    if ((st = check_tensor(ctx, dfilter, "dfilter", 4, 4)) != TFJSB_OK) return st;
    ConvGeom g;
    if ((st = grad_geometry(ctx, x, dfilter, dy, strides, pad, dilations, false, &g)) != TFJSB_OK) return st;
    if (overlaps(dfilter, dy) || overlaps(dfilter, x)) return fail(ctx, TFJSB_ERR_INVALID_ARG, "dfilter aliases an input");
    if (numel(dfilter) == 0) return TFJSB_OK;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const float* px = static_cast<const float*>(x->data);
    const float* pg = static_cast<const float*>(dy->data);
    float* pdf = static_cast<float*>(dfilter->data);
    cudaError_t e;
    const int64_t pixels = g.N * g.Ho * g.Wo;
    if (pixels == 0) {
        e = cudaMemsetAsync(pdf, 0, (size_t)numel(dfilter) * 4, s);
        return e == cudaSuccess ? TFJSB_OK : cuda_fail(ctx, e, "cudaMemsetAsync");
    }
    const bool pointwise = g.fh == 1 && g.fw == 1 && g.sh == 1 && g.sw == 1;
    if (pointwise && ctx->math == TFJSB_MATH_TF32 && ctx->encode_tiled) {
        // df [Cin, Cout] = x^T . dy, a product whose summed index is the pixel.  The pixels are cut into B
        // slices; slice b of x and of dy is transposed into scratch ([Cin, M/B] and [Cout, M/B]), the B small
        // products run as one batched launch of the tensor-core GEMM (their tiles share the SMs), and the B
        // partial results are added in slice order.
        const int64_t M = pixels;
        const int64_t tiles = ((g.C + 127) / 128) * ((g.Co + 31) / 32);
        int64_t B = 0;
        for (int64_t cand = 1024; cand >= 1; cand >>= 1) {
            if (M % cand != 0 || (M / cand) % 4 != 0 || (cand > 1 && M / cand < 256)) continue;
            if (cand > 1 && cand * tiles > 8 * (int64_t)ctx->sm_count) continue;
            B = cand;
            break;
        }
        if (B >= 1 && gemm_tf32_supported(g.C, g.Co, M / B) && M / B <= 65535LL * 32) {
            const int64_t Ms = M / B;
            if ((st = ensure_scratch(ctx, &ctx->scratch_a, (size_t)M * g.C * 4)) != TFJSB_OK) return st;
            if ((st = ensure_scratch(ctx, &ctx->scratch_b, (size_t)M * g.Co * 4)) != TFJSB_OK) return st;
            if (B > 1 && (st = ensure_scratch(ctx, &ctx->scratch_c, (size_t)B * g.C * g.Co * 4)) != TFJSB_OK) return st;
            if ((e = launch_transpose_batched(px, ctx->scratch_a.ptr, B, Ms, g.C, s, &ctx->launches)) != cudaSuccess)
                return cuda_fail(ctx, e, "transpose(x)");
            if ((e = launch_transpose_batched(pg, ctx->scratch_b.ptr, B, Ms, g.Co, s, &ctx->launches)) != cudaSuccess)
                return cuda_fail(ctx, e, "transpose(dy)");
            GemmTf32Plan plan;
            float* target = B > 1 ? ctx->scratch_c.ptr : pdf;
            if ((st = gemm_tf32_plan(ctx, ctx->scratch_a.ptr, ctx->scratch_b.ptr, target, g.C, g.Co, Ms, &plan, B)) != TFJSB_OK) return st;
            if ((e = launch_gemm_tf32(plan, nullptr, TFJSB_ACT_NONE, ctx->dev_status, s, &ctx->launches)) != cudaSuccess)
                return cuda_fail(ctx, e, "tf32 gemm launch");
            if (B > 1 && (e = launch_sum_rows(ctx->scratch_c.ptr, pdf, nullptr, B, (int64_t)g.C * g.Co, 1, s, &ctx->launches)) != cudaSuccess)
                return cuda_fail(ctx, e, "partial-sum launch");
            return TFJSB_OK;
        }
    }
    int slices = backprop_slices(pixels, ctx->sm_count);
    const int64_t tile_blocks = (int64_t)g.fh * g.fw * ((g.C + 31) / 32) * ((g.Co + 31) / 32);
    while (slices > 1 && tile_blocks * slices > 16 * (int64_t)ctx->sm_count) slices >>= 1;
    if (slices > 1 && (st = ensure_scratch(ctx, &ctx->scratch_c, (size_t)slices * numel(dfilter) * 4)) != TFJSB_OK) return st;
    if ((e = launch_conv2d_backprop_filter(px, pg, pdf, ctx->scratch_c.ptr, slices, g, s, &ctx->launches)) != cudaSuccess)
        return cuda_fail(ctx, e, "conv2d_backprop_filter launch");
    return TFJSB_OK;
}

tfjsb_status tfjsb_depthwise_conv2d_backprop_input(tfjsb_ctx* ctx, const tfjsb_tensor* dy, const tfjsb_tensor* filter,
                                                   const int strides[2], tfjsb_pad pad, const int dilations[2], tfjsb_tensor* dx,
                                                   void* stream) {
    TFJSB_REQUIRE_CTX(ctx);
    tfjsb_status st;
    if ((st = check_tensor(ctx, dy, "dy", 4, 4)) != TFJSB_OK) return st;
    if ((st = check_tensor(ctx, filter, "filter", 4, 4)) != TFJSB_OK) return st;
    if ((st = check_tensor(ctx, dx, "dx", 4, 4)) != TFJSB_OK) return st;
    ConvGeom g;
    if ((st = grad_geometry(ctx, dx, filter, dy, strides, pad, dilations, true, &g)) != TFJSB_OK) return st;
    if (overlaps(dx, dy) || overlaps(dx, filter)) return fail(ctx, TFJSB_ERR_INVALID_ARG, "dx aliases an input");
    if (numel(dx) == 0) return TFJSB_OK;
    cudaError_t e = launch_depthwise_backprop_input(static_cast<const float*>(dy->data), static_cast<const float*>(filter->data),
                                                    static_cast<float*>(dx->data), g, ctx->sm_count,
                                                    static_cast<cudaStream_t>(stream), &ctx->launches);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "depthwise_backprop_input launch");
    return TFJSB_OK;
}

tfjsb_status tfjsb_depthwise_conv2d_backprop_filter(tfjsb_ctx* ctx, const tfjsb_tensor* x, const tfjsb_tensor* dy,
                                                    const int strides[2], tfjsb_pad pad, const int dilations[2],
                                                    tfjsb_tensor* dfilter, void* stream) {
    TFJSB_REQUIRE_CTX(ctx);
    tfjsb_status st;
    if ((st = check_tensor(ctx, x, "x", 4, 4)) != TFJSB_OK) return st;
    if ((st = check_tensor(ctx, dy, "dy", 4, 4)) != TFJSB_OK) return st;
    if ((st = check_tensor(ctx, dfilter, "dfilter", 4, 4)) != TFJSB_OK) return st;
    ConvGeom g;
    if ((st = grad_geometry(ctx, x, dfilter, dy, strides, pad, dilations, true, &g)) != TFJSB_OK) return st;
    if (overlaps(dfilter, dy) || overlaps(dfilter, x)) return fail(ctx, TFJSB_ERR_INVALID_ARG, "dfilter aliases an input");
    if (numel(dfilter) == 0) return TFJSB_OK;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int64_t pixels = g.N * g.Ho * g.Wo;
    if (pixels == 0) {
        cudaError_t e = cudaMemsetAsync(dfilter->data, 0, (size_t)numel(dfilter) * 4, s);
        return e == cudaSuccess ? TFJSB_OK : cuda_fail(ctx, e, "cudaMemsetAsync");
    }
    int slices = backprop_slices(pixels, ctx->sm_count);
    if (slices > 1 && (st = ensure_scratch(ctx, &ctx->scratch_c, (size_t)slices * numel(dfilter) * 4)) != TFJSB_OK) return st;
    cudaError_t e = launch_depthwise_backprop_filter(static_cast<const float*>(x->data), static_cast<const float*>(dy->data),
                                                     static_cast<float*>(dfilter->data), ctx->scratch_c.ptr, slices, g, s,
                                                     &ctx->launches);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "depthwise_backprop_filter launch");
    return TFJSB_OK;
}

tfjsb_status tfjsb_act_backprop(tfjsb_ctx* ctx, const tfjsb_tensor* y, const tfjsb_tensor* dy, tfjsb_act act, tfjsb_tensor* dz,
                                void* stream) {
    TFJSB_REQUIRE_CTX(ctx);
    tfjsb_status st;
    if (act != TFJSB_ACT_NONE && act != TFJSB_ACT_RELU && act != TFJSB_ACT_RELU6) return fail(ctx, TFJSB_ERR_INVALID_ARG, "unknown activation");
    if ((st = check_tensor(ctx, y, "y", 1, 4)) != TFJSB_OK) return st;
    if ((st = check_tensor(ctx, dy, "dy", 1, 4)) != TFJSB_OK) return st;
    if ((st = check_tensor(ctx, dz, "dz", 1, 4)) != TFJSB_OK) return st;
    if (dy->rank != y->rank || dz->rank != y->rank) return fail(ctx, TFJSB_ERR_SHAPE, "y, dy and dz must have one shape");
    for (int i = 0; i < y->rank; ++i)
        if (dy->dims[i] != y->dims[i] || dz->dims[i] != y->dims[i]) return fail(ctx, TFJSB_ERR_SHAPE, "y, dy and dz must have one shape");
    if (overlaps(dz, y) || overlaps(dz, dy)) return fail(ctx, TFJSB_ERR_INVALID_ARG, "dz aliases an input");
    if (numel(y) == 0) return TFJSB_OK;
    cudaError_t e = launch_act_backprop(static_cast<const float*>(y->data), static_cast<const float*>(dy->data),
                                        static_cast<float*>(dz->data), numel(y), act, ctx->sm_count,
                                        static_cast<cudaStream_t>(stream), &ctx->launches);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "act_backprop launch");
    return TFJSB_OK;
}

tfjsb_status tfjsb_bias_backprop(tfjsb_ctx* ctx, const tfjsb_tensor* dz, tfjsb_tensor* dbias, void* stream) {
    TFJSB_REQUIRE_CTX(ctx);
    tfjsb_status st;
    if ((st = check_tensor(ctx, dz, "dz", 1, 4)) != TFJSB_OK) return st;
    if ((st = check_tensor(ctx, dbias, "dbias", 1, 1)) != TFJSB_OK) return st;
    const int64_t C = dz->dims[dz->rank - 1];
    if (dbias->dims[0] != C) return fail(ctx, TFJSB_ERR_SHAPE, "dbias must have the length of dz's last dimension");
    if (overlaps(dbias, dz)) return fail(ctx, TFJSB_ERR_INVALID_ARG, "dbias aliases the input");
    if (C == 0) return TFJSB_OK;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int64_t rows = numel(dz) / C;
    if (rows == 0) {
        cudaError_t e = cudaMemsetAsync(dbias->data, 0, (size_t)C * 4, s);
        return e == cudaSuccess ? TFJSB_OK : cuda_fail(ctx, e, "cudaMemsetAsync");
    }
    const int slices = backprop_slices(rows, ctx->sm_count);
    if (slices > 1 && (st = ensure_scratch(ctx, &ctx->scratch_c, (size_t)slices * C * 4)) != TFJSB_OK) return st;
    cudaError_t e = launch_sum_rows(static_cast<const float*>(dz->data), static_cast<float*>(dbias->data), ctx->scratch_c.ptr, rows, C,
                                    slices, s, &ctx->launches);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "bias_backprop launch");
    return TFJSB_OK;
}

}  // extern "C"

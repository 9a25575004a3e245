// Shared declarations of the CUDA library: context, error helpers, the fused epilogue,
// and the host-side launchers each kernel file exports to the API layer.
#pragma once

#include <cuda_runtime.h>
#include <cuda.h>
#include <stdint.h>

#include <string>
#include <utility>
#include <vector>

#include "tfjsb.h"

namespace tfjsb {

// ---- device status word -------------------------------------------------------------------
// Kernels with bounded waits OR a code into this word when a wait gives up; the host reads it
// in tfjsb_check_device_status.
enum : unsigned int {
    DEV_STATUS_OK = 0u,
    DEV_STATUS_TIMEOUT_PRODUCER = 1u,  // TMA producer waited too long for a free stage
    DEV_STATUS_TIMEOUT_MMA = 2u,       // MMA issuer waited too long for data or for a free accumulator
    DEV_STATUS_TIMEOUT_EPILOGUE = 4u,  // epilogue waited too long for an accumulator
    DEV_STATUS_TIMEOUT_DRAIN = 8u,     // teardown waited too long for copies in flight
    DEV_STATUS_TIMEOUT_DEPTHWISE = 16u // depthwise kernel waited too long for an input tile
};

// ---- fused epilogue (bias add, then activation), identical in every kernel -----------------
//   v = acc + bias ; relu: v > 0 ? v : +0 (NaN stays NaN, -0 -> +0) ; relu6: min(relu(v), 6)
// max.NaN / min.NaN return NaN when an input is NaN and order -0 below +0, which is exactly that
// definition in two instructions (a compare-and-select chain costs four times as many, and the
// bandwidth-bound kernels turned out to be bound by instruction issue).
__device__ __forceinline__ float relu_nan(float v) {
    float r;
    asm("max.NaN.f32 %0, %1, 0f00000000;" : "=f"(r) : "f"(v));
    return r;
}
__device__ __forceinline__ float relu6_nan(float v) {
    float r;
    asm("max.NaN.f32 %0, %1, 0f00000000;\n\tmin.NaN.f32 %0, %0, 0f40C00000;" : "=f"(r) : "f"(v));
    return r;
}
__device__ __forceinline__ float apply_act(float v, int act) {
    const float r = relu_nan(v);
    const float r6 = relu6_nan(v);
    return act == TFJSB_ACT_NONE ? v : (act == TFJSB_ACT_RELU6 ? r6 : r);
}
// Two independent fp32 FMAs in one instruction (sm_100 packed fp32): acc.{x,y} += a.{x,y} * b.{x,y},
// each lane rounded exactly like a scalar fmaf.  Halves the issue slots of the CUDA-core kernels,
// which are bound by instruction issue.
__device__ __forceinline__ void fma2(float2& acc, const float2& a, const float2& b) {
    unsigned long long& d = reinterpret_cast<unsigned long long&>(acc);
    asm("fma.rn.f32x2 %0, %1, %2, %0;"
        : "+l"(d)
        : "l"(reinterpret_cast<const unsigned long long&>(a)), "l"(reinterpret_cast<const unsigned long long&>(b)));
}
__device__ __forceinline__ void fma4_packed(float4& acc, const float4& a, const float4& b) {
    fma2(reinterpret_cast<float2*>(&acc)[0], reinterpret_cast<const float2*>(&a)[0], reinterpret_cast<const float2*>(&b)[0]);
    fma2(reinterpret_cast<float2*>(&acc)[1], reinterpret_cast<const float2*>(&a)[1], reinterpret_cast<const float2*>(&b)[1]);
}

template <int ACT>
__device__ __forceinline__ float apply_act_t(float v) {
    if (ACT == TFJSB_ACT_NONE) return v;
    if (ACT == TFJSB_ACT_RELU6) return relu6_nan(v);
    return relu_nan(v);
}

// ---- context --------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct Scratch {
    float* ptr = nullptr;
    size_t bytes = 0;
};

}  // namespace tfjsb

struct tfjsb_ctx {
    int device = 0;
    int sm_count = 0;
    tfjsb_math math = TFJSB_MATH_TF32;
    std::string last_error;
    unsigned int* dev_status = nullptr;  // device status word
    tfjsb::EncodeTiledFn encode_tiled = nullptr;
    tfjsb::Scratch scratch_a, scratch_b;  // transposed operands of tfjsb_matmul
    tfjsb::Scratch scratch_c;             // partial sums of the filter / bias gradients
    std::vector<void*> retired;            // outgrown scratch blocks, freed at shutdown
    int64_t launches = 0;
    int live_models = 0;
};

namespace tfjsb {

tfjsb_status fail(tfjsb_ctx* ctx, tfjsb_status st, const std::string& msg);
tfjsb_status cuda_fail(tfjsb_ctx* ctx, cudaError_t err, const char* what);
// Grows `s` to at least `bytes`.  Never synchronises: an outgrown block may still be read by kernels in
// flight on any stream, so it is kept until tfjsb_shutdown; growth is geometric, so all outgrown blocks
// together are smaller than the live one.  tfjsb_reserve_scratch sizes the blocks up front.
tfjsb_status ensure_scratch(tfjsb_ctx* ctx, Scratch* s, size_t bytes);

// Raises a kernel's dynamic shared-memory limit once per (kernel, device): function attributes belong to
// a device's copy of the function, and contexts on several devices or host threads may launch the same kernel.
cudaError_t smem_attr_once(const void* kernel, int bytes);
// Number of SMs of the current device (cached per device): grid caps of the grid-stride kernels.
int current_sm_count();

// ---- kernel launch with optional programmatic dependent launch --------------------------------------
// The executor sets this while it enqueues a model: its kernels all call pdl_wait() before reading
// their inputs, so each may be launched while the previous one drains and only its prologue
// (barrier set-up, tensor-map prefetch, TMEM allocation) overlaps.  Off for stand-alone op calls.
extern thread_local bool g_launch_pdl;

template <typename... KArgs, typename... Args>
cudaError_t launch_k(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = g_launch_pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}

// The same launch without the attribute, whatever the executor's setting: for kernels made of many
// small blocks with little shared memory.  Launched early, their first blocks become resident beside
// the predecessor's CTAs and wait there, and that costs the predecessor more than the overlap returns
// (measured: a model whose depthwise layers are such kernels ran 4 % slower with the attribute on
// them, and the fp32 model 9 % slower when its depthwise layers were swapped for such a kernel; the
// persistent kernels with large shared-memory footprints cannot become resident early and only
// overlap their prologue).  Such a kernel still executes griddepcontrol.launch_dependents, so its
// successor may start early.
template <typename... KArgs, typename... Args>
cudaError_t launch_k_serial(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cfg.attrs = nullptr;
    cfg.numAttrs = 0;
    return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}

// ---- geometry of one convolution / pooling call -----------------------------------------------
struct ConvGeom {
    int64_t N;
    int H, W, C;        // input
    int fh, fw;         // filter window
    int Co;             // output channels (conv: Cout; depthwise: C*mult; pool: C)
    int mult;           // depthwise channel multiplier (1 otherwise)
    int sh, sw, dh, dw; // strides, dilations
    int pt, pl;         // padding before (top, left)
    int Ho, Wo;
};

// ---- launchers (each returns the CUDA launch error; `launches` is incremented per kernel) -----
cudaError_t launch_bias_act(const float* x, const float* bias, float* y, int64_t rows, int64_t C, int act,
                            cudaStream_t s, int64_t* launches);
cudaError_t launch_avg_pool(const float* x, float* y, const ConvGeom& g, cudaStream_t s, int64_t* launches);
cudaError_t launch_softmax(const float* x, float* y, int64_t rows, int64_t cols, cudaStream_t s, int64_t* launches);
cudaError_t launch_max_pool(const float* x, float* y, const ConvGeom& g, cudaStream_t s, int64_t* launches);
// out[i] = a[i] op b[i % b_len] (op: tfjsb_binary_op)
cudaError_t launch_binary(int op, const float* a, const float* b, float* out, int64_t n, int64_t b_len, cudaStream_t s,
                          int64_t* launches);
// out[c, r] = in[r, c] for in of shape [rows, cols]
cudaError_t launch_transpose(const float* in, float* out, int64_t rows, int64_t cols, cudaStream_t s,
                             int64_t* launches);

// C[M,N] = act(A' B' + bias), CUDA-core fp32.  A' element (i,k) at a[i*a_rs + k*a_cs]; B' element
// (k,j) at b[k*b_rs + j*b_cs]; C row pitch ldc.
cudaError_t launch_gemm_fp32(const float* a, int64_t a_rs, int64_t a_cs, const float* b, int64_t b_rs, int64_t b_cs,
                             const float* bias, int act, float* c, int64_t ldc, int64_t M, int64_t N, int64_t K,
                             cudaStream_t s, int64_t* launches);

// Direct convolution on CUDA cores (any window, stride, dilation).  filter [fh,fw,Cin,Cout].
cudaError_t launch_conv2d_fp32(const float* x, const float* f, const float* bias, int act, float* y,
                               const ConvGeom& g, cudaStream_t s, int64_t* launches);

// Depthwise convolution.  filter [fh,fw,C,mult].  A plan picks the kernel and, for the bulk-copy
// pipelined 3x3 kernel, holds the tensor map of the input; it stays valid while `x` and the
// geometry stay the same.
struct DepthwisePlan {
    int variant = -1;  // -1: register kernel / scalar kernel; >= 0: index of the pipelined instance
    CUtensorMap map_x;
    int tiles_x = 0, tiles_y = 0, c_blocks = 0;
    int64_t num_tiles = 0;
    int grid = 0, stages = 0;
    size_t smem_bytes = 0;
    bool narrow = false;  // planned for bfloat16 storage
};
// `narrow`: x is bfloat16 (narrow storage); the plan then runs through launch_depthwise_tma_narrow, and
// variant stays -1 where the pipelined kernel has no instance for the shape.
tfjsb_status depthwise_plan(tfjsb_ctx* ctx, const void* x, const ConvGeom& g, DepthwisePlan* plan, bool narrow = false);
cudaError_t launch_depthwise_tma_narrow(const DepthwisePlan& plan, const float* f, const float* bias, int act, void* y,
                                        bool y_is_bf16, const ConvGeom& g, unsigned int* dev_status, cudaStream_t s,
                                        int64_t* launches);
cudaError_t launch_depthwise(const DepthwisePlan& plan, const float* x, const float* f, const float* bias, int act,
                             float* y, const ConvGeom& g, unsigned int* dev_status, cudaStream_t s,
                             int64_t* launches);

// Tensor-core GEMM: C[M,N] = act(A[M,K] . Bt[N,K]^T + bias); all three row-major with K (resp. N)
// contiguous.  A plan holds the tensor maps and tile choice; it can be built once and reused while
// the pointers stay the same.
struct GemmTf32Plan {
    CUtensorMap map_a, map_b, map_c;
    int64_t M, N, K;
    int64_t batches = 1;  // independent products of this shape in one launch (single-CTA kernel only)
    int block_n;       // 32..256
    int stages;
    int acc_stages;
    int num_tiles;
    int grid;
    size_t smem_bytes;
    // CTA-pair kernel (gemm_pair.cu): 256 x block_n tiles shared by two CTAs
    bool pair = false;
    // cluster split-K kernel (gemm_tf32_splitk.cu): `splits` CTAs per tile, reduced through shared memory
    bool cluster_split = false;
    int splits = 1, kb_per_split = 0;  // slices of the K loop (= cluster size) and k-blocks per slice
    float* c = nullptr;                // C, which that kernel stores directly
    // implicit-GEMM convolution: A is gathered from x by the kernel instead of copied
    bool gather = false;
    const float* x = nullptr;
    ConvGeom g{};
};
bool gemm_tf32_supported(int64_t M, int64_t N, int64_t K);
// `batches` > 1: that many products of the same shape, operands and results stored one after the other.
tfjsb_status gemm_tf32_plan(tfjsb_ctx* ctx, const float* a, const float* bt, float* c, int64_t M, int64_t N,
                            int64_t K, GemmTf32Plan* plan, int64_t batches = 1);
// The same GEMM on CTA pairs; gemm_tf32_plan picks it where it is the faster kernel (environment
// variable TFJSB_GEMM_PAIR: 0 = never, 1 = wherever the shape allows, unset = by shape).
bool gemm_tf32_pair_preferred(int64_t M, int64_t N, int64_t K, int sm_count);
tfjsb_status gemm_tf32_pair_plan(tfjsb_ctx* ctx, const float* a, const float* bt, float* c, int64_t M, int64_t N,
                                 int64_t K, GemmTf32Plan* plan);
cudaError_t launch_gemm_tf32_pair(const GemmTf32Plan& plan, const float* bias, int act, unsigned int* dev_status,
                                  cudaStream_t s, int64_t* launches);
// Split K across the CTAs of a cluster, for GEMMs with too few tiles for the SMs (gemm_tf32_splitk.cu).
bool gemm_tf32_splitk_choice(int64_t M, int64_t N, int64_t K, int sm_count, int* block_n, int* splits);
tfjsb_status gemm_tf32_splitk_plan(tfjsb_ctx* ctx, const float* a, const float* bt, float* c, int64_t M, int64_t N,
                                   int64_t K, int block_n, int splits, GemmTf32Plan* plan);
cudaError_t launch_gemm_tf32_splitk(const GemmTf32Plan& plan, const float* bias, int act, unsigned int* dev_status,
                                    cudaStream_t s, int64_t* launches);
// Implicit-GEMM convolution on the same kernel: M = N*Ho*Wo output pixels, K = fh*fw*Cin, N = Cout.
// `bt` is the filter packed as [Cout, k_pad] (K-contiguous, zero padded to a multiple of 32).
bool conv_igemm_supported(const ConvGeom& g);
int64_t conv_igemm_k_pad(const ConvGeom& g);
tfjsb_status conv_igemm_plan(tfjsb_ctx* ctx, const float* x, const float* bt, float* y, const ConvGeom& g,
                             GemmTf32Plan* plan);
// out[n, k] = k < K ? f[k, n] : 0 for f of shape [K, N], out of shape [N, k_pad]
cudaError_t launch_pack_filter(const float* f, float* out, int64_t K, int64_t N, int64_t k_pad, cudaStream_t s,
                               int64_t* launches);
cudaError_t launch_gemm_tf32(const GemmTf32Plan& plan, const float* bias, int act, unsigned int* dev_status,
                             cudaStream_t s, int64_t* launches);

// ---- narrow storage (bfloat16 in memory, fp32 sums) -------------------------------------------------
// Tensor-core GEMM on bfloat16 operands: C[M,N] = act(A[M,K] . Bt[N,K]^T + bias), C bfloat16 or fp32.
struct GemmBf16Plan {
    CUtensorMap map_a, map_b, map_c;
    int64_t M = 0, N = 0, K = 0;
    bool c_is_bf16 = true;
    bool pair = false;  // CTA-pair kernel (gemm_pair.cu): 256 x block_n tiles shared by two CTAs
    int block_n = 0, stages = 0, acc_stages = 0, num_tiles = 0, grid = 0;
    int epi_warps = 16;  // epilogue warps of the single-CTA kernel: 16 for short K loops, 8 otherwise
    size_t smem_bytes = 0;
};
bool gemm_bf16_supported(int64_t M, int64_t N, int64_t K);
tfjsb_status gemm_bf16_plan(tfjsb_ctx* ctx, const void* a, const void* bt, void* c, bool c_is_bf16, int64_t M, int64_t N,
                            int64_t K, GemmBf16Plan* plan);
cudaError_t launch_gemm_bf16(const GemmBf16Plan& plan, const float* bias, int act, unsigned int* dev_status,
                             cudaStream_t s, int64_t* launches);
// The same GEMM (bfloat16 output only) on CTA pairs; gemm_bf16_plan picks it where it is the faster
// kernel (TFJSB_GEMM_PAIR: 0 = never, 1 = wherever the shape allows, unset = by shape).
bool gemm_bf16_pair_preferred(int64_t M, int64_t N, int64_t K, int sm_count);
tfjsb_status gemm_bf16_pair_plan(tfjsb_ctx* ctx, const void* a, const void* bt, void* c, int64_t M, int64_t N, int64_t K,
                                 GemmBf16Plan* plan);
cudaError_t launch_gemm_bf16_pair(const GemmBf16Plan& plan, const float* bias, int act, unsigned int* dev_status,
                                  cudaStream_t s, int64_t* launches);
// CUDA-core layers of the same mode.  Filters are fp32 arrays holding bfloat16 values.
cudaError_t launch_conv_narrow(const void* x, bool x_is_f32, const float* f, const float* bias, int act, void* y,
                               bool y_is_bf16, const ConvGeom& g, cudaStream_t s, int64_t* launches);
bool depthwise_narrow_supported(const ConvGeom& g);
cudaError_t launch_depthwise_narrow(const void* x, const float* f, const float* bias, int act, void* y, bool y_is_bf16,
                                    const ConvGeom& g, cudaStream_t s, int64_t* launches);
cudaError_t launch_avg_pool_global_narrow(const void* x, void* y, bool y_is_bf16, int64_t images, int positions, int C,
                                          cudaStream_t s, int64_t* launches);
cudaError_t launch_f32_to_bf16(const float* in, void* out, int64_t n, cudaStream_t s, int64_t* launches);
cudaError_t launch_bf16_to_f32(const void* in, float* out, int64_t n, cudaStream_t s, int64_t* launches);
cudaError_t launch_round_to_bf16_in_place(float* v, int64_t n, cudaStream_t s, int64_t* launches);
// out [r*N, r*K] = r copies of km [N, K] down the diagonal, zeros elsewhere
cudaError_t launch_block_diagonal(const float* km, float* out, int64_t N, int64_t K, int r, cudaStream_t s, int64_t* launches);

// ---- gradients (backprop.cu) ----------------------------------------------------------------------
// `g` is the geometry of the FORWARD op (H, W, C the forward input; Ho, Wo, Co the forward output).
int backprop_slices(int64_t rows, int sm_count);
cudaError_t launch_conv2d_backprop_input(const float* dy, const float* f, float* dx, const ConvGeom& g, int sm_count,
                                         cudaStream_t s, int64_t* launches);
// `partial` holds slices * fh*fw*C*Co floats (unused when slices == 1)
cudaError_t launch_conv2d_backprop_filter(const float* x, const float* dy, float* df, float* partial, int slices,
                                          const ConvGeom& g, cudaStream_t s, int64_t* launches);
cudaError_t launch_depthwise_backprop_input(const float* dy, const float* f, float* dx, const ConvGeom& g, int sm_count,
                                            cudaStream_t s, int64_t* launches);
// `partial` holds slices * fh*fw*Co floats (unused when slices == 1)
cudaError_t launch_depthwise_backprop_filter(const float* x, const float* dy, float* df, float* partial, int slices,
                                             const ConvGeom& g, cudaStream_t s, int64_t* launches);
cudaError_t launch_act_backprop(const float* y, const float* dy, float* dz, int64_t n, int act, int sm_count, cudaStream_t s,
                                int64_t* launches);
// out[c] = sum_r in[r, c]; with slices > 1 in two steps through `partial` (slices * C floats)
cudaError_t launch_sum_rows(const float* in, float* out, float* partial, int64_t rows, int64_t C, int slices, cudaStream_t s,
                            int64_t* launches);
// out[b, c, r] = in[b, r, c] for `batches` matrices [rows, cols] stored one after the other
cudaError_t launch_transpose_batched(const float* in, float* out, int64_t batches, int64_t rows, int64_t cols, cudaStream_t s,
                                     int64_t* launches);

// Fused depthwise 3x3 (stride 1) + pointwise block: the depthwise output is produced straight into
// the tensor-core operand layout in shared memory and never written to global memory.
// `bt` is the pointwise filter stored [Cout, Cin] (K-contiguous).
struct DwPwPlan {
    CUtensorMap map_x, map_b, map_y;
    ConvGeom g{};   // geometry of the depthwise layer
    int Co = 0;
    int block_n = 0, n_sub = 1, acc_stages = 0, patch_stages = 0, a_stages = 0, b_stages = 0;
    bool b_resident = false;  // the B ring holds all of Bt for the whole kernel
    bool wide_epi = false;    // sixteen epilogue warps and one depthwise group (one k-block per tile)
    int tiles_x = 0, tiles_y = 0, num_tiles = 0, grid = 0;
    size_t smem_bytes = 0;
    int patch_bytes = 0, patch_stride = 0;
    // small-window convolution mode of the same kernel
    bool conv = false;
    bool y_bf16 = false;  // the output tensor is bfloat16 (narrow storage): small-window mode only
    int row_floats = 0, patch_rows = 0;
};
bool dwpw_fused_supported(const ConvGeom& dw, int64_t Cout);
// `narrow`: x and y are bfloat16 (narrow storage), bt holds bfloat16 values as fp32
tfjsb_status dwpw_fused_plan(tfjsb_ctx* ctx, const void* x, const float* bt, void* y, const ConvGeom& dw,
                             int64_t Cout, DwPwPlan* plan, bool narrow = false);
// conv2d with fh*fw*Cin <= 32 on the same kernel (input patch by bulk tensor copy, im2col in shared
// memory); `bt` is the filter packed [Cout, 32].  Launched with launch_dwpw_fused (pw_bias / pw_act = the
// convolution's bias and activation; the depthwise arguments are ignored).
bool conv_patch_supported(const ConvGeom& g);
tfjsb_status conv_patch_plan(tfjsb_ctx* ctx, const float* x, const float* bt, void* y, const ConvGeom& g, DwPwPlan* plan,
                             bool y_bf16 = false);
cudaError_t launch_dwpw_fused(const DwPwPlan& plan, const float* dw_filter, const float* dw_bias, int dw_act,
                              const float* pw_bias, int pw_act, unsigned int* dev_status, cudaStream_t s,
                              int64_t* launches);

}  // namespace tfjsb

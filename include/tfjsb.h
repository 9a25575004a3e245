/*
 * tfjsb — op kernels and a small graph executor for a TensorFlow.js-style inference path,
 * written for NVIDIA B200 (sm_100a).  C ABI of libtfjsb.so.
 *
 * The op list follows the ops API of "TensorFlow.js: Machine Learning for the Web and
 * Beyond" (arxiv 1901.05350): operations are device-independent calls that dispatch to
 * device kernels (Sec. 3.3); tf.matMul and tf.conv2d are the ops the paper names
 * (Sec. 3.6, Sec. 4.1, Listing 2); the model the paper times is MobileNet v1 (Table 1,
 * Sec. 3.9), which also needs depthwiseConv2d, the fused bias + relu/relu6 epilogue,
 * avgPool and softmax.  The paper does not define those ops' arithmetic; this library
 * follows TensorFlow's definitions (cross-correlation, NHWC, HWIO filters, 'same' padding
 * with the odd element after, avgPool dividing by the in-bounds count).
 *
 * Conventions shared by every call
 *   Tensors   fp32, dense, row-major, last dimension contiguous; 4-D tensors are NHWC.
 *             `tfjsb_tensor.data` is a DEVICE pointer unless a parameter says "host".
 *             It must be 16-byte aligned.  The caller owns every tensor it passes; `out`
 *             must be pre-allocated with exactly the inferred shape and must not alias an
 *             input (tensors are immutable, ops are functional: Sec. 3.7).
 *             A reshape is the caller changing `rank`/`dims` over the same `data`
 *             (reshape is free: Sec. 3.4).
 *   Async     Every op enqueues its kernels on `stream` (a cudaStream_t passed as void*;
 *             NULL = the legacy default stream) and returns without synchronising, like
 *             the paper's ops returning a handle before the GPU is done (Sec. 4.1.1).
 *             Results are valid once the caller synchronises the stream.
 *   Errors    Every call returns a tfjsb_status.  All argument checks happen on the host
 *             before anything is launched; on error nothing has been enqueued.
 *             `tfjsb_last_error` gives a message for the last failing call on that context
 *             (valid until the next call on the context).  No CPU fallback exists: with no
 *             usable CUDA device `tfjsb_init` fails with TFJSB_ERR_CUDA.
 *   Threads   A context may be used from one host thread at a time.
 *   Streams   The kernels are written to have the GPU to themselves: persistent grids sized to all SMs,
 *             tensor memory and most of an SM's shared memory per CTA.  Enqueue the work of a process on one
 *             stream at a time, or order the streams with events; kernels of two streams that run side by
 *             side on the same SMs are not a supported configuration (copies on a second stream are fine:
 *             `tfjsb_run_model_host_async` does that itself).
 */
#ifndef TFJSB_H_
#define TFJSB_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct tfjsb_ctx tfjsb_ctx;
typedef struct tfjsb_model tfjsb_model;

typedef struct {
    void* data;      /* device pointer to fp32 elements, 16-byte aligned */
    int32_t rank;    /* 1..4 */
    int64_t dims[4]; /* dims[0..rank-1]; the rest ignored */
} tfjsb_tensor;

typedef enum {
    TFJSB_OK = 0,
    TFJSB_ERR_INVALID_ARG = 1, /* null pointer, bad enum, bad rank, misaligned pointer, aliasing */
    TFJSB_ERR_SHAPE = 2,       /* dimensions inconsistent with each other or with `out` */
    TFJSB_ERR_UNSUPPORTED = 3, /* valid in principle, not implemented (e.g. stride>1 with dilation>1) */
    TFJSB_ERR_CUDA = 4,        /* a CUDA runtime/driver call failed; message holds the CUDA error */
    TFJSB_ERR_TIMEOUT = 5,     /* a bounded device-side wait gave up (reported by tfjsb_check_device_status) */
    TFJSB_ERR_OOM = 6          /* device allocation failed */
} tfjsb_status;

typedef enum { TFJSB_PAD_VALID = 0, TFJSB_PAD_SAME = 1 } tfjsb_pad;
typedef enum { TFJSB_ACT_NONE = 0, TFJSB_ACT_RELU = 1, TFJSB_ACT_RELU6 = 2 } tfjsb_act;

/* Which multiplier the GEMM-shaped ops (matMul, conv2d, dense) use.
 *   TF32  tensor cores (tcgen05, operands read as TF32, fp32 accumulation in tensor memory)
 *         wherever the shape allows, CUDA cores otherwise.  Default.
 *   FP32  CUDA-core FFMA everywhere: the variant kept for exactness checks.
 *   BF16  narrow storage (the counterpart of the paper's 16-bit float textures, Sec. 4.1.3): a model
 *         created in this mode keeps its filters and every layer output except dense / softmax
 *         outputs and its final result as bfloat16 in device memory (rounded to nearest even, once,
 *         when stored); products of stored values are exact, sums are fp32, biases stay fp32, and
 *         1x1 convolutions and dense layers run on the tensor cores (tcgen05 kind::f16).  The model's
 *         input and output tensors stay fp32 (the input is rounded as it is read).  Supported layers:
 *         conv2d (must come first), depthwise 3x3 (stride 1 or 2, no dilation, multiplier 1, channels
 *         a multiple of 8), global avgPool, dense, softmax after dense.  The op entry points that
 *         take fp32 tensors run their FP32 path in this mode. */
typedef enum { TFJSB_MATH_TF32 = 0, TFJSB_MATH_FP32 = 1, TFJSB_MATH_BF16 = 2 } tfjsb_math;
typedef enum { TFJSB_BINARY_ADD = 0, TFJSB_BINARY_SUB = 1, TFJSB_BINARY_MUL = 2 } tfjsb_binary_op;

/* ---- context ------------------------------------------------------------------------ */

/* Creates a context on CUDA device `device` (makes it current for the calling thread).
 * Allocates a small device status word and, lazily, scratch memory for transposes.
 * Fails with TFJSB_ERR_CUDA when there is no such device or it is not compute capability 10.x. */
tfjsb_status tfjsb_init(int device, tfjsb_ctx** ctx);
/* Synchronises the device, frees everything the context owns.  Models must be destroyed first. */
tfjsb_status tfjsb_shutdown(tfjsb_ctx* ctx);
tfjsb_status tfjsb_set_math(tfjsb_ctx* ctx, tfjsb_math mode);
const char* tfjsb_last_error(tfjsb_ctx* ctx);
/* Synchronises `stream`, then reads the device status word that kernels with bounded waits
 * write.  Returns TFJSB_ERR_TIMEOUT (and clears the word) if any wait gave up since the last
 * check, TFJSB_OK otherwise. */
tfjsb_status tfjsb_check_device_status(tfjsb_ctx* ctx, void* stream);
/* Sizes the context's three scratch blocks (transposed matMul operands, partial sums of the filter and
 * bias gradients) to at least `bytes` each, so that later op calls find them large enough.  An op that
 * needs more grows its block by allocating a larger one (cudaMalloc, no synchronisation; the old block is
 * kept until tfjsb_shutdown because kernels in flight may still read it). */
tfjsb_status tfjsb_reserve_scratch(tfjsb_ctx* ctx, int64_t bytes);
/* Number of kernels this context (and its models) has launched since creation. */
int64_t tfjsb_launch_count(tfjsb_ctx* ctx);

/* ---- shape inference (pure host arithmetic) ------------------------------------------ */

/* One spatial dimension of a convolution or pooling window.
 *   ek = (k-1)*dilation + 1
 *   VALID: out = floor((in - ek)/stride) + 1, no padding; in < ek is TFJSB_ERR_SHAPE
 *   SAME : out = ceil(in/stride); total = max((out-1)*stride + ek - in, 0);
 *          pad_before = floor(total/2); pad_after = total - pad_before.
 * Any of out / pad_before / pad_after may be NULL. */
tfjsb_status tfjsb_window_out_shape(int64_t in, int k, int stride, int dilation, tfjsb_pad pad,
                                    int64_t* out, int* pad_before, int* pad_after);

/* ---- ops ---------------------------------------------------------------------------- */

/* tf.matMul (Sec. 3.6; Listing 2 is the no-transpose case).
 *   out[M,N] = op(a) . op(b);  a is [M,K], or [K,M] when transpose_a; b is [K,N], or [N,K]
 *   when transpose_b.  Rank 2 only.  Inner-dimension or `out` mismatch: TFJSB_ERR_SHAPE.
 * TF32 mode uses the tensor-core kernel when K % 4 == 0 and N % 4 == 0 (row pitches must be
 * multiples of 16 bytes for the bulk tensor copies); operands that are not already K-contiguous
 * are transposed into context-owned scratch first (grown on demand without synchronising, see
 * tfjsb_reserve_scratch).  Other shapes, and FP32 mode, run on CUDA cores. */
tfjsb_status tfjsb_matmul(tfjsb_ctx* ctx, const tfjsb_tensor* a, const tfjsb_tensor* b, int transpose_a,
                          int transpose_b, tfjsb_tensor* out, void* stream);

/* The same operation as tfjsb_matmul for callers that must not allocate device memory; the
 * paper has no counterpart of this call.  tfjsb_matmul transposes operands that are not
 * K-contiguous into scratch memory it takes from cudaMalloc.  Some callers cannot afford that
 * where they call the library: a real-time loop that may not block on the allocator or on the
 * device synchronisation an allocation can imply, a service whose device-memory budget was
 * fixed at start-up, any code that runs at a point where cudaMalloc is not permitted.  Here the
 * scratch is a fixed 16 MiB array that is part of the library's device image on every GPU that
 * loads it (held until the process exits), and the call never allocates or frees anything.
 * Create `ctx` at start-up, while allocating is still allowed.
 *   Limit     (a's elements if transpose_a) + (b's elements if not transpose_b), each rounded up
 *             to 64, must not exceed 4 Mi floats; otherwise TFJSB_ERR_UNSUPPORTED with the sizes
 *             in the message and nothing launched.  Operands already K-contiguous need no scratch.
 *   Sharing   one array per GPU, shared by all calls and contexts and never cleared (every
 *             element read is overwritten first).  Calls whose kernels may overlap on the GPU
 *             race on it: keep them on one stream or order them with events.
 *   Set-up    the first call on a GPU looks up the array's device address
 *             (cudaGetSymbolAddress); make that first call before any stream capture starts.
 * Arguments, results and every other rule are those of tfjsb_matmul. */
tfjsb_status tfjsb_matmul_static_scratch(tfjsb_ctx* ctx, const tfjsb_tensor* a, const tfjsb_tensor* b,
                                         int transpose_a, int transpose_b, tfjsb_tensor* out, void* stream);

/* tf.conv2d with an optional fused bias and activation.
 *   x [N,H,W,Cin], filter [fh,fw,Cin,Cout], bias NULL or [Cout], out [N,Ho,Wo,Cout]
 *   out[n,oy,ox,co] = act( bias[co] + sum_{ky,kx,ci} x[n, oy*sh - pt + ky*dh, ox*sw - pl + kx*dw, ci]
 *                                                  * filter[ky,kx,ci,co] ),   outside the image = 0
 *   strides = {sh, sw}, dilations = {dh, dw}; Ho/Wo/pt/pl from tfjsb_window_out_shape.
 * A stride > 1 together with a dilation > 1 is TFJSB_ERR_UNSUPPORTED.
 * 1x1 / stride 1 filters run as a GEMM over x viewed as [N*H*W, Cin]. */
tfjsb_status tfjsb_conv2d(tfjsb_ctx* ctx, const tfjsb_tensor* x, const tfjsb_tensor* filter, const int strides[2],
                          tfjsb_pad pad, const int dilations[2], const tfjsb_tensor* bias, tfjsb_act act,
                          tfjsb_tensor* out, void* stream);

/* tf.depthwiseConv2d with an optional fused bias and activation.
 *   x [N,H,W,C], filter [fh,fw,C,mult], bias NULL or [C*mult], out [N,Ho,Wo,C*mult]
 *   out[n,oy,ox,c*mult+q] = act( bias[c*mult+q] + sum_{ky,kx} x[n,iy,ix,c] * filter[ky,kx,c,q] )
 * Always fp32 CUDA-core arithmetic (not a dense contraction).  Same stride/dilation rule as conv2d. */
tfjsb_status tfjsb_depthwise_conv2d(tfjsb_ctx* ctx, const tfjsb_tensor* x, const tfjsb_tensor* filter,
                                    const int strides[2], tfjsb_pad pad, const int dilations[2],
                                    const tfjsb_tensor* bias, tfjsb_act act, tfjsb_tensor* out, void* stream);

/* tf.avgPool.  x [N,H,W,C] -> out [N,Ho,Wo,C]; each output is the sum of the in-bounds
 * window elements divided by their number (padding never counts). */
tfjsb_status tfjsb_avg_pool(tfjsb_ctx* ctx, const tfjsb_tensor* x, const int filter_size[2], const int strides[2],
                            tfjsb_pad pad, tfjsb_tensor* out, void* stream);

/* tf.maxPool.  x [N,H,W,C] -> out [N,Ho,Wo,C]; each output is the largest in-bounds window element
 * (padding never takes part; a NaN in the window gives NaN).  Not defined in the paper: TensorFlow's
 * definition, with the window geometry of tfjsb_window_out_shape. */
tfjsb_status tfjsb_max_pool(tfjsb_ctx* ctx, const tfjsb_tensor* x, const int filter_size[2], const int strides[2],
                            tfjsb_pad pad, tfjsb_tensor* out, void* stream);

/* tf.add / tf.sub / tf.mul: out = a op b, elementwise (the addition shader of Fig. 3, Sec. 4.1, computes
 * one output value per invocation; here one per thread, four per thread when the sizes allow).
 * a, out: rank 1..4, same shape.  b: a's shape, or a rank-1 vector of a's last dimension, broadcast
 * along every other dimension.  One fp32 operation per element, rounded to nearest: exact parity with
 * any IEEE implementation.  `out` may not alias an input. */
tfjsb_status tfjsb_binary(tfjsb_ctx* ctx, tfjsb_binary_op op, const tfjsb_tensor* a, const tfjsb_tensor* b,
                          tfjsb_tensor* out, void* stream);

/* matMul on bfloat16 storage with the fused epilogue (the GEMM of the BF16 math mode, exposed for
 * tensors the caller already holds in that format):
 *   out[M,N] = act( a[M,K] . bt[N,K]^T + bias[N] )
 * a and bt are DEVICE pointers to bfloat16 (2 bytes per element, row-major, K contiguous: bt is the
 * right-hand operand stored transposed); bias is a DEVICE pointer to N fp32 values or NULL; out is a
 * DEVICE pointer to M*N bfloat16 (out_is_bf16 != 0; the sum is rounded to nearest even once, after
 * bias and activation) or fp32 values.  Products are exact, sums fp32 in tensor memory.  All pointers
 * 16-byte aligned, K and N multiples of 8; TFJSB_ERR_UNSUPPORTED otherwise.  Enqueues on `stream`
 * and returns; the caller keeps ownership of every buffer. */
tfjsb_status tfjsb_matmul_bf16(tfjsb_ctx* ctx, const void* a, const void* bt, const float* bias, tfjsb_act act,
                               void* out, int out_is_bf16, int64_t M, int64_t N, int64_t K, void* stream);

/* tf.matMul on rank-3 tensors (Sec. 3.3 names the op; Listing 2 prints the rank-2 case): one rank-2
 * product per leading index.  a [B,M,K] (or [B,K,M] if transpose_a), b [B,K,N] (or [B,N,K] if
 * transpose_b), out [B,M,N].  Same math mode and tolerances as tfjsb_matmul.  With K and N multiples
 * of 4 all B products run as ONE launch of the tensor-core kernel (the batch is a third dimension of
 * its tensor maps, tile = (product, rows, columns)); otherwise each product runs on its own, on the
 * CUDA-core fp32 kernel where its slices are not 16-byte aligned. */
tfjsb_status tfjsb_batch_matmul(tfjsb_ctx* ctx, const tfjsb_tensor* a, const tfjsb_tensor* b, int transpose_a,
                                int transpose_b, tfjsb_tensor* out, void* stream);

/* tf.softmax over the last dimension of a rank 1..4 tensor:
 *   out[..., j] = exp(x[..., j] - max_j x) / sum_k exp(x[..., k] - max_j x). */
tfjsb_status tfjsb_softmax(tfjsb_ctx* ctx, const tfjsb_tensor* logits, tfjsb_tensor* out, void* stream);

/* The elementwise epilogue on its own (the paper's elementwise shader, Fig. 3):
 *   out[..., c] = act(x[..., c] + bias[c]);  bias NULL or [last dim].
 *   relu(v) = v > 0 ? v : +0 (so -0 -> +0), NaN stays NaN; relu6(v) = min(relu(v), 6).
 * One fp32 add and one clamp per element: results are bit-identical to the definition. */
tfjsb_status tfjsb_bias_act(tfjsb_ctx* ctx, const tfjsb_tensor* x, const tfjsb_tensor* bias, tfjsb_act act,
                            tfjsb_tensor* out, void* stream);

/* ---- gradients ---------------------------------------------------------------------- */

/* The paper differentiates eagerly: each kernel has a gradient function that the backward pass calls
 * (Sec. 3.5; model.fit of Sec. 3.2 rests on it).  It names no gradient op and gives none of their
 * arithmetic; the calls below are the adjoints of the forward definitions above, with TensorFlow's
 * names.  Geometry arguments (strides, pad, dilations) are those of the FORWARD call; `dy` has the
 * forward output's shape, which is checked.  Sums over pixels are taken in a fixed order: results do
 * not depend on scheduling.  1x1 / stride-1 convolutions run their two gradients as matrix products on
 * the tensor cores in TF32 mode (channel counts multiples of 4; for the filter gradient the pixel count
 * a multiple of 4); every other case runs on CUDA cores in fp32.  All enqueue on `stream` and return;
 * the filter and bias gradients use context-owned scratch (see tfjsb_reserve_scratch). */

/* dx[n,iy,ix,ci] = sum over (oy,ky), (ox,kx) with oy*sh - pt + ky*dh = iy and ox*sw - pl + kx*dw = ix, and co,
 *                  of dy[n,oy,ox,co] * filter[ky,kx,ci,co].
 * dy [N,Ho,Wo,Cout], filter [fh,fw,Cin,Cout], dx [N,H,W,Cin] (dx's shape names the forward input's). */
tfjsb_status tfjsb_conv2d_backprop_input(tfjsb_ctx* ctx, const tfjsb_tensor* dy, const tfjsb_tensor* filter,
                                         const int strides[2], tfjsb_pad pad, const int dilations[2], tfjsb_tensor* dx,
                                         void* stream);
/* dfilter[ky,kx,ci,co] = sum_{n,oy,ox} x[n, oy*sh - pt + ky*dh, ox*sw - pl + kx*dw, ci] * dy[n,oy,ox,co]
 * (samples outside the image are zero).  dfilter's shape names the filter's. */
tfjsb_status tfjsb_conv2d_backprop_filter(tfjsb_ctx* ctx, const tfjsb_tensor* x, const tfjsb_tensor* dy,
                                          const int strides[2], tfjsb_pad pad, const int dilations[2],
                                          tfjsb_tensor* dfilter, void* stream);
/* The same two gradients of tf.depthwiseConv2d: filter [fh,fw,C,mult], dy [N,Ho,Wo,C*mult], output
 * channel c*mult+q pairs with input channel c. */
tfjsb_status tfjsb_depthwise_conv2d_backprop_input(tfjsb_ctx* ctx, const tfjsb_tensor* dy, const tfjsb_tensor* filter,
                                                   const int strides[2], tfjsb_pad pad, const int dilations[2],
                                                   tfjsb_tensor* dx, void* stream);
tfjsb_status tfjsb_depthwise_conv2d_backprop_filter(tfjsb_ctx* ctx, const tfjsb_tensor* x, const tfjsb_tensor* dy,
                                                    const int strides[2], tfjsb_pad pad, const int dilations[2],
                                                    tfjsb_tensor* dfilter, void* stream);
/* Gradient through the fused epilogue y = act(z + bias), given the forward OUTPUT y:
 *   dz = dy where the activation passed its input through (none: everywhere; relu: y > 0;
 *   relu6: 0 < y < 6), +0 elsewhere.  Bit-exact.  y, dy, dz: one shape, rank 1..4. */
tfjsb_status tfjsb_act_backprop(tfjsb_ctx* ctx, const tfjsb_tensor* y, const tfjsb_tensor* dy, tfjsb_act act,
                                tfjsb_tensor* dz, void* stream);
/* dbias[c] = sum of dz[..., c] over every other dimension.  dz rank 1..4, dbias [last dim of dz]. */
tfjsb_status tfjsb_bias_backprop(tfjsb_ctx* ctx, const tfjsb_tensor* dz, tfjsb_tensor* dbias, void* stream);

/* ---- models ------------------------------------------------------------------------- */

typedef enum {
    TFJSB_LAYER_CONV2D = 0,          /* filter [fh,fw,Cin,out_channels] */
    TFJSB_LAYER_DEPTHWISE_CONV2D = 1,/* filter [fh,fw,C,out_channels] (out_channels = channel multiplier) */
    TFJSB_LAYER_AVG_POOL = 2,        /* filter_hw = window; {0,0} = global pool ('valid', window = H x W),
                                        whose output is viewed as [N, C] */
    TFJSB_LAYER_DENSE = 3,           /* input viewed as [N, K]; filter [K,out_channels]; bias; act */
    TFJSB_LAYER_SOFTMAX = 4
} tfjsb_layer_kind;

typedef struct {
    int32_t kind;          /* tfjsb_layer_kind */
    int32_t filter_hw[2];
    int32_t strides[2];
    int32_t dilations[2];
    int32_t pad;           /* tfjsb_pad */
    int32_t act;           /* tfjsb_act */
    int32_t out_channels;
    const float* filter;   /* HOST pointer, copied (and re-laid out) at model creation; NULL for pool/softmax */
    const float* bias;     /* HOST pointer or NULL */
} tfjsb_layer_desc;

/* Builds an executor for a straight-line model: shape inference for every layer, weights
 * copied to the device (1x1-conv and dense filters are also stored K-contiguous for the
 * tensor-core kernel), one arena for all intermediates (two ping-pong regions, reused across
 * layers and runs, like the paper's texture recycler, Sec. 4.1.2), tensor maps encoded once.
 * `input_dims` is the NHWC input shape; the batch size is fixed per model.
 * The math mode in force on `ctx` at creation is baked into the model. */
tfjsb_status tfjsb_model_create(tfjsb_ctx* ctx, const tfjsb_layer_desc* layers, int n_layers,
                                const int64_t input_dims[4], tfjsb_model** model);
tfjsb_status tfjsb_model_destroy(tfjsb_model* model);
/* Shape of the model's final output. */
tfjsb_status tfjsb_model_output_shape(tfjsb_model* model, int32_t* rank, int64_t dims[4]);
/* Number of kernels one run launches. */
int32_t tfjsb_model_launches_per_run(tfjsb_model* model);

/* Runs every layer in order on `stream` and returns without synchronising (Sec. 4.1.1).
 * `input` and `output` are device tensors with the model's input / output shapes. */
tfjsb_status tfjsb_run_model(tfjsb_model* model, const tfjsb_tensor* input, tfjsb_tensor* output, void* stream);

/* The same run from HOST memory: copies `host_input` (input-shape fp32, ideally pinned) to the
 * device, runs the model, copies the output to `host_output`, and synchronises `stream` before
 * returning (the blocking dataSync() of Sec. 3.6).  Batches of 32 images or more (a multiple of 4)
 * are pipelined in 4 slices: slice c+1 is copied on an internal stream while slice c is computed
 * on `stream` as a graph replay (images are independent, so the result is that of the whole-batch
 * run). */
tfjsb_status tfjsb_run_model_host(tfjsb_model* model, const float* host_input, float* host_output, void* stream);

/* The asynchronous form of the same run (the data() promise of Sec. 3.6 beside the blocking
 * dataSync()): enqueues the copy of `host_input` to the device, the run and the copy of the result to
 * `host_output`, and returns without waiting.  The model keeps two sets of device staging buffers and
 * alternates between them, so the input copy of one run overlaps the computation of the run before
 * it; a third call first waits for the first to finish.  `host_input` must be ready when the call is
 * made (the copy does not wait for work queued on `stream`), and neither buffer may be touched until
 * tfjsb_model_host_wait has returned (or a later call has had to wait for that run).  Runs complete in
 * the order of the calls; use one `stream` for all of them. */
tfjsb_status tfjsb_run_model_host_async(tfjsb_model* model, const float* host_input, float* host_output, void* stream);
/* Blocks until every run enqueued by tfjsb_run_model_host_async has delivered its output. */
tfjsb_status tfjsb_model_host_wait(tfjsb_model* model);

/* A stride-1 3x3 depthwise layer followed by a pointwise layer (<= 512 output channels, depthwise
 * channels a multiple of 32) can run as ONE kernel that keeps the depthwise output in shared
 * memory as the tensor-core operand, so the intermediate tensor is neither written nor read back.
 * mode 0: never; 1 (default): where the pair has enough 8x16-pixel tiles for the fused kernel to be
 * the faster choice; 2: wherever the shapes allow.  In the fp32 storage modes results are bit-identical
 * in every mode.  Models in the BF16 storage mode have the same kernel in that format (bfloat16 in and
 * out, the depthwise result rounded to bfloat16 on its way into the operand tile); there it is never
 * the default (the separate narrow kernels are faster) and agrees with the separate kernels to the
 * rounding of a stored value, not bit for bit.  The keep-all debug mode always runs the layers
 * separately. */
tfjsb_status tfjsb_model_set_fusion(tfjsb_model* model, int mode);

/* Replays one run as a CUDA graph instead of enqueueing the layers one by one (the enqueue cost per
 * program is what the paper's async design hides, Sec. 4.1.1; a graph removes it from the host).
 * The graph is captured on a private stream at the next tfjsb_run_model, for the input / output
 * buffers of that call, and re-captured when they change.  Run the model once without the graph
 * first.  Off by default. */
tfjsb_status tfjsb_model_set_graph(tfjsb_model* model, int use_graph);

/* Debug aid (the paper's debug mode downloads every intermediate, Sec. 3.8): a view of the
 * output of layer `layer` as left by the last run.  With the ping-pong arena only the most
 * recent layers survive a full run, so call tfjsb_model_set_keep_all(model, 1) before the run
 * to give every layer its own buffer. */
tfjsb_status tfjsb_model_set_keep_all(tfjsb_model* model, int keep_all);
tfjsb_status tfjsb_model_layer_output(tfjsb_model* model, int layer, tfjsb_tensor* view);
/* The same read as fp32 values whatever the layer's storage format: writes the layer's output
 * (converted from bfloat16 where the model stores it so) into `dst`, a DEVICE buffer of as many
 * floats as the layer has outputs, on `stream`.  tfjsb_model_layer_output refuses a layer that is
 * stored as bfloat16 (its view would mislabel the data) with TFJSB_ERR_UNSUPPORTED. */
tfjsb_status tfjsb_model_layer_output_f32(tfjsb_model* model, int layer, float* dst, void* stream);
/* Shape of the output of layer `layer`. */
tfjsb_status tfjsb_model_layer_shape(tfjsb_model* model, int layer, int32_t* rank, int64_t dims[4]);

/* Name of the kernel that runs layer `layer` in the model's current mode, as planned for the buffers
 * of the last run (the per-kernel view of the paper's profiler, Sec. 3.8): written to `name` (a HOST
 * buffer of `name_len` bytes, NUL-terminated, truncated if too short).  The second layer of a fused
 * depthwise + pointwise pair reports "(in the previous layer's kernel)".  TFJSB_ERR_INVALID_ARG before
 * the first run. */
tfjsb_status tfjsb_model_layer_kernel(tfjsb_model* model, int layer, char* name, int32_t name_len);

/* Per-layer device timing (the paper's per-kernel profile, Sec. 3.8): runs the model `reps`
 * times with a CUDA event pair around every layer, synchronises, and writes the mean
 * milliseconds per layer into ms_per_layer[0..n_layers-1] (host). */
tfjsb_status tfjsb_model_profile(tfjsb_model* model, const tfjsb_tensor* input, tfjsb_tensor* output, int reps,
                                 float* ms_per_layer, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* TFJSB_H_ */

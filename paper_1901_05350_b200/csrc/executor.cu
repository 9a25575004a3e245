// Graph executor: a straight-line model (list of layer records) planned once and run as a
// sequence of kernel launches on one stream.
//
// Planning (tfjsb_model_create): shape inference per layer, weights copied to the device (the
// filters of GEMM-shaped layers are additionally stored [Cout, Cin], K-contiguous, for the
// tensor-core kernel), one arena holding two ping-pong regions for the intermediates (a layer
// reads one region and writes the other; the regions are reused by every run, in the spirit of
// the paper's texture recycler, Sec. 4.1.2), tensor maps encoded once against those fixed
// addresses.  Running (tfjsb_run_model) therefore does no allocation, no shape arithmetic and
// no synchronisation: it enqueues the kernels and returns (Sec. 4.1.1).
#include <cstdio>
#include <cstdlib>
#include <vector>

#include "common.cuh"

using namespace tfjsb;

namespace {

enum StepKind {
    STEP_GEMM_TF32, STEP_GEMM_FP32, STEP_CONV_TF32, STEP_CONV_FP32, STEP_DEPTHWISE, STEP_POOL, STEP_SOFTMAX,
    // narrow-storage mode (activations and filters bfloat16 in memory, fp32 sums)
    STEP_GEMM_NARROW, STEP_CONV_NARROW, STEP_DEPTHWISE_NARROW, STEP_POOL_NARROW
};

struct Step {
    StepKind kind;
    ConvGeom g{};                // conv / depthwise / pool
    int64_t M = 0, N = 0, K = 0;  // gemm; softmax: M rows, N cols
    int act = TFJSB_ACT_NONE;
    float* filter = nullptr;     // device, as given ([fh,fw,Cin,Cout] / [K,N])
    float* filter_km = nullptr;  // device, [N,K] (tensor-core layers only)
    float* bias = nullptr;       // device or null
    GemmTf32Plan plan{};
    DepthwisePlan dw_plan{};
    bool plan_built = false;
    // a depthwise layer followed by a pointwise layer can run as one fused kernel (the pointwise step
    // is then skipped); the separate plans are kept for the keep-all debug mode
    bool conv_patch = false;  // STEP_CONV_TF32 through the patch kernel (whole im2col row in one k-block)
    bool fuse_next = false;
    bool fusable = false;     // the pair's shapes fit the fused kernel
    bool fuse_pays = false;   // and there are enough tiles for it to be the faster choice
    DwPwPlan fused_plan{};
    // narrow-storage mode: which of the layer's tensors are bfloat16, and the GEMM's bfloat16 filter [N,K]
    bool is_dense = false;
    bool in_f32 = true;
    bool out_bf16 = false;
    void* filter16 = nullptr;
    GemmBf16Plan plan16{};
    // A pointwise layer with fewer than 64 input channels (K = 8, 16, 32) runs as the GEMM of r = 64 / K
    // pixels at a time: A [M, K] read as [M / r, 64] (r pixels fill one 128-byte row), the filter laid r
    // times down the diagonal of a [r N, 64] matrix, and C [M / r, r N] is C [M, N] as it lies in memory.
    // The tensor core multiplies the zeros too, which such a layer (bound by its memory traffic) can
    // afford; a k-block of which the copy engine has to zero-fill half is several times slower.
    int pack_r = 1;
    float* bias_packed = nullptr;
    int32_t out_rank = 4;
    int64_t out_dims[4] = {0, 0, 0, 0};
    int64_t out_elems = 0;
    float* out = nullptr;        // where this layer writes (arena or, for the last layer, the caller's output)
    const float* in = nullptr;   // where it reads (arena or, for the first layer, the caller's input)
};

}  // namespace

struct tfjsb_model {
    tfjsb_ctx* ctx = nullptr;
    std::vector<Step> steps;
    std::vector<float*> owned;  // every device allocation of this model
    int64_t in_dims[4] = {0, 0, 0, 0};
    int64_t in_elems = 0;
    float* arena = nullptr;
    size_t region_elems = 0;     // elements per ping-pong region
    float* keep_all_arena = nullptr;
    bool keep_all = false;
    // Host-buffer runs (tfjsb_run_model_host / _async) alternate between two sets of device staging
    // buffers, so that the input copy of one run can overlap the computation of the run before it.
    float* staged_in[2] = {nullptr, nullptr};
    float* staged_out[2] = {nullptr, nullptr};
    cudaEvent_t host_run_done[2] = {nullptr, nullptr};  // recorded after a run's output copy
    bool host_run_pending[2] = {false, false};
    int next_staging = 0;
    bool use_tf32 = true;
    bool narrow = false;  // bfloat16 storage (TFJSB_MATH_BF16 at creation)
    // caller buffers the first/last tensor maps were last encoded for
    const void* bound_in = nullptr;
    void* bound_out = nullptr;
    // Host-buffer runs pipeline the batch in slices: slice c+1 is copied to the device on a stream
    // of its own while slice c is computed.  Each slice has a view of this model with a smaller
    // batch: the same weights and arena, its own shapes, plans and fixed staging addresses.  There is
    // one set of views and events per staging buffer: entry b * n_slices + c.
    std::vector<tfjsb_model*> slices;
    std::vector<cudaEvent_t> slice_copied;
    int n_slices = 0;
    cudaStream_t copy_stream = nullptr;
    bool is_view = false;
    // optional CUDA-graph replay of one run (tfjsb_model_set_graph): captured for the current binding
    // programmatic dependent launch between the layers' kernels (each waits before reading its input)
    bool use_pdl = true;
    bool use_graph = false;
    cudaGraphExec_t graph_exec = nullptr;
    cudaStream_t capture_stream = nullptr;
};

namespace {

tfjsb_status dev_alloc(tfjsb_model* m, size_t elems, float** out) {
    *out = nullptr;
    if (elems == 0) elems = 4;
    cudaError_t e = cudaMalloc(out, elems * sizeof(float));
    if (e != cudaSuccess) {
        (void)cudaGetLastError();
        return fail(m->ctx, TFJSB_ERR_OOM, "could not allocate " + std::to_string(elems * 4) + " bytes on the device");
    }
    m->owned.push_back(*out);
    return TFJSB_OK;
}

tfjsb_status upload(tfjsb_model* m, const float* host, size_t elems, float** out) {
    tfjsb_status st = dev_alloc(m, elems, out);
    if (st != TFJSB_OK) return st;
    cudaError_t e = cudaMemcpy(*out, host, elems * sizeof(float), cudaMemcpyHostToDevice);
    if (e != cudaSuccess) return cuda_fail(m->ctx, e, "copying weights to the device");
    return TFJSB_OK;
}

bool window(int64_t in, int k, int s, int d, int pad, int* out, int* before) {
    int64_t o;
    int a;
    if (tfjsb_window_out_shape(in, k, s, d, (tfjsb_pad)pad, &o, before, &a) != TFJSB_OK) return false;
    *out = (int)o;
    return true;
}

// (Re)binds the addresses a step reads and writes; tensor-core plans depend on them.
tfjsb_status bind_step(tfjsb_model* m, Step& st, const float* in, float* out) {
    const bool changed = st.in != in || st.out != out;
    st.in = in;
    st.out = out;
    if (st.kind == STEP_GEMM_TF32 && (changed || !st.plan_built)) {
        tfjsb_status rc = gemm_tf32_plan(m->ctx, in, st.filter_km, out, st.M, st.N, st.K, &st.plan);
        if (rc != TFJSB_OK) return rc;
        st.plan_built = true;
    }
    if (st.kind == STEP_CONV_TF32 && (changed || !st.plan_built)) {
        tfjsb_status rc = st.conv_patch ? conv_patch_plan(m->ctx, in, st.filter_km, out, st.g, &st.fused_plan)
                                        : conv_igemm_plan(m->ctx, in, st.filter_km, out, st.g, &st.plan);
        if (rc != TFJSB_OK) return rc;
        st.plan_built = true;
    }
    if (st.kind == STEP_GEMM_NARROW && (changed || !st.plan_built)) {
        tfjsb_status rc = gemm_bf16_plan(m->ctx, in, st.filter16, out, st.out_bf16, st.M / st.pack_r, st.N * st.pack_r,
                                         st.K * st.pack_r, &st.plan16);
        if (rc != TFJSB_OK) return rc;
        st.plan_built = true;
    }
    if (st.kind == STEP_CONV_NARROW && st.conv_patch && (changed || !st.plan_built)) {
        tfjsb_status rc = conv_patch_plan(m->ctx, in, st.filter_km, out, st.g, &st.fused_plan, true);
        if (rc != TFJSB_OK) return rc;
        st.plan_built = true;
    }
    if (st.kind == STEP_DEPTHWISE && (changed || !st.plan_built)) {
        tfjsb_status rc = depthwise_plan(m->ctx, in, st.g, &st.dw_plan);
        if (rc != TFJSB_OK) return rc;
        st.plan_built = true;
    }
    if (st.kind == STEP_DEPTHWISE_NARROW && (changed || !st.plan_built)) {
        // the pipelined kernel where it has an instance for the shape (variant >= 0), else the register kernel
        tfjsb_status rc = depthwise_plan(m->ctx, in, st.g, &st.dw_plan, !st.in_f32);
        if (rc != TFJSB_OK) return rc;
        if (st.in_f32) st.dw_plan.variant = -1;
        st.plan_built = true;
    }
    return TFJSB_OK;
}

// Assigns buffers: layer i reads the previous layer's output; intermediates alternate between the
// two arena regions (or get a region each in keep-all mode); the ends use the caller's tensors.
tfjsb_status bind_all(tfjsb_model* m, const float* input, float* output) {
    const int n = (int)m->steps.size();
    const float* cur = input;
    size_t keep_off = 0;
    int region = 0;  // arena region the next launched kernel writes
    for (int i = 0; i < n; ++i) {
        Step& st = m->steps[i];
        float* dst;
        if (i == n - 1) dst = output;
        else if (m->keep_all) {
            dst = m->keep_all_arena + keep_off;
            keep_off += (size_t)((st.out_elems + 63) / 64 * 64);
        } else {
            dst = m->arena + (size_t)region * m->region_elems;
            // A fused pair is one kernel: it reads the first layer's input and writes the second
            // layer's output, so the pair takes one region (the first layer's own output buffer is
            // never written) and the region flips once per kernel, not once per layer.
            if (!st.fuse_next) region ^= 1;
        }
        tfjsb_status rc = bind_step(m, st, cur, dst);
        if (rc != TFJSB_OK) return rc;
        cur = dst;
    }
    if (!m->keep_all) {
        for (int i = 0; i + 1 < n; ++i) {
            Step& st = m->steps[i];
            if (!st.fuse_next) continue;
            Step& pw = m->steps[i + 1];
            tfjsb_status rc = dwpw_fused_plan(m->ctx, st.in, pw.filter_km, pw.out, st.g, pw.N, &st.fused_plan, m->narrow);
            if (rc != TFJSB_OK) return rc;
        }
    }
    m->bound_in = input;
    m->bound_out = output;
    return TFJSB_OK;
}

cudaError_t launch_step(tfjsb_model* m, const Step& st, cudaStream_t s) {
    tfjsb_ctx* ctx = m->ctx;
    switch (st.kind) {
        case STEP_CONV_TF32:
            if (st.conv_patch)
                return launch_dwpw_fused(st.fused_plan, nullptr, nullptr, TFJSB_ACT_NONE, st.bias, st.act, ctx->dev_status, s,
                                         &ctx->launches);
            return launch_gemm_tf32(st.plan, st.bias, st.act, ctx->dev_status, s, &ctx->launches);
        case STEP_GEMM_TF32:
            return launch_gemm_tf32(st.plan, st.bias, st.act, ctx->dev_status, s, &ctx->launches);
        case STEP_GEMM_FP32:
            return launch_gemm_fp32(st.in, st.K, 1, st.filter, st.N, 1, st.bias, st.act, st.out, st.N, st.M, st.N, st.K,
                                    s, &ctx->launches);
        case STEP_CONV_FP32:
            return launch_conv2d_fp32(st.in, st.filter, st.bias, st.act, st.out, st.g, s, &ctx->launches);
        case STEP_DEPTHWISE:
            return launch_depthwise(st.dw_plan, st.in, st.filter, st.bias, st.act, st.out, st.g, ctx->dev_status, s,
                                    &ctx->launches);
        case STEP_POOL:
            return launch_avg_pool(st.in, st.out, st.g, s, &ctx->launches);
        case STEP_SOFTMAX:
            return launch_softmax(st.in, st.out, st.M, st.N, s, &ctx->launches);
        case STEP_GEMM_NARROW:
            return launch_gemm_bf16(st.plan16, st.pack_r > 1 ? st.bias_packed : st.bias, st.act, ctx->dev_status, s,
                                    &ctx->launches);
        case STEP_CONV_NARROW:
            if (st.conv_patch)
                return launch_dwpw_fused(st.fused_plan, nullptr, nullptr, TFJSB_ACT_NONE, st.bias, st.act, ctx->dev_status, s,
                                         &ctx->launches);
            return launch_conv_narrow(st.in, st.in_f32, st.filter, st.bias, st.act, st.out, st.out_bf16, st.g, s,
                                      &ctx->launches);
        case STEP_DEPTHWISE_NARROW:
            if (st.dw_plan.variant >= 0)
                return launch_depthwise_tma_narrow(st.dw_plan, st.filter, st.bias, st.act, st.out, st.out_bf16, st.g, ctx->dev_status, s,
                                                   &ctx->launches);
            return launch_depthwise_narrow(st.in, st.filter, st.bias, st.act, st.out, st.out_bf16, st.g, s, &ctx->launches);
        case STEP_POOL_NARROW:
            return launch_avg_pool_global_narrow(st.in, st.out, st.out_bf16, st.g.N, st.g.H * st.g.W, st.g.C, s,
                                                 &ctx->launches);
    }
    return cudaErrorUnknown;
}

// A view of `parent` for a batch of `n` images: steps copied with every batch-proportional size scaled.
tfjsb_model* make_batch_view(tfjsb_model* parent, int64_t n) {
    const int64_t pn = parent->in_dims[0];
    tfjsb_model* v = new tfjsb_model();
    v->ctx = parent->ctx;
    v->is_view = true;
    v->use_tf32 = parent->use_tf32;
    v->narrow = parent->narrow;
    v->use_pdl = parent->use_pdl;
    v->arena = parent->arena;
    v->region_elems = parent->region_elems;
    v->steps = parent->steps;
    for (int i = 0; i < 4; ++i) v->in_dims[i] = parent->in_dims[i];
    v->in_dims[0] = n;
    v->in_elems = parent->in_elems / pn * n;
    for (Step& st : v->steps) {
        st.g.N = n;
        st.M = st.M / pn * n;  // GEMM rows and softmax rows are both proportional to the batch
        st.out_dims[0] = n;
        st.out_elems = st.out_elems / pn * n;
        st.plan_built = false;
        st.in = nullptr;
        st.out = nullptr;
    }
    return v;
}

cudaError_t launch_layers(tfjsb_model* m, int i, cudaStream_t s, int* consumed);
int launches_per_run(const tfjsb_model* m);

void drop_graph(tfjsb_model* m) {
    if (m->graph_exec) {
        cudaGraphExecDestroy(m->graph_exec);
        m->graph_exec = nullptr;
    }
}

// Records one run (every layer's launch, in order) into a graph on a private stream.  Nothing
// executes during the capture; the first launch of every kernel must already have happened
// outside a capture (function attributes are set then), which a warm-up run guarantees.
tfjsb_status capture_graph(tfjsb_model* m) {
    tfjsb_ctx* ctx = m->ctx;
    cudaError_t e;
    if (!m->capture_stream && (e = cudaStreamCreateWithFlags(&m->capture_stream, cudaStreamNonBlocking)) != cudaSuccess)
        return cuda_fail(ctx, e, "cudaStreamCreate");
    if ((e = cudaStreamBeginCapture(m->capture_stream, cudaStreamCaptureModeRelaxed)) != cudaSuccess)
        return cuda_fail(ctx, e, "cudaStreamBeginCapture");
    const int64_t before = ctx->launches;
    cudaError_t launch_err = cudaSuccess;
    for (int i = 0, used = 1; i < (int)m->steps.size(); i += used)
        if ((launch_err = launch_layers(m, i, m->capture_stream, &used)) != cudaSuccess) break;
    ctx->launches = before;  // recorded, not run
    cudaGraph_t graph = nullptr;
    e = cudaStreamEndCapture(m->capture_stream, &graph);
    if (launch_err != cudaSuccess || e != cudaSuccess) {
        if (graph) cudaGraphDestroy(graph);
        (void)cudaGetLastError();
        return cuda_fail(ctx, launch_err != cudaSuccess ? launch_err : e, "capturing the model into a graph");
    }
    e = cudaGraphInstantiate(&m->graph_exec, graph, 0);
    cudaGraphDestroy(graph);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "cudaGraphInstantiate");
    return TFJSB_OK;
}

// Launches layer i (and, when it is fused with its successor, that one too); returns how many layers ran.
struct PdlScope {
    explicit PdlScope(bool on) { g_launch_pdl = on; }
    ~PdlScope() { g_launch_pdl = false; }
};

cudaError_t launch_layers(tfjsb_model* m, int i, cudaStream_t s, int* consumed) {
    const Step& st = m->steps[i];
    PdlScope pdl(m->use_pdl);
    if (st.fuse_next && !m->keep_all) {
        const Step& pw = m->steps[i + 1];
        *consumed = 2;
        return launch_dwpw_fused(st.fused_plan, st.filter, st.bias, st.act, pw.bias, pw.act, m->ctx->dev_status, s,
                                 &m->ctx->launches);
    }
    *consumed = 1;
    return launch_step(m, st, s);
}

int launches_per_run(const tfjsb_model* m) {
    int n = (int)m->steps.size();
    if (!m->keep_all)
        for (const Step& st : m->steps) n -= st.fuse_next ? 1 : 0;
    return n;
}

tfjsb_status check_io(tfjsb_model* m, const tfjsb_tensor* input, const tfjsb_tensor* output) {
    tfjsb_ctx* ctx = m->ctx;
    if (!input || !output || !input->data || !output->data) return fail(ctx, TFJSB_ERR_INVALID_ARG, "input / output is null");
    if (input->rank != 4) return fail(ctx, TFJSB_ERR_SHAPE, "input must be rank 4 (NHWC)");
    for (int i = 0; i < 4; ++i)
        if (input->dims[i] != m->in_dims[i]) return fail(ctx, TFJSB_ERR_SHAPE, "input shape differs from the model's");
    const Step& last = m->steps.back();
    if (output->rank != last.out_rank) return fail(ctx, TFJSB_ERR_SHAPE, "output rank differs from the model's");
    for (int i = 0; i < last.out_rank; ++i)
        if (output->dims[i] != last.out_dims[i]) return fail(ctx, TFJSB_ERR_SHAPE, "output shape differs from the model's");
    if ((reinterpret_cast<uintptr_t>(input->data) & 15u) || (reinterpret_cast<uintptr_t>(output->data) & 15u))
        return fail(ctx, TFJSB_ERR_INVALID_ARG, "input / output must be 16-byte aligned");
    if (input->data == output->data) return fail(ctx, TFJSB_ERR_INVALID_ARG, "output aliases the input");
    return TFJSB_OK;
}

}  // namespace

extern "C" {

tfjsb_status tfjsb_model_create(tfjsb_ctx* ctx, const tfjsb_layer_desc* layers, int n_layers,
                                const int64_t input_dims[4], tfjsb_model** out) {
    if (!ctx) return TFJSB_ERR_INVALID_ARG;
    if (!out) return fail(ctx, TFJSB_ERR_INVALID_ARG, "model out-pointer is null");
    *out = nullptr;
    if (!layers || n_layers < 1 || !input_dims) return fail(ctx, TFJSB_ERR_INVALID_ARG, "no layers / no input shape");
    for (int i = 0; i < 4; ++i)
        if (input_dims[i] < 1 || input_dims[i] > 0x3fffffff) return fail(ctx, TFJSB_ERR_SHAPE, "input dimensions must be in [1, 2^30]");

    tfjsb_model* m = new tfjsb_model();
    m->ctx = ctx;
    m->use_tf32 = ctx->math == TFJSB_MATH_TF32 && ctx->encode_tiled != nullptr;
    m->narrow = ctx->math == TFJSB_MATH_BF16;
    if (m->narrow && !ctx->encode_tiled) {
        delete m;
        return fail(ctx, TFJSB_ERR_CUDA, "cuTensorMapEncodeTiled is not available");
    }
    m->use_pdl = getenv("TFJSB_NO_PDL") == nullptr;
    for (int i = 0; i < 4; ++i) m->in_dims[i] = input_dims[i];
    m->in_elems = input_dims[0] * input_dims[1] * input_dims[2] * input_dims[3];

    // running shape: rank 4 [N,H,W,C] or rank 2 [N,F]
    int rank = 4;
    int64_t d[4] = {input_dims[0], input_dims[1], input_dims[2], input_dims[3]};
    tfjsb_status st = TFJSB_OK;
    auto bail = [&](tfjsb_status code, const std::string& msg) {
        fail(ctx, code, msg);
        for (float* p : m->owned) cudaFree(p);
        delete m;
        return code;
    };

    for (int li = 0; li < n_layers; ++li) {
        const tfjsb_layer_desc& L = layers[li];
        const std::string where = "layer " + std::to_string(li) + ": ";
        Step step;
        step.act = L.act;
        if (L.act != TFJSB_ACT_NONE && L.act != TFJSB_ACT_RELU && L.act != TFJSB_ACT_RELU6)
            return bail(TFJSB_ERR_INVALID_ARG, where + "unknown activation");
        switch (L.kind) {
            case TFJSB_LAYER_CONV2D:
            case TFJSB_LAYER_DEPTHWISE_CONV2D: {
                if (rank != 4) return bail(TFJSB_ERR_SHAPE, where + "needs a rank-4 input");
                if (!L.filter) return bail(TFJSB_ERR_INVALID_ARG, where + "filter is null");
                if (L.filter_hw[0] < 1 || L.filter_hw[1] < 1 || L.strides[0] < 1 || L.strides[1] < 1 ||
                    L.dilations[0] < 1 || L.dilations[1] < 1 || L.out_channels < 1)
                    return bail(TFJSB_ERR_INVALID_ARG, where + "window, strides, dilations and out_channels must be >= 1");
                if ((L.strides[0] > 1 || L.strides[1] > 1) && (L.dilations[0] > 1 || L.dilations[1] > 1))
                    return bail(TFJSB_ERR_UNSUPPORTED, where + "a stride > 1 together with a dilation > 1 is not supported");
                if (L.pad != TFJSB_PAD_VALID && L.pad != TFJSB_PAD_SAME) return bail(TFJSB_ERR_INVALID_ARG, where + "unknown padding mode");
                const bool dw = L.kind == TFJSB_LAYER_DEPTHWISE_CONV2D;
                ConvGeom g;
                g.N = d[0]; g.H = (int)d[1]; g.W = (int)d[2]; g.C = (int)d[3];
                g.fh = L.filter_hw[0]; g.fw = L.filter_hw[1];
                g.sh = L.strides[0]; g.sw = L.strides[1]; g.dh = L.dilations[0]; g.dw = L.dilations[1];
                g.mult = dw ? L.out_channels : 1;
                const int64_t co = dw ? (int64_t)g.C * L.out_channels : L.out_channels;
                if (co > 0x3fffffff) return bail(TFJSB_ERR_UNSUPPORTED, where + "too many output channels");
                g.Co = (int)co;
                if (!window(g.H, g.fh, g.sh, g.dh, L.pad, &g.Ho, &g.pt) || !window(g.W, g.fw, g.sw, g.dw, L.pad, &g.Wo, &g.pl))
                    return bail(TFJSB_ERR_SHAPE, where + "the filter window does not fit the input under 'valid' padding");
                step.g = g;
                const size_t f_elems = (size_t)g.fh * g.fw * g.C * (dw ? g.mult : g.Co);
                if ((st = upload(m, L.filter, f_elems, &step.filter)) != TFJSB_OK) return bail(st, ctx->last_error);
                if (L.bias && (st = upload(m, L.bias, (size_t)g.Co, &step.bias)) != TFJSB_OK) return bail(st, ctx->last_error);
                if (m->narrow) {
                    // what is stored is a bfloat16: the filter is rounded once, here
                    cudaError_t e = launch_round_to_bf16_in_place(step.filter, (int64_t)f_elems, 0, &ctx->launches);
                    if (e != cudaSuccess) return bail(TFJSB_ERR_CUDA, std::string("rounding weights: ") + cudaGetErrorString(e));
                    if (dw) {
                        if (li == 0) return bail(TFJSB_ERR_UNSUPPORTED, where + "in the bfloat16 storage mode the first layer must be a conv2d");
                        if (!depthwise_narrow_supported(g))
                            return bail(TFJSB_ERR_UNSUPPORTED, where + "the bfloat16 storage mode has depthwise 3x3, stride 1 or 2, "
                                                                       "no dilation, multiplier 1, channels a multiple of 8");
                        step.kind = STEP_DEPTHWISE_NARROW;
                    } else if (li > 0 && g.fh == 1 && g.fw == 1 && g.sh == 1 && g.sw == 1 &&
                               gemm_bf16_supported(g.N * g.H * g.W, g.Co, g.C)) {
                        step.M = g.N * g.H * g.W; step.K = g.C; step.N = g.Co;
                        step.kind = STEP_GEMM_NARROW;
                    } else step.kind = STEP_CONV_NARROW;
                } else if (dw) step.kind = STEP_DEPTHWISE;
                else if (g.fh == 1 && g.fw == 1 && g.sh == 1 && g.sw == 1) {
                    step.M = g.N * g.H * g.W; step.K = g.C; step.N = g.Co;
                    step.kind = (m->use_tf32 && gemm_tf32_supported(step.M, step.N, step.K)) ? STEP_GEMM_TF32 : STEP_GEMM_FP32;
                } else step.kind = (m->use_tf32 && conv_igemm_supported(g)) ? STEP_CONV_TF32 : STEP_CONV_FP32;
                step.out_rank = 4;
                step.out_dims[0] = g.N; step.out_dims[1] = g.Ho; step.out_dims[2] = g.Wo; step.out_dims[3] = g.Co;
                break;
            }
            case TFJSB_LAYER_AVG_POOL: {
                if (rank != 4) return bail(TFJSB_ERR_SHAPE, where + "needs a rank-4 input");
                const bool global = L.filter_hw[0] == 0 && L.filter_hw[1] == 0;
                ConvGeom g;
                g.N = d[0]; g.H = (int)d[1]; g.W = (int)d[2]; g.C = (int)d[3];
                g.Co = g.C; g.mult = 1; g.dh = g.dw = 1;
                if (global) {
                    g.fh = g.H; g.fw = g.W; g.sh = g.sw = 1; g.pt = g.pl = 0; g.Ho = g.Wo = 1;
                } else {
                    if (L.filter_hw[0] < 1 || L.filter_hw[1] < 1 || L.strides[0] < 1 || L.strides[1] < 1)
                        return bail(TFJSB_ERR_INVALID_ARG, where + "window and strides must be >= 1");
                    if (L.pad != TFJSB_PAD_VALID && L.pad != TFJSB_PAD_SAME) return bail(TFJSB_ERR_INVALID_ARG, where + "unknown padding mode");
                    g.fh = L.filter_hw[0]; g.fw = L.filter_hw[1]; g.sh = L.strides[0]; g.sw = L.strides[1];
                    if (!window(g.H, g.fh, g.sh, 1, L.pad, &g.Ho, &g.pt) || !window(g.W, g.fw, g.sw, 1, L.pad, &g.Wo, &g.pl))
                        return bail(TFJSB_ERR_SHAPE, where + "the pooling window does not fit the input under 'valid' padding");
                }
                step.kind = STEP_POOL;
                if (m->narrow) {
                    if (li == 0 || !global || (g.C % 8) != 0)
                        return bail(TFJSB_ERR_UNSUPPORTED, where + "the bfloat16 storage mode has the global average pool only "
                                                                   "(channels a multiple of 8, not as the first layer)");
                    step.kind = STEP_POOL_NARROW;
                }
                step.g = g;
                if (global) {
                    step.out_rank = 2;
                    step.out_dims[0] = g.N; step.out_dims[1] = g.C;
                } else {
                    step.out_rank = 4;
                    step.out_dims[0] = g.N; step.out_dims[1] = g.Ho; step.out_dims[2] = g.Wo; step.out_dims[3] = g.C;
                }
                break;
            }
            case TFJSB_LAYER_DENSE: {
                if (!L.filter) return bail(TFJSB_ERR_INVALID_ARG, where + "filter is null");
                if (L.out_channels < 1) return bail(TFJSB_ERR_INVALID_ARG, where + "out_channels must be >= 1");
                int64_t feat = 1;
                for (int i = 1; i < rank; ++i) feat *= d[i];
                step.M = d[0]; step.K = feat; step.N = L.out_channels;
                if ((st = upload(m, L.filter, (size_t)(step.K * step.N), &step.filter)) != TFJSB_OK) return bail(st, ctx->last_error);
                if (L.bias && (st = upload(m, L.bias, (size_t)step.N, &step.bias)) != TFJSB_OK) return bail(st, ctx->last_error);
                step.kind = (m->use_tf32 && gemm_tf32_supported(step.M, step.N, step.K)) ? STEP_GEMM_TF32 : STEP_GEMM_FP32;
                if (m->narrow) {
                    if (li == 0) return bail(TFJSB_ERR_UNSUPPORTED, where + "in the bfloat16 storage mode the first layer must be a conv2d");
                    cudaError_t e = launch_round_to_bf16_in_place(step.filter, step.K * step.N, 0, &ctx->launches);
                    if (e != cudaSuccess) return bail(TFJSB_ERR_CUDA, std::string("rounding weights: ") + cudaGetErrorString(e));
                    step.is_dense = true;
                    if (gemm_bf16_supported(step.M, step.N, step.K)) step.kind = STEP_GEMM_NARROW;
                    else {
                        // a 1x1 convolution over [M,1,1,K]: the filter [K,N] already has that layout
                        if (step.K > 0x3fffffff || step.N > 0x3fffffff) return bail(TFJSB_ERR_UNSUPPORTED, where + "too wide");
                        ConvGeom g{};
                        g.N = step.M; g.H = g.W = 1; g.C = (int)step.K; g.fh = g.fw = 1; g.Co = (int)step.N; g.mult = 1;
                        g.sh = g.sw = g.dh = g.dw = 1; g.pt = g.pl = 0; g.Ho = g.Wo = 1;
                        step.g = g;
                        step.kind = STEP_CONV_NARROW;
                    }
                }
                step.out_rank = 2;
                step.out_dims[0] = step.M; step.out_dims[1] = step.N;
                break;
            }
            case TFJSB_LAYER_SOFTMAX: {
                step.kind = STEP_SOFTMAX;
                if (m->narrow && (li == 0 || !(m->steps.back().is_dense || m->steps.back().kind == STEP_SOFTMAX)))
                    return bail(TFJSB_ERR_UNSUPPORTED, where + "in the bfloat16 storage mode softmax follows a dense layer");
                step.N = d[rank - 1];
                step.M = 1;
                for (int i = 0; i < rank - 1; ++i) step.M *= d[i];
                step.out_rank = rank;
                for (int i = 0; i < rank; ++i) step.out_dims[i] = d[i];
                break;
            }
            default:
                return bail(TFJSB_ERR_INVALID_ARG, where + "unknown layer kind");
        }
        if (step.kind == STEP_CONV_TF32) {
            step.conv_patch = conv_patch_supported(step.g) && !getenv("TFJSB_NO_PATCH_CONV");
            // filter [fh*fw*Cin, Cout] -> [Cout, k_pad] once, on the device
            const int64_t k_pad = conv_igemm_k_pad(step.g);
            if ((st = dev_alloc(m, (size_t)(k_pad * step.g.Co), &step.filter_km)) != TFJSB_OK) return bail(st, ctx->last_error);
            cudaError_t e = launch_pack_filter(step.filter, step.filter_km, (int64_t)step.g.fh * step.g.fw * step.g.C,
                                               step.g.Co, k_pad, 0, &ctx->launches);
            if (e != cudaSuccess) return bail(TFJSB_ERR_CUDA, std::string("packing weights: ") + cudaGetErrorString(e));
        }
        if (step.kind == STEP_GEMM_NARROW) {
            // weights [K,N] fp32 -> [N,K] bfloat16 once, on the device
            int r = (!step.is_dense && step.K < 64 && 64 % step.K == 0) ? (int)(64 / step.K) : 1;
            if (r > 1 && (((int64_t)step.g.H * step.g.W) % r != 0 || !gemm_bf16_supported(step.M / r, step.N * r, 64))) r = 1;
            step.pack_r = r;
            const size_t w_elems = (size_t)(step.K * step.N) * r * r;
            float* km32 = nullptr;
            if ((st = dev_alloc(m, (size_t)(step.K * step.N), &km32)) != TFJSB_OK) return bail(st, ctx->last_error);
            float* km16 = nullptr;
            if ((st = dev_alloc(m, (w_elems + 1) / 2, &km16)) != TFJSB_OK) return bail(st, ctx->last_error);
            cudaError_t e = launch_transpose(step.filter, km32, step.K, step.N, 0, &ctx->launches);
            step.filter_km = km32;  // [N, K] fp32 holding bfloat16 values: the B operand of the fused block kernel
            if (r > 1) {
                float* diag = nullptr;
                if ((st = dev_alloc(m, w_elems, &diag)) != TFJSB_OK) return bail(st, ctx->last_error);
                if (e == cudaSuccess) e = launch_block_diagonal(km32, diag, step.N, step.K, r, 0, &ctx->launches);
                km32 = diag;
                if (step.bias) {
                    if ((st = dev_alloc(m, (size_t)step.N * r, &step.bias_packed)) != TFJSB_OK) return bail(st, ctx->last_error);
                    for (int j = 0; j < r && e == cudaSuccess; ++j)
                        e = cudaMemcpy(step.bias_packed + (size_t)j * step.N, step.bias, (size_t)step.N * 4, cudaMemcpyDeviceToDevice);
                }
            }
            if (e == cudaSuccess) e = launch_f32_to_bf16(km32, km16, (int64_t)w_elems, 0, &ctx->launches);
            if (e != cudaSuccess) return bail(TFJSB_ERR_CUDA, std::string("converting weights: ") + cudaGetErrorString(e));
            step.filter16 = km16;
        }
        if (step.kind == STEP_GEMM_TF32) {
            // weights [K,N] -> [N,K] once, on the device
            if ((st = dev_alloc(m, (size_t)(step.K * step.N), &step.filter_km)) != TFJSB_OK) return bail(st, ctx->last_error);
            cudaError_t e = launch_transpose(step.filter, step.filter_km, step.K, step.N, 0, &ctx->launches);
            if (e != cudaSuccess) return bail(TFJSB_ERR_CUDA, std::string("transposing weights: ") + cudaGetErrorString(e));
        }
        step.out_elems = 1;
        for (int i = 0; i < step.out_rank; ++i) step.out_elems *= step.out_dims[i];
        rank = step.out_rank;
        for (int i = 0; i < 4; ++i) d[i] = i < rank ? step.out_dims[i] : 0;
        m->steps.push_back(step);
    }

    if (m->narrow) {
        // every layer output is stored narrow except dense and softmax outputs and the model's result
        const size_t n = m->steps.size();
        for (size_t i = 0; i < n; ++i) {
            Step& sp = m->steps[i];
            sp.out_bf16 = !sp.is_dense && sp.kind != STEP_SOFTMAX && i + 1 != n;
            sp.in_f32 = i == 0 || !m->steps[i - 1].out_bf16;
            if (sp.in_f32 && (sp.kind == STEP_GEMM_NARROW || sp.kind == STEP_DEPTHWISE_NARROW || sp.kind == STEP_POOL_NARROW))
                return bail(TFJSB_ERR_UNSUPPORTED, "layer " + std::to_string(i) + ": in the bfloat16 storage mode only conv2d and "
                                                   "softmax layers read an fp32 tensor");
            // A small-window first layer (the 3x3 stem on RGB input) runs on the tensor cores: the patch kernel
            // rounds the fp32 image as it builds the operand tile, multiplies in TF32 (exact for bfloat16
            // values) and stores bfloat16.
            if (sp.kind == STEP_CONV_NARROW && sp.in_f32 && sp.out_bf16 && !sp.is_dense && sp.g.Co % 8 == 0 &&
                conv_patch_supported(sp.g) && !getenv("TFJSB_NO_PATCH_CONV")) {
                const int64_t k_pad = conv_igemm_k_pad(sp.g);
                if ((st = dev_alloc(m, (size_t)(k_pad * sp.g.Co), &sp.filter_km)) != TFJSB_OK) return bail(st, ctx->last_error);
                cudaError_t e = launch_pack_filter(sp.filter, sp.filter_km, (int64_t)sp.g.fh * sp.g.fw * sp.g.C, sp.g.Co, k_pad, 0,
                                                   &ctx->launches);
                if (e != cudaSuccess) return bail(TFJSB_ERR_CUDA, std::string("packing weights: ") + cudaGetErrorString(e));
                sp.conv_patch = true;
            }
        }
    }
    // arena: two regions, each large enough for the largest intermediate
    int64_t largest = 0;
    for (size_t i = 0; i + 1 < m->steps.size(); ++i)
        if (m->steps[i].out_elems > largest) largest = m->steps[i].out_elems;
    m->region_elems = (size_t)((largest + 63) / 64 * 64);
    if (m->use_tf32 && !getenv("TFJSB_NO_FUSION")) {
        for (size_t i = 0; i + 1 < m->steps.size(); ++i) {
            Step& dw = m->steps[i];
            const Step& pw = m->steps[i + 1];
            if (dw.kind == STEP_DEPTHWISE && pw.kind == STEP_GEMM_TF32 && pw.K == dw.g.Co &&
                pw.M == dw.g.N * dw.g.Ho * dw.g.Wo && dwpw_fused_supported(dw.g, pw.N)) {
                // The fused kernel has one unit of parallelism per 8 x 16 pixel tile: it pays off when
                // there are several waves of tiles; with few tiles (small batches, 14 x 14 images) the
                // stand-alone kernels spread channel blocks and column tiles over more SMs.
                const int64_t tiles = dw.g.N * ((dw.g.Ho + 7) / 8) * ((dw.g.Wo + 15) / 16);
                dw.fusable = true;
                dw.fuse_pays = tiles >= 4 * (int64_t)ctx->sm_count;
                dw.fuse_next = dw.fuse_pays;
            }
        }
    }
    if (m->narrow && !getenv("TFJSB_NO_FUSION")) {
        // The same fused kernel in the narrow format: bfloat16 patches in, the depthwise result rounded to
        // bfloat16 on its way into the operand tile, TF32 multiplies (exact for bfloat16 values), bfloat16 out.
        for (size_t i = 0; i + 1 < m->steps.size(); ++i) {
            Step& dw = m->steps[i];
            const Step& pw = m->steps[i + 1];
            if (dw.kind == STEP_DEPTHWISE_NARROW && pw.kind == STEP_GEMM_NARROW && !pw.is_dense && pw.filter_km && pw.K == dw.g.Co &&
                pw.M == dw.g.N * dw.g.Ho * dw.g.Wo && pw.N % 8 == 0 && dw.out_bf16 && pw.out_bf16 && dwpw_fused_supported(dw.g, pw.N)) {
                const int64_t tiles = dw.g.N * ((dw.g.Ho + 7) / 8) * ((dw.g.Wo + 15) / 16);
                // Available (tfjsb_model_set_fusion(model, 2)) but not chosen: the fused kernel is paced by its own
                // pipeline, not by memory traffic, so halving the bytes does not speed it up, while the separate
                // narrow kernels do gain from it (batch 128: 118 / 106 / 66 us fused against 66+55 / 63+37 / 35+26).
                (void)tiles;
                dw.fusable = true;
                dw.fuse_pays = false;
                dw.fuse_next = false;
            }
        }
    }
    if ((st = dev_alloc(m, 2 * m->region_elems, &m->arena)) != TFJSB_OK) return bail(st, ctx->last_error);
    cudaError_t e = cudaDeviceSynchronize();  // weight transposes done
    if (e != cudaSuccess) return bail(TFJSB_ERR_CUDA, std::string("model set-up: ") + cudaGetErrorString(e));
    ++ctx->live_models;
    *out = m;
    return TFJSB_OK;
}

tfjsb_status tfjsb_model_destroy(tfjsb_model* m) {
    if (!m) return TFJSB_ERR_INVALID_ARG;
    cudaDeviceSynchronize();
    drop_graph(m);
    if (m->capture_stream) cudaStreamDestroy(m->capture_stream);
    for (tfjsb_model* v : m->slices) {
        drop_graph(v);
        if (v->capture_stream) cudaStreamDestroy(v->capture_stream);
        delete v;
    }
    for (cudaEvent_t e : m->slice_copied) cudaEventDestroy(e);
    for (cudaEvent_t e : m->host_run_done)
        if (e) cudaEventDestroy(e);
    if (m->copy_stream) cudaStreamDestroy(m->copy_stream);
    for (float* p : m->owned) cudaFree(p);
    --m->ctx->live_models;
    delete m;
    return TFJSB_OK;
}

tfjsb_status tfjsb_model_output_shape(tfjsb_model* m, int32_t* rank, int64_t dims[4]) {
    if (!m || !rank || !dims) return TFJSB_ERR_INVALID_ARG;
    const Step& last = m->steps.back();
    *rank = last.out_rank;
    for (int i = 0; i < 4; ++i) dims[i] = i < last.out_rank ? last.out_dims[i] : 0;
    return TFJSB_OK;
}

int32_t tfjsb_model_launches_per_run(tfjsb_model* m) { return m ? (int32_t)launches_per_run(m) : -1; }

tfjsb_status tfjsb_run_model(tfjsb_model* m, const tfjsb_tensor* input, tfjsb_tensor* output, void* stream) {
    if (!m) return TFJSB_ERR_INVALID_ARG;
    tfjsb_status st = check_io(m, input, output);
    if (st != TFJSB_OK) return st;
    if (m->bound_in != input->data || m->bound_out != output->data) {
        if ((st = bind_all(m, static_cast<const float*>(input->data), static_cast<float*>(output->data))) != TFJSB_OK) return st;
        drop_graph(m);  // the captured launches point at the old buffers
    }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (m->use_graph) {
        if (!m->graph_exec && (st = capture_graph(m)) != TFJSB_OK) return st;
        cudaError_t e = cudaGraphLaunch(m->graph_exec, s);
        if (e != cudaSuccess) return cuda_fail(m->ctx, e, "cudaGraphLaunch");
        m->ctx->launches += launches_per_run(m);
        return TFJSB_OK;
    }
    for (int i = 0, used = 1; i < (int)m->steps.size(); i += used) {
        cudaError_t e = launch_layers(m, i, s, &used);
        if (e != cudaSuccess) return cuda_fail(m->ctx, e, "layer launch");
    }
    return TFJSB_OK;
}

tfjsb_status tfjsb_model_set_fusion(tfjsb_model* m, int mode) {
    if (!m) return TFJSB_ERR_INVALID_ARG;
    if (mode < 0 || mode > 2) return fail(m->ctx, TFJSB_ERR_INVALID_ARG, "fusion mode must be 0 (off), 1 (auto) or 2 (always)");
    for (Step& st : m->steps) st.fuse_next = st.fusable && (mode == 2 || (mode == 1 && st.fuse_pays));
    for (tfjsb_model* v : m->slices) {
        for (Step& st : v->steps) st.fuse_next = st.fusable && (mode == 2 || (mode == 1 && st.fuse_pays));
        v->bound_in = nullptr; v->bound_out = nullptr;
        drop_graph(v);
    }
    m->bound_in = nullptr;  // buffers and plans are re-assigned on the next run
    m->bound_out = nullptr;
    drop_graph(m);
    return TFJSB_OK;
}

tfjsb_status tfjsb_model_set_graph(tfjsb_model* m, int use_graph) {
    if (!m) return TFJSB_ERR_INVALID_ARG;
    m->use_graph = use_graph != 0;
    if (!m->use_graph) drop_graph(m);
    return TFJSB_OK;
}

}  // extern "C"

namespace {

// Enqueues one run from / to host memory on staging set `b` and records host_run_done[b]; no waiting
// except for the run that last used the same staging set.
tfjsb_status enqueue_host_run(tfjsb_model* m, const float* host_input, float* host_output, cudaStream_t s, int b) {
    tfjsb_ctx* ctx = m->ctx;
    tfjsb_status st;
    cudaError_t e;
    const Step& last = m->steps.back();
    if (m->host_run_pending[b]) {  // its output has been delivered and its staging buffers are free after this
        if ((e = cudaEventSynchronize(m->host_run_done[b])) != cudaSuccess) return cuda_fail(ctx, e, "cudaEventSynchronize");
        m->host_run_pending[b] = false;
    }
    if (!m->staged_in[b]) {
        if ((st = dev_alloc(m, (size_t)m->in_elems, &m->staged_in[b])) != TFJSB_OK) return st;
        if ((st = dev_alloc(m, (size_t)last.out_elems, &m->staged_out[b])) != TFJSB_OK) return st;
        if ((e = cudaEventCreateWithFlags(&m->host_run_done[b], cudaEventDisableTiming)) != cudaSuccess)
            return cuda_fail(ctx, e, "cudaEventCreate");
    }
    if (m->keep_all) {
        // debug mode: the whole batch through the model itself, so that every layer's output stays readable
        e = cudaMemcpyAsync(m->staged_in[b], host_input, (size_t)m->in_elems * 4, cudaMemcpyHostToDevice, s);
        if (e != cudaSuccess) return cuda_fail(ctx, e, "host-to-device copy of the input");
        tfjsb_tensor in{m->staged_in[b], 4, {m->in_dims[0], m->in_dims[1], m->in_dims[2], m->in_dims[3]}};
        tfjsb_tensor out{m->staged_out[b], last.out_rank, {last.out_dims[0], last.out_dims[1], last.out_dims[2], last.out_dims[3]}};
        if ((st = tfjsb_run_model(m, &in, &out, s)) != TFJSB_OK) return st;
    } else {
        if (m->slices.empty()) {
            const int64_t n = m->in_dims[0];
            // four slices: more of them lose more to per-launch fixed costs than the extra overlap returns
            int n_slices = (n % 4 == 0 && n >= 32) ? 4 : 1;
            if (const char* env = getenv("TFJSB_HOST_SLICES")) {  // tuning knob: 1 disables the slicing
                const int v = atoi(env);
                if (v >= 1 && n % v == 0) n_slices = v;
            }
            if ((e = cudaStreamCreateWithFlags(&m->copy_stream, cudaStreamNonBlocking)) != cudaSuccess)
                return cuda_fail(ctx, e, "cudaStreamCreate");
            for (int i = 0; i < 2 * n_slices; ++i) {
                cudaEvent_t ev;
                if ((e = cudaEventCreateWithFlags(&ev, cudaEventDisableTiming)) != cudaSuccess)
                    return cuda_fail(ctx, e, "cudaEventCreate");
                m->slice_copied.push_back(ev);
                m->slices.push_back(make_batch_view(m, n / n_slices));
            }
            m->n_slices = n_slices;
        }
        const int n_slices = m->n_slices;
        const int64_t in_slice = m->in_elems / n_slices, out_slice = last.out_elems / n_slices;
        // The copies wait for nothing on `stream`: the staging set is free (checked above), so they may
        // run while an earlier run is still computing.
        for (int c = 0; c < n_slices; ++c) {
            e = cudaMemcpyAsync(m->staged_in[b] + c * in_slice, host_input + c * in_slice, (size_t)in_slice * 4,
                                cudaMemcpyHostToDevice, m->copy_stream);
            if (e != cudaSuccess) return cuda_fail(ctx, e, "host-to-device copy of the input");
            if ((e = cudaEventRecord(m->slice_copied[b * n_slices + c], m->copy_stream)) != cudaSuccess)
                return cuda_fail(ctx, e, "cudaEventRecord");
        }
        for (int c = 0; c < n_slices; ++c) {
            tfjsb_model* v = m->slices[b * n_slices + c];
            if ((e = cudaStreamWaitEvent(s, m->slice_copied[b * n_slices + c], 0)) != cudaSuccess)
                return cuda_fail(ctx, e, "cudaStreamWaitEvent");
            tfjsb_tensor in{m->staged_in[b] + c * in_slice, 4, {v->in_dims[0], v->in_dims[1], v->in_dims[2], v->in_dims[3]}};
            const Step& vl = v->steps.back();
            tfjsb_tensor out{m->staged_out[b] + c * out_slice, vl.out_rank, {vl.out_dims[0], vl.out_dims[1], vl.out_dims[2], vl.out_dims[3]}};
            if ((st = tfjsb_run_model(v, &in, &out, s)) != TFJSB_OK) return st;
            v->use_graph = true;  // the first pass ran launch by launch; later passes replay a graph
        }
    }
    e = cudaMemcpyAsync(host_output, m->staged_out[b], (size_t)last.out_elems * 4, cudaMemcpyDeviceToHost, s);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "device-to-host copy of the output");
    if ((e = cudaEventRecord(m->host_run_done[b], s)) != cudaSuccess) return cuda_fail(ctx, e, "cudaEventRecord");
    m->host_run_pending[b] = true;
    return TFJSB_OK;
}

}  // namespace

extern "C" {

tfjsb_status tfjsb_run_model_host_async(tfjsb_model* m, const float* host_input, float* host_output, void* stream) {
    if (!m) return TFJSB_ERR_INVALID_ARG;
    if (!host_input || !host_output) return fail(m->ctx, TFJSB_ERR_INVALID_ARG, "host_input / host_output is null");
    const int b = m->next_staging;
    tfjsb_status st = enqueue_host_run(m, host_input, host_output, static_cast<cudaStream_t>(stream), b);
    if (st == TFJSB_OK) m->next_staging = b ^ 1;
    return st;
}

tfjsb_status tfjsb_model_host_wait(tfjsb_model* m) {
    if (!m) return TFJSB_ERR_INVALID_ARG;
    for (int k = 0; k < 2; ++k) {
        const int b = (m->next_staging + k) & 1;  // older run first
        if (!m->host_run_pending[b]) continue;
        cudaError_t e = cudaEventSynchronize(m->host_run_done[b]);
        if (e != cudaSuccess) return cuda_fail(m->ctx, e, "cudaEventSynchronize");
        m->host_run_pending[b] = false;
    }
    return TFJSB_OK;
}

tfjsb_status tfjsb_run_model_host(tfjsb_model* m, const float* host_input, float* host_output, void* stream) {
    tfjsb_status st = tfjsb_run_model_host_async(m, host_input, host_output, stream);
    if (st != TFJSB_OK) return st;
    if ((st = tfjsb_model_host_wait(m)) != TFJSB_OK) return st;
    cudaError_t e = cudaStreamSynchronize(static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_fail(m->ctx, e, "cudaStreamSynchronize");
    return TFJSB_OK;
}

tfjsb_status tfjsb_model_set_keep_all(tfjsb_model* m, int keep_all) {
    if (!m) return TFJSB_ERR_INVALID_ARG;
    if (keep_all && !m->keep_all_arena) {
        size_t total = 0;
        for (size_t i = 0; i + 1 < m->steps.size(); ++i) total += (size_t)((m->steps[i].out_elems + 63) / 64 * 64);
        tfjsb_status st = dev_alloc(m, total, &m->keep_all_arena);
        if (st != TFJSB_OK) return st;
    }
    m->keep_all = keep_all != 0;
    drop_graph(m);
    m->bound_in = nullptr;  // force a re-bind on the next run
    m->bound_out = nullptr;
    return TFJSB_OK;
}

tfjsb_status tfjsb_model_layer_output(tfjsb_model* m, int layer, tfjsb_tensor* view) {
    if (!m || !view) return TFJSB_ERR_INVALID_ARG;
    if (layer < 0 || layer >= (int)m->steps.size()) return fail(m->ctx, TFJSB_ERR_INVALID_ARG, "no such layer");
    const Step& st = m->steps[layer];
    if (!st.out) return fail(m->ctx, TFJSB_ERR_INVALID_ARG, "the model has not run yet");
    if (st.out_bf16)
        return fail(m->ctx, TFJSB_ERR_UNSUPPORTED, "this layer's output is stored as bfloat16: read it with tfjsb_model_layer_output_f32");
    view->data = st.out;
    view->rank = st.out_rank;
    for (int i = 0; i < 4; ++i) view->dims[i] = i < st.out_rank ? st.out_dims[i] : 0;
    return TFJSB_OK;
}

tfjsb_status tfjsb_model_layer_kernel(tfjsb_model* m, int layer, char* name, int32_t name_len) {
    if (!m || !name || name_len < 1) return TFJSB_ERR_INVALID_ARG;
    if (layer < 0 || layer >= (int)m->steps.size()) return fail(m->ctx, TFJSB_ERR_INVALID_ARG, "no such layer");
    const Step& st = m->steps[layer];
    if (!st.out) return fail(m->ctx, TFJSB_ERR_INVALID_ARG, "the model has not run yet");
    const bool fused_mode = !m->keep_all;
    const char* k = "?";
    if (fused_mode && layer > 0 && m->steps[layer - 1].fuse_next) k = "(in the previous layer's kernel)";
    else if (fused_mode && st.fuse_next) k = "dwpw_fused_kernel<false>";
    else switch (st.kind) {
        case STEP_GEMM_TF32:
            k = st.plan.pair ? "gemm_pair_kernel<false>" : st.plan.cluster_split ? "gemm_tf32_splitk_kernel" : "gemm_tf32_kernel<false>";
            break;
        case STEP_CONV_TF32: k = st.conv_patch ? "dwpw_fused_kernel<true>" : "gemm_tf32_kernel<true>"; break;
        case STEP_GEMM_FP32: k = "gemm_fp32_kernel"; break;
        case STEP_CONV_FP32: k = "conv2d_fp32_kernel"; break;
        case STEP_DEPTHWISE: k = st.dw_plan.variant >= 0 ? "depthwise3x3_tma_kernel" : "depthwise3x3_kernel"; break;
        case STEP_POOL: k = (st.g.Ho == 1 && st.g.Wo == 1 && st.g.fh == st.g.H && st.g.fw == st.g.W) ? "avg_pool_global_kernel" : "avg_pool_window_kernel"; break;
        case STEP_SOFTMAX: k = "softmax_rows_kernel"; break;
        case STEP_GEMM_NARROW: k = st.plan16.pair ? "gemm_pair_kernel<true>" : "gemm_bf16_kernel"; break;
        case STEP_CONV_NARROW: k = st.conv_patch ? "dwpw_fused_kernel<true, true>" : "conv_narrow_kernel"; break;
        case STEP_DEPTHWISE_NARROW: k = st.dw_plan.variant >= 0 ? "depthwise3x3_tma_kernel" : "depthwise3x3_narrow_kernel"; break;
        case STEP_POOL_NARROW: k = "avg_pool_global_narrow_kernel"; break;
    }
    snprintf(name, (size_t)name_len, "%s", k);
    return TFJSB_OK;
}

tfjsb_status tfjsb_model_layer_shape(tfjsb_model* m, int layer, int32_t* rank, int64_t dims[4]) {
    if (!m || !rank || !dims) return TFJSB_ERR_INVALID_ARG;
    if (layer < 0 || layer >= (int)m->steps.size()) return fail(m->ctx, TFJSB_ERR_INVALID_ARG, "no such layer");
    const Step& st = m->steps[layer];
    *rank = st.out_rank;
    for (int i = 0; i < 4; ++i) dims[i] = i < st.out_rank ? st.out_dims[i] : 0;
    return TFJSB_OK;
}

tfjsb_status tfjsb_model_layer_output_f32(tfjsb_model* m, int layer, float* dst, void* stream) {
    if (!m) return TFJSB_ERR_INVALID_ARG;
    if (!dst) return fail(m->ctx, TFJSB_ERR_INVALID_ARG, "dst is null");
    if (layer < 0 || layer >= (int)m->steps.size()) return fail(m->ctx, TFJSB_ERR_INVALID_ARG, "no such layer");
    const Step& st = m->steps[layer];
    if (!st.out) return fail(m->ctx, TFJSB_ERR_INVALID_ARG, "the model has not run yet");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    cudaError_t e = st.out_bf16 ? launch_bf16_to_f32(st.out, dst, st.out_elems, s, &m->ctx->launches)
                                : cudaMemcpyAsync(dst, st.out, (size_t)st.out_elems * 4, cudaMemcpyDeviceToDevice, s);
    if (e != cudaSuccess) return cuda_fail(m->ctx, e, "reading a layer's output");
    return TFJSB_OK;
}

tfjsb_status tfjsb_model_profile(tfjsb_model* m, const tfjsb_tensor* input, tfjsb_tensor* output, int reps,
                                 float* ms_per_layer, void* stream) {
    if (!m) return TFJSB_ERR_INVALID_ARG;
    tfjsb_ctx* ctx = m->ctx;
    if (!ms_per_layer || reps < 1) return fail(ctx, TFJSB_ERR_INVALID_ARG, "ms_per_layer is null or reps < 1");
    tfjsb_status st = check_io(m, input, output);
    if (st != TFJSB_OK) return st;
    if (m->bound_in != input->data || m->bound_out != output->data) {
        if ((st = bind_all(m, static_cast<const float*>(input->data), static_cast<float*>(output->data))) != TFJSB_OK) return st;
    }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int n = (int)m->steps.size();
    std::vector<cudaEvent_t> ev((size_t)n + 1);
    for (auto& e : ev)
        if (cudaEventCreate(&e) != cudaSuccess) return fail(ctx, TFJSB_ERR_CUDA, "cudaEventCreate failed");
    std::vector<double> sum((size_t)n, 0.0);
    tfjsb_status rc = TFJSB_OK;
    for (int r = 0; r < reps && rc == TFJSB_OK; ++r) {
        cudaEventRecord(ev[0], s);
        for (int i = 0, used = 1; i < n; i += used) {
            cudaError_t e = launch_layers(m, i, s, &used);
            if (e != cudaSuccess) { rc = cuda_fail(ctx, e, "layer launch"); break; }
            // a fused pair reports its whole time under the first layer and zero under the second
            for (int k = 1; k <= used; ++k) cudaEventRecord(ev[i + k], s);
        }
        cudaError_t e = cudaStreamSynchronize(s);
        if (e != cudaSuccess) { rc = cuda_fail(ctx, e, "cudaStreamSynchronize"); break; }
        if (rc != TFJSB_OK) break;
        for (int i = 0; i < n; ++i) {
            float ms = 0.f;
            cudaEventElapsedTime(&ms, ev[i], ev[i + 1]);
            sum[i] += ms;
        }
    }
    for (auto& e : ev) cudaEventDestroy(e);
    if (rc == TFJSB_OK)
        for (int i = 0; i < n; ++i) ms_per_layer[i] = (float)(sum[i] / reps);
    return rc;
}

}  // extern "C"

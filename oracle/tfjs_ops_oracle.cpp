// CPU oracle for the op kernels of a TensorFlow.js-style inference path.
//
// TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what each op
// computes; it shares no code with the CUDA library and is never on the product path.
// It is called from the test-suite, from the smoke check and from the benchmark's
// cpu-baseline leg, and from nowhere else.
//
// What it follows.  The paper (arxiv 1901.05350) names the ops (`tf.matMul`, Sec. 3.6;
// `tf.conv2d` sampling a 4-D tensor by (batch, row, column, depth), Sec. 4.1) and prints one
// kernel, the matMul shader of Listing 2; it does not define conv2d, depthwiseConv2d,
// avgPool, softmax, relu6 or 'same'/'valid' padding.  Those are written here as TensorFlow
// defines them (the reading this project takes of "as TF.js defines it"):
//   * tensors are fp32, dense, row-major, NHWC; filters are [fh, fw, Cin, Cout]
//     (depthwise: [fh, fw, C, multiplier]);
//   * conv2d is a cross-correlation (no filter flip); positions outside the image read as 0;
//   * 'same' puts the odd padding element after (bottom / right);
//   * avgPool divides by the number of in-bounds window elements;
//   * softmax subtracts the row maximum before exponentiating.
//
// Arithmetic.  None of the ops is an approximation, so every function is the plain
// definition: the sum is accumulated in double in the order the definition names its
// indices, rounded once to fp32; bias is then added in fp32 and the activation applied in
// fp32.  No blocking, no reordering.  `#pragma omp parallel for` over the outermost
// independent index only spreads output elements over threads; each element's arithmetic
// is unchanged.
//
// Gradients (Sec. 3.5: eager differentiation calls a gradient function per kernel).  The paper names no
// gradient op; each one here is the adjoint of the forward definition above, written as a gather over
// the forward op's index relation: every (output, tap) pair that read an input sample in the forward
// pass sends its gradient back to it, nothing else does.
//
// Parity pins (tests/test_oracle_*.py): integer-exact inputs against exact integer
// arithmetic; torch/scipy library routines on the special cases that reduce to them;
// an independently written scatter-form evaluator on tiny shapes; identity/delta filters;
// hand-derived padding tables; algebraic identities; softmax/relu6 invariants; the
// Listing 2 arithmetic restated in fp32.  Gradients: the adjoint identity <op(x), g> = <x, op^T(g)>
// on integers (exact), central finite differences of the forward oracle, torch fp64 autograd.
// Parity unpinned: nothing in this file.  (The seeded number generator is not part of the
// oracle; both sides consume the same bytes.)

#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>

#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

enum { PAD_VALID = 0, PAD_SAME = 1 };
enum { ACT_NONE = 0, ACT_RELU = 1, ACT_RELU6 = 2 };
enum { OPERAND_FP32 = 0, OPERAND_TF32_RNA = 1, OPERAND_TF32_RZ = 2 };

// Output extent and padding of one spatial dimension (TensorFlow's formulas).
//   effective kernel  ek = (k-1)*d + 1
//   valid: out = floor((in - ek)/s) + 1, no padding
//   same : out = ceil(in/s); total = max((out-1)*s + ek - in, 0); before = total/2 (floor)
bool window_geometry(int in, int k, int s, int d, int pad_mode, int* out, int* before, int* after) {
    if (in < 1 || k < 1 || s < 1 || d < 1) return false;
    const int ek = (k - 1) * d + 1;
    if (pad_mode == PAD_VALID) {
        if (in < ek) return false;
        *out = (in - ek) / s + 1;
        *before = 0;
        *after = 0;
        return true;
    }
    if (pad_mode == PAD_SAME) {
        *out = (in + s - 1) / s;
        int total = (*out - 1) * s + ek - in;
        if (total < 0) total = 0;
        *before = total / 2;
        *after = total - *before;
        return true;
    }
    return false;
}

// Optional emulation of the operand rounding a TF32 multiplier applies (10 explicit
// mantissa bits): RNA = nearest, ties away from zero; RZ = truncate.  Diagnostic only.
inline double operand(float v, int mode) {
    if (mode == OPERAND_FP32) return (double)v;
    uint32_t bits;
    std::memcpy(&bits, &v, 4);
    if ((bits & 0x7F800000u) == 0x7F800000u) return (double)v;  // inf / nan unchanged
    if (mode == OPERAND_TF32_RNA) bits += 0x00001000u;
    bits &= 0xFFFFE000u;
    float r;
    std::memcpy(&r, &bits, 4);
    return (double)r;
}

// bias add (one fp32 add) then activation, both in fp32.
// relu(v) = v > 0 ? v : +0 except that NaN stays NaN; relu6(v) = min(relu(v), 6).
inline float bias_then_act(float acc, const float* bias, int64_t c, int act) {
    float v = acc;
    if (bias) v = v + bias[c];
    if (act == ACT_NONE) return v;
    if (v != v) return v;  // NaN propagates
    float r = v > 0.0f ? v : 0.0f;
    if (act == ACT_RELU6 && r > 6.0f) r = 6.0f;
    return r;
}

}  // namespace

extern "C" {

void orc_set_threads(int n) {
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
#else
    (void)n;
#endif
}

int orc_get_threads() {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

int orc_window_geometry(int in, int k, int s, int d, int pad_mode, int* out, int* before, int* after) {
    return window_geometry(in, k, s, d, pad_mode, out, before, after) ? 0 : 1;
}

// C[i,j] = fl32( sum_k A'[i,k] * B'[k,j] ),  A' = tA ? A^T : A,  B' = tB ? B^T : B.
// a is stored [M,K] (or [K,M] when tA), b is stored [K,N] (or [N,K] when tB).
int orc_matmul(const float* a, const float* b, int64_t M, int64_t K, int64_t N, int tA, int tB,
               float* c, int operand_mode) {
    if (!a || !b || !c || M < 0 || K < 0 || N < 0) return 1;
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < M; ++i) {
        for (int64_t j = 0; j < N; ++j) {
            double acc = 0.0;
            for (int64_t k = 0; k < K; ++k) {
                const float av = tA ? a[k * M + i] : a[i * K + k];
                const float bv = tB ? b[j * K + k] : b[k * N + j];
                acc += operand(av, operand_mode) * operand(bv, operand_mode);
            }
            c[i * N + j] = (float)acc;
        }
    }
    return 0;
}

// y[n,oy,ox,co] = act( fl32( sum_{ky,kx,ci} x[n, oy*sh - pt + ky*dh, ox*sw - pl + kx*dw, ci]
//                                          * f[ky,kx,ci,co] ) + bias[co] )
int orc_conv2d(const float* x, int64_t N, int H, int W, int Cin, const float* f, int fh, int fw, int Cout,
               int sh, int sw, int pad_mode, int dh, int dw, const float* bias, int act, float* y,
               int operand_mode) {
    int Ho, Wo, pt, pb, pl, pr;
    if (!x || !f || !y) return 1;
    if (!window_geometry(H, fh, sh, dh, pad_mode, &Ho, &pt, &pb)) return 2;
    if (!window_geometry(W, fw, sw, dw, pad_mode, &Wo, &pl, &pr)) return 2;
#pragma omp parallel for collapse(2) schedule(static)
    for (int64_t n = 0; n < N; ++n) {
        for (int oy = 0; oy < Ho; ++oy) {
            for (int ox = 0; ox < Wo; ++ox) {
                for (int co = 0; co < Cout; ++co) {
                    double acc = 0.0;
                    for (int ky = 0; ky < fh; ++ky) {
                        const int iy = oy * sh - pt + ky * dh;
                        if (iy < 0 || iy >= H) continue;
                        for (int kx = 0; kx < fw; ++kx) {
                            const int ix = ox * sw - pl + kx * dw;
                            if (ix < 0 || ix >= W) continue;
                            const float* xp = x + ((n * H + iy) * (int64_t)W + ix) * Cin;
                            const float* fp = f + ((int64_t)(ky * fw + kx) * Cin) * Cout + co;
                            for (int ci = 0; ci < Cin; ++ci)
                                acc += operand(xp[ci], operand_mode) * operand(fp[(int64_t)ci * Cout], operand_mode);
                        }
                    }
                    y[((n * Ho + oy) * (int64_t)Wo + ox) * Cout + co] = bias_then_act((float)acc, bias, co, act);
                }
            }
        }
    }
    return 0;
}

// y[n,oy,ox,c*mult+q] = act( fl32( sum_{ky,kx} x[n,iy,ix,c] * f[ky,kx,c,q] ) + bias[c*mult+q] )
int orc_depthwise_conv2d(const float* x, int64_t N, int H, int W, int C, const float* f, int fh, int fw,
                         int mult, int sh, int sw, int pad_mode, int dh, int dw, const float* bias, int act,
                         float* y) {
    int Ho, Wo, pt, pb, pl, pr;
    if (!x || !f || !y || mult < 1) return 1;
    if (!window_geometry(H, fh, sh, dh, pad_mode, &Ho, &pt, &pb)) return 2;
    if (!window_geometry(W, fw, sw, dw, pad_mode, &Wo, &pl, &pr)) return 2;
    const int64_t Co = (int64_t)C * mult;
#pragma omp parallel for collapse(2) schedule(static)
    for (int64_t n = 0; n < N; ++n) {
        for (int oy = 0; oy < Ho; ++oy) {
            for (int ox = 0; ox < Wo; ++ox) {
                for (int c = 0; c < C; ++c) {
                    for (int q = 0; q < mult; ++q) {
                        double acc = 0.0;
                        for (int ky = 0; ky < fh; ++ky) {
                            const int iy = oy * sh - pt + ky * dh;
                            if (iy < 0 || iy >= H) continue;
                            for (int kx = 0; kx < fw; ++kx) {
                                const int ix = ox * sw - pl + kx * dw;
                                if (ix < 0 || ix >= W) continue;
                                acc += (double)x[((n * H + iy) * (int64_t)W + ix) * C + c] *
                                       (double)f[((int64_t)(ky * fw + kx) * C + c) * mult + q];
                            }
                        }
                        const int64_t oc = (int64_t)c * mult + q;
                        y[((n * Ho + oy) * (int64_t)Wo + ox) * Co + oc] = bias_then_act((float)acc, bias, oc, act);
                    }
                }
            }
        }
    }
    return 0;
}

// y[r, c] = act(x[r, c] + bias[c]) over `rows` rows of C channels (channels last).
int orc_bias_act(const float* x, int64_t rows, int64_t C, const float* bias, int act, float* y) {
    if (!x || !y) return 1;
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t c = 0; c < C; ++c) y[r * C + c] = bias_then_act(x[r * C + c], bias, c, act);
    return 0;
}

// y[n,oy,ox,c] = (sum of in-bounds window elements) / (number of in-bounds window elements)
int orc_avg_pool(const float* x, int64_t N, int H, int W, int C, int fh, int fw, int sh, int sw, int pad_mode,
                 float* y) {
    int Ho, Wo, pt, pb, pl, pr;
    if (!x || !y) return 1;
    if (!window_geometry(H, fh, sh, 1, pad_mode, &Ho, &pt, &pb)) return 2;
    if (!window_geometry(W, fw, sw, 1, pad_mode, &Wo, &pl, &pr)) return 2;
#pragma omp parallel for collapse(2) schedule(static)
    for (int64_t n = 0; n < N; ++n) {
        for (int oy = 0; oy < Ho; ++oy) {
            for (int ox = 0; ox < Wo; ++ox) {
                for (int c = 0; c < C; ++c) {
                    double acc = 0.0;
                    int64_t count = 0;
                    for (int ky = 0; ky < fh; ++ky) {
                        const int iy = oy * sh - pt + ky;
                        if (iy < 0 || iy >= H) continue;
                        for (int kx = 0; kx < fw; ++kx) {
                            const int ix = ox * sw - pl + kx;
                            if (ix < 0 || ix >= W) continue;
                            acc += (double)x[((n * H + iy) * (int64_t)W + ix) * C + c];
                            ++count;
                        }
                    }
                    y[((n * Ho + oy) * (int64_t)Wo + ox) * C + c] = (float)(acc / (double)count);
                }
            }
        }
    }
    return 0;
}

// y[n,oy,ox,c] = largest in-bounds window element (padding never takes part; a NaN in the window gives NaN).
// tf.maxPool: not defined in the paper; TensorFlow's definition, with the window geometry above.
int orc_max_pool(const float* x, int64_t N, int H, int W, int C, int fh, int fw, int sh, int sw, int pad_mode,
                 float* y) {
    int Ho, Wo, pt, pb, pl, pr;
    if (!x || !y) return 1;
    if (!window_geometry(H, fh, sh, 1, pad_mode, &Ho, &pt, &pb)) return 2;
    if (!window_geometry(W, fw, sw, 1, pad_mode, &Wo, &pl, &pr)) return 2;
#pragma omp parallel for collapse(2) schedule(static)
    for (int64_t n = 0; n < N; ++n) {
        for (int oy = 0; oy < Ho; ++oy) {
            for (int ox = 0; ox < Wo; ++ox) {
                for (int c = 0; c < C; ++c) {
                    float m = -std::numeric_limits<float>::infinity();
                    for (int ky = 0; ky < fh; ++ky) {
                        const int iy = oy * sh - pt + ky;
                        if (iy < 0 || iy >= H) continue;
                        for (int kx = 0; kx < fw; ++kx) {
                            const int ix = ox * sw - pl + kx;
                            if (ix < 0 || ix >= W) continue;
                            const float v = x[((n * H + iy) * (int64_t)W + ix) * C + c];
                            if (v > m || v != v) m = v;  // once m is NaN no comparison replaces it
                        }
                    }
                    y[((n * Ho + oy) * (int64_t)Wo + ox) * C + c] = m;
                }
            }
        }
    }
    return 0;
}

// Elementwise binary op of Sec. 4.1 (the addition shader of Fig. 3 computes one output value per
// invocation): out[i] = a[i] op b[i % b_len], one fp32 operation per element.  b_len = n: same
// shapes; b_len = the last dimension: b is a vector broadcast along every other dimension.
// op: 0 add, 1 subtract, 2 multiply.
int orc_binary(int op, const float* a, const float* b, int64_t n, int64_t b_len, float* out) {
    if (!a || !b || !out || b_len < 1 || op < 0 || op > 2) return 1;
    for (int64_t i = 0; i < n; ++i) {
        const float u = a[i], v = b[i % b_len];
        out[i] = op == 0 ? u + v : (op == 1 ? u - v : u * v);
    }
    return 0;
}

// p[r, j] = exp(x[r,j] - max_r) / sum_k exp(x[r,k] - max_r), over the last dimension.
int orc_softmax(const float* x, int64_t rows, int64_t cols, float* y) {
    if (!x || !y || cols < 1) return 1;
    for (int64_t r = 0; r < rows; ++r) {
        const float* xr = x + r * cols;
        float m = -std::numeric_limits<float>::infinity();
        for (int64_t j = 0; j < cols; ++j)
            if (xr[j] > m) m = xr[j];
        double sum = 0.0;
        for (int64_t j = 0; j < cols; ++j) sum += std::exp((double)xr[j] - (double)m);
        for (int64_t j = 0; j < cols; ++j) y[r * cols + j] = (float)(std::exp((double)xr[j] - (double)m) / sum);
    }
    return 0;
}

// ---- gradients ------------------------------------------------------------------------------------

// dx[n,iy,ix,ci] = fl32( sum over (oy,ky), (ox,kx), co with oy*sh - pt + ky*dh = iy and ox*sw - pl + kx*dw = ix
//                        of dy[n,oy,ox,co] * f[ky,kx,ci,co] )
// The gradient of conv2d with respect to its input (x has shape [N,H,W,Cin]; dy the forward output's shape).
int orc_conv2d_backprop_input(const float* dy, int64_t N, int H, int W, int Cin, const float* f, int fh, int fw, int Cout,
                              int sh, int sw, int pad_mode, int dh, int dw, float* dx, int operand_mode) {
    int Ho, Wo, pt, pb, pl, pr;
    if (!dy || !f || !dx) return 1;
    if (!window_geometry(H, fh, sh, dh, pad_mode, &Ho, &pt, &pb)) return 2;
    if (!window_geometry(W, fw, sw, dw, pad_mode, &Wo, &pl, &pr)) return 2;
#pragma omp parallel for collapse(2) schedule(static)
    for (int64_t n = 0; n < N; ++n) {
        for (int iy = 0; iy < H; ++iy) {
            for (int ix = 0; ix < W; ++ix) {
                for (int ci = 0; ci < Cin; ++ci) {
                    double acc = 0.0;
                    for (int ky = 0; ky < fh; ++ky) {
                        const int ty = iy + pt - ky * dh;  // = oy*sh
                        if (ty < 0 || ty % sh != 0 || ty / sh >= Ho) continue;
                        const int oy = ty / sh;
                        for (int kx = 0; kx < fw; ++kx) {
                            const int tx = ix + pl - kx * dw;
                            if (tx < 0 || tx % sw != 0 || tx / sw >= Wo) continue;
                            const int ox = tx / sw;
                            const float* gp = dy + ((n * Ho + oy) * (int64_t)Wo + ox) * Cout;
                            const float* fp = f + ((int64_t)(ky * fw + kx) * Cin + ci) * Cout;
                            for (int co = 0; co < Cout; ++co)
                                acc += operand(gp[co], operand_mode) * operand(fp[co], operand_mode);
                        }
                    }
                    dx[((n * H + iy) * (int64_t)W + ix) * Cin + ci] = (float)acc;
                }
            }
        }
    }
    return 0;
}

// df[ky,kx,ci,co] = fl32( sum_{n,oy,ox} x[n, oy*sh - pt + ky*dh, ox*sw - pl + kx*dw, ci] * dy[n,oy,ox,co] )
// (samples outside the image are zero and add nothing).  The gradient of conv2d with respect to its filter.
int orc_conv2d_backprop_filter(const float* x, int64_t N, int H, int W, int Cin, const float* dy, int fh, int fw, int Cout,
                               int sh, int sw, int pad_mode, int dh, int dw, float* df, int operand_mode) {
    int Ho, Wo, pt, pb, pl, pr;
    if (!x || !dy || !df) return 1;
    if (!window_geometry(H, fh, sh, dh, pad_mode, &Ho, &pt, &pb)) return 2;
    if (!window_geometry(W, fw, sw, dw, pad_mode, &Wo, &pl, &pr)) return 2;
#pragma omp parallel for collapse(3) schedule(static)
    for (int ky = 0; ky < fh; ++ky) {
        for (int kx = 0; kx < fw; ++kx) {
            for (int ci = 0; ci < Cin; ++ci) {
                for (int co = 0; co < Cout; ++co) {
                    double acc = 0.0;
                    for (int64_t n = 0; n < N; ++n) {
                        for (int oy = 0; oy < Ho; ++oy) {
                            const int iy = oy * sh - pt + ky * dh;
                            if (iy < 0 || iy >= H) continue;
                            for (int ox = 0; ox < Wo; ++ox) {
                                const int ix = ox * sw - pl + kx * dw;
                                if (ix < 0 || ix >= W) continue;
                                acc += operand(x[((n * H + iy) * (int64_t)W + ix) * Cin + ci], operand_mode) *
                                       operand(dy[((n * Ho + oy) * (int64_t)Wo + ox) * Cout + co], operand_mode);
                            }
                        }
                    }
                    df[((int64_t)(ky * fw + kx) * Cin + ci) * Cout + co] = (float)acc;
                }
            }
        }
    }
    return 0;
}

// dx[n,iy,ix,c] = fl32( sum over (oy,ky), (ox,kx) meeting (iy,ix) as above, and q, of dy[n,oy,ox,c*mult+q] * f[ky,kx,c,q] )
int orc_depthwise_backprop_input(const float* dy, int64_t N, int H, int W, int C, const float* f, int fh, int fw, int mult,
                                 int sh, int sw, int pad_mode, int dh, int dw, float* dx) {
    int Ho, Wo, pt, pb, pl, pr;
    if (!dy || !f || !dx || mult < 1) return 1;
    if (!window_geometry(H, fh, sh, dh, pad_mode, &Ho, &pt, &pb)) return 2;
    if (!window_geometry(W, fw, sw, dw, pad_mode, &Wo, &pl, &pr)) return 2;
    const int64_t Co = (int64_t)C * mult;
#pragma omp parallel for collapse(2) schedule(static)
    for (int64_t n = 0; n < N; ++n) {
        for (int iy = 0; iy < H; ++iy) {
            for (int ix = 0; ix < W; ++ix) {
                for (int c = 0; c < C; ++c) {
                    double acc = 0.0;
                    for (int ky = 0; ky < fh; ++ky) {
                        const int ty = iy + pt - ky * dh;
                        if (ty < 0 || ty % sh != 0 || ty / sh >= Ho) continue;
                        const int oy = ty / sh;
                        for (int kx = 0; kx < fw; ++kx) {
                            const int tx = ix + pl - kx * dw;
                            if (tx < 0 || tx % sw != 0 || tx / sw >= Wo) continue;
                            const int ox = tx / sw;
                            for (int q = 0; q < mult; ++q)
                                acc += (double)dy[((n * Ho + oy) * (int64_t)Wo + ox) * Co + (int64_t)c * mult + q] *
                                       (double)f[((int64_t)(ky * fw + kx) * C + c) * mult + q];
                        }
                    }
                    dx[((n * H + iy) * (int64_t)W + ix) * C + c] = (float)acc;
                }
            }
        }
    }
    return 0;
}

// df[ky,kx,c,q] = fl32( sum_{n,oy,ox} x[n, oy*sh - pt + ky*dh, ox*sw - pl + kx*dw, c] * dy[n,oy,ox,c*mult+q] )
int orc_depthwise_backprop_filter(const float* x, int64_t N, int H, int W, int C, const float* dy, int fh, int fw, int mult,
                                  int sh, int sw, int pad_mode, int dh, int dw, float* df) {
    int Ho, Wo, pt, pb, pl, pr;
    if (!x || !dy || !df || mult < 1) return 1;
    if (!window_geometry(H, fh, sh, dh, pad_mode, &Ho, &pt, &pb)) return 2;
    if (!window_geometry(W, fw, sw, dw, pad_mode, &Wo, &pl, &pr)) return 2;
    const int64_t Co = (int64_t)C * mult;
#pragma omp parallel for collapse(3) schedule(static)
    for (int ky = 0; ky < fh; ++ky) {
        for (int kx = 0; kx < fw; ++kx) {
            for (int c = 0; c < C; ++c) {
                for (int q = 0; q < mult; ++q) {
                    double acc = 0.0;
                    for (int64_t n = 0; n < N; ++n) {
                        for (int oy = 0; oy < Ho; ++oy) {
                            const int iy = oy * sh - pt + ky * dh;
                            if (iy < 0 || iy >= H) continue;
                            for (int ox = 0; ox < Wo; ++ox) {
                                const int ix = ox * sw - pl + kx * dw;
                                if (ix < 0 || ix >= W) continue;
                                acc += (double)x[((n * H + iy) * (int64_t)W + ix) * C + c] *
                                       (double)dy[((n * Ho + oy) * (int64_t)Wo + ox) * Co + (int64_t)c * mult + q];
                            }
                        }
                    }
                    df[((int64_t)(ky * fw + kx) * C + c) * mult + q] = (float)acc;
                }
            }
        }
    }
    return 0;
}

// Gradient through the fused epilogue y = act(z + bias):  dz[r,c] = dy[r,c] where the activation passed its
// input through, +0 elsewhere (relu: y > 0; relu6: 0 < y < 6, the clamp's flat parts have zero slope;
// none: everywhere), written in terms of the forward OUTPUT y, which is what a caller keeps.
int orc_act_backprop(const float* y, const float* dy, int64_t n, int act, float* dz) {
    if (!y || !dy || !dz) return 1;
    for (int64_t i = 0; i < n; ++i) {
        bool pass = true;
        if (act == ACT_RELU) pass = y[i] > 0.0f;
        if (act == ACT_RELU6) pass = y[i] > 0.0f && y[i] < 6.0f;
        dz[i] = pass ? dy[i] : 0.0f;
    }
    return 0;
}

// db[c] = fl32( sum_r dz[r,c] ): the bias is added to every row, so its gradient is the column sum.
int orc_bias_backprop(const float* dz, int64_t rows, int64_t C, float* db) {
    if (!dz || !db) return 1;
    for (int64_t c = 0; c < C; ++c) {
        double acc = 0.0;
        for (int64_t r = 0; r < rows; ++r) acc += (double)dz[r * C + c];
        db[c] = (float)acc;
    }
    return 0;
}

}  // extern "C"

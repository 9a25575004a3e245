"""GPU parity of the tensor-core (tcgen05, TF32) GEMM path: matMul, 1x1 conv2d, fused epilogue.

Tolerances.  TF32 keeps 10 explicit mantissa bits of each operand, so against the exact
(double-accumulate) oracle the per-op bar is a relative Frobenius error <= 5e-3.  Against the
oracle run with the same operand rounding (products and sums still in double) only fp32
accumulation order remains, and the bar is 2e-5; whichever of truncation / round-to-nearest
matches tells how the hardware reads fp32 bits.  Small integers are exact in TF32 and every
partial sum is exact in fp32, so there the result must be bit-identical: a zero-tolerance
check of descriptors, swizzles, tile tails and the epilogue's addressing.
"""
import numpy as np
import pytest

import seeded_inputs as si
from helpers import dev, host, rel_fro, same_bits

pytestmark = pytest.mark.gpu

TF32_TOL = 5e-3
MATCHED_TOL = 2e-5

GEMM_SHAPES = [
    # M, K, N
    (128, 32, 32),        # one tile, one k-block, one MMA group
    (128, 64, 64),
    (512, 512, 512),      # config 1
    (300, 100, 72),       # ragged in M, K and N
    (1, 1024, 1000),      # batch-1 dense layer
    (128, 1024, 1000),    # batch-128 dense layer: N tail inside a 32-column chunk
    (12544, 32, 64),      # config 2 pointwise step
    (3136, 128, 128),
    (1000, 8, 16),        # K and N below one tile
    (4100, 36, 260),      # N just above one 256 tile
    (49, 1024, 1024),     # many k-blocks: the stage ring wraps several times
    (20000, 256, 512),    # more tiles than SMs: persistent loop, both accumulator stages reused
    (6272, 512, 1024),    # 196 tiles of 256 columns on 148 SMs: the 192-column tile is chosen instead
]


@pytest.mark.parametrize("mkn", GEMM_SHAPES)
def test_matmul_tf32_integer_exact(ctx, oracle, mkn):
    M, K, N = mkn
    a = si.small_integers(301, 0, (M, K), -8, 8)
    b = si.small_integers(301, 1, (K, N), -8, 8)
    got = host(ctx.matmul(dev(a), dev(b)))
    ctx.check_device_status()
    want = (a.astype(np.int64) @ b.astype(np.int64)).astype(np.float32)
    assert same_bits(got, want)


@pytest.mark.parametrize("mkn", GEMM_SHAPES)
def test_matmul_tf32_parity(ctx, oracle, mkn):
    M, K, N = mkn
    a = si.uniform(302, 0, (M, K), -1, 1)
    b = si.uniform(302, 1, (K, N), -1, 1)
    got = host(ctx.matmul(dev(a), dev(b)))
    ctx.check_device_status()
    if M * K * N <= 600_000_000:
        want = oracle.matmul(a, b)
        assert rel_fro(got, want) <= TF32_TOL
        matched = min(rel_fro(got, oracle.matmul(a, b, operand="tf32_rz")),
                      rel_fro(got, oracle.matmul(a, b, operand="tf32_rna")))
        assert matched <= MATCHED_TOL
    else:  # sampled rows, each computed one by one by the oracle
        rows = np.unique(np.linspace(0, M - 1, 257).astype(np.int64))
        want = oracle.matmul(a[rows], b)
        assert rel_fro(got[rows], want) <= TF32_TOL


SPLIT_K_SHAPES = [
    # M, K, N: few output tiles and a long K loop, so the planner cuts K into slices (work item = tile x slice)
    (128, 1024, 1000),   # dense layer at batch 128
    (1, 1024, 1000),     # dense layer at batch 1
    (49, 1024, 1024),    # pw13 at batch 1
    (196, 512, 512),     # pw7 at batch 1: two row tiles, the second mostly empty
    (300, 4100, 72),     # K not a multiple of the slice length: the last slice is short and ragged
    (512, 512, 512),     # config 1
]


@pytest.mark.parametrize("mkn", SPLIT_K_SHAPES)
def test_matmul_split_k_agrees_with_unsplit_and_oracle(ctx, oracle, monkeypatch, mkn):
    M, K, N = mkn
    a = si.uniform(311, 0, (M, K), -1, 1)
    b = si.uniform(311, 1, (K, N), -1, 1)
    monkeypatch.delenv("TFJSB_NO_SPLIT_K", raising=False)
    split = host(ctx.matmul(dev(a), dev(b)))
    again = host(ctx.matmul(dev(a), dev(b)))
    monkeypatch.setenv("TFJSB_NO_SPLIT_K", "1")
    whole = host(ctx.matmul(dev(a), dev(b)))
    ctx.check_device_status()
    assert not same_bits(split, whole)                    # another summation order: K really was cut
    assert same_bits(split, again)                        # slices are added in a fixed order, whichever finishes first
    want = oracle.matmul(a, b)
    assert rel_fro(split, want) <= TF32_TOL and rel_fro(whole, want) <= TF32_TOL
    assert rel_fro(split, oracle.matmul(a, b, operand="tf32_rz")) <= MATCHED_TOL
    ai = si.small_integers(312, 0, (M, K), -8, 8)
    bi = si.small_integers(312, 1, (K, N), -8, 8)
    monkeypatch.delenv("TFJSB_NO_SPLIT_K", raising=False)
    assert same_bits(host(ctx.matmul(dev(ai), dev(bi))), (ai.astype(np.int64) @ bi.astype(np.int64)).astype(np.float32))


def test_dense_split_k_fused_bias_and_activation(ctx, oracle):
    # the reduction applies bias and activation: [128,1,1,1024] x [1,1,1024,1000] + bias, relu6
    x = si.uniform(313, 0, (128, 1, 1, 1024), 0, 1)
    f = si.normal(313, 1, (1, 1, 1024, 1000), 0, float(np.sqrt(2.0 / 1024)))
    b = si.normal(313, 2, (1000,), 0, 0.5)
    for act in ("none", "relu6"):
        got = host(ctx.conv2d(dev(x), dev(f), bias=dev(b), act=act))
        assert rel_fro(got, oracle.conv2d(x, f, bias=b, act=act)) <= TF32_TOL
    ctx.check_device_status()


@pytest.mark.parametrize("ta,tb", [(False, True), (True, False), (True, True)])
def test_matmul_tf32_transposes(ctx, oracle, ta, tb):
    M, K, N = 260, 96, 132
    a = si.uniform(303, 0, (K, M) if ta else (M, K), -1, 1)
    b = si.uniform(303, 1, (N, K) if tb else (K, N), -1, 1)
    got = host(ctx.matmul(dev(a), dev(b), ta, tb))
    ctx.check_device_status()
    assert rel_fro(got, oracle.matmul(a, b, ta, tb)) <= TF32_TOL
    ai = si.small_integers(304, 0, a.shape, -8, 8)
    bi = si.small_integers(304, 1, b.shape, -8, 8)
    assert same_bits(host(ctx.matmul(dev(ai), dev(bi), ta, tb)), oracle.matmul(ai, bi, ta, tb))


def test_matmul_unaligned_shapes_take_the_cuda_core_path(ctx, oracle):
    a = si.uniform(305, 0, (70, 27), -1, 1)   # K % 4 != 0
    b = si.uniform(305, 1, (27, 33), -1, 1)   # N % 4 != 0
    got = host(ctx.matmul(dev(a), dev(b)))
    assert rel_fro(got, oracle.matmul(a, b)) <= 1e-5


@pytest.mark.parametrize("act", ["none", "relu", "relu6"])
@pytest.mark.parametrize("shape", [(1, 112, 112, 32, 64), (2, 14, 14, 512, 512), (1, 7, 7, 1024, 1024),
                                   (3, 9, 5, 8, 16), (1, 28, 28, 128, 256)])
def test_pointwise_conv_tf32_fused_epilogue(ctx, oracle, shape, act):
    N, H, W, Cin, Cout = shape
    x = si.uniform(306, 0, (N, H, W, Cin), 0, 6)
    f = si.normal(306, 1, (1, 1, Cin, Cout), 0, float(np.sqrt(2.0 / Cin)))
    b = si.normal(306, 2, (Cout,), 0, 0.5)
    got = host(ctx.conv2d(dev(x), dev(f), bias=dev(b), act=act))
    ctx.check_device_status()
    want = oracle.conv2d(x, f, bias=b, act=act)
    assert got.shape == want.shape
    assert rel_fro(got, want) <= TF32_TOL
    if act == "relu6":
        assert got.min() >= 0 and got.max() <= 6
    xi = si.small_integers(307, 0, x.shape, -8, 8)
    fi = si.small_integers(307, 1, f.shape, -8, 8)
    bi = si.small_integers(307, 2, b.shape, -8, 8)
    assert same_bits(host(ctx.conv2d(dev(xi), dev(fi), bias=dev(bi), act=act)),
                     oracle.conv2d(xi, fi, bias=bi, act=act))


IGEMM_CASES = [
    # N, H, W, Cin, fh, fw, Cout, strides, pad, dilations: conv2d as an implicit GEMM on the tensor cores
    (1, 224, 224, 3, 3, 3, 32, (2, 2), "same", (1, 1)),   # the stem of the 224 models (K = 27, scalar gather)
    (2, 33, 29, 3, 3, 3, 8, (2, 2), "same", (1, 1)),
    (1, 17, 19, 5, 3, 3, 40, (1, 1), "same", (1, 1)),     # K = 45: two k-blocks, the second mostly padding
    (1, 20, 20, 16, 3, 3, 36, (2, 2), "valid", (1, 1)),   # Cin % 4 == 0: float4 gather, K = 144
    (1, 15, 15, 4, 3, 3, 8, (1, 1), "same", (2, 2)),      # dilation
    (1, 12, 14, 7, 5, 3, 12, (3, 2), "same", (1, 1)),     # 5x3 window, unequal strides
    (3, 9, 9, 30, 1, 1, 52, (2, 2), "same", (1, 1)),      # strided 1x1
    (1, 6, 6, 72, 3, 3, 4, (1, 1), "valid", (1, 1)),      # K = 648: the stage ring wraps
    (5, 40, 40, 8, 3, 3, 260, (1, 1), "same", (1, 1)),    # Cout just above one 256-wide tile, many pixel tiles
    (3, 37, 50, 3, 3, 3, 16, (2, 2), "valid", (1, 1)),    # patch kernel: ragged tiles, 'valid'
    (2, 30, 30, 3, 3, 3, 8, (1, 1), "valid", (1, 1)),     # patch kernel: stride 1
    (1, 19, 23, 4, 2, 2, 12, (1, 1), "same", (1, 1)),     # patch kernel: 2x2 window, Cin 4, pad after only
    (2, 21, 21, 1, 5, 5, 32, (2, 2), "valid", (1, 1)),    # patch kernel: one input channel, 5x5 (K = 25)
]


@pytest.mark.parametrize("case", IGEMM_CASES)
def test_conv2d_implicit_gemm_tf32(ctx, oracle, case):
    N, H, W, Cin, fh, fw, Cout, strides, pad, dil = case
    x = si.uniform(309, 0, (N, H, W, Cin), -1, 1)
    f = si.normal(309, 1, (fh, fw, Cin, Cout), 0, float(np.sqrt(2.0 / (fh * fw * Cin))))
    b = si.normal(309, 2, (Cout,), 0, 0.5)
    got = host(ctx.conv2d(dev(x), dev(f), strides, pad, dil, dev(b), "relu6"))
    ctx.check_device_status()
    want = oracle.conv2d(x, f, strides, pad, dil, b, "relu6")
    assert got.shape == want.shape
    assert rel_fro(got, want) <= TF32_TOL
    matched = oracle.conv2d(x, f, strides, pad, dil, b, "relu6", operand="tf32_rz")
    assert rel_fro(got, matched) <= MATCHED_TOL
    xi = si.small_integers(310, 0, x.shape, -4, 4)
    fi = si.small_integers(310, 1, f.shape, -4, 4)
    assert same_bits(host(ctx.conv2d(dev(xi), dev(fi), strides, pad, dil)), oracle.conv2d(xi, fi, strides, pad, dil))
    ctx.check_device_status()


def test_separable_block_config2(ctx, oracle):
    x, layers = si.config_separable_block()
    dw, pw = layers
    y1 = ctx.depthwise_conv2d(dev(x), dev(dw.filter), dw.strides, dw.pad, dw.dilations, dev(dw.bias), dw.act)
    y2 = host(ctx.conv2d(y1, dev(pw.filter), pw.strides, pw.pad, pw.dilations, dev(pw.bias), pw.act))
    ctx.check_device_status()
    w1 = oracle.depthwise_conv2d(x, dw.filter, dw.strides, dw.pad, dw.dilations, dw.bias, dw.act)
    w2 = oracle.conv2d(w1, pw.filter, pw.strides, pw.pad, pw.dilations, pw.bias, pw.act)
    assert rel_fro(host(y1), w1) <= 1e-6
    assert rel_fro(y2, w2) <= TF32_TOL


def test_tf32_result_is_deterministic(ctx):
    a = dev(si.uniform(308, 0, (5000, 256), -1, 1))
    b = dev(si.uniform(308, 1, (256, 512), -1, 1))
    first = host(ctx.matmul(a, b))
    for _ in range(3):
        assert same_bits(host(ctx.matmul(a, b)), first)
    ctx.check_device_status()


FUSED_BLOCK_CASES = [
    # N, H, W, C, Cout, pad: depthwise 3x3 stride 1 + pointwise, run by the executor as one fused kernel
    (1, 112, 112, 32, 64, "same"),     # config 2
    (2, 20, 37, 32, 8, "same"),        # ragged tiles in both directions, Cout below one chunk
    (3, 14, 14, 128, 128, "same"),     # four k-blocks, image smaller than the 16-wide tile
    (2, 7, 7, 256, 256, "same"),       # eight k-blocks, 256-wide accumulator (two stages)
    (1, 30, 33, 64, 100, "valid"),     # 'valid': no padding offset, Cout not a multiple of 32
    (5, 56, 56, 96, 36, "same"),       # more tiles than SMs, three k-blocks
    (2, 14, 14, 512, 512, "same"),     # two 256-wide accumulator halves sharing each A tile, 16 k-blocks
    (1, 9, 20, 64, 320, "same"),       # second half partly empty (320 = 256 + 64)
]


@pytest.mark.parametrize("case", FUSED_BLOCK_CASES)
def test_fused_depthwise_pointwise_block(ctx, oracle, monkeypatch, case):
    from seeded_inputs.workloads import Layer

    N, H, W, C, Cout, pad = case
    x = si.uniform(311, 0, (N, H, W, C), 0, 6)
    layers = [Layer("depthwise_conv2d", (3, 3), (1, 1), (1, 1), pad, "relu6", 1, "dw"),
              Layer("conv2d", (1, 1), (1, 1), (1, 1), "same", "relu6", Cout, "pw")]
    si.make_model_weights(layers, C, 311)
    model = ctx.model(layers, x.shape)
    model.set_fusion("always")                  # small cases: 'auto' would keep the layers apart
    assert model.launches_per_run == 1          # the two layers run as one kernel
    got = host(model.run(dev(x)))
    ctx.check_device_status()
    want = oracle.run_model(layers, x)
    assert got.shape == want.shape
    assert rel_fro(got, want) <= TF32_TOL
    monkeypatch.setenv("TFJSB_NO_SPLIT_K", "1")  # (a pointwise GEMM cut along K adds in another order)
    model.set_keep_all(True)                    # debug mode: the two stand-alone kernels
    unfused = host(model.run(dev(x)))
    assert model.launches_per_run == 2
    assert same_bits(got, unfused)              # same arithmetic in the same order
    monkeypatch.delenv("TFJSB_NO_SPLIT_K")
    model.close()
    # small integers: exact in TF32 and fp32, so bit-identical to the oracle
    xi = si.small_integers(312, 0, x.shape, 0, 3)
    for layer in layers:
        layer.filter = si.small_integers(312, 1, layer.filter.shape, -2, 2)
        layer.bias = si.small_integers(312, 2, layer.bias.shape, -2, 2)
        layer.act = "none"
    model = ctx.model(layers, x.shape)
    model.set_fusion("always")
    assert same_bits(host(model.run(dev(xi))), oracle.run_model(layers, xi))
    ctx.check_device_status()
    model.close()

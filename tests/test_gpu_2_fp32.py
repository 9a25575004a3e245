"""GPU parity of the CUDA-core fp32 kernels: matMul (all transposes), conv2d, depthwiseConv2d.

Tolerances: these kernels accumulate in fp32 with FMA, in an order that differs from the
oracle's double accumulation, so they are compared by relative Frobenius error <= 1e-5 (the
worst-case bound for K <= 1152 products is K * 2^-24 ~ 7e-5 per element; the norm-wise error
behaves like sqrt(K) * 2^-24 ~ 2e-6).  On small-integer inputs every partial sum is exact in
fp32, so the result must be bit-identical to exact integer arithmetic.
"""
import itertools

import numpy as np
import pytest

import seeded_inputs as si
from helpers import dev, host, rel_fro, same_bits

pytestmark = pytest.mark.gpu

FP32_TOL = 1e-5


@pytest.fixture()
def fp32(ctx):
    ctx.set_math("fp32")
    yield ctx
    ctx.set_math("tf32")


@pytest.mark.parametrize("ta,tb", list(itertools.product([False, True], repeat=2)))
@pytest.mark.parametrize("mkn", [(7, 13, 5), (128, 128, 128), (300, 100, 72), (1, 1024, 1000), (513, 31, 257)])
def test_matmul_fp32_all_transposes(fp32, oracle, ta, tb, mkn):
    M, K, N = mkn
    a = si.uniform(201, 0, (K, M) if ta else (M, K), -1, 1)
    b = si.uniform(201, 1, (N, K) if tb else (K, N), -1, 1)
    got = host(fp32.matmul(dev(a), dev(b), ta, tb))
    want = oracle.matmul(a, b, ta, tb)
    assert got.shape == want.shape
    assert rel_fro(got, want) <= FP32_TOL
    ai = si.small_integers(202, 0, a.shape, -8, 8)
    bi = si.small_integers(202, 1, b.shape, -8, 8)
    assert same_bits(host(fp32.matmul(dev(ai), dev(bi), ta, tb)), oracle.matmul(ai, bi, ta, tb))


def test_matmul_fp32_config1(fp32, oracle):
    a, b = si.config_matmul(512)
    got = host(fp32.matmul(dev(a), dev(b)))
    assert rel_fro(got, oracle.matmul(a, b)) <= FP32_TOL


CONV_CASES = [
    # N, H, W, Cin, fh, fw, Cout, strides, pad, dilations
    (1, 224, 224, 3, 3, 3, 32, (2, 2), "same", (1, 1)),  # the stem of the 224 models
    (2, 33, 29, 3, 3, 3, 8, (2, 2), "same", (1, 1)),
    (1, 17, 19, 5, 3, 3, 40, (1, 1), "same", (1, 1)),
    (1, 20, 20, 16, 3, 3, 33, (2, 2), "valid", (1, 1)),
    (1, 15, 15, 4, 3, 3, 6, (1, 1), "same", (2, 2)),
    (1, 12, 14, 7, 5, 3, 9, (3, 2), "same", (1, 1)),
    (3, 9, 9, 30, 1, 1, 50, (2, 2), "same", (1, 1)),     # strided 1x1 is not a GEMM view
    (1, 6, 6, 70, 3, 3, 4, (1, 1), "valid", (1, 1)),     # more filter rows than one shared-memory slice
]


@pytest.mark.parametrize("case", CONV_CASES)
def test_conv2d_fp32_parity(fp32, oracle, case):
    N, H, W, Cin, fh, fw, Cout, strides, pad, dil = case
    x = si.uniform(203, 0, (N, H, W, Cin), -1, 1)
    f = si.normal(203, 1, (fh, fw, Cin, Cout), 0, float(np.sqrt(2.0 / (fh * fw * Cin))))
    b = si.normal(203, 2, (Cout,), 0, 0.5)
    got = host(fp32.conv2d(dev(x), dev(f), strides, pad, dil, dev(b), "relu6"))
    want = oracle.conv2d(x, f, strides, pad, dil, b, "relu6")
    assert got.shape == want.shape
    assert rel_fro(got, want) <= FP32_TOL
    xi = si.small_integers(204, 0, x.shape, -4, 4)
    fi = si.small_integers(204, 1, f.shape, -4, 4)
    assert same_bits(host(fp32.conv2d(dev(xi), dev(fi), strides, pad, dil)), oracle.conv2d(xi, fi, strides, pad, dil))


def test_pointwise_conv_fp32_is_matmul_on_reshaped_input(fp32, oracle):
    x = si.uniform(205, 0, (2, 14, 14, 48), 0, 6)
    f = si.normal(205, 1, (1, 1, 48, 96), 0, 0.2)
    b = si.normal(205, 2, (96,), 0, 0.01)
    y = host(fp32.conv2d(dev(x), dev(f), bias=dev(b), act="relu6"))
    assert rel_fro(y, oracle.conv2d(x, f, bias=b, act="relu6")) <= FP32_TOL
    c = host(fp32.matmul(dev(x.reshape(-1, 48)), dev(f.reshape(48, 96))))
    raw = host(fp32.conv2d(dev(x), dev(f)))
    assert same_bits(raw.reshape(-1, 96), c)


DW_CASES = [
    # N, H, W, C, fh, fw, mult, strides, pad, dilations
    (1, 112, 112, 32, 3, 3, 1, (1, 1), "same", (1, 1)),   # config 2, step 1
    (2, 56, 56, 64, 3, 3, 1, (2, 2), "same", (1, 1)),
    (1, 14, 14, 512, 3, 3, 1, (1, 1), "same", (1, 1)),
    (1, 7, 7, 1024, 3, 3, 1, (1, 1), "same", (1, 1)),
    (2, 20, 37, 48, 3, 3, 1, (1, 1), "same", (1, 1)),     # pipelined kernel: ragged tiles, partial channel block
    (1, 14, 14, 64, 3, 3, 1, (1, 1), "same", (1, 1)),     # pipelined kernel: whole 14-row image in one tile
    (3, 7, 7, 96, 3, 3, 1, (1, 1), "same", (1, 1)),       # pipelined kernel: narrow-image instance
    (2, 29, 31, 32, 3, 3, 1, (2, 2), "same", (1, 1)),     # pipelined kernel: stride 2, odd sizes
    (1, 14, 14, 160, 3, 3, 1, (2, 2), "same", (1, 1)),    # pipelined kernel: stride 2, narrow output
    (1, 9, 40, 32, 3, 3, 1, (1, 1), "valid", (1, 1)),     # pipelined kernel: 'valid' (no padding offset)
    # the 64-channel instances of the pipelined kernel (channel count a multiple of 64)
    (2, 21, 37, 128, 3, 3, 1, (1, 1), "same", (1, 1)),    # large stride-1 images: ragged tiles both ways, two channel blocks
    (3, 13, 20, 128, 3, 3, 1, (1, 1), "same", (1, 1)),    # 9..14 rows: two tiles down, two across, ragged
    (3, 7, 7, 192, 3, 3, 1, (1, 1), "same", (1, 1)),      # whole 7 x 7 image per tile, three channel blocks
    (2, 11, 6, 64, 3, 3, 1, (1, 1), "same", (1, 1)),      # narrow image taller than one tile
    (2, 29, 47, 64, 3, 3, 1, (2, 2), "same", (1, 1)),     # stride 2, 8-wide tiles (24 outputs across), odd sizes
    (1, 33, 50, 128, 3, 3, 1, (2, 2), "valid", (1, 1)),   # stride 2, 'valid', 8-wide tiles
    (5, 33, 18, 36, 3, 3, 1, (2, 2), "valid", (1, 1)),
    (3, 13, 11, 24, 3, 3, 1, (1, 1), "same", (1, 1)),     # channel quads not a power of two, ragged rows
    (2, 15, 9, 8, 3, 3, 1, (2, 2), "same", (1, 1)),       # odd sizes at stride 2 (symmetric padding)
    (1, 10, 10, 16, 3, 3, 1, (1, 1), "valid", (1, 1)),
    (1, 9, 9, 6, 3, 3, 1, (1, 1), "same", (1, 1)),        # C % 4 != 0 -> scalar kernel
    (1, 9, 8, 4, 3, 3, 2, (1, 1), "same", (1, 1)),        # channel multiplier
    (1, 11, 11, 8, 3, 3, 1, (1, 1), "same", (2, 2)),      # dilation
    (1, 8, 8, 8, 5, 5, 1, (1, 1), "same", (1, 1)),        # 5x5 window
    (1, 9, 9, 8, 3, 3, 1, (2, 1), "same", (1, 1)),        # unequal strides
]


@pytest.mark.parametrize("case", DW_CASES)
def test_depthwise_parity(ctx, oracle, case):
    N, H, W, C, fh, fw, mult, strides, pad, dil = case
    x = si.uniform(206, 0, (N, H, W, C), 0, 6)
    f = si.normal(206, 1, (fh, fw, C, mult), 0, float(np.sqrt(2.0 / (fh * fw))))
    b = si.normal(206, 2, (C * mult,), 0, 0.01)
    got = host(ctx.depthwise_conv2d(dev(x), dev(f), strides, pad, dil, dev(b), "relu6"))
    want = oracle.depthwise_conv2d(x, f, strides, pad, dil, b, "relu6")
    assert got.shape == want.shape
    assert rel_fro(got, want) <= 1e-6
    assert np.max(np.abs(got - want)) <= 1e-5
    xi = si.small_integers(207, 0, x.shape, -8, 8)
    fi = si.small_integers(207, 1, f.shape, -8, 8)
    assert same_bits(host(ctx.depthwise_conv2d(dev(xi), dev(fi), strides, pad, dil)),
                     oracle.depthwise_conv2d(xi, fi, strides, pad, dil))


def test_depthwise_shifted_delta_taps_on_gpu(ctx):
    """The padding offsets once more, on the device: a single-tap filter must pick
    x[oy*s - pt + ky, ox*s - pl + kx]; even size at stride 2 pads nothing before."""
    size, C = 8, 4
    x = si.uniform(208, 0, (1, size, size, C), 1, 2)
    for stride, before in [(1, 1), (2, 0)]:
        out = -(-size // stride)
        for ky in range(3):
            for kx in range(3):
                f = np.zeros((3, 3, C, 1), np.float32)
                f[ky, kx, :, 0] = 1.0
                y = host(ctx.depthwise_conv2d(dev(x), dev(f), (stride, stride), "same"))
                for oy in range(out):
                    for ox in range(out):
                        iy, ix = oy * stride - before + ky, ox * stride - before + kx
                        want = x[0, iy, ix] if (0 <= iy < size and 0 <= ix < size) else np.zeros(C, np.float32)
                        assert np.array_equal(y[0, oy, ox], want)

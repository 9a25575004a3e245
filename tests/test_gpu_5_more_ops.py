"""GPU parity of the ops beyond the MobileNet path: maxPool, elementwise add / sub / mul, rank-3 matMul,
dilated depthwise convolution and the atrous (output stride 16 / 8) MobileNet variants built from it.

Tolerances.  maxPool selects an input value and add / sub / mul are one correctly rounded fp32
operation per element, so both must match the oracle bit for bit (NaNs in the same places).  A
rank-3 matMul is one rank-2 product per leading index through the same kernels as tfjsb_matmul:
relative Frobenius error <= 5e-3 against the exact oracle on the tensor cores, <= 1e-5 in fp32 mode,
bit-identical on small integers.
"""
import numpy as np
import pytest

import seeded_inputs as si
from helpers import dev, host, rel_fro, same_bits

pytestmark = pytest.mark.gpu

POOL_CASES = [
    # N, H, W, C, window, strides, pad
    (2, 112, 112, 32, (3, 3), (2, 2), "same"),    # even size, stride 2: padding after only
    (1, 7, 7, 1024, (7, 7), (1, 1), "valid"),     # global
    (3, 13, 17, 5, (2, 3), (2, 1), "valid"),      # unequal window and strides, odd channel count
    (1, 9, 9, 8, (3, 3), (1, 1), "same"),
    (1, 1, 1, 4, (3, 3), (1, 1), "same"),         # window mostly outside the image
    (2, 33, 20, 64, (5, 5), (3, 3), "same"),
]


def same_bits_or_both_nan(a, b):
    a, b = np.ascontiguousarray(a, np.float32), np.ascontiguousarray(b, np.float32)
    nan = np.isnan(a)
    return a.shape == b.shape and np.array_equal(nan, np.isnan(b)) and np.array_equal(a[~nan].view(np.uint32), b[~nan].view(np.uint32))


@pytest.mark.parametrize("case", POOL_CASES)
def test_max_pool_bit_exact(ctx, oracle, case):
    N, H, W, C, k, s, pad = case
    x = si.normal(501, 0, (N, H, W, C), -1, 2)   # mostly negative: zero padding would win wrongly
    got = host(ctx.max_pool(dev(x), k, s, pad))
    want = oracle.max_pool(x, k, s, pad)
    assert got.shape == want.shape and same_bits(got, want)
    x.reshape(-1)[::97] = np.nan                  # NaNs reach exactly the windows that contain them
    assert same_bits_or_both_nan(host(ctx.max_pool(dev(x), k, s, pad)), oracle.max_pool(x, k, s, pad))


def test_max_pool_rejects_bad_arguments(ctx, tfjsb):
    import torch

    x = torch.zeros(1, 4, 4, 4, device="cuda")
    with pytest.raises(tfjsb.TfjsbError) as err:
        ctx.max_pool(x, (5, 5), (1, 1), "valid")                       # window larger than the image
    assert err.value.status_name == "SHAPE"
    with pytest.raises(tfjsb.TfjsbError):
        ctx.max_pool(x, (2, 2), (2, 2), "valid", out=torch.zeros(1, 3, 3, 4, device="cuda"))  # wrong out shape


BINARY_SHAPES = [(4, 56, 56, 64), (3, 5, 7, 6), (1000,), (2, 3, 5), (1, 1, 1, 4), (128, 1000), (7, 13, 3)]


@pytest.mark.parametrize("op", ["add", "sub", "mul"])
@pytest.mark.parametrize("shape", BINARY_SHAPES)
def test_binary_ops_bit_exact(ctx, oracle, op, shape):
    a = si.normal(502, 0, shape, 0, 10)
    b = si.normal(502, 1, shape, 0, 10)
    v = si.normal(502, 2, (shape[-1],), 0, 10)
    a.reshape(-1)[::53] = np.nan
    b.reshape(-1)[::71] = np.inf
    assert same_bits_or_both_nan(host(ctx.binary(op, dev(a), dev(b))), oracle.binary(op, a, b))
    assert same_bits_or_both_nan(host(ctx.binary(op, dev(a), dev(v))), oracle.binary(op, a, v))


def test_binary_rejects_bad_arguments(ctx, tfjsb):
    import torch

    a = torch.zeros(2, 8, device="cuda")
    with pytest.raises(tfjsb.TfjsbError) as err:
        ctx.binary("add", a, torch.zeros(2, 4, device="cuda"))
    assert err.value.status_name == "SHAPE"
    with pytest.raises(tfjsb.TfjsbError) as err:
        ctx.binary("add", a, torch.zeros(8, device="cuda"), out=a)     # out aliases an input
    assert err.value.status_name == "INVALID_ARG"
    assert ctx.binary("mul", torch.zeros(0, 8, device="cuda"), torch.zeros(8, device="cuda")).shape == (0, 8)


BATCH_MATMUL_CASES = [
    # B, M, K, N, transpose_a, transpose_b
    (4, 128, 64, 64, False, False),
    (3, 300, 100, 72, False, True),
    (2, 49, 1024, 256, True, False),     # few tiles, long K: each product is cut along K
    (5, 9, 13, 5, False, False),         # slices not 16-byte aligned: CUDA-core kernel
    (1, 512, 512, 512, True, True),
]


@pytest.mark.parametrize("case", BATCH_MATMUL_CASES)
def test_batch_matmul_parity(ctx, oracle, case):
    B, M, K, N, ta, tb = case
    a = si.uniform(503, 0, (B, K, M) if ta else (B, M, K), -1, 1)
    b = si.uniform(503, 1, (B, N, K) if tb else (B, K, N), -1, 1)
    got = host(ctx.batch_matmul(dev(a), dev(b), ta, tb))
    ctx.check_device_status()
    want = oracle.batch_matmul(a, b, ta, tb)
    assert got.shape == (B, M, N)
    for i in range(B):  # per product, so that one bad slice cannot hide among good ones
        assert rel_fro(got[i], want[i]) <= 5e-3
    ai = si.small_integers(504, 0, a.shape, -8, 8)
    bi = si.small_integers(504, 1, b.shape, -8, 8)
    assert same_bits(host(ctx.batch_matmul(dev(ai), dev(bi), ta, tb)), oracle.batch_matmul(ai, bi, ta, tb))
    ctx.set_math("fp32")
    try:
        got32 = host(ctx.batch_matmul(dev(a), dev(b), ta, tb))
    finally:
        ctx.set_math("tf32")
    assert rel_fro(got32, want) <= 1e-5


def test_batch_matmul_rejects_bad_arguments(ctx, tfjsb):
    import torch

    with pytest.raises(tfjsb.TfjsbError) as err:
        ctx.batch_matmul(torch.zeros(2, 4, 8, device="cuda"), torch.zeros(3, 8, 4, device="cuda"))
    assert err.value.status_name == "SHAPE"
    with pytest.raises(tfjsb.TfjsbError) as err:
        ctx.batch_matmul(torch.zeros(2, 4, 8, device="cuda"), torch.zeros(2, 7, 4, device="cuda"))
    assert err.value.status_name == "SHAPE"


DILATED_DW_CASES = [
    # N, H, W, C, dilation: 3x3 depthwise, stride 1, 'same' (the atrous layers of output-stride-16 / -8 models)
    (2, 14, 14, 512, 2),
    (1, 28, 28, 256, 4),
    (3, 9, 11, 32, 2),     # image barely larger than the dilated window
    (1, 5, 5, 8, 4),       # dilated window larger than the image: most taps fall outside
    (2, 14, 14, 6, 2),     # channel count not a multiple of 4: the general kernel
]


@pytest.mark.parametrize("case", DILATED_DW_CASES)
def test_dilated_depthwise_parity(ctx, oracle, case):
    N, H, W, C, d = case
    x = si.uniform(505, 0, (N, H, W, C), 0, 6)
    f = si.normal(505, 1, (3, 3, C, 1), 0, 0.47)
    b = si.normal(505, 2, (C,), 0, 0.5)
    got = host(ctx.depthwise_conv2d(dev(x), dev(f), (1, 1), "same", (d, d), dev(b), "relu6"))
    want = oracle.depthwise_conv2d(x, f, (1, 1), "same", (d, d), b, "relu6")
    assert got.shape == want.shape and rel_fro(got, want) <= 1e-6
    xi = si.small_integers(506, 0, x.shape, -8, 8)
    fi = si.small_integers(506, 1, f.shape, -8, 8)
    assert same_bits(host(ctx.depthwise_conv2d(dev(xi), dev(fi), (1, 1), "same", (d, d))),
                     oracle.depthwise_conv2d(xi, fi, (1, 1), "same", (d, d)))


@pytest.mark.parametrize("output_stride", [16, 8])
def test_atrous_mobilenet_every_layer(ctx, oracle, output_stride):
    """alpha 0.25, 96x96 input, batch 2, output stride 16 / 8: every layer's output against the oracle."""
    x, layers = si.config_mobilenet_atrous(0.25, 96, 2, output_stride, seed=4243, classes=100)
    dilations = sorted({l.dilations[0] for l in layers if l.kind == "depthwise_conv2d"})
    assert dilations == ([1, 2] if output_stride == 16 else [1, 2, 4])
    want = oracle.run_model(layers, x, keep_all=True)
    assert want[-4].shape[1] == 96 // output_stride          # spatial size of the last block's output
    model = ctx.model(layers, x.shape)
    model.set_keep_all(True)
    probs = host(model.run(dev(x)))
    ctx.check_device_status()
    for i, layer in enumerate(layers):
        got = host(model.layer_output(i)) if i < len(layers) - 1 else probs
        assert got.shape == want[i].shape, layer.name
        assert rel_fro(got, want[i]) <= 2e-2, f"layer {i} ({layer.name}) diverges: {rel_fro(got, want[i]):.3e}"
    span = float(want[-2].max() - want[-2].min())
    assert np.max(np.abs(host(model.layer_output(len(layers) - 2)) - want[-2])) <= 1e-2 * span
    model.set_keep_all(False)
    assert same_bits(host(model.run(dev(x))), probs)          # the ping-pong run gives the same bits
    model.close()

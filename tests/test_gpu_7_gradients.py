"""GPU parity of the gradient ops (conv2d / depthwiseConv2d / epilogue gradients, Sec. 3.5) against the oracle.

Bars: bit-identical on small integers (every product and partial sum exact in fp32 and in TF32, whatever the
order); fp32 CUDA-core kernels rel. Frobenius <= 1e-5; the pointwise gradients on the tensor cores <= 5e-3
against the exact oracle and <= 2e-5 against the oracle with truncated TF32 operands; the activation
gradient bit-exact.
"""
import numpy as np
import pytest

import seeded_inputs as si
from helpers import dev, host, rel_fro, same_bits

pytestmark = pytest.mark.gpu

CONV_CASES = [
    # N, H, W, Cin, Cout, fh, fw, stride, dilation, pad
    (2, 9, 11, 5, 7, 3, 3, 1, 1, "same"),
    (3, 14, 14, 8, 12, 3, 3, 2, 1, "same"),     # even size, stride 2: odd padding element after
    (2, 13, 10, 3, 32, 3, 3, 2, 1, "valid"),
    (1, 12, 12, 6, 4, 3, 3, 1, 2, "same"),      # dilated
    (2, 8, 9, 40, 36, 5, 3, 1, 1, "same"),      # more than one 32-channel tile, ragged
    (4, 31, 29, 16, 24, 3, 3, 1, 1, "same"),    # thousands of pixels: several slices in the filter gradient
    (2, 7, 5, 6, 10, 1, 1, 1, 1, "same"),       # pointwise with channel counts the tensor-core path cannot take
    (2, 9, 9, 8, 8, 1, 1, 2, 1, "same"),        # 1x1 with stride 2: not a plain matrix product
]


def geometry(oracle, H, W, fh, fw, s, d, pad):
    return oracle.window_geometry(H, fh, s, d, pad)[0], oracle.window_geometry(W, fw, s, d, pad)[0]


@pytest.mark.parametrize("case", CONV_CASES)
def test_conv2d_gradients(ctx, oracle, case):
    N, H, W, Cin, Cout, fh, fw, s, d, pad = case
    Ho, Wo = geometry(oracle, H, W, fh, fw, s, d, pad)
    ctx.set_math("fp32")
    try:
        # small integers: bit-identical
        x = si.small_integers(81, 0, (N, H, W, Cin), -3, 3)
        f = si.small_integers(81, 1, (fh, fw, Cin, Cout), -3, 3)
        g = si.small_integers(81, 2, (N, Ho, Wo, Cout), -3, 3)
        dx = host(ctx.conv2d_backprop_input(x.shape, dev(f), dev(g), (s, s), pad, (d, d)))
        df = host(ctx.conv2d_backprop_filter(dev(x), f.shape, dev(g), (s, s), pad, (d, d)))
        ctx.check_device_status()
        assert same_bits(dx, oracle.conv2d_backprop_input(x.shape, f, g, (s, s), pad, (d, d)))
        assert same_bits(df, oracle.conv2d_backprop_filter(x, f.shape, g, (s, s), pad, (d, d)))
        # random values
        x = si.uniform(82, 0, (N, H, W, Cin), -1, 1)
        f = si.normal(82, 1, (fh, fw, Cin, Cout), 0, 0.3)
        g = si.normal(82, 2, (N, Ho, Wo, Cout), 0, 1)
        dx = host(ctx.conv2d_backprop_input(x.shape, dev(f), dev(g), (s, s), pad, (d, d)))
        df = host(ctx.conv2d_backprop_filter(dev(x), f.shape, dev(g), (s, s), pad, (d, d)))
        ctx.check_device_status()
        assert rel_fro(dx, oracle.conv2d_backprop_input(x.shape, f, g, (s, s), pad, (d, d))) <= 1e-5
        assert rel_fro(df, oracle.conv2d_backprop_filter(x, f.shape, g, (s, s), pad, (d, d))) <= 1e-5
    finally:
        ctx.set_math("tf32")


@pytest.mark.parametrize("case", CONV_CASES[:6])
@pytest.mark.parametrize("mult", [1, 2])
def test_depthwise_gradients(ctx, oracle, case, mult):
    N, H, W, C, _, fh, fw, s, d, pad = case
    Ho, Wo = geometry(oracle, H, W, fh, fw, s, d, pad)
    x = si.small_integers(83, 0, (N, H, W, C), -3, 3)
    f = si.small_integers(83, 1, (fh, fw, C, mult), -3, 3)
    g = si.small_integers(83, 2, (N, Ho, Wo, C * mult), -3, 3)
    dx = host(ctx.depthwise_conv2d_backprop_input(x.shape, dev(f), dev(g), (s, s), pad, (d, d)))
    df = host(ctx.depthwise_conv2d_backprop_filter(dev(x), f.shape, dev(g), (s, s), pad, (d, d)))
    ctx.check_device_status()
    assert same_bits(dx, oracle.depthwise_conv2d_backprop_input(x.shape, f, g, (s, s), pad, (d, d)))
    assert same_bits(df, oracle.depthwise_conv2d_backprop_filter(x, f.shape, g, (s, s), pad, (d, d)))
    x = si.uniform(84, 0, (N, H, W, C), -1, 1)
    f = si.normal(84, 1, (fh, fw, C, mult), 0, 0.5)
    g = si.normal(84, 2, (N, Ho, Wo, C * mult), 0, 1)
    dx = host(ctx.depthwise_conv2d_backprop_input(x.shape, dev(f), dev(g), (s, s), pad, (d, d)))
    df = host(ctx.depthwise_conv2d_backprop_filter(dev(x), f.shape, dev(g), (s, s), pad, (d, d)))
    ctx.check_device_status()
    assert rel_fro(dx, oracle.depthwise_conv2d_backprop_input(x.shape, f, g, (s, s), pad, (d, d))) <= 1e-6
    assert rel_fro(df, oracle.depthwise_conv2d_backprop_filter(x, f.shape, g, (s, s), pad, (d, d))) <= 1e-5


POINTWISE_CASES = [
    # N, H, W, Cin, Cout: gradients of a 1x1 convolution as matrix products on the tensor cores
    (1, 8, 8, 32, 64),        # 64 pixels: a single slice, K = 64
    (2, 28, 28, 128, 256),    # pw4 of the 224 model at batch 2: 1568 pixels
    (8, 56, 56, 64, 128),     # pw2 at batch 8: 25088 pixels cut into slices, batched launch + ordered sum
    (3, 15, 15, 36, 20),      # 675 pixels: not a multiple of 4, so the filter gradient falls back to CUDA cores
    (2, 14, 14, 512, 512),    # pw7-pw11
]


@pytest.mark.parametrize("case", POINTWISE_CASES)
def test_pointwise_gradients_on_the_tensor_cores(ctx, oracle, case):
    N, H, W, Cin, Cout = case
    before = ctx.launch_count
    x = si.small_integers(85, 0, (N, H, W, Cin), -2, 2)
    f = si.small_integers(85, 1, (1, 1, Cin, Cout), -2, 2)
    g = si.small_integers(85, 2, (N, H, W, Cout), -2, 2)
    dx = host(ctx.conv2d_backprop_input(x.shape, dev(f), dev(g)))
    df = host(ctx.conv2d_backprop_filter(dev(x), f.shape, dev(g)))
    ctx.check_device_status()
    assert ctx.launch_count > before
    # |sums| <= 4 * max(Cout, N*H*W) < 2^24: exact whatever the order and the multiplier
    assert same_bits(dx, oracle.conv2d_backprop_input(x.shape, f, g))
    assert same_bits(df, oracle.conv2d_backprop_filter(x, f.shape, g))
    x = si.uniform(86, 0, (N, H, W, Cin), -1, 1)
    f = si.normal(86, 1, (1, 1, Cin, Cout), 0, 0.3)
    g = si.normal(86, 2, (N, H, W, Cout), 0, 1)
    dx = host(ctx.conv2d_backprop_input(x.shape, dev(f), dev(g)))
    df = host(ctx.conv2d_backprop_filter(dev(x), f.shape, dev(g)))
    ctx.check_device_status()
    assert rel_fro(dx, oracle.conv2d_backprop_input(x.shape, f, g)) <= 5e-3
    assert rel_fro(df, oracle.conv2d_backprop_filter(x, f.shape, g)) <= 5e-3
    # against the oracle whose operands are truncated the way the tensor core reads them
    assert rel_fro(dx, oracle.conv2d_backprop_input(x.shape, f, g, operand="tf32_rz")) <= 2e-5
    if (N * H * W) % 4 == 0:
        assert rel_fro(df, oracle.conv2d_backprop_filter(x, f.shape, g, operand="tf32_rz")) <= 2e-5
    else:
        assert rel_fro(df, oracle.conv2d_backprop_filter(x, f.shape, g)) <= 1e-5


def test_epilogue_gradients(ctx, oracle):
    y = np.array([-0.0, 0.0, 1e-30, 0.5, 5.999999, 6.0, 3.0, 0.0], np.float32)
    dy = np.array([1, 2, 3, 4, 5, 6, -7, np.nan], np.float32)
    for act in ("none", "relu", "relu6"):
        assert same_bits(host(ctx.act_backprop(dev(y), dev(dy), act)), oracle.act_backprop(y, dy, act)), act
    z = si.uniform(87, 0, (5, 17, 13, 24), -3, 9)
    g = si.normal(87, 1, z.shape, 0, 1)
    for act in ("relu", "relu6"):
        yv = oracle.bias_act(z, None, act)
        assert same_bits(host(ctx.act_backprop(dev(yv), dev(g), act)), oracle.act_backprop(yv, g, act)), act
    # bias gradient: exact on integers (one slice and many), 1e-6 otherwise
    for shape in [(3, 4, 5, 6), (64, 28, 28, 40), (7, 1000)]:
        dz = si.small_integers(88, 0, shape, -8, 8)
        assert same_bits(host(ctx.bias_backprop(dev(dz))), oracle.bias_backprop(dz)), shape
        dz = si.normal(88, 1, shape, 0, 1)
        want = oracle.bias_backprop(dz)
        assert np.max(np.abs(host(ctx.bias_backprop(dev(dz))) - want)) <= 1e-5 * np.sqrt(dz.size / shape[-1]), shape
    ctx.check_device_status()


def test_gradients_reject_bad_arguments(ctx, tfjsb):
    import torch

    f = torch.zeros(3, 3, 4, 8, device="cuda")
    with pytest.raises(tfjsb.TfjsbError) as e:  # dy does not have the forward output's shape
        ctx.conv2d_backprop_input((1, 8, 8, 4), f, torch.zeros(1, 8, 8, 6, device="cuda"))
    assert e.value.status_name == "SHAPE"
    with pytest.raises(tfjsb.TfjsbError) as e:  # filter channels differ from x's
        ctx.conv2d_backprop_filter(torch.zeros(1, 8, 8, 5, device="cuda"), (3, 3, 4, 8), torch.zeros(1, 8, 8, 8, device="cuda"))
    assert e.value.status_name == "SHAPE"
    with pytest.raises(tfjsb.TfjsbError) as e:
        ctx.depthwise_conv2d_backprop_input((1, 8, 8, 4), torch.zeros(3, 3, 4, 1, device="cuda"),
                                            torch.zeros(1, 4, 4, 4, device="cuda"), (2, 2), "same", (2, 2))
    assert e.value.status_name == "UNSUPPORTED"
    with pytest.raises(tfjsb.TfjsbError) as e:
        ctx.bias_backprop(torch.zeros(4, 6, device="cuda"), out=torch.zeros(5, device="cuda"))
    assert e.value.status_name == "SHAPE"
    with pytest.raises(tfjsb.TfjsbError) as e:
        ctx.act_backprop(torch.zeros(4, 6, device="cuda"), torch.zeros(4, 7, device="cuda"), "relu")
    assert e.value.status_name == "SHAPE"
    # scratch sized up front: a later call finds it large enough and allocates nothing
    ctx.reserve_scratch(8 << 20)
    x = torch.ones(2, 16, 16, 32, device="cuda")
    out = torch.empty(1, 1, 32, 64, device="cuda")
    dy = torch.ones(2, 16, 16, 64, device="cuda")
    ctx.conv2d_backprop_filter(x, (1, 1, 32, 64), dy, out=out)  # first use loads the kernels' code
    torch.cuda.synchronize()
    free0 = torch.cuda.mem_get_info()[0]
    ctx.conv2d_backprop_filter(x, (1, 1, 32, 64), dy, out=out.zero_())
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free0
    assert torch.equal(out, torch.full_like(out, 512.0))

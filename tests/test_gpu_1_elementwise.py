"""GPU parity, bandwidth-bound ops: bias+activation (bit-exact), avgPool, softmax; argument checks."""
import numpy as np
import pytest

import seeded_inputs as si
from helpers import dev, host, rel_fro, same_bits

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("shape", [(1, 112, 112, 32), (3, 7, 5, 20), (2, 9, 13), (1000,), (5, 3, 3, 7), (64, 1000)])
@pytest.mark.parametrize("act", ["none", "relu", "relu6"])
def test_bias_act_bit_exact(ctx, oracle, shape, act):
    x = si.uniform(101, 0, shape, -8, 8)
    b = si.normal(101, 1, (shape[-1],), 0, 1)
    assert same_bits(host(ctx.bias_act(dev(x), dev(b), act)), oracle.bias_act(x, b, act))
    assert same_bits(host(ctx.bias_act(dev(x), None, act)), oracle.bias_act(x, None, act))


def test_bias_act_special_values_bit_exact(ctx, oracle):
    x = np.array([[-1.0, -0.0, 0.0, 0.5, 5.5, 6.0, 7.0, np.nan, np.inf, -np.inf, 1e-40, -1e-40]], np.float32)
    b = np.zeros(12, np.float32)
    for act in ("none", "relu", "relu6"):
        got = host(ctx.bias_act(dev(x), dev(b), act))
        want = oracle.bias_act(x, b, act)
        fin = ~np.isnan(want)
        assert same_bits(got[fin], want[fin])
        assert np.array_equal(np.isnan(got), np.isnan(want))


def test_bias_act_large_spans_many_blocks(ctx, oracle):
    x = si.uniform(102, 0, (4, 112, 112, 64), -8, 8)  # 3.2M elements, ragged vs the grid
    b = si.normal(102, 1, (64,), 0, 1)
    assert same_bits(host(ctx.bias_act(dev(x), dev(b), "relu6")), oracle.bias_act(x, b, "relu6"))


@pytest.mark.parametrize("case", [
    # N, H, W, C, window, strides, pad
    (2, 7, 7, 1024, (7, 7), (1, 1), "valid"),   # the models' global pool
    (1, 4, 4, 256, (4, 4), (1, 1), "valid"),
    (3, 9, 8, 10, (3, 3), (2, 2), "same"),
    (1, 8, 6, 5, (2, 2), (2, 2), "valid"),
    (2, 5, 5, 33, (3, 2), (1, 2), "same"),
    (1, 30, 30, 40, (30, 30), (1, 1), "valid"),  # global pool with a large window
])
def test_avg_pool_parity(ctx, oracle, case):
    N, H, W, C, k, s, pad = case
    x = si.uniform(103, 0, (N, H, W, C), 0, 6)
    got = host(ctx.avg_pool(dev(x), k, s, pad))
    want = oracle.avg_pool(x, k, s, pad)
    assert got.shape == want.shape
    # fp32 running sum of <= 900 values of magnitude <= 6: error well below 900 * 2^-24 * 6
    np.testing.assert_allclose(got, want, rtol=0, atol=2e-5)


@pytest.mark.parametrize("shape", [(1, 1000), (128, 1000), (7, 33), (3, 5, 17), (4097,), (2, 2, 2, 300)])
def test_softmax_parity(ctx, oracle, shape):
    x = si.normal(104, 0, shape, 0, 3)
    got = host(ctx.softmax(dev(x)))
    want = oracle.softmax(x)
    np.testing.assert_allclose(got, want, rtol=2e-5, atol=1e-10)
    assert np.all(np.abs(got.astype(np.float64).sum(-1) - 1) <= 1e-5)
    assert np.array_equal(got.argmax(-1), want.argmax(-1))


def test_softmax_extreme_logits(ctx, oracle):
    x = np.array([[1000.0, 999.0, -1000.0, 0.0], [-50.0, -50.0, -50.0, -50.0]], np.float32)
    got = host(ctx.softmax(dev(x)))
    np.testing.assert_allclose(got, oracle.softmax(x), rtol=2e-6, atol=1e-30)


def test_argument_errors_are_reported_before_any_launch(ctx, tfjsb):
    import torch

    before = ctx.launch_count
    a = torch.zeros(4, 8, device="cuda")
    b = torch.zeros(6, 4, device="cuda")
    with pytest.raises(tfjsb.TfjsbError) as e:
        ctx.matmul(a, b)
    assert e.value.status_name == "SHAPE"
    with pytest.raises(tfjsb.TfjsbError) as e:
        ctx.matmul(a, torch.zeros(8, 4, device="cuda"), out=torch.zeros(5, 4, device="cuda"))
    assert e.value.status_name == "SHAPE"
    x = torch.zeros(1, 8, 8, 4, device="cuda")
    f = torch.zeros(3, 3, 5, 2, device="cuda")
    with pytest.raises(tfjsb.TfjsbError) as e:
        ctx.conv2d(x, f)
    assert e.value.status_name == "SHAPE"
    f = torch.zeros(3, 3, 4, 2, device="cuda")
    with pytest.raises(tfjsb.TfjsbError) as e:
        ctx.conv2d(x, f, strides=(2, 2), dilations=(2, 2), out=torch.zeros(1, 4, 4, 2, device="cuda"))
    assert e.value.status_name == "UNSUPPORTED"
    with pytest.raises(tfjsb.TfjsbError) as e:
        ctx.conv2d(x, f, bias=torch.zeros(3, device="cuda"))
    assert e.value.status_name == "SHAPE"
    with pytest.raises(tfjsb.TfjsbError) as e:
        ctx.conv2d(x, f, strides=(0, 1), out=torch.zeros(1, 8, 8, 2, device="cuda"))
    assert e.value.status_name == "INVALID_ARG"
    with pytest.raises(tfjsb.TfjsbError) as e:
        ctx.bias_act(x, out=x)
    assert e.value.status_name == "INVALID_ARG"
    with pytest.raises(tfjsb.TfjsbError) as e:
        ctx.depthwise_conv2d(torch.zeros(1, 2, 2, 4, device="cuda"), torch.zeros(3, 3, 4, 1, device="cuda"),
                             pad="valid", out=torch.zeros(1, 1, 1, 4, device="cuda"))
    assert e.value.status_name == "SHAPE"
    with pytest.raises(tfjsb.TfjsbError) as e:
        ctx.matmul(torch.zeros(64, device="cuda")[1:13].view(3, 4), torch.zeros(4, 4, device="cuda"))
    assert e.value.status_name == "INVALID_ARG"  # misaligned data pointer
    assert ctx.launch_count == before


def test_empty_tensors_are_a_no_op(ctx):
    import torch

    out = ctx.bias_act(torch.zeros(0, 8, device="cuda"), None, "relu")
    assert out.shape == (0, 8)
    c = ctx.matmul(torch.zeros(0, 8, device="cuda"), torch.zeros(8, 4, device="cuda"))
    assert c.shape == (0, 4)

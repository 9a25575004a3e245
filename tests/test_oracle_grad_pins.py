"""Pins of the oracle's gradient functions (the per-kernel gradients that eager differentiation calls,
Sec. 3.5 of the paper, which names no gradient op and prints no worked example).

What fixes them from outside the oracle:
  * the adjoint identity  <op(x), g> = <x, op^T(g)>  on small integers, where every sum is exact, so both
    sides must be the same integer: any wrong index, stride, padding side or dropped tap breaks it;
  * central differences of the forward oracle: the forward ops are linear in x and in the filter, so on
    integers  L(v + e_i) - L(v - e_i) = 2 dL/dv_i  exactly;
  * torch fp64 autograd of torch's own conv2d on input padded by hand the TensorFlow way;
  * the 1x1 case written as two matrix products; relu / relu6 slopes at the kinks; column sums.
"""
import itertools

import numpy as np
import pytest

import seeded_inputs as si

CASES = [
    # H, W, Cin, Cout, fh, fw, stride, dilation, pad
    (5, 5, 2, 3, 3, 3, 1, 1, "same"),
    (5, 4, 3, 2, 3, 3, 2, 1, "same"),     # even width, stride 2: the odd padding element goes after
    (6, 5, 2, 2, 3, 3, 2, 1, "valid"),
    (7, 7, 1, 2, 3, 3, 1, 2, "same"),     # dilated
    (5, 6, 2, 3, 1, 1, 1, 1, "same"),     # pointwise
    (6, 6, 2, 2, 2, 3, 3, 1, "same"),     # even window, stride larger than the window's overlap
    (6, 5, 3, 1, 5, 3, 1, 1, "valid"),
]


def ints(seed, stream, shape, lo=-3, hi=3):
    return si.small_integers(seed, stream, shape, lo, hi)


def dot(a, b):
    return int(np.sum(a.astype(np.int64) * b.astype(np.int64)))


@pytest.mark.parametrize("case", CASES)
def test_conv2d_gradients_are_the_adjoints_of_the_forward_op(oracle, case):
    H, W, Cin, Cout, fh, fw, s, d, pad = case
    x = ints(71, 0, (2, H, W, Cin))
    f = ints(71, 1, (fh, fw, Cin, Cout))
    y = oracle.conv2d(x, f, (s, s), pad, (d, d))
    g = ints(71, 2, y.shape)
    dx = oracle.conv2d_backprop_input(x.shape, f, g, (s, s), pad, (d, d))
    df = oracle.conv2d_backprop_filter(x, f.shape, g, (s, s), pad, (d, d))
    assert dx.shape == x.shape and df.shape == f.shape
    assert dot(y, g) == dot(x, dx) == dot(f, df)
    # a second, independent x and f against the same gradients' linearity: <conv(x2, f), g> = <x2, dx>
    x2 = ints(71, 3, x.shape)
    f2 = ints(71, 4, f.shape)
    assert dot(oracle.conv2d(x2, f, (s, s), pad, (d, d)), g) == dot(x2, dx)
    assert dot(oracle.conv2d(x, f2, (s, s), pad, (d, d)), g) == dot(f2, df)


@pytest.mark.parametrize("case", CASES)
@pytest.mark.parametrize("mult", [1, 2])
def test_depthwise_gradients_are_the_adjoints_of_the_forward_op(oracle, case, mult):
    H, W, C, _, fh, fw, s, d, pad = case
    x = ints(72, 0, (2, H, W, C))
    f = ints(72, 1, (fh, fw, C, mult))
    y = oracle.depthwise_conv2d(x, f, (s, s), pad, (d, d))
    g = ints(72, 2, y.shape)
    dx = oracle.depthwise_conv2d_backprop_input(x.shape, f, g, (s, s), pad, (d, d))
    df = oracle.depthwise_conv2d_backprop_filter(x, f.shape, g, (s, s), pad, (d, d))
    assert dot(y, g) == dot(x, dx) == dot(f, df)
    x2, f2 = ints(72, 3, x.shape), ints(72, 4, f.shape)
    assert dot(oracle.depthwise_conv2d(x2, f, (s, s), pad, (d, d)), g) == dot(x2, dx)
    assert dot(oracle.depthwise_conv2d(x, f2, (s, s), pad, (d, d)), g) == dot(f2, df)


@pytest.mark.parametrize("case", CASES[:4])
def test_gradients_equal_central_differences_of_the_forward_oracle(oracle, case):
    """Element by element (the adjoint identity above only fixes inner products)."""
    H, W, Cin, Cout, fh, fw, s, d, pad = case
    x = ints(73, 0, (1, H, W, Cin))
    f = ints(73, 1, (fh, fw, Cin, Cout))
    g = ints(73, 2, oracle.conv2d(x, f, (s, s), pad, (d, d)).shape)
    dx = oracle.conv2d_backprop_input(x.shape, f, g, (s, s), pad, (d, d))
    df = oracle.conv2d_backprop_filter(x, f.shape, g, (s, s), pad, (d, d))

    def loss(xv, fv):
        return dot(oracle.conv2d(xv, fv, (s, s), pad, (d, d)), g)

    for idx in itertools.product(*(range(n) for n in x.shape)):
        e = np.zeros_like(x)
        e[idx] = 1
        assert loss(x + e, f) - loss(x - e, f) == 2 * int(dx[idx]), idx
    for idx in itertools.product(*(range(n) for n in f.shape)):
        e = np.zeros_like(f)
        e[idx] = 1
        assert loss(x, f + e) - loss(x, f - e) == 2 * int(df[idx]), idx
    # depthwise, multiplier 2, the same way
    fd = ints(73, 3, (fh, fw, Cin, 2))
    gd = ints(73, 4, oracle.depthwise_conv2d(x, fd, (s, s), pad, (d, d)).shape)
    ddx = oracle.depthwise_conv2d_backprop_input(x.shape, fd, gd, (s, s), pad, (d, d))
    ddf = oracle.depthwise_conv2d_backprop_filter(x, fd.shape, gd, (s, s), pad, (d, d))

    def dloss(xv, fv):
        return dot(oracle.depthwise_conv2d(xv, fv, (s, s), pad, (d, d)), gd)

    for idx in itertools.product(*(range(n) for n in x.shape)):
        e = np.zeros_like(x)
        e[idx] = 1
        assert dloss(x + e, fd) - dloss(x - e, fd) == 2 * int(ddx[idx]), idx
    for idx in itertools.product(*(range(n) for n in fd.shape)):
        e = np.zeros_like(fd)
        e[idx] = 1
        assert dloss(x, fd + e) - dloss(x, fd - e) == 2 * int(ddf[idx]), idx


@pytest.mark.parametrize("case", CASES)
def test_gradients_against_torch_fp64_autograd(oracle, case):
    import torch

    H, W, Cin, Cout, fh, fw, s, d, pad = case
    x = si.uniform(74, 0, (2, H, W, Cin), -1, 1)
    f = si.normal(74, 1, (fh, fw, Cin, Cout), 0, 0.5)
    Ho, pt, pb = oracle.window_geometry(H, fh, s, d, pad)
    Wo, pl, pr = oracle.window_geometry(W, fw, s, d, pad)
    g = si.normal(74, 2, (2, Ho, Wo, Cout), 0, 1)

    def torch_grads(xn, fn, gn, groups):
        xt = torch.from_numpy(xn.astype(np.float64)).permute(0, 3, 1, 2).requires_grad_(True)
        ft = torch.from_numpy(fn.astype(np.float64)).requires_grad_(True)
        # HWIO -> OIHW; for a depthwise filter [fh,fw,C,m] the output channel c*m+q has one input channel
        w = ft.permute(3, 2, 0, 1) if groups == 1 else ft.reshape(fn.shape[0], fn.shape[1], -1).permute(2, 0, 1).unsqueeze(1)
        w = w.contiguous()  # one of torch's CPU convolution paths insists on it
        xp = torch.nn.functional.pad(xt, (pl, pr, pt, pb))
        y = torch.nn.functional.conv2d(xp, w, stride=s, dilation=d, groups=groups)
        y.backward(torch.from_numpy(gn.astype(np.float64)).permute(0, 3, 1, 2))
        return xt.grad.permute(0, 2, 3, 1).numpy(), ft.grad.numpy()

    want_dx, want_df = torch_grads(x, f, g, 1)
    dx = oracle.conv2d_backprop_input(x.shape, f, g, (s, s), pad, (d, d))
    df = oracle.conv2d_backprop_filter(x, f.shape, g, (s, s), pad, (d, d))
    np.testing.assert_allclose(dx, want_dx, rtol=2e-6, atol=2e-6)
    np.testing.assert_allclose(df, want_df, rtol=2e-6, atol=2e-6)
    fd = si.normal(74, 3, (fh, fw, Cin, 2), 0, 0.5)
    gd = si.normal(74, 4, (2, Ho, Wo, Cin * 2), 0, 1)
    want_dx, want_df = torch_grads(x, fd, gd, Cin)
    np.testing.assert_allclose(oracle.depthwise_conv2d_backprop_input(x.shape, fd, gd, (s, s), pad, (d, d)), want_dx,
                               rtol=2e-6, atol=2e-6)
    np.testing.assert_allclose(oracle.depthwise_conv2d_backprop_filter(x, fd.shape, gd, (s, s), pad, (d, d)), want_df,
                               rtol=2e-6, atol=2e-6)


def test_pointwise_gradients_are_two_matrix_products(oracle):
    """conv 1x1 is a matMul over [N*H*W, Cin] (reshape is free, Sec. 3.4); so are its gradients:
    dx = dy . f^T and df = x^T . dy."""
    x = si.uniform(75, 0, (2, 6, 5, 12), -1, 1)
    f = si.normal(75, 1, (1, 1, 12, 20), 0, 0.3)
    g = si.normal(75, 2, (2, 6, 5, 20), 0, 1)
    dx = oracle.conv2d_backprop_input(x.shape, f, g)
    df = oracle.conv2d_backprop_filter(x, f.shape, g)
    assert np.array_equal(dx.reshape(-1, 12), oracle.matmul(g.reshape(-1, 20), f.reshape(12, 20), transpose_b=True))
    assert np.array_equal(df.reshape(12, 20), oracle.matmul(x.reshape(-1, 12), g.reshape(-1, 20), transpose_a=True))


def test_gradient_shape_checks(oracle):
    x = np.zeros((1, 5, 5, 2), np.float32)
    f = np.zeros((3, 3, 2, 4), np.float32)
    with pytest.raises(ValueError):
        oracle.conv2d_backprop_input(x.shape, f, np.zeros((1, 5, 5, 3), np.float32))
    with pytest.raises(ValueError):
        oracle.conv2d_backprop_filter(x, (3, 3, 3, 4), np.zeros((1, 5, 5, 4), np.float32))
    with pytest.raises(ValueError):
        oracle.depthwise_conv2d_backprop_input(x.shape, np.zeros((3, 3, 2, 1), np.float32), np.zeros((1, 4, 5, 2), np.float32))


def test_activation_and_bias_gradients(oracle):
    import torch

    y = np.array([-0.0, 0.0, 1e-30, 0.5, 5.999999, 6.0, 3.0, 0.0], np.float32)
    dy = np.array([1, 2, 3, 4, 5, 6, -7, -8], np.float32)
    assert np.array_equal(oracle.act_backprop(y, dy, "none"), dy)
    assert np.array_equal(oracle.act_backprop(y, dy, "relu"), np.array([0, 0, 3, 4, 5, 6, -7, 0], np.float32))
    assert np.array_equal(oracle.act_backprop(y, dy, "relu6"), np.array([0, 0, 3, 4, 5, 0, -7, 0], np.float32))
    # against torch's own relu6 gradient, through the pre-activation value
    z = si.uniform(76, 0, (4, 7, 5), -3, 9)
    g = si.normal(76, 1, z.shape, 0, 1)
    zt = torch.from_numpy(z).requires_grad_(True)
    torch.nn.functional.relu6(zt).backward(torch.from_numpy(g))
    assert np.array_equal(oracle.act_backprop(oracle.bias_act(z, None, "relu6"), g, "relu6"), zt.grad.numpy())
    zt = torch.from_numpy(z).requires_grad_(True)
    torch.relu(zt).backward(torch.from_numpy(g))
    assert np.array_equal(oracle.act_backprop(oracle.bias_act(z, None, "relu"), g, "relu"), zt.grad.numpy())
    # the bias gradient is the column sum: exact on integers, and within half an ulp of fp64 otherwise
    dz = si.small_integers(76, 2, (3, 4, 5, 6), -8, 8)
    assert np.array_equal(oracle.bias_backprop(dz), dz.reshape(-1, 6).astype(np.int64).sum(0).astype(np.float32))
    dz = si.normal(76, 3, (50, 7), 0, 1)
    assert np.array_equal(oracle.bias_backprop(dz), dz.astype(np.float64).sum(0).astype(np.float32))

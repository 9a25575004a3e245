"""Pins for the CPU oracle: every check compares it with something other than itself.

The paper prints no worked numeric example for these ops, so the pins are: hand-derived
tables (tests/golden), exact integer arithmetic, library routines (torch fp64 conv / pooling,
scipy softmax, numpy fp64 matmul) on the cases that reduce to them, an independently
written scatter-form evaluator, identity / delta filters, algebraic identities, and the
arithmetic of the paper's matMul shader (Listing 2) restated in fp32.
"""
import itertools
import os

import numpy as np
import pytest
import torch
import torch.nn.functional as F

import seeded_inputs as si

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rows(name):
    with open(os.path.join(GOLDEN, name)) as fh:
        for line in fh:
            line = line.strip()
            if line and not line.startswith("#"):
                yield line.split()


def rel_fro(a, b):
    a = np.asarray(a, np.float64)
    b = np.asarray(b, np.float64)
    d = np.linalg.norm((a - b).ravel())
    n = np.linalg.norm(b.ravel())
    return d / n if n > 0 else d


# ------------------------------------------------------------------ shapes and padding
def test_window_geometry_table(oracle):
    n = 0
    for in_, k, s, d, pad, out, before, after in _rows("window_geometry.txt"):
        got = oracle.window_geometry(int(in_), int(k), int(s), int(d), pad)
        assert got == (int(out), int(before), int(after)), (in_, k, s, d, pad, got)
        n += 1
    assert n >= 30


def test_valid_window_larger_than_input_is_an_error(oracle):
    with pytest.raises(ValueError):
        oracle.window_geometry(2, 3, 1, 1, "valid")
    with pytest.raises(ValueError):
        oracle.window_geometry(4, 3, 1, 2, "valid")


# ------------------------------------------------------------------ matmul
@pytest.mark.parametrize("ta,tb", list(itertools.product([False, True], repeat=2)))
def test_matmul_integer_exact_all_transposes(oracle, ta, tb):
    M, K, N = 7, 13, 5
    a = si.small_integers(11, 0, (M, K), -8, 8)
    b = si.small_integers(11, 1, (K, N), -8, 8)
    want = (a.astype(np.int64) @ b.astype(np.int64)).astype(np.float32)
    a_in = np.ascontiguousarray(a.T) if ta else a
    b_in = np.ascontiguousarray(b.T) if tb else b
    got = oracle.matmul(a_in, b_in, ta, tb)
    assert got.shape == (M, N)
    assert np.array_equal(got, want)


def test_matmul_matches_fp64_library_product(oracle):
    a = si.uniform(3, 0, (33, 70), -1, 1)
    b = si.uniform(3, 1, (70, 21), -1, 1)
    want = a.astype(np.float64) @ b.astype(np.float64)
    got = oracle.matmul(a, b)
    # double accumulation then one rounding: within half an fp32 ulp of the fp64 product
    assert np.all(np.abs(got.astype(np.float64) - want) <= np.spacing(np.abs(want).astype(np.float32)) * 0.5001 + 1e-12)


def test_matmul_identity_and_transpose_identity(oracle):
    a = si.uniform(4, 0, (9, 9), -1, 1)
    b = si.uniform(4, 1, (9, 6), -1, 1)
    eye = np.eye(9, dtype=np.float32)
    assert np.array_equal(oracle.matmul(a, eye), a)
    assert np.array_equal(oracle.matmul(eye, b), b)
    # (A B)^T = B^T A^T: feeding b as "A transposed" and a as "B transposed"
    ab = oracle.matmul(a, b)
    assert np.array_equal(oracle.matmul(b, a, True, True), ab.T)


def test_matmul_inner_dim_mismatch_rejected(oracle):
    with pytest.raises(ValueError):
        oracle.matmul(np.zeros((3, 4), np.float32), np.zeros((5, 2), np.float32))


def test_matmul_agrees_with_shader_arithmetic_listing2(oracle):
    """Listing 2 of the paper: each output is an fp32 running sum of 4-wide dot products over
    the shared dimension (a multiple of 4).  Restated here in fp32; the oracle (double
    accumulate) must agree to fp32 summation error, ~ sqrt(K) * 2^-24 relative."""
    M, K, N = 12, 64, 10
    a = si.uniform(5, 0, (M, K), -1, 1)
    b = si.uniform(5, 1, (K, N), -1, 1)
    shader = np.zeros((M, N), np.float32)
    for row in range(M):
        for col in range(N):
            result = np.float32(0.0)
            for i in range(0, K, 4):
                va, vb = a[row, i:i + 4], b[i:i + 4, col]
                dot = np.float32(0.0)
                for t in range(4):
                    dot = np.float32(dot + np.float32(va[t] * vb[t]))
                result = np.float32(result + dot)
            shader[row, col] = result
    got = oracle.matmul(a, b)
    assert rel_fro(got, shader) <= 1e-6 * np.sqrt(K)
    assert np.max(np.abs(got - shader)) <= 64 * 2.0 ** -24 * np.sqrt(K) * 4


def test_tf32_operand_modes_on_hand_picked_bit_patterns(oracle):
    one = np.float32(1.0)
    tie = np.float32(1.0 + 2.0 ** -11)  # exactly halfway between two TF32 values
    above = np.float32(1.0 + 2.0 ** -11 + 2.0 ** -20)
    below = np.float32(1.0 + 2.0 ** -12)
    for v, rna, rz in [(tie, 1 + 2.0 ** -10, 1.0), (above, 1 + 2.0 ** -10, 1.0), (below, 1.0, 1.0),
                       (-tie, -(1 + 2.0 ** -10), -1.0)]:
        a = np.array([[v]], np.float32)
        b = np.array([[one]], np.float32)
        assert oracle.matmul(a, b, operand="tf32_rna")[0, 0] == np.float32(rna)
        assert oracle.matmul(a, b, operand="tf32_rz")[0, 0] == np.float32(rz)
        assert oracle.matmul(a, b, operand="fp32")[0, 0] == v


# ------------------------------------------------------------------ conv2d
def _torch_conv(x, f, strides, pad, dilations, groups=1):
    """fp64 library convolution with TensorFlow-style explicit padding done by hand here."""
    N, H, W, C = x.shape
    fh, fw = f.shape[:2]

    def geom(in_, k, s, d):
        ek = (k - 1) * d + 1
        if pad == "valid":
            return 0, 0
        out = -(-in_ // s)
        total = max((out - 1) * s + ek - in_, 0)
        return total // 2, total - total // 2

    pt, pb = geom(H, fh, strides[0], dilations[0])
    pl, pr = geom(W, fw, strides[1], dilations[1])
    xt = torch.from_numpy(x.astype(np.float64)).permute(0, 3, 1, 2)
    xt = F.pad(xt, (pl, pr, pt, pb))
    if groups == 1:
        wt = torch.from_numpy(f.astype(np.float64)).permute(3, 2, 0, 1)  # [Cout, Cin, fh, fw]
    else:
        # depthwise filter [fh, fw, C, mult] -> [C*mult, 1, fh, fw], output channel c*mult+q
        mult = f.shape[3]
        wt = torch.from_numpy(f.astype(np.float64)).permute(2, 3, 0, 1).reshape(C * mult, 1, fh, fw)
    y = F.conv2d(xt, wt, None, stride=strides, padding=0, dilation=dilations, groups=groups)
    return y.permute(0, 2, 3, 1).numpy()


CONV_CASES = [
    # N, H, W, Cin, fh, fw, Cout, strides, pad, dilations
    (2, 7, 6, 3, 3, 3, 4, (1, 1), "same", (1, 1)),
    (1, 8, 8, 3, 3, 3, 5, (2, 2), "same", (1, 1)),
    (1, 9, 7, 2, 3, 3, 3, (2, 2), "same", (1, 1)),
    (1, 9, 8, 2, 3, 3, 3, (2, 1), "valid", (1, 1)),
    (1, 9, 9, 2, 3, 3, 2, (1, 1), "same", (2, 2)),
    (1, 10, 9, 2, 3, 2, 2, (1, 1), "valid", (2, 1)),
    (2, 5, 5, 4, 1, 1, 6, (1, 1), "same", (1, 1)),
    (1, 6, 7, 3, 5, 3, 2, (3, 2), "same", (1, 1)),
    (1, 4, 4, 1, 4, 4, 1, (1, 1), "valid", (1, 1)),
]


@pytest.mark.parametrize("case", CONV_CASES)
def test_conv2d_matches_fp64_library_convolution(oracle, case):
    N, H, W, Cin, fh, fw, Cout, strides, pad, dil = case
    x = si.uniform(21, 0, (N, H, W, Cin), -1, 1)
    f = si.normal(21, 1, (fh, fw, Cin, Cout), 0, 0.5)
    want = _torch_conv(x, f, strides, pad, dil)
    got = oracle.conv2d(x, f, strides, pad, dil)
    assert got.shape == want.shape
    np.testing.assert_allclose(got, want, rtol=0, atol=2e-6)


def _scatter_conv(x, f, strides, pad_before, out_hw, dilations):
    """Definition written the other way round: every input element is pushed through every
    filter tap into the output it contributes to (fp64)."""
    N, H, W, Cin = x.shape
    fh, fw, _, Cout = f.shape
    Ho, Wo = out_hw
    y = np.zeros((N, Ho, Wo, Cout), np.float64)
    for n in range(N):
        for iy in range(H):
            for ix in range(W):
                for ky in range(fh):
                    ty = iy + pad_before[0] - ky * dilations[0]
                    if ty < 0 or ty % strides[0]:
                        continue
                    oy = ty // strides[0]
                    if oy >= Ho:
                        continue
                    for kx in range(fw):
                        tx = ix + pad_before[1] - kx * dilations[1]
                        if tx < 0 or tx % strides[1]:
                            continue
                        ox = tx // strides[1]
                        if ox >= Wo:
                            continue
                        y[n, oy, ox, :] += x[n, iy, ix, :].astype(np.float64) @ f[ky, kx].astype(np.float64)
    return y


@pytest.mark.parametrize("strides,pad,dil", [((1, 1), "same", (1, 1)), ((2, 2), "same", (1, 1)),
                                             ((2, 2), "valid", (1, 1)), ((1, 1), "same", (2, 2)),
                                             ((1, 2), "valid", (1, 1)), ((3, 3), "same", (1, 1))])
@pytest.mark.parametrize("hw", [(5, 5), (4, 5), (6, 4)])
def test_conv2d_matches_scatter_form_on_tiny_shapes(oracle, strides, pad, dil, hw):
    H, W = hw
    x = si.uniform(22, 0, (1, H, W, 3), -1, 1)
    f = si.normal(22, 1, (3, 3, 3, 4), 0, 0.5)
    try:
        Ho, pt, _ = oracle.window_geometry(H, 3, strides[0], dil[0], pad)
        Wo, pl, _ = oracle.window_geometry(W, 3, strides[1], dil[1], pad)
    except ValueError:
        pytest.skip("window larger than input")
    want = _scatter_conv(x, f, strides, (pt, pl), (Ho, Wo), dil)
    got = oracle.conv2d(x, f, strides, pad, dil)
    np.testing.assert_allclose(got, want, rtol=0, atol=2e-6)


def test_conv2d_integer_exact_against_library(oracle):
    x = si.small_integers(23, 0, (2, 9, 8, 5), -8, 8)
    f = si.small_integers(23, 1, (3, 3, 5, 7), -8, 8)
    for strides, pad in [((1, 1), "same"), ((2, 2), "same"), ((2, 2), "valid")]:
        want = _torch_conv(x, f, strides, pad, (1, 1))
        got = oracle.conv2d(x, f, strides, pad)
        assert np.array_equal(got.astype(np.float64), want)


def test_centre_delta_filter_returns_input(oracle):
    x = si.uniform(24, 0, (2, 6, 7, 3), -1, 1)
    f = np.zeros((3, 3, 3, 3), np.float32)
    for c in range(3):
        f[1, 1, c, c] = 1.0
    assert np.array_equal(oracle.conv2d(x, f, (1, 1), "same"), x)
    d = np.zeros((3, 3, 3, 1), np.float32)
    d[1, 1, :, 0] = 1.0
    assert np.array_equal(oracle.depthwise_conv2d(x, d, (1, 1), "same"), x)
    eye = np.eye(3, dtype=np.float32).reshape(1, 1, 3, 3)
    assert np.array_equal(oracle.conv2d(x, eye), x)


@pytest.mark.parametrize("size,stride", [(8, 2), (7, 2), (8, 1), (9, 3)])
def test_shifted_delta_taps_pin_same_padding_offsets(oracle, size, stride):
    """A filter that is 1 at a single tap (ky,kx) must read x[oy*s - pt + ky, ox*s - pl + kx]
    (0 outside).  For an even size and stride 2 'same' pads nothing before, so tap (0,0)
    reads x[2oy, 2ox]."""
    x = si.uniform(25, 0, (1, size, size, 1), 1, 2)
    out, before, _ = oracle.window_geometry(size, 3, stride, 1, "same")
    if size % 2 == 0 and stride == 2:
        assert before == 0
    for ky in range(3):
        for kx in range(3):
            f = np.zeros((3, 3, 1, 1), np.float32)
            f[ky, kx, 0, 0] = 1.0
            y = oracle.conv2d(x, f, (stride, stride), "same")
            yd = oracle.depthwise_conv2d(x, f, (stride, stride), "same")
            for oy in range(out):
                for ox in range(out):
                    iy, ix = oy * stride - before + ky, ox * stride - before + kx
                    want = x[0, iy, ix, 0] if (0 <= iy < size and 0 <= ix < size) else 0.0
                    assert y[0, oy, ox, 0] == want
                    assert yd[0, oy, ox, 0] == want


def test_pointwise_conv_is_matmul_on_reshaped_input(oracle):
    """Reshape is free (Sec. 3.4): a 1x1 conv is matMul of x viewed as [N*H*W, Cin]."""
    x = si.uniform(26, 0, (2, 5, 4, 6), -1, 1)
    f = si.normal(26, 1, (1, 1, 6, 9), 0, 0.5)
    y = oracle.conv2d(x, f)
    c = oracle.matmul(x.reshape(-1, 6), f.reshape(6, 9))
    assert np.array_equal(y.reshape(-1, 9), c)


def test_conv2d_bias_and_activation_order(oracle):
    x = si.uniform(27, 0, (1, 5, 5, 2), -1, 1)
    f = si.normal(27, 1, (3, 3, 2, 3), 0, 1.0)
    b = np.array([0.5, -0.25, 7.0], np.float32)
    raw = oracle.conv2d(x, f)
    want = np.minimum(np.maximum(raw + b, np.float32(0)), np.float32(6))
    assert np.array_equal(oracle.conv2d(x, f, bias=b, act="relu6"), want)
    assert np.array_equal(oracle.conv2d(x, f, bias=b, act="relu"), np.maximum(raw + b, np.float32(0)))
    assert np.array_equal(oracle.conv2d(x, f, bias=b), raw + b)


def test_conv2d_is_linear_in_input(oracle):
    x = si.small_integers(28, 0, (1, 6, 6, 2), -4, 4)
    z = si.small_integers(28, 1, (1, 6, 6, 2), -4, 4)
    f = si.small_integers(28, 2, (3, 3, 2, 3), -4, 4)
    lhs = oracle.conv2d(2 * x + 3 * z, f, (2, 2), "same")
    rhs = 2 * oracle.conv2d(x, f, (2, 2), "same") + 3 * oracle.conv2d(z, f, (2, 2), "same")
    assert np.array_equal(lhs, rhs)


def test_conv2d_channel_mismatch_rejected(oracle):
    with pytest.raises(ValueError):
        oracle.conv2d(np.zeros((1, 4, 4, 3), np.float32), np.zeros((3, 3, 2, 4), np.float32))


# ------------------------------------------------------------------ depthwise
DW_CASES = [
    (2, 7, 6, 4, 3, 3, 1, (1, 1), "same", (1, 1)),
    (1, 8, 8, 4, 3, 3, 1, (2, 2), "same", (1, 1)),
    (1, 9, 7, 3, 3, 3, 2, (2, 2), "same", (1, 1)),
    (1, 9, 8, 3, 3, 3, 3, (1, 1), "valid", (1, 1)),
    (1, 9, 9, 2, 3, 3, 1, (1, 1), "same", (2, 2)),
    (1, 6, 6, 5, 5, 5, 1, (1, 1), "same", (1, 1)),
]


@pytest.mark.parametrize("case", DW_CASES)
def test_depthwise_matches_fp64_grouped_library_convolution(oracle, case):
    N, H, W, C, fh, fw, mult, strides, pad, dil = case
    x = si.uniform(31, 0, (N, H, W, C), -1, 1)
    f = si.normal(31, 1, (fh, fw, C, mult), 0, 0.5)
    want = _torch_conv(x, f, strides, pad, dil, groups=C)
    got = oracle.depthwise_conv2d(x, f, strides, pad, dil)
    assert got.shape == want.shape
    np.testing.assert_allclose(got, want, rtol=0, atol=2e-6)


def test_depthwise_equals_conv2d_with_channel_diagonal_filter(oracle):
    C = 4
    x = si.small_integers(32, 0, (1, 7, 7, C), -8, 8)
    f = si.small_integers(32, 1, (3, 3, C, 1), -8, 8)
    full = np.zeros((3, 3, C, C), np.float32)
    for c in range(C):
        full[:, :, c, c] = f[:, :, c, 0]
    for strides in [(1, 1), (2, 2)]:
        assert np.array_equal(oracle.depthwise_conv2d(x, f, strides, "same"), oracle.conv2d(x, full, strides, "same"))


def test_depthwise_equals_per_channel_single_channel_conv(oracle):
    C, mult = 3, 2
    x = si.small_integers(33, 0, (1, 6, 5, C), -8, 8)
    f = si.small_integers(33, 1, (3, 3, C, mult), -8, 8)
    y = oracle.depthwise_conv2d(x, f, (1, 1), "same")
    for c in range(C):
        for q in range(mult):
            single = oracle.conv2d(x[..., c:c + 1], f[:, :, c:c + 1, q:q + 1], (1, 1), "same")
            assert np.array_equal(y[..., c * mult + q], single[..., 0])


# ------------------------------------------------------------------ bias / activation
def test_bias_act_hand_values_signed_zero_and_nan(oracle):
    x = np.array([[-1.0, -0.0, 0.0, 0.5, 5.5, 6.0, 7.0, np.nan, np.inf, -np.inf]], np.float32)
    b = np.zeros(10, np.float32)
    r = oracle.bias_act(x, b, "relu")[0]
    r6 = oracle.bias_act(x, b, "relu6")[0]
    assert list(r[:7]) == [0.0, 0.0, 0.0, 0.5, 5.5, 6.0, 7.0]
    assert list(r6[:7]) == [0.0, 0.0, 0.0, 0.5, 5.5, 6.0, 6.0]
    assert not np.signbit(r[1]) and not np.signbit(r[0]) and not np.signbit(r6[1])
    assert np.isnan(r[7]) and np.isnan(r6[7])
    assert r[8] == np.inf and r6[8] == 6.0 and r[9] == 0.0 and r6[9] == 0.0
    none = oracle.bias_act(x, None, "none")[0]
    assert np.array_equal(none[:7], x[0, :7]) and np.signbit(none[1])


def test_bias_act_is_one_fp32_add_then_clamp(oracle):
    x = si.uniform(41, 0, (5, 7, 16), -8, 8)
    b = si.normal(41, 1, (16,), 0, 1)
    s = (x + b).astype(np.float32)  # numpy fp32 add = one IEEE add
    assert np.array_equal(oracle.bias_act(x, b, "none"), s)
    r6 = oracle.bias_act(x, b, "relu6")
    assert np.array_equal(r6, np.clip(s, np.float32(0), np.float32(6)))
    assert r6.min() >= 0 and r6.max() <= 6
    assert np.array_equal(oracle.bias_act(r6, None, "relu6"), r6)  # idempotent, identity on [0,6]


# ------------------------------------------------------------------ avgPool
@pytest.mark.parametrize("H,W,k,s,pad", [(7, 7, 7, 1, "valid"), (8, 6, 2, 2, "valid"), (7, 7, 3, 1, "same"),
                                         (9, 9, 3, 2, "same"), (6, 5, 3, 1, "valid")])
def test_avg_pool_matches_library_pooling(oracle, H, W, k, s, pad):
    x = si.uniform(51, 0, (2, H, W, 3), -1, 1)
    got = oracle.avg_pool(x, (k, k), (s, s), pad)
    xt = torch.from_numpy(x.astype(np.float64)).permute(0, 3, 1, 2)
    if pad == "same":
        # symmetric cases only ((k-1) even and sizes chosen so before == after)
        _, before, after = oracle.window_geometry(H, k, s, 1, pad)
        assert before == after
        want = F.avg_pool2d(xt, k, s, padding=before, count_include_pad=False)
    else:
        want = F.avg_pool2d(xt, k, s)
    want = want.permute(0, 2, 3, 1).numpy()
    assert got.shape == want.shape
    np.testing.assert_allclose(got, want, rtol=0, atol=1e-6)


def test_avg_pool_constant_and_global_mean(oracle):
    c = np.full((1, 6, 6, 2), 3.25, np.float32)
    for pad, k, s in [("same", 3, 2), ("same", 2, 1), ("valid", 2, 2)]:
        assert np.all(oracle.avg_pool(c, (k, k), (s, s), pad) == np.float32(3.25))
    x = si.uniform(52, 0, (3, 7, 7, 5), 0, 6)
    g = oracle.avg_pool(x, (7, 7), (1, 1), "valid")
    assert g.shape == (3, 1, 1, 5)
    np.testing.assert_allclose(g[:, 0, 0, :], x.astype(np.float64).mean(axis=(1, 2)), rtol=0, atol=5e-7)


def test_avg_pool_asymmetric_same_padding_divisor(oracle):
    # in=4, k=3, s=2, 'same': out=2, pad 0 before / 1 after; the last window holds 2 in-bounds rows
    x = np.arange(16, dtype=np.float32).reshape(1, 4, 4, 1)
    y = oracle.avg_pool(x, (3, 3), (2, 2), "same")
    assert y.shape == (1, 2, 2, 1)
    assert y[0, 0, 0, 0] == np.float32(x[0, 0:3, 0:3, 0].mean())
    assert y[0, 1, 1, 0] == np.float32(x[0, 2:4, 2:4, 0].mean())
    assert y[0, 0, 1, 0] == np.float32(x[0, 0:3, 2:4, 0].mean())


# ------------------------------------------------------------------ maxPool, elementwise binary ops, rank-3 matMul
@pytest.mark.parametrize("H,W,k,s,pad", [(7, 7, 7, 1, "valid"), (8, 6, 2, 2, "valid"), (7, 7, 3, 1, "same"),
                                         (9, 9, 3, 2, "same"), (8, 8, 3, 2, "same"), (6, 5, 3, 1, "valid")])
def test_max_pool_matches_library_pooling_on_explicitly_padded_input(oracle, H, W, k, s, pad):
    x = si.uniform(53, 0, (2, H, W, 3), -1, 1)
    got = oracle.max_pool(x, (k, k), (s, s), pad)
    xt = torch.from_numpy(x).permute(0, 3, 1, 2)
    if pad == "same":  # TF padding built by hand (extra element after), filled with -inf so it never wins
        _, pt, pb = oracle.window_geometry(H, k, s, 1, pad)
        _, pl, pr = oracle.window_geometry(W, k, s, 1, pad)
        xt = F.pad(xt, (pl, pr, pt, pb), value=float("-inf"))
    want = F.max_pool2d(xt, k, s).permute(0, 2, 3, 1).numpy()
    assert got.shape == want.shape
    assert np.array_equal(got, want)  # a selection: exact


def test_max_pool_hand_values_asymmetric_padding_and_nan(oracle):
    # in=4, k=3, s=2, 'same': out=2, pad 0 before / 1 after
    x = np.arange(16, dtype=np.float32).reshape(1, 4, 4, 1)
    y = oracle.max_pool(x, (3, 3), (2, 2), "same")
    assert y[0, :, :, 0].tolist() == [[10.0, 11.0], [14.0, 15.0]]
    neg = -np.abs(si.uniform(54, 0, (1, 5, 5, 2), 1, 2))          # all negative: zero padding would win wrongly
    assert oracle.max_pool(neg, (3, 3), (1, 1), "same").max() < 0
    x[0, 3, 3, 0] = np.nan                                         # a NaN wins its windows and no other
    y = oracle.max_pool(x, (3, 3), (2, 2), "same")
    assert np.isnan(y[0, 1, 1, 0]) and y[0, 0, 0, 0] == 10.0 and y[0, 0, 1, 0] == 11.0 and y[0, 1, 0, 0] == 14.0
    assert np.array_equal(oracle.max_pool(x[:, :3, :3], (1, 1), (1, 1), "valid"), x[:, :3, :3])  # 1x1 window: identity


@pytest.mark.parametrize("op,fn", [("add", np.add), ("sub", np.subtract), ("mul", np.multiply)])
def test_binary_ops_are_one_fp32_operation_per_element(oracle, op, fn):
    a = si.normal(55, 0, (3, 5, 7, 6), 0, 10)
    b = si.normal(55, 1, (3, 5, 7, 6), 0, 10)
    assert np.array_equal(oracle.binary(op, a, b), fn(a, b))                    # numpy fp32: the same single rounding
    v = si.normal(55, 2, (6,), 0, 10)
    assert np.array_equal(oracle.binary(op, a, v), fn(a, v[None, None, None, :]))  # vector along the last dimension
    exact = fn(a.astype(np.float64), b.astype(np.float64))
    assert np.all(np.abs(oracle.binary(op, a, b) - exact) <= np.spacing(np.abs(exact).astype(np.float32)) / 2 + 0)
    assert np.array_equal(oracle.binary("add", a, np.zeros_like(a)), a)
    assert np.array_equal(oracle.binary("mul", a, np.ones(6, np.float32)), a)
    assert np.array_equal(oracle.binary("sub", a, a), np.zeros_like(a))


def test_batch_matmul_is_one_product_per_leading_index(oracle):
    a = si.uniform(56, 0, (4, 9, 13), -1, 1)
    b = si.uniform(56, 1, (4, 13, 5), -1, 1)
    got = oracle.batch_matmul(a, b)
    want = np.einsum("bik,bkj->bij", a.astype(np.float64), b.astype(np.float64))
    assert got.shape == (4, 9, 5)
    np.testing.assert_allclose(got, want, rtol=0, atol=2e-7 * 13)
    ai = si.small_integers(57, 0, (3, 6, 8), -8, 8)
    bi = si.small_integers(57, 1, (3, 7, 8), -8, 8)
    want_i = np.einsum("bik,bjk->bij", ai.astype(np.int64), bi.astype(np.int64)).astype(np.float32)
    assert np.array_equal(oracle.batch_matmul(ai, bi, transpose_b=True), want_i)
    # a product must not see its neighbours: permuting the leading index permutes the result
    perm = [2, 0, 3, 1]
    assert np.array_equal(oracle.batch_matmul(a[perm], b[perm]), got[perm])


# ------------------------------------------------------------------ softmax
def test_softmax_invariants_and_library(oracle):
    from scipy.special import softmax as sp_softmax

    x = si.normal(61, 0, (6, 1000), 0, 3)
    p = oracle.softmax(x)
    assert np.all(np.abs(p.astype(np.float64).sum(-1) - 1) <= 1e-6)
    assert np.array_equal(p.argmax(-1), x.argmax(-1))
    np.testing.assert_allclose(p, sp_softmax(x.astype(np.float64), axis=-1), rtol=1e-6, atol=1e-12)
    shifted = oracle.softmax(x + np.float32(8.0))  # exact shift for these magnitudes? compare loosely
    np.testing.assert_allclose(shifted, p, rtol=2e-5, atol=1e-10)
    u = oracle.softmax(np.full((2, 8), 1.5, np.float32))
    assert np.all(u == np.float32(0.125))
    big = oracle.softmax(np.array([[1000.0, 999.0, -1000.0]], np.float32))
    assert np.isfinite(big).all() and abs(big[0, 0] - 1 / (1 + np.exp(-1.0))) < 1e-7
    r3 = oracle.softmax(x.reshape(2, 3, 1000))
    assert np.array_equal(r3.reshape(6, 1000), p)


# ------------------------------------------------------------------ whole model
@pytest.mark.parametrize("alpha,hw,macs,params", [(float(a), int(h), int(m), int(p))
                                                  for a, h, m, p in _rows("mobilenet_v1_counts.txt")])
def test_model_counts_from_layer_list(oracle, alpha, hw, macs, params):
    layers = si.make_model_weights(si.mobilenet_v1_layers(alpha), 3, seed=1)
    chans = si.layer_channels(layers, 3)
    h = w = hw
    total_macs = 0
    total_params = 0
    spatial = []
    for layer, (cin, cout) in zip(layers, chans):
        if layer.kind in ("conv2d", "depthwise_conv2d"):
            fh, fw = layer.filter_hw
            h, _, _ = oracle.window_geometry(h, fh, layer.strides[0], 1, layer.pad)
            w, _, _ = oracle.window_geometry(w, fw, layer.strides[1], 1, layer.pad)
            per_out = fh * fw * (cin if layer.kind == "conv2d" else 1)
            total_macs += h * w * cout * per_out
            spatial.append(h)
        elif layer.kind == "dense":
            total_macs += cin * cout
        if layer.filter is not None:
            total_params += layer.filter.size + layer.bias.size
    assert total_macs == macs
    assert total_params == params
    first = hw // 2  # 224 -> 112 -> 112 -> 56 -> 56 -> 28 -> 28 -> 14 (x6 blocks) -> 7 -> 7
    assert spatial == [first] * 3 + [first // 2] * 4 + [first // 4] * 4 + [first // 8] * 12 + [first // 16] * 4


def test_small_model_invariants(oracle):
    x, layers = si.config_mobilenet(0.25, 32, 2, seed=77, classes=10)
    outs = oracle.run_model(layers, x, keep_all=True)
    assert outs[0].shape == (2, 16, 16, 8)
    assert outs[-3].shape == (2, 256) and outs[-2].shape == (2, 10) and outs[-1].shape == (2, 10)
    for layer, out in zip(layers, outs):
        if layer.act == "relu6":
            assert out.min() >= 0 and out.max() <= 6
    assert np.all(np.abs(outs[-1].astype(np.float64).sum(-1) - 1) <= 1e-6)
    assert np.array_equal(outs[-1].argmax(-1), outs[-2].argmax(-1))
    # images are independent: running one image alone gives the same bits
    solo = oracle.run_model(layers, x[1:2])
    assert np.array_equal(solo[0], outs[-1][1])
    # thread count never changes a bit
    oracle.set_threads(1)
    again = oracle.run_model(layers, x)
    oracle.set_threads(os.cpu_count() or 1)
    assert np.array_equal(again, outs[-1])


# ------------------------------------------------------------------ narrow (bfloat16) storage
def test_round_bf16_hand_values_ties_and_specials(oracle):
    # bfloat16 keeps 8 significand bits: the spacing in [1, 2) is 2^-7
    cases = [
        (1.0, 1.0),
        (1.0 + 2.0 ** -8, 1.0),                      # exactly halfway between 1 and 1 + 2^-7: to the even one
        (1.0 + 2.0 ** -8 + 2.0 ** -23, 1.0 + 2.0 ** -7),  # just above halfway
        (1.0 + 3 * 2.0 ** -8, 1.0 + 2.0 ** -6),      # halfway between 1 + 2^-7 (odd) and 1 + 2^-6 (even)
        (3.14159265, 3.140625),                      # pi: 0x40490FDB -> 0x4049
        (-2.71828183, -2.71875),                     # -e: 0xC02DF854 -> 0xC02E
        (0.1, 0.10009765625),                        # 0x3DCCCCCD -> 0x3DCD
        (256.0 + 1.0, 256.0),                        # spacing 2 in [256, 512): 257 is halfway, 256 is even
        (256.0 + 3.0, 260.0),                        # halfway between 258 (odd) and 260 (even)
        (3.3895313892515355e38, 3.3895313892515355e38),  # the largest bfloat16, 0x7F7F0000
        (3.4028234663852886e38, np.inf),             # the largest fp32 rounds up past it
        (1e-40, 9.9e-41),                            # subnormal: 0x000116C2 -> 0x0001 0000 = 9.18e-41
        (0.0, 0.0),
    ]
    x = np.array([c[0] for c in cases], dtype=np.float32)
    got = oracle.round_bf16(x)
    for (src, want), g in zip(cases, got):
        if src == 1e-40:
            assert g.view(np.uint32) == 0x00010000
        else:
            assert g == np.float32(want), (src, g, want)
    sp = oracle.round_bf16(np.array([np.inf, -np.inf, np.nan, -0.0], dtype=np.float32))
    assert sp[0] == np.inf and sp[1] == -np.inf and np.isnan(sp[2]) and sp[3] == 0 and np.signbit(sp[3])
    # a NaN whose payload sits only in the dropped bits must not turn into an infinity
    sneaky = np.array([0x7F800001], dtype=np.uint32).view(np.float32)
    assert np.isnan(oracle.round_bf16(sneaky)[0])


def test_round_bf16_matches_library_conversion(oracle):
    x = np.concatenate([
        si.normal(91, 0, (100000,), 0, 3),
        si.uniform(91, 1, (50000,), -1e-3, 1e-3),
        (si.uniform(91, 2, (50000,), -1, 1).astype(np.float64) * 1e30).astype(np.float32),
        np.arange(0, 70000, dtype=np.uint32).view(np.float32),          # subnormals and their ties
        (np.arange(0, 70000, dtype=np.uint32) + 0x3F7F0000).view(np.float32),  # around 1.0, every low-bit pattern
    ])
    want = torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy()
    got = oracle.round_bf16(x)
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))
    assert np.array_equal(oracle.round_bf16(got), got)  # idempotent
    assert np.all((got.view(np.uint32) & 0xFFFF) == 0)


def test_narrow_storage_model_is_the_fp32_model_on_stored_values(oracle):
    x, layers = si.config_mobilenet(0.25, 32, 2, seed=78, classes=10)
    outs = oracle.run_model(layers, x, keep_all=True, storage="bf16")
    # what is stored is a bfloat16; dense, softmax and the last layer stay fp32
    for layer, out in zip(layers[:-2], outs[:-2]):
        assert np.all((out.view(np.uint32) & 0xFFFF) == 0), layer.kind
    assert np.any((outs[-2].view(np.uint32) & 0xFFFF) != 0)
    # layer by layer: the fp32 op on the stored input and the stored filter, then one rounding
    stored = oracle.round_bf16
    first = oracle.conv2d(stored(x), stored(layers[0].filter), layers[0].strides, layers[0].pad, layers[0].dilations,
                          layers[0].bias, layers[0].act)
    assert np.array_equal(outs[0], stored(first))
    dw = oracle.depthwise_conv2d(outs[0], stored(layers[1].filter), layers[1].strides, layers[1].pad,
                                 layers[1].dilations, layers[1].bias, layers[1].act)
    assert np.array_equal(outs[1], stored(dw))
    n, h, w, c = outs[-4].shape
    assert np.array_equal(outs[-3], stored(oracle.avg_pool(outs[-4], (h, w), (1, 1), "valid").reshape(n, c)))
    # on values every format holds exactly (small integers, sums below 256) both modes agree bit for bit
    xi = si.small_integers(79, 0, (1, 8, 8, 4), -2, 2)
    li = [si.Layer(kind="conv2d", filter_hw=(3, 3), strides=(1, 1), pad="same", act="relu", out_channels=4,
                   filter=si.small_integers(79, 1, (3, 3, 4, 4), -1, 1), bias=si.small_integers(79, 2, (4,), -3, 3)),
          si.Layer(kind="depthwise_conv2d", filter_hw=(3, 3), strides=(1, 1), pad="same", act="relu6", out_channels=1,
                   filter=si.small_integers(79, 3, (3, 3, 4, 1), -1, 1), bias=None)]
    assert np.array_equal(oracle.run_model(li, xi, storage="bf16"), oracle.run_model(li, xi))
    # and close to the fp32 model overall: storage error is 2^-9 relative per stored value
    full = oracle.run_model(layers, x, keep_all=True)
    assert rel_fro(outs[-2], full[-2]) < 3e-2
    assert rel_fro(outs[0], full[0]) < 2.0 ** -7


def test_generator_moments_and_reproducibility():
    u = si.uniform(9, 0, (200000,), -1, 1)
    assert u.min() >= -1 and u.max() < 1 and abs(u.mean()) < 5e-3 and abs(u.var() - 1 / 3) < 5e-3
    g = si.normal(9, 1, (200000,), 0, 2)
    assert abs(g.mean()) < 2e-2 and abs(g.std() - 2) < 2e-2
    assert np.array_equal(si.uniform(9, 0, (200000,), -1, 1), u)
    assert not np.array_equal(si.uniform(9, 2, (200000,), -1, 1), u)
    six = si.uniform(10, 0, (100000,), 0, 6)
    assert six.min() >= 0 and six.max() < 6
    k = si.small_integers(3, 0, (10000,), -8, 8)
    assert k.min() == -8 and k.max() == 8 and np.all(k == np.round(k))

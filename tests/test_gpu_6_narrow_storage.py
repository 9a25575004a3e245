"""GPU parity of the narrow-storage mode: bfloat16 in memory, exact products, fp32 sums, one rounding
(to nearest even) when a result is stored (the counterpart of the paper's 16-bit float textures,
Sec. 4.1.3).

Tolerances.  Products of two bfloat16 values are exact in fp32, so kernel and oracle differ only in
how the sum is rounded: the tensor core adds in fp32 in an order and with an alignment of its own
(the same accumulator as the TF32 kernel, which agrees with its operand-matched oracle to 2e-5), the
oracle adds in fp64 and rounds once.
  * fp32 output: relative Frobenius error <= 2e-5.
  * bfloat16 output: the two sums round to the same bfloat16 except when they straddle a rounding
    boundary, so at most one bfloat16 step (2^-7 relative) per element, plus the summation error
    itself where the terms cancel to a value far below them, and at most 2 % of the elements off at
    all.
  * small integers: every product, sum and stored value is exact, results must agree bit for bit.
  * a model: storing a value re-quantises it, and that amplifies a small difference between two
    computations: a pre-rounding gap of d (relative, below the step 2^-8) flips the rounding with
    probability d / 2^-8 and then costs a whole step, an RMS error of sqrt(d * 2^-8) >> d.  Layer after
    layer the difference between kernel and oracle therefore climbs towards the quantisation noise
    itself (2^-9 / sqrt(3) ~ 1e-3 per stored tensor, adding like a random walk over the layers) and
    stays there; it cannot be bounded below that level.  The bars: the first three layers, which see no
    accumulated noise, at most one step on at most 1 % of the elements; every layer a relative
    Frobenius error <= 1e-2 (a little above one step, 2^-7); a small-integer model bit for bit; and the
    whole-model bar of the fp32 modes (max logit error <= 1e-2 of the logit span; same top-1 wherever
    the oracle's own top-1 margin is at least 4x that tolerance, so that the comparison is not luck).
"""
import numpy as np
import pytest

import seeded_inputs as si
from helpers import dev, host, rel_fro, same_bits

pytestmark = pytest.mark.gpu

SHAPES = [
    # M, K, N   (K and N multiples of 8: 16-byte row pitches)
    (128, 64, 32),       # one tile, one k-block
    (128, 8, 8),         # the smallest K and N
    (300, 104, 72),      # ragged in M, K (a k-block with 40 live columns) and N
    (4100, 40, 264),     # N just above one 256 tile
    (520, 1024, 512),    # sixteen k-blocks: the stage ring wraps
    (1000, 1024, 1000),  # the dense layer's width, N tail inside a 32-column chunk
    (20000, 256, 512),   # more tiles than SMs: persistent loop, accumulator stages reused
    (25088, 512, 512),   # pw7-pw11 of the 224 model at batch 128
]


def bf16_dev(a):
    """A bfloat16 CUDA tensor holding `a`, whose values must already be bfloat16."""
    import torch

    t = torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).cuda()
    h = t.to(torch.bfloat16)
    assert torch.equal(h.to(torch.float32), t), "values are not representable"
    return h


def widen(t):
    import torch

    return t.to(torch.float32).cpu().numpy()


def bf16_steps(got, want):
    """Distance in bfloat16 steps between two arrays of bfloat16 values held as fp32 (same-sign values)."""
    g = (np.ascontiguousarray(got, np.float32).view(np.uint32) >> 16).astype(np.int64)
    w = (np.ascontiguousarray(want, np.float32).view(np.uint32) >> 16).astype(np.int64)
    # map the sign-magnitude patterns onto a line
    g = np.where(g & 0x8000, -(g & 0x7FFF), g)
    w = np.where(w & 0x8000, -(w & 0x7FFF), w)
    return np.abs(g - w)


@pytest.mark.parametrize("mkn", SHAPES)
def test_matmul_bf16_integer_exact(ctx, oracle, mkn):
    import torch

    M, K, N = mkn
    a = si.small_integers(601, 0, (M, K), -8, 8)
    bt = si.small_integers(601, 1, (N, K), -8, 8)
    exact = (a.astype(np.int64) @ bt.astype(np.int64).T).astype(np.float32)  # |sums| <= 64 K < 2^24
    wide = widen(ctx.matmul_bf16(bf16_dev(a), bf16_dev(bt), out_dtype=torch.float32))
    narrow = widen(ctx.matmul_bf16(bf16_dev(a), bf16_dev(bt)))
    ctx.check_device_status()
    assert same_bits(wide, exact)
    assert same_bits(narrow, oracle.round_bf16(exact))


@pytest.mark.parametrize("mkn", SHAPES)
def test_matmul_bf16_parity_with_fused_epilogue(ctx, oracle, mkn):
    import torch

    M, K, N = mkn
    a = oracle.round_bf16(si.uniform(602, 0, (M, K), -1, 1))
    bt = oracle.round_bf16(si.uniform(602, 1, (N, K), -1, 1))
    bias = si.normal(602, 2, (N,), 0, 2.0)
    ad, bd, biasd = bf16_dev(a), bf16_dev(bt), dev(bias)
    rows = np.arange(M) if M * K * N <= 600_000_000 else np.unique(np.linspace(0, M - 1, 257).astype(np.int64))
    # Elementwise bound for a stored result: one bfloat16 step of the value, plus the fp32 summation
    # error, which is absolute (about 2^-23 of the norm of the K terms, sqrt(K) / 3 here): where the
    # terms cancel to a value far below them, that error is many steps of the tiny result.
    def check_stored(got, want32):
        want = oracle.round_bf16(want32)
        assert np.all(np.abs(got - want) <= 2.0 ** -7 * np.abs(want) + 4e-6 * np.sqrt(K))
        assert np.count_nonzero(got != want) <= 0.02 * want.size
        assert np.all((got.view(np.uint32) & 0xFFFF) == 0)

    for act in ("none", "relu6"):
        want = oracle.bias_act(oracle.matmul(a[rows], bt, transpose_b=True), bias, act)
        wide = widen(ctx.matmul_bf16(ad, bd, bias=biasd, act=act, out_dtype=torch.float32))[rows]
        narrow = widen(ctx.matmul_bf16(ad, bd, bias=biasd, act=act))[rows]
        ctx.check_device_status()
        assert rel_fro(wide, want) <= 2e-5
        check_stored(narrow, want)
        if act == "relu6":
            assert narrow.min() >= 0 and narrow.max() <= 6
    # without a bias the rounding of the plain product is what is stored
    check_stored(widen(ctx.matmul_bf16(ad, bd))[rows], oracle.matmul(a[rows], bt, transpose_b=True))


PAIR_SHAPES = [
    (256, 64, 64),       # one pair tile, one k-block, 32 Bt rows per CTA
    (128, 128, 256),     # the odd CTA's rows are all outside the matrix
    (300, 104, 72),      # ragged in M, K and N
    (4100, 40, 264),     # a second tile along N with 8 live columns
    (520, 1024, 512),    # sixteen k-blocks: the stage ring wraps
    (20000, 256, 512),   # more tiles than SM pairs: persistent loop, accumulator stages reused
    (25088, 512, 512),   # pw7-pw11 of the 224 model at batch 128: the shape the planner gives to this kernel
]


@pytest.mark.parametrize("mkn", PAIR_SHAPES)
def test_matmul_bf16_pair_kernel(ctx, oracle, monkeypatch, mkn):
    """The CTA-pair kernel (forced on with TFJSB_GEMM_PAIR=1): exact on small integers, within the
    stored-result bound on random values, and bit-identical to the single-CTA kernel, which adds the
    same k-blocks in the same order."""
    M, K, N = mkn
    ai = bf16_dev(si.small_integers(603, 0, (M, K), -8, 8))
    bi = bf16_dev(si.small_integers(603, 1, (N, K), -8, 8))
    a = oracle.round_bf16(si.uniform(604, 0, (M, K), -1, 1))
    bt = oracle.round_bf16(si.uniform(604, 1, (N, K), -1, 1))
    bias = si.normal(604, 2, (N,), 0, 2.0)
    ad, bd, biasd = bf16_dev(a), bf16_dev(bt), dev(bias)
    monkeypatch.setenv("TFJSB_GEMM_PAIR", "1")
    exact = widen(ctx.matmul_bf16(ai, bi))
    pair = widen(ctx.matmul_bf16(ad, bd, bias=biasd, act="relu6"))
    monkeypatch.setenv("TFJSB_GEMM_PAIR", "0")
    single = widen(ctx.matmul_bf16(ad, bd, bias=biasd, act="relu6"))
    ctx.check_device_status()
    want_int = (widen(ai).astype(np.int64) @ widen(bi).astype(np.int64).T).astype(np.float32)
    assert same_bits(exact, oracle.round_bf16(want_int))
    assert same_bits(pair, single)
    rows = np.arange(M) if M * K * N <= 600_000_000 else np.unique(np.linspace(0, M - 1, 257).astype(np.int64))
    want = oracle.round_bf16(oracle.bias_act(oracle.matmul(a[rows], bt, transpose_b=True), bias, "relu6"))
    assert np.all(np.abs(pair[rows] - want) <= 2.0 ** -7 * np.abs(want) + 4e-6 * np.sqrt(K))
    assert np.count_nonzero(pair[rows] != want) <= 0.02 * want.size


def test_matmul_bf16_rejects_what_it_cannot_run(ctx, tfjsb):
    import torch

    a = torch.zeros(64, 36, dtype=torch.bfloat16, device="cuda")  # K = 36: row pitch 72 bytes
    bt = torch.zeros(32, 36, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(tfjsb.TfjsbError) as e:
        ctx.matmul_bf16(a, bt)
    assert e.value.status_name == "UNSUPPORTED"
    a = torch.zeros(64, 64, dtype=torch.bfloat16, device="cuda")
    bt = torch.zeros(36, 64, dtype=torch.bfloat16, device="cuda")  # N = 36
    with pytest.raises(tfjsb.TfjsbError) as e:
        ctx.matmul_bf16(a, bt)
    assert e.value.status_name == "UNSUPPORTED"
    with pytest.raises(TypeError):
        ctx.matmul_bf16(a.to(torch.float32), bt)
    # nothing to compute: no launch, no error
    before = ctx.launch_count
    empty = ctx.matmul_bf16(torch.zeros(0, 64, dtype=torch.bfloat16, device="cuda"), bt[:32].contiguous())
    assert tuple(empty.shape) == (0, 32) and ctx.launch_count == before


def narrow_model(ctx, layers, shape):
    ctx.set_math("bf16")
    try:
        return ctx.model(layers, shape)
    finally:
        ctx.set_math("tf32")


def check_logits(got_logits, got_probs, want_logits, want_probs, rel=1e-2, min_decided=1):
    decided = 0
    for i in range(want_logits.shape[0]):
        span = float(want_logits[i].max() - want_logits[i].min())
        tol = rel * span
        top = np.sort(want_logits[i])
        err = float(np.max(np.abs(got_logits[i] - want_logits[i])))
        assert err <= tol, f"image {i}: max logit error {err:.3e} > {tol:.3e}"
        if top[-1] - top[-2] >= 4 * tol:
            decided += 1
            assert int(got_logits[i].argmax()) == int(want_logits[i].argmax())
            assert int(got_probs[i].argmax()) == int(want_probs[i].argmax())
        assert abs(float(got_probs[i].astype(np.float64).sum()) - 1) <= 1e-5
    assert decided >= min_decided, f"only {decided} images with a clear top-1 in the oracle; pick another seed"


def test_small_model_every_layer(ctx, oracle):
    """A reduced model (alpha 0.25, 64x64 input, batch 3, 100 classes: the dense layer's width is not a
    multiple of 8, so it runs on the CUDA-core kernel): every layer's output against the oracle."""
    x, layers = si.config_mobilenet(0.25, 64, 3, seed=4243, classes=100)
    want = oracle.run_model(layers, x, keep_all=True, storage="bf16")
    model = narrow_model(ctx, layers, x.shape)
    model.set_keep_all(True)
    probs = host(model.run(dev(x)))
    ctx.check_device_status()
    assert model.launches_per_run == len(layers) == 30
    for i, layer in enumerate(layers):
        got = host(model.layer_output_f32(i)) if i < len(layers) - 1 else probs
        assert got.shape == want[i].shape, layer.name
        assert rel_fro(got, want[i]) <= 1e-2, f"layer {i} ({layer.name}) diverges: {rel_fro(got, want[i]):.3e}"
        if i < len(layers) - 2:  # what is stored is a bfloat16
            assert np.all((got.view(np.uint32) & 0xFFFF) == 0), layer.name
        if layer.act == "relu6":
            assert got.min() >= 0 and got.max() <= 6
    # the first layers see no accumulated noise: at most one bfloat16 step, on few elements
    for i in (0, 1, 2):
        steps = bf16_steps(host(model.layer_output_f32(i)), want[i])
        assert steps.max() <= 1 and np.count_nonzero(steps) <= 0.01 * steps.size, i
    check_logits(host(model.layer_output_f32(28)), probs, want[28], want[29])
    # ping-pong arena and keep-all buffers give the same bits
    model.set_keep_all(False)
    assert same_bits(host(model.run(dev(x))), probs)
    model.close()


def test_small_integer_model_is_bit_exact(ctx, oracle):
    """Small integers everywhere (inputs, filters, biases; sums below 2^8 where they are stored): both
    sides compute and store exact values."""
    x = si.small_integers(610, 0, (2, 13, 11, 3), -2, 2)
    layers = [
        si.Layer(kind="conv2d", filter_hw=(3, 3), strides=(2, 2), pad="same", act="relu6", out_channels=16,
                 filter=si.small_integers(610, 1, (3, 3, 3, 16), -1, 1), bias=si.small_integers(610, 2, (16,), -2, 2)),
        si.Layer(kind="depthwise_conv2d", filter_hw=(3, 3), strides=(1, 1), pad="same", act="relu6", out_channels=1,
                 filter=si.small_integers(610, 3, (3, 3, 16, 1), -1, 1), bias=si.small_integers(610, 4, (16,), -2, 2)),
        si.Layer(kind="conv2d", filter_hw=(1, 1), strides=(1, 1), pad="same", act="relu6", out_channels=24,
                 filter=si.small_integers(610, 5, (1, 1, 16, 24), -1, 1), bias=si.small_integers(610, 6, (24,), -2, 2)),
        si.Layer(kind="depthwise_conv2d", filter_hw=(3, 3), strides=(2, 2), pad="same", act="relu6", out_channels=1,
                 filter=si.small_integers(610, 7, (3, 3, 24, 1), -1, 1), bias=None),
        si.Layer(kind="conv2d", filter_hw=(1, 1), strides=(1, 1), pad="same", act="none", out_channels=8,
                 filter=si.small_integers(610, 8, (1, 1, 24, 8), -1, 1), bias=None),
    ]
    want = oracle.run_model(layers, x, keep_all=True, storage="bf16")
    assert all(np.array_equal(a, b) for a, b in zip(want, oracle.run_model(layers, x, keep_all=True)))
    model = narrow_model(ctx, layers, x.shape)
    model.set_keep_all(True)
    out = host(model.run(dev(x)))
    ctx.check_device_status()
    for i in range(len(layers) - 1):
        assert same_bits(host(model.layer_output_f32(i)), want[i]), i
    assert same_bits(out, want[-1])
    model.close()


FUSED_BLOCKS = [
    # N, H, W, C, Cout: depthwise 3x3 + pointwise as ONE kernel in the narrow format
    (2, 40, 52, 32, 64),     # one k-block per tile: the sixteen-epilogue-warp instance; ragged tiles (40 = 5 x 8, 52 = 3 x 16 + 4)
    (2, 24, 40, 128, 128),   # four k-blocks, weights resident in shared memory
    (1, 20, 24, 256, 256),   # eight k-blocks, weights streamed per tile
    (3, 9, 17, 64, 40),      # images barely larger than a tile, Cout not a power of two
]


def block_model(si_mod, seed, N, H, W, C, Cout, integers):
    """conv 3x3 (3 -> C) -> depthwise 3x3 -> pointwise (C -> Cout) -> global pool; the pair in the middle fuses."""
    L = si_mod.Layer
    layers = [L(kind="conv2d", filter_hw=(3, 3), strides=(1, 1), pad="same", act="relu6", out_channels=C, name="stem"),
              L(kind="depthwise_conv2d", filter_hw=(3, 3), strides=(1, 1), pad="same", act="relu6", out_channels=1, name="dw"),
              L(kind="conv2d", filter_hw=(1, 1), strides=(1, 1), pad="same", act="relu6", out_channels=Cout, name="pw"),
              L(kind="global_avg_pool", name="pool")]
    if integers:
        x = si_mod.small_integers(seed, 0, (N, H, W, 3), -2, 2)
        # sparse small filters keep every sum an integer below 2^8, which bfloat16 holds exactly
        layers[0].filter = si_mod.small_integers(seed, 1, (3, 3, 3, C), -1, 1)
        layers[0].bias = si_mod.small_integers(seed, 2, (C,), -1, 1)
        layers[1].filter = si_mod.small_integers(seed, 3, (3, 3, C, 1), -1, 1) * (si_mod.small_integers(seed, 4, (3, 3, C, 1), 0, 2) == 0)
        layers[1].bias = si_mod.small_integers(seed, 5, (C,), -1, 1)
        layers[2].filter = si_mod.small_integers(seed, 6, (1, 1, C, Cout), -1, 1) * (si_mod.small_integers(seed, 7, (1, 1, C, Cout), 0, 7) == 0)
        layers[2].bias = si_mod.small_integers(seed, 8, (Cout,), -1, 1)
    else:
        x = si_mod.uniform(seed, 0, (N, H, W, 3), -1, 1)
        si_mod.make_model_weights(layers, 3, seed)
    return x, layers


@pytest.mark.parametrize("case", FUSED_BLOCKS)
def test_fused_depthwise_pointwise_block_narrow(ctx, oracle, case):
    """The fused block kernel in the narrow format (bfloat16 patches in, depthwise result rounded to bfloat16 into
    the operand tile, TF32 multiplies of bfloat16 values, bfloat16 out): bit for bit on small integers, within the
    stored-result bars on random values, and against the same model run layer by layer."""
    N, H, W, C, Cout = case
    # small integers: every product, sum and stored value is exact on both sides
    x, layers = block_model(si, 620, N, H, W, C, Cout, integers=True)
    want = oracle.run_model(layers, x, keep_all=True, storage="bf16")
    assert all(np.array_equal(a, b) for a, b in zip(want, oracle.run_model(layers, x, keep_all=True)))
    assert np.abs(want[2]).max() > 0
    model = narrow_model(ctx, layers, x.shape)
    model.set_fusion("always")
    out = host(model.run(dev(x)))
    ctx.check_device_status()
    assert model.layer_kernels()[1:3] == ["dwpw_fused_kernel<false>", "(in the previous layer's kernel)"]
    assert model.launches_per_run == 3
    assert same_bits(host(model.layer_output_f32(2)), want[2])
    assert same_bits(out, want[3])
    model.close()
    # random values
    x, layers = block_model(si, 621, N, H, W, C, Cout, integers=False)
    want = oracle.run_model(layers, x, keep_all=True, storage="bf16")
    model = narrow_model(ctx, layers, x.shape)
    model.set_fusion("always")
    out = host(model.run(dev(x)))
    fused_pw = host(model.layer_output_f32(2))
    ctx.check_device_status()
    assert np.all((fused_pw.view(np.uint32) & 0xFFFF) == 0)
    assert rel_fro(fused_pw, want[2]) <= 1e-2
    assert fused_pw.min() >= 0 and fused_pw.max() <= 6
    assert rel_fro(out, want[3]) <= 5e-3
    # the pointwise layer on the input it actually saw: the oracle's pointwise layer applied to the oracle's
    # depthwise layer of the GPU's own first-layer output (one bfloat16 step plus the fp32 summation error)
    model.set_keep_all(True)
    model.run(dev(x))
    stem = host(model.layer_output_f32(0))
    unfused_pw = host(model.layer_output_f32(2))
    alone = oracle.run_model(layers[1:3], stem, keep_all=True, storage="bf16")
    alone_pw = oracle.round_bf16(alone[1])
    for got in (fused_pw, unfused_pw):
        assert rel_fro(got, alone_pw) <= 4e-3
        assert np.count_nonzero(np.abs(got - alone_pw) > 2.0 ** -6 * np.abs(alone_pw) + 2e-5 * np.abs(alone_pw).max()) <= 2e-3 * got.size
    model.close()


def test_depthwise_as_last_layer_narrow_writes_fp32(ctx, oracle):
    """A bfloat16-storage model hands its result back as fp32: a depthwise layer in last place runs on the
    pipelined kernel with bfloat16 patches and an fp32 store, without the rounding of a stored activation."""
    L = si.Layer
    x = si.small_integers(640, 0, (2, 15, 22, 3), -2, 2)
    layers = [L(kind="conv2d", filter_hw=(3, 3), strides=(1, 1), pad="same", act="relu6", out_channels=64, name="stem",
                filter=si.small_integers(640, 1, (3, 3, 3, 64), -1, 1), bias=si.small_integers(640, 2, (64,), -1, 1)),
              L(kind="depthwise_conv2d", filter_hw=(3, 3), strides=(1, 1), pad="same", act="none", out_channels=1, name="dw",
                filter=si.small_integers(640, 3, (3, 3, 64, 1), -2, 2), bias=si.small_integers(640, 4, (64,), -2, 2))]
    want = oracle.run_model(layers, x, keep_all=True, storage="bf16")
    model = narrow_model(ctx, layers, x.shape)
    out = host(model.run(dev(x)))
    ctx.check_device_status()
    assert model.layer_kernels()[1] == "depthwise3x3_tma_kernel"
    assert out.dtype == np.float32 and same_bits(out, want[1])
    # random values: sums that a bfloat16 could not hold come back unrounded
    x = si.uniform(641, 0, x.shape, -1, 1)
    si.make_model_weights(layers, 3, 641)
    model.close()
    model = narrow_model(ctx, layers, x.shape)
    model.set_keep_all(True)
    out = host(model.run(dev(x)))
    stem = host(model.layer_output_f32(0))
    alone = oracle.run_model(layers[1:2], stem, keep_all=True, storage="bf16")[0]
    assert rel_fro(out, alone) <= 1e-6
    assert np.any((out.view(np.uint32) & 0xFFFF) != 0)
    model.close()


NARROW_DEPTHWISE = [
    # N, H, W, C, stride: one case per instance of the pipelined depthwise kernel in the narrow format
    (2, 21, 37, 128, 1),   # 64-channel tiles, large stride-1 image, ragged tiles both ways
    (3, 13, 20, 64, 1),    # 9..14 rows: two tiles down
    (3, 7, 7, 192, 1),     # whole 7 x 7 image per tile, three channel blocks
    (2, 11, 6, 64, 1),     # narrow image taller than one tile
    (2, 29, 47, 64, 2),    # stride 2, 8-wide tiles
    (1, 40, 61, 128, 2),   # stride 2, 16-wide tiles
    (2, 21, 37, 40, 1),    # 32-channel tiles (channel count not a multiple of 64), partial channel block
    (3, 13, 20, 96, 1),
    (3, 7, 7, 40, 1),
    (2, 29, 47, 32, 2),
    (1, 40, 61, 48, 2),
]


@pytest.mark.parametrize("case", NARROW_DEPTHWISE)
def test_depthwise_pipelined_kernel_narrow(ctx, oracle, case):
    """conv 3x3 -> depthwise 3x3 -> global pool with bfloat16 storage; the depthwise layer runs on the bulk-copy
    pipelined kernel: bit for bit on small integers, and on random values against the oracle's depthwise layer
    applied to the GPU's own first-layer output (fp32 sums in another order, then one rounding to bfloat16)."""
    N, H, W, C, stride = case
    L = si.Layer

    def build(seed, integers):
        layers = [L(kind="conv2d", filter_hw=(3, 3), strides=(1, 1), pad="same", act="relu6", out_channels=C, name="stem"),
                  L(kind="depthwise_conv2d", filter_hw=(3, 3), strides=(stride, stride), pad="same", act="relu6", out_channels=1, name="dw"),
                  L(kind="global_avg_pool", name="pool")]
        if integers:
            x = si.small_integers(seed, 0, (N, H, W, 3), -2, 2)
            layers[0].filter = si.small_integers(seed, 1, (3, 3, 3, C), -1, 1)
            layers[0].bias = si.small_integers(seed, 2, (C,), -1, 1)
            layers[1].filter = si.small_integers(seed, 3, (3, 3, C, 1), -2, 2)
            layers[1].bias = si.small_integers(seed, 4, (C,), -2, 2)
        else:
            x = si.uniform(seed, 0, (N, H, W, 3), -1, 1)
            si.make_model_weights(layers, 3, seed)
        return x, layers

    x, layers = build(630, True)
    want = oracle.run_model(layers, x, keep_all=True, storage="bf16")
    assert all(np.array_equal(a, b) for a, b in zip(want[:2], oracle.run_model(layers, x, keep_all=True)[:2]))
    model = narrow_model(ctx, layers, x.shape)
    model.set_keep_all(True)
    model.run(dev(x))
    ctx.check_device_status()
    assert model.layer_kernels()[1] == "depthwise3x3_tma_kernel"
    assert same_bits(host(model.layer_output_f32(1)), want[1])
    model.close()

    x, layers = build(631, False)
    model = narrow_model(ctx, layers, x.shape)
    model.set_keep_all(True)
    model.run(dev(x))
    ctx.check_device_status()
    stem = host(model.layer_output_f32(0))
    got = host(model.layer_output_f32(1))
    alone = oracle.round_bf16(oracle.run_model(layers[1:2], stem, keep_all=True, storage="bf16")[0])
    assert got.shape == alone.shape
    assert np.all((got.view(np.uint32) & 0xFFFF) == 0)
    steps = bf16_steps(got, alone)
    assert steps.max() <= 1 and np.count_nonzero(steps) <= 0.01 * steps.size
    model.close()


def test_config3_mobilenet_025_128_narrow(ctx, oracle):
    x, layers = si.config_mobilenet(0.25, 128, 1, seed=si.CONFIG_SEEDS["mobilenet_025_128"])
    want = oracle.run_model(layers, x, keep_all=True, storage="bf16")
    model = narrow_model(ctx, layers, x.shape)
    model.set_keep_all(True)
    probs = host(model.run(dev(x)))
    ctx.check_device_status()
    for i in range(len(layers) - 1):
        got = host(model.layer_output_f32(i))
        assert rel_fro(got, want[i]) <= 1e-2, f"layer {i} diverges: {rel_fro(got, want[i]):.3e}"
    check_logits(host(model.layer_output_f32(28)), probs, want[28], want[29])
    model.close()


def test_config4_mobilenet_100_224_narrow_every_layer(ctx, oracle):
    """Config 4 (batch 1, 224 x 224, alpha 1.0) layer by layer: the full-size kernel instances the narrow mode's
    throughput rests on (the 32-channel first layer, the 2 x 2-tile depthwise at 112 x 112 and 56 x 56)."""
    x, layers = si.config_mobilenet(1.0, 224, 1, seed=si.CONFIG_SEEDS["mobilenet_100_224"])
    want = oracle.run_model(layers, x, keep_all=True, storage="bf16")
    model = narrow_model(ctx, layers, x.shape)
    model.set_keep_all(True)
    probs = host(model.run(dev(x)))
    ctx.check_device_status()
    for i, layer in enumerate(layers[:-1]):
        got = host(model.layer_output_f32(i))
        assert got.shape == want[i].shape, layer.name
        assert rel_fro(got, want[i]) <= 1e-2, f"layer {i} ({layer.name}) diverges: {rel_fro(got, want[i]):.3e}"
        if i < len(layers) - 2:
            assert np.all((got.view(np.uint32) & 0xFFFF) == 0), layer.name
    # Each of the first layers on its own: the oracle applied to the input the GPU layer actually read (its own
    # previous output), so that a one-step difference in an earlier layer, which a later sum can turn into
    # several steps of a small result, is not in the comparison.  What remains is one bfloat16 step of the value
    # plus the fp32 summation error (absolute, relative to the largest values of the layer), on few elements.
    prev = x
    for i in (0, 1, 2, 3, 4):
        got = host(model.layer_output_f32(i))
        alone = oracle.round_bf16(oracle.run_model([layers[i]], prev, storage="bf16"))
        assert np.all(np.abs(got - alone) <= 2.0 ** -7 * np.abs(alone) + 2e-6 * np.abs(alone).max()), layers[i].name
        assert np.count_nonzero(got != alone) <= 0.01 * got.size, layers[i].name
        prev = got
    steps = bf16_steps(host(model.layer_output_f32(0)), want[0])
    assert steps.max() <= 1 and np.count_nonzero(steps) <= 0.01 * steps.size
    check_logits(host(model.layer_output_f32(28)), probs, want[28], want[29])
    model.close()


def test_integer_model_full_width_first_layer_and_wide_depthwise(ctx, oracle):
    """Bit for bit on small integers through the kernel instances of the full-size model: a first layer with
    32 output channels on an odd-sized image, depthwise layers 57 and 61 pixels wide (stride 1 and 2: the
    2 x 2 and 1 x 2 register tiles meet a ragged right and bottom edge) and the pixel-packed 32-channel
    pointwise layer."""
    x = si.small_integers(611, 0, (2, 115, 121, 3), -2, 2)
    layers = [
        si.Layer(kind="conv2d", filter_hw=(3, 3), strides=(2, 2), pad="same", act="relu6", out_channels=32,
                 filter=si.small_integers(611, 1, (3, 3, 3, 32), -1, 1), bias=si.small_integers(611, 2, (32,), -2, 2)),
        si.Layer(kind="depthwise_conv2d", filter_hw=(3, 3), strides=(1, 1), pad="same", act="relu6", out_channels=1,
                 filter=si.small_integers(611, 3, (3, 3, 32, 1), -1, 1), bias=si.small_integers(611, 4, (32,), -2, 2)),
        si.Layer(kind="conv2d", filter_hw=(1, 1), strides=(1, 1), pad="same", act="relu6", out_channels=64,
                 filter=si.small_integers(611, 5, (1, 1, 32, 64), -1, 1), bias=si.small_integers(611, 6, (64,), -2, 2)),
        si.Layer(kind="depthwise_conv2d", filter_hw=(3, 3), strides=(2, 2), pad="same", act="relu6", out_channels=1,
                 filter=si.small_integers(611, 7, (3, 3, 64, 1), -1, 1), bias=None),
        si.Layer(kind="conv2d", filter_hw=(1, 1), strides=(1, 1), pad="same", act="none", out_channels=16,
                 filter=si.small_integers(611, 8, (1, 1, 64, 16), -1, 1), bias=None),
    ]
    want = oracle.run_model(layers, x, keep_all=True, storage="bf16")
    assert all(np.array_equal(a, b) for a, b in zip(want, oracle.run_model(layers, x, keep_all=True)))
    model = narrow_model(ctx, layers, x.shape)
    model.set_keep_all(True)
    out = host(model.run(dev(x)))
    ctx.check_device_status()
    assert want[0].shape == (2, 58, 61, 32) and want[3].shape == (2, 29, 31, 64)
    for i in range(len(layers) - 1):
        assert same_bits(host(model.layer_output_f32(i)), want[i]), i
    assert same_bits(out, want[-1])
    model.close()


def test_config5_mobilenet_100_224_batch128_narrow_all_images(ctx, oracle, tfjsb):
    """The benchmark's model and batch in the narrow-storage mode, every image against the oracle; top-1 is
    compared on every image whose oracle margin allows, which holds for all 128 with this seed."""
    import torch

    x, layers = si.config_mobilenet(1.0, 224, 128, seed=si.CONFIG_SEEDS["mobilenet_100_224_b128"])
    model = narrow_model(ctx, layers, x.shape)
    xd = dev(x)
    probs = model.run(xd)
    logits = host(model.layer_output_f32(model.n_layers - 2))
    ctx.check_device_status()
    probs = host(probs)
    assert probs.shape == (128, 1000)
    want = oracle.run_model(layers, x, keep_all=True, storage="bf16")
    check_logits(logits, probs, want[-2], want[-1], min_decided=128)
    # a bfloat16 layer cannot be viewed as fp32
    with pytest.raises(tfjsb.TfjsbError) as e:
        model.layer_output(3)
    assert e.value.status_name == "UNSUPPORTED"
    # host-buffer entry point (sliced, graph replays) and whole-batch graph replay: same bits
    hin = torch.from_numpy(x).pin_memory()
    hout = torch.empty(128, 1000).pin_memory()
    model.run_host(hin, hout)
    assert same_bits(hout.numpy(), probs)
    model.run_host(hin, hout.zero_())
    assert same_bits(hout.numpy(), probs)
    out2 = torch.empty(128, 1000, device="cuda")
    model.set_graph(True)
    model.run(xd, out=out2)
    model.run(xd, out=out2)
    assert same_bits(host(out2), probs)
    model.close()


def test_narrow_mode_rejects_layers_it_does_not_have(ctx, tfjsb):
    x, layers = si.config_mobilenet(0.25, 32, 1, seed=5, classes=16)
    with pytest.raises(tfjsb.TfjsbError) as e:
        narrow_model(ctx, layers[1:], (1, 16, 16, 8))  # starts with a depthwise layer
    assert e.value.status_name == "UNSUPPORTED"
    dilated = si.mobilenet_v1_layers(0.25, 16, output_stride=16)
    si.make_model_weights(dilated, 3, 5)
    with pytest.raises(tfjsb.TfjsbError) as e:
        narrow_model(ctx, dilated, x.shape)  # dilated depthwise layers
    assert e.value.status_name == "UNSUPPORTED"
    # the context is left in its default mode and still builds the default model
    ctx.model(layers, x.shape).close()

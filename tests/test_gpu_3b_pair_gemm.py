"""GPU parity of the CTA-pair tensor-core GEMM (tcgen05 cta_group::2: two CTAs share a 256-row tile).

The library picks this kernel by shape (long K loops, wide N, enough tiles for every SM pair); the
environment variable TFJSB_GEMM_PAIR forces it on (1) or off (0) when the plan is made, which lets the
same shape run through both kernels.  Tolerances as for the single-CTA kernel: bit-identical on small
integers (all products and partial sums exact), relative Frobenius error <= 5e-3 against the exact
oracle, <= 2e-5 against the oracle with truncated TF32 operands.  Both kernels add the k-blocks in the
same order into fp32 accumulators, so on the same inputs they must agree bit for bit.
"""
import numpy as np
import pytest

import seeded_inputs as si
from helpers import dev, host, rel_fro, same_bits

pytestmark = pytest.mark.gpu

TF32_TOL = 5e-3
MATCHED_TOL = 2e-5

PAIR_SHAPES = [
    # M, K, N
    (256, 32, 64),        # one pair tile, one k-block, 32 Bt rows per CTA
    (256, 64, 256),       # full-width tile, two k-blocks
    (128, 128, 256),      # the odd CTA's rows are all outside the matrix
    (300, 100, 72),       # ragged in M, K and N
    (4100, 36, 260),      # N just above one 256 tile: a second tile with 4 live columns
    (520, 512, 512),      # sixteen k-blocks: the stage ring wraps
    (1000, 1024, 1000),   # N tail inside a 32-column chunk, 32 k-blocks
    (20000, 256, 512),    # more tiles than SM pairs: persistent loop, accumulator stages reused
    (6272, 512, 1024),    # pw12 of the 224 model at batch 128: last 256-row tile half empty
]


@pytest.fixture
def pair_on(monkeypatch):
    monkeypatch.setenv("TFJSB_GEMM_PAIR", "1")


@pytest.mark.parametrize("mkn", PAIR_SHAPES)
def test_pair_gemm_integer_exact(ctx, pair_on, mkn):
    M, K, N = mkn
    a = si.small_integers(321, 0, (M, K), -8, 8)
    b = si.small_integers(321, 1, (K, N), -8, 8)
    got = host(ctx.matmul(dev(a), dev(b)))
    ctx.check_device_status()
    want = (a.astype(np.int64) @ b.astype(np.int64)).astype(np.float32)
    assert same_bits(got, want)


@pytest.mark.parametrize("mkn", PAIR_SHAPES)
def test_pair_gemm_parity(ctx, oracle, pair_on, mkn):
    M, K, N = mkn
    a = si.uniform(322, 0, (M, K), -1, 1)
    b = si.uniform(322, 1, (K, N), -1, 1)
    got = host(ctx.matmul(dev(a), dev(b)))
    ctx.check_device_status()
    if M * K * N <= 600_000_000:
        assert rel_fro(got, oracle.matmul(a, b)) <= TF32_TOL
        assert rel_fro(got, oracle.matmul(a, b, operand="tf32_rz")) <= MATCHED_TOL
    else:  # sampled rows, each computed one by one by the oracle
        rows = np.unique(np.linspace(0, M - 1, 257).astype(np.int64))
        assert rel_fro(got[rows], oracle.matmul(a[rows], b)) <= TF32_TOL
        assert rel_fro(got[rows], oracle.matmul(a[rows], b, operand="tf32_rz")) <= MATCHED_TOL


@pytest.mark.parametrize("act", ["none", "relu6"])
def test_pair_gemm_fused_epilogue_and_single_cta_agreement(ctx, oracle, monkeypatch, act):
    # pw7 of the 224 model at batch 8: [8,14,14,512] x [1,1,512,512] + bias, both kernels
    x = si.uniform(323, 0, (8, 14, 14, 512), 0, 6)
    f = si.normal(323, 1, (1, 1, 512, 512), 0, float(np.sqrt(2.0 / 512)))
    b = si.normal(323, 2, (512,), 0, 0.5)
    monkeypatch.setenv("TFJSB_GEMM_PAIR", "1")
    pair = host(ctx.conv2d(dev(x), dev(f), bias=dev(b), act=act))
    monkeypatch.setenv("TFJSB_GEMM_PAIR", "0")
    single = host(ctx.conv2d(dev(x), dev(f), bias=dev(b), act=act))
    ctx.check_device_status()
    assert rel_fro(pair, oracle.conv2d(x, f, bias=b, act=act)) <= TF32_TOL
    assert same_bits(pair, single)


def test_pair_gemm_default_choice_and_determinism(ctx, monkeypatch):
    # pw7..pw11 of the 224 model at batch 128 ([25088,512] x [512,512]): whichever kernel the planner
    # takes by itself, forcing the pair kernel must give the same bits, and so must repeating the call.
    monkeypatch.delenv("TFJSB_GEMM_PAIR", raising=False)
    a = dev(si.uniform(324, 0, (25088, 512), -1, 1))
    b = dev(si.uniform(324, 1, (512, 512), -1, 1))
    default = host(ctx.matmul(a, b))
    monkeypatch.setenv("TFJSB_GEMM_PAIR", "1")
    forced = host(ctx.matmul(a, b))
    again = host(ctx.matmul(a, b))
    ctx.check_device_status()
    assert same_bits(default, forced) and same_bits(forced, again)

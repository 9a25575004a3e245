"""The benchmark's algorithmic-work accounting (host arithmetic only) against hand-derived figures.

The roofline fractions the benchmark prints divide by these byte and flop counts, so a slip here would
flatter or slander every kernel.  Figures for MobileNet v1 1.0 at 224 x 224, batch 128: each tensor read
or written exactly once; 4 bytes per value with fp32 storage; with narrow storage 2 bytes per filter
and activation value, 4 for the model input, biases, logits and probabilities.
"""
import importlib.util
import os

import pytest

import seeded_inputs as si

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def bench():
    spec = importlib.util.spec_from_file_location("bench_module", os.path.join(ROOT, "bench.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    return mod


def test_fp32_accounting_matches_hand_figures(bench, oracle):
    layers = si.mobilenet_v1_layers(1.0, 1000)
    rows = {r["name"]: r for r in bench.layer_work(layers, (128, 224, 224, 3), oracle.window_geometry)}
    assert len(rows) == 30
    # stem: [128,224,224,3] -> [128,112,112,32], 3x3x3x32 filter
    px = 128 * 112 * 112
    assert rows["stem"]["flops"] == 2 * px * 32 * 27
    assert rows["stem"]["bytes"] == 4 * (128 * 224 * 224 * 3 + 27 * 32 + 32 + px * 32)
    # pw7: [25088, 512] x [512, 512]
    assert rows["pw7"]["flops"] == 2 * 25088 * 512 * 512
    assert rows["pw7"]["bytes"] == 4 * (25088 * 512 + 512 * 512 + 512 + 25088 * 512)
    # dw2: stride 2, 64 channels, 112 -> 56: 18 flop per output, input read once
    assert rows["dw2"]["flops"] == 18 * 128 * 56 * 56 * 64
    assert rows["dw2"]["bytes"] == 4 * (128 * 112 * 112 * 64 + 9 * 64 + 64 + 128 * 56 * 56 * 64)
    total_flops = sum(r["flops"] for r in rows.values())
    assert abs(total_flops / 128 - 1.138e9) < 5e6  # the model's ~569 M multiply-adds per image


def test_narrow_accounting_halves_what_is_stored_narrow(bench, oracle):
    layers = si.mobilenet_v1_layers(1.0, 1000)
    wide = bench.layer_work(layers, (128, 224, 224, 3), oracle.window_geometry)
    narrow = bench.narrow_layer_work(layers, (128, 224, 224, 3), oracle.window_geometry)
    assert [r["name"] for r in narrow] == [r["name"] for r in wide]
    by = {r["name"]: r for r in narrow}
    px = 128 * 112 * 112
    # the first layer reads the fp32 image and writes bfloat16
    assert by["stem"]["bytes"] == 4 * 128 * 224 * 224 * 3 + 2 * 27 * 32 + 4 * 32 + 2 * px * 32
    # a middle layer: everything but the bias is two bytes
    assert by["pw7"]["bytes"] == 2 * (25088 * 512 + 512 * 512 + 25088 * 512) + 4 * 512
    assert by["dw2"]["bytes"] == 2 * (128 * 112 * 112 * 64 + 9 * 64 + 128 * 56 * 56 * 64) + 4 * 64
    # the dense layer reads bfloat16 and writes fp32 logits; softmax is fp32 in and out
    assert by["dense"]["bytes"] == 2 * (128 * 1024 + 1024 * 1000) + 4 * 1000 + 4 * 128 * 1000
    assert by["softmax"]["bytes"] == 8 * 128 * 1000
    for w, n in zip(wide, narrow):
        assert n["flops"] == w["flops"]
        assert n["bytes"] <= w["bytes"]
    assert by["pw7"]["tensor"] and by["dense"]["tensor"] and not by["dw2"]["tensor"] and not by["stem"]["tensor"]


def test_roofline_bound_of_the_kernels_the_library_names(bench):
    """The compute leg of a row's roofline uses the tensor-core peak exactly for the kernels that run on
    the tensor cores: a GEMM kernel left off that list would be judged against the CUDA-core peak and read
    several times above its roofline."""
    peaks = {"hbm_gbs": 6500.0, "bf16_tflops": 1600.0, "bf16_tflops_sustained": 1400.0}
    pw7 = dict(name="pw7", flops=2 * 25088 * 512 * 512, bytes=4 * (2 * 25088 * 512 + 512 * 512 + 512), units=25088 * 512)
    for kernel in ("gemm_pair_kernel<false>", "gemm_pair_kernel<true>", "gemm_tf32_kernel<false>", "gemm_tf32_kernel<true>",
                   "gemm_tf32_splitk_kernel", "gemm_bf16_kernel", "dwpw_fused_kernel<false>", "dwpw_fused_kernel<true, true>"):
        (row,) = bench.roofline_rows([dict(pw7, kernel=kernel)], [0.030], peaks, fp32_tflops=75.0)
        assert row["bound"] == "tensor", kernel
        assert abs(row["roofline_us"] - pw7["flops"] / 800e12 * 1e6) < 1e-6, kernel
        assert row["frac"] < 1.0
    for kernel in ("gemm_fp32_kernel", "conv2d_fp32_kernel"):
        (row,) = bench.roofline_rows([dict(pw7, kernel=kernel)], [0.300], peaks, fp32_tflops=75.0)
        assert row["bound"] == "alu", kernel
    dw = dict(name="dw7", flops=18 * 25088 * 512, bytes=4 * (2 * 25088 * 512 + 10 * 512), units=25088 * 512)
    (row,) = bench.roofline_rows([dict(dw, kernel="depthwise3x3_tma_kernel")], [0.020], peaks, fp32_tflops=75.0)
    assert row["bound"] == "hbm"

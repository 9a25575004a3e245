"""CPU-side checks of the boundary: the shared library builds, loads without a GPU, exports
every symbol include/tfjsb.h declares, and its host-only arithmetic agrees with the oracle."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def pkg():
    import paper_1901_05350_b200 as p

    return p


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "tfjsb.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(tfjsb_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(pkg):
    declared = _declared_symbols()
    assert len(declared) >= 20
    for name in declared:
        assert hasattr(pkg.lib, name), f"{name} is declared in tfjsb.h but not exported"
    assert sorted(pkg.EXPORTS) == declared


def test_window_out_shape_matches_golden_table_and_oracle(pkg, oracle):
    golden = os.path.join(ROOT, "tests", "golden", "window_geometry.txt")
    for line in open(golden):
        if line.startswith("#") or not line.strip():
            continue
        in_, k, s, d, pad, out, before, after = line.split()
        got = pkg.window_out_shape(int(in_), int(k), int(s), int(d), pad)
        assert got == (int(out), int(before), int(after))
    for in_ in range(1, 40):
        for k in (1, 2, 3, 5):
            for s in (1, 2, 3):
                for d in (1, 2):
                    for pad in ("same", "valid"):
                        try:
                            want = oracle.window_geometry(in_, k, s, d, pad)
                        except ValueError:
                            with pytest.raises(pkg.TfjsbError) as err:
                                pkg.window_out_shape(in_, k, s, d, pad)
                            assert err.value.status_name == "SHAPE"
                            continue
                        assert pkg.window_out_shape(in_, k, s, d, pad) == want


def test_no_gpu_means_a_loud_failure_not_a_fallback(pkg):
    import torch

    if torch.cuda.is_available():
        pytest.skip("a CUDA device is present")
    with pytest.raises(RuntimeError):
        pkg.Context(0)
    handle = ctypes.c_void_p()
    assert pkg.lib.tfjsb_init(0, ctypes.byref(handle)) == 4  # TFJSB_ERR_CUDA
    assert not handle.value


def test_null_context_is_rejected(pkg):
    assert pkg.lib.tfjsb_set_math(None, 0) == 1
    assert pkg.lib.tfjsb_matmul(None, None, None, 0, 0, None, None) == 1
    assert pkg.lib.tfjsb_run_model(None, None, None, None) == 1
    assert pkg.lib.tfjsb_launch_count(None) == -1


def test_product_path_never_imports_the_oracle():
    pkg_dir = os.path.join(ROOT, "paper_1901_05350_b200")
    for base, _, files in os.walk(pkg_dir):
        if "_build" in base:
            continue
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h", ".cpp")):
                text = open(os.path.join(base, f)).read()
                assert "oracle" not in text.lower(), f"{f} mentions the oracle"
    orc = open(os.path.join(ROOT, "oracle", "__init__.py")).read() + open(
        os.path.join(ROOT, "oracle", "tfjs_ops_oracle.cpp")).read()
    assert "paper_1901_05350_b200" not in orc and "tfjsb" not in orc

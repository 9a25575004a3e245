"""Python face of the CPU oracle (test infrastructure only; never on the product path).

The arithmetic lives in `tfjs_ops_oracle.cpp` (plain loops, double accumulation, one
rounding to fp32).  This file compiles it with g++ on first use, marshals numpy arrays to
it, and chains the ops of a layer list (`run_model`).  Nothing here imports, links or
calls the CUDA library, and the CUDA library never reaches this package.

Only the test-suite, the smoke check and the benchmark's cpu-baseline leg may import it.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import List, Optional, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "tfjs_ops_oracle.cpp")
_LIB = os.path.join(_HERE, "libtfjs_ops_oracle.so")

PAD = {"valid": 0, "same": 1}
ACT = {"none": 0, "relu": 1, "relu6": 2}
OPERAND = {"fp32": 0, "tf32_rna": 1, "tf32_rz": 2}

_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle into a shared library beside its source (g++, OpenMP, no fp contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["g++", "-O2", "-fopenmp", "-ffp-contract=off", "-fno-fast-math", "-shared", "-fPIC",
               "-o", _LIB, _SRC]
        subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        i32, i64, fp = ctypes.c_int, ctypes.c_int64, ctypes.c_void_p
        ip = ctypes.POINTER(ctypes.c_int)
        lib.orc_set_threads.argtypes = [i32]
        lib.orc_get_threads.restype = i32
        lib.orc_window_geometry.argtypes = [i32, i32, i32, i32, i32, ip, ip, ip]
        lib.orc_matmul.argtypes = [fp, fp, i64, i64, i64, i32, i32, fp, i32]
        lib.orc_conv2d.argtypes = [fp, i64, i32, i32, i32, fp, i32, i32, i32, i32, i32, i32, i32, i32, fp, i32,
                                   fp, i32]
        lib.orc_depthwise_conv2d.argtypes = [fp, i64, i32, i32, i32, fp, i32, i32, i32, i32, i32, i32, i32, i32,
                                             fp, i32, fp]
        lib.orc_bias_act.argtypes = [fp, i64, i64, fp, i32, fp]
        lib.orc_avg_pool.argtypes = [fp, i64, i32, i32, i32, i32, i32, i32, i32, i32, fp]
        lib.orc_softmax.argtypes = [fp, i64, i64, fp]
        lib.orc_max_pool.argtypes = [fp, i64, i32, i32, i32, i32, i32, i32, i32, i32, fp]
        lib.orc_binary.argtypes = [i32, fp, fp, i64, i64, fp]
        conv_grad = [fp, i64, i32, i32, i32, fp, i32, i32, i32, i32, i32, i32, i32, i32, fp]
        lib.orc_conv2d_backprop_input.argtypes = conv_grad + [i32]
        lib.orc_conv2d_backprop_filter.argtypes = conv_grad + [i32]
        lib.orc_depthwise_backprop_input.argtypes = conv_grad
        lib.orc_depthwise_backprop_filter.argtypes = conv_grad
        lib.orc_act_backprop.argtypes = [fp, fp, i64, i32, fp]
        lib.orc_bias_backprop.argtypes = [fp, i64, i64, fp]
        _lib = lib
    return _lib


def _f32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float32)


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def set_threads(n: int) -> None:
    _load().orc_set_threads(int(n))


def get_threads() -> int:
    return int(_load().orc_get_threads())


def window_geometry(size: int, k: int, stride: int, dilation: int, pad: str) -> Tuple[int, int, int]:
    """(out, pad_before, pad_after) of one spatial dimension; raises on an impossible window."""
    o, b, a = ctypes.c_int(), ctypes.c_int(), ctypes.c_int()
    rc = _load().orc_window_geometry(size, k, stride, dilation, PAD[pad], ctypes.byref(o), ctypes.byref(b),
                                     ctypes.byref(a))
    if rc:
        raise ValueError(f"no output for in={size} k={k} s={stride} d={dilation} pad={pad}")
    return o.value, b.value, a.value


def matmul(a, b, transpose_a: bool = False, transpose_b: bool = False, operand: str = "fp32") -> np.ndarray:
    a, b = _f32(a), _f32(b)
    if a.ndim != 2 or b.ndim != 2:
        raise ValueError("matmul takes rank-2 tensors")
    M, K = (a.shape[1], a.shape[0]) if transpose_a else a.shape
    Kb, N = (b.shape[1], b.shape[0]) if transpose_b else b.shape
    if K != Kb:
        raise ValueError(f"inner dimensions differ: {K} vs {Kb}")
    c = np.empty((M, N), dtype=np.float32)
    rc = _load().orc_matmul(_ptr(a), _ptr(b), M, K, N, int(transpose_a), int(transpose_b), _ptr(c),
                            OPERAND[operand])
    if rc:
        raise RuntimeError(f"orc_matmul failed ({rc})")
    return c


def conv2d(x, f, strides=(1, 1), pad="same", dilations=(1, 1), bias=None, act="none",
           operand: str = "fp32") -> np.ndarray:
    x, f = _f32(x), _f32(f)
    bias = None if bias is None else _f32(bias)
    N, H, W, Cin = x.shape
    fh, fw, fc, Cout = f.shape
    if fc != Cin:
        raise ValueError(f"filter has {fc} input channels, x has {Cin}")
    if bias is not None and bias.shape != (Cout,):
        raise ValueError("bias length must equal Cout")
    Ho, _, _ = window_geometry(H, fh, strides[0], dilations[0], pad)
    Wo, _, _ = window_geometry(W, fw, strides[1], dilations[1], pad)
    y = np.empty((N, Ho, Wo, Cout), dtype=np.float32)
    rc = _load().orc_conv2d(_ptr(x), N, H, W, Cin, _ptr(f), fh, fw, Cout, strides[0], strides[1], PAD[pad],
                            dilations[0], dilations[1], _ptr(bias), ACT[act], _ptr(y), OPERAND[operand])
    if rc:
        raise RuntimeError(f"orc_conv2d failed ({rc})")
    return y


def depthwise_conv2d(x, f, strides=(1, 1), pad="same", dilations=(1, 1), bias=None, act="none") -> np.ndarray:
    x, f = _f32(x), _f32(f)
    bias = None if bias is None else _f32(bias)
    N, H, W, C = x.shape
    fh, fw, fc, mult = f.shape
    if fc != C:
        raise ValueError(f"filter has {fc} channels, x has {C}")
    if bias is not None and bias.shape != (C * mult,):
        raise ValueError("bias length must equal C*multiplier")
    Ho, _, _ = window_geometry(H, fh, strides[0], dilations[0], pad)
    Wo, _, _ = window_geometry(W, fw, strides[1], dilations[1], pad)
    y = np.empty((N, Ho, Wo, C * mult), dtype=np.float32)
    rc = _load().orc_depthwise_conv2d(_ptr(x), N, H, W, C, _ptr(f), fh, fw, mult, strides[0], strides[1],
                                      PAD[pad], dilations[0], dilations[1], _ptr(bias), ACT[act], _ptr(y))
    if rc:
        raise RuntimeError(f"orc_depthwise_conv2d failed ({rc})")
    return y


def bias_act(x, bias=None, act="none") -> np.ndarray:
    x = _f32(x)
    bias = None if bias is None else _f32(bias)
    C = x.shape[-1]
    if bias is not None and bias.shape != (C,):
        raise ValueError("bias length must equal the last dimension")
    y = np.empty_like(x)
    rc = _load().orc_bias_act(_ptr(x), x.size // C if C else 0, C, _ptr(bias), ACT[act], _ptr(y))
    if rc:
        raise RuntimeError(f"orc_bias_act failed ({rc})")
    return y


def avg_pool(x, filter_size, strides, pad="valid") -> np.ndarray:
    x = _f32(x)
    N, H, W, C = x.shape
    Ho, _, _ = window_geometry(H, filter_size[0], strides[0], 1, pad)
    Wo, _, _ = window_geometry(W, filter_size[1], strides[1], 1, pad)
    y = np.empty((N, Ho, Wo, C), dtype=np.float32)
    rc = _load().orc_avg_pool(_ptr(x), N, H, W, C, filter_size[0], filter_size[1], strides[0], strides[1],
                              PAD[pad], _ptr(y))
    if rc:
        raise RuntimeError(f"orc_avg_pool failed ({rc})")
    return y


def max_pool(x, filter_size, strides, pad="valid") -> np.ndarray:
    x = _f32(x)
    N, H, W, C = x.shape
    Ho, _, _ = window_geometry(H, filter_size[0], strides[0], 1, pad)
    Wo, _, _ = window_geometry(W, filter_size[1], strides[1], 1, pad)
    y = np.empty((N, Ho, Wo, C), dtype=np.float32)
    rc = _load().orc_max_pool(_ptr(x), N, H, W, C, filter_size[0], filter_size[1], strides[0], strides[1],
                              PAD[pad], _ptr(y))
    if rc:
        raise RuntimeError(f"orc_max_pool failed ({rc})")
    return y


BINARY_OP = {"add": 0, "sub": 1, "mul": 2}


def binary(op: str, a, b) -> np.ndarray:
    """a op b, elementwise; b has a's shape or is a vector of a's last dimension."""
    a, b = _f32(a), _f32(b)
    if b.shape != a.shape and b.shape != (a.shape[-1],):
        raise ValueError("b must have a's shape or be a vector of a's last dimension")
    out = np.empty_like(a)
    rc = _load().orc_binary(BINARY_OP[op], _ptr(a), _ptr(b), a.size, b.size, _ptr(out))
    if rc:
        raise RuntimeError(f"orc_binary failed ({rc})")
    return out


def batch_matmul(a, b, transpose_a: bool = False, transpose_b: bool = False, operand: str = "fp32") -> np.ndarray:
    """Rank-3 matMul: one rank-2 product per leading index."""
    a, b = _f32(a), _f32(b)
    if a.ndim != 3 or b.ndim != 3 or a.shape[0] != b.shape[0]:
        raise ValueError("batch_matmul takes rank-3 tensors with equal leading dimensions")
    return np.stack([matmul(a[i], b[i], transpose_a, transpose_b, operand) for i in range(a.shape[0])])


def _grad_geometry(x_shape, fh, fw, strides, pad, dilations, dy_shape, out_channels):
    N, H, W, _ = x_shape
    Ho, _, _ = window_geometry(H, fh, strides[0], dilations[0], pad)
    Wo, _, _ = window_geometry(W, fw, strides[1], dilations[1], pad)
    if tuple(dy_shape) != (N, Ho, Wo, out_channels):
        raise ValueError(f"dy has shape {tuple(dy_shape)}, the forward output has {(N, Ho, Wo, out_channels)}")


def conv2d_backprop_input(x_shape, f, dy, strides=(1, 1), pad="same", dilations=(1, 1), operand: str = "fp32") -> np.ndarray:
    """Gradient of conv2d with respect to its input: the adjoint of x -> conv2d(x, f) applied to dy."""
    f, dy = _f32(f), _f32(dy)
    N, H, W, Cin = (int(v) for v in x_shape)
    fh, fw, fc, Cout = f.shape
    if fc != Cin:
        raise ValueError(f"filter has {fc} input channels, x has {Cin}")
    _grad_geometry(x_shape, fh, fw, strides, pad, dilations, dy.shape, Cout)
    dx = np.empty((N, H, W, Cin), dtype=np.float32)
    rc = _load().orc_conv2d_backprop_input(_ptr(dy), N, H, W, Cin, _ptr(f), fh, fw, Cout, strides[0], strides[1], PAD[pad],
                                           dilations[0], dilations[1], _ptr(dx), OPERAND[operand])
    if rc:
        raise RuntimeError(f"orc_conv2d_backprop_input failed ({rc})")
    return dx


def conv2d_backprop_filter(x, filter_shape, dy, strides=(1, 1), pad="same", dilations=(1, 1), operand: str = "fp32") -> np.ndarray:
    """Gradient of conv2d with respect to its filter [fh, fw, Cin, Cout]."""
    x, dy = _f32(x), _f32(dy)
    N, H, W, Cin = x.shape
    fh, fw, fc, Cout = (int(v) for v in filter_shape)
    if fc != Cin:
        raise ValueError(f"filter has {fc} input channels, x has {Cin}")
    _grad_geometry(x.shape, fh, fw, strides, pad, dilations, dy.shape, Cout)
    df = np.empty((fh, fw, Cin, Cout), dtype=np.float32)
    rc = _load().orc_conv2d_backprop_filter(_ptr(x), N, H, W, Cin, _ptr(dy), fh, fw, Cout, strides[0], strides[1], PAD[pad],
                                            dilations[0], dilations[1], _ptr(df), OPERAND[operand])
    if rc:
        raise RuntimeError(f"orc_conv2d_backprop_filter failed ({rc})")
    return df


def depthwise_conv2d_backprop_input(x_shape, f, dy, strides=(1, 1), pad="same", dilations=(1, 1)) -> np.ndarray:
    f, dy = _f32(f), _f32(dy)
    N, H, W, C = (int(v) for v in x_shape)
    fh, fw, fc, mult = f.shape
    if fc != C:
        raise ValueError(f"filter has {fc} channels, x has {C}")
    _grad_geometry(x_shape, fh, fw, strides, pad, dilations, dy.shape, C * mult)
    dx = np.empty((N, H, W, C), dtype=np.float32)
    rc = _load().orc_depthwise_backprop_input(_ptr(dy), N, H, W, C, _ptr(f), fh, fw, mult, strides[0], strides[1], PAD[pad],
                                              dilations[0], dilations[1], _ptr(dx))
    if rc:
        raise RuntimeError(f"orc_depthwise_backprop_input failed ({rc})")
    return dx


def depthwise_conv2d_backprop_filter(x, filter_shape, dy, strides=(1, 1), pad="same", dilations=(1, 1)) -> np.ndarray:
    x, dy = _f32(x), _f32(dy)
    N, H, W, C = x.shape
    fh, fw, fc, mult = (int(v) for v in filter_shape)
    if fc != C:
        raise ValueError(f"filter has {fc} channels, x has {C}")
    _grad_geometry(x.shape, fh, fw, strides, pad, dilations, dy.shape, C * mult)
    df = np.empty((fh, fw, C, mult), dtype=np.float32)
    rc = _load().orc_depthwise_backprop_filter(_ptr(x), N, H, W, C, _ptr(dy), fh, fw, mult, strides[0], strides[1], PAD[pad],
                                               dilations[0], dilations[1], _ptr(df))
    if rc:
        raise RuntimeError(f"orc_depthwise_backprop_filter failed ({rc})")
    return df


def act_backprop(y, dy, act="none") -> np.ndarray:
    """Gradient through y = act(z): dy where the activation passed z through (relu: y > 0; relu6: 0 < y < 6), else 0."""
    y, dy = _f32(y), _f32(dy)
    if y.shape != dy.shape:
        raise ValueError("y and dy must have one shape")
    dz = np.empty_like(y)
    rc = _load().orc_act_backprop(_ptr(y), _ptr(dy), y.size, ACT[act], _ptr(dz))
    if rc:
        raise RuntimeError(f"orc_act_backprop failed ({rc})")
    return dz


def bias_backprop(dz) -> np.ndarray:
    """Gradient of a bias added along the last dimension: the sum of dz over every other dimension."""
    dz = _f32(dz)
    C = dz.shape[-1]
    db = np.empty((C,), dtype=np.float32)
    rc = _load().orc_bias_backprop(_ptr(dz), dz.size // C, C, _ptr(db))
    if rc:
        raise RuntimeError(f"orc_bias_backprop failed ({rc})")
    return db


def softmax(x) -> np.ndarray:
    x = _f32(x)
    cols = x.shape[-1]
    y = np.empty_like(x)
    rc = _load().orc_softmax(_ptr(x), x.size // cols, cols, _ptr(y))
    if rc:
        raise RuntimeError(f"orc_softmax failed ({rc})")
    return y


def round_bf16(x) -> np.ndarray:
    """Each fp32 value rounded to the nearest bfloat16 (8 significand bits, ties to even), returned as
    fp32.  Infinities stay, finite values beyond the largest bfloat16 become infinite, NaN stays NaN.

    This is the 16-bit storage format of the narrow-storage mode (the paper's 16-bit float textures,
    Sec. 4.1.3, carried over to the format this hardware's tensor cores read).
    """
    x = _f32(x)
    u = x.view(np.uint32).astype(np.uint64)
    kept_lsb = (u >> np.uint64(16)) & np.uint64(1)
    r = (u + np.uint64(0x7FFF) + kept_lsb) & np.uint64(0xFFFF0000)
    out = r.astype(np.uint32).view(np.float32).reshape(x.shape)
    return np.where(np.isnan(x), np.float32(np.nan), out).astype(np.float32)


def run_model(layers: Sequence, x, operand: str = "fp32", keep_all: bool = False, storage: str = "fp32"):
    """Run a layer list (records with kind / filter_hw / strides / dilations / pad / act /
    out_channels / filter / bias) op by op; every layer's fp32 output feeds the next.

    Returns the list of all layer outputs when `keep_all`, else the last one.
    global_avg_pool is a 'valid' avgPool whose window is the remaining H x W, followed by the
    free reshape to [batch, C]; dense is matMul then a bias add with no activation.

    storage="bf16": the narrow-storage mode.  Everything that is stored is a bfloat16: the model
    input, every filter, and the output of every layer except dense and softmax layers and the
    model's last layer, which stay fp32.  Biases stay fp32 (they are added to the wide sum).  The
    arithmetic in between is the exact one of the fp32 mode: exact products of the stored values,
    a wide sum, one rounding to fp32, and then the rounding to the stored format.
    """
    if storage not in ("fp32", "bf16"):
        raise ValueError(f"unknown storage {storage!r}")
    narrow = storage == "bf16"
    if narrow and operand != "fp32":
        raise ValueError("narrow storage has no operand rounding of its own: bfloat16 products are exact")
    stored = round_bf16 if narrow else (lambda t: t)
    outs: List[np.ndarray] = []
    cur = stored(_f32(x))
    layers = list(layers)
    for li, layer in enumerate(layers):
        kind = layer.kind
        if kind == "conv2d":
            cur = conv2d(cur, stored(layer.filter), layer.strides, layer.pad, layer.dilations, layer.bias, layer.act,
                         operand)
        elif kind == "depthwise_conv2d":
            cur = depthwise_conv2d(cur, stored(layer.filter), layer.strides, layer.pad, layer.dilations, layer.bias,
                                   layer.act)
        elif kind == "global_avg_pool":
            n, h, w, c = cur.shape
            cur = avg_pool(cur, (h, w), (1, 1), "valid").reshape(n, c)
        elif kind == "dense":
            cur = bias_act(matmul(cur.reshape(cur.shape[0], -1), stored(layer.filter), operand=operand), layer.bias,
                           layer.act)
        elif kind == "softmax":
            cur = softmax(cur)
        else:
            raise ValueError(f"unknown layer kind {kind!r}")
        if narrow and kind not in ("dense", "softmax") and li != len(layers) - 1:
            cur = round_bf16(cur)
        if keep_all:
            outs.append(cur)
    return outs if keep_all else cur

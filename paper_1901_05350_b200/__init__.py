"""Python binding of libtfjsb.so: the same calls as include/tfjsb.h, argument marshalling only.

Every step of the op path runs in the CUDA library; PyTorch supplies device memory
(`torch.empty`), streams and nothing else.  There is no CPU fallback: if the shared library
cannot be built or loaded, importing this package raises.

    import paper_1901_05350_b200 as tfjsb
    ctx = tfjsb.Context(0)
    c = ctx.matmul(a, b)                       # torch CUDA fp32 tensors in, torch tensor out
    y = ctx.conv2d(x, f, (2, 2), "same", bias=b, act="relu6")
    model = ctx.model(layers, input_shape)      # layers: records with kind/filter_hw/.../filter/bias
    probs = model.run(x)
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

from . import build as _build

PAD = {"valid": 0, "same": 1}
ACT = {"none": 0, "relu": 1, "relu6": 2}
MATH = {"tf32": 0, "fp32": 1, "bf16": 2}
BINARY_OP = {"add": 0, "sub": 1, "mul": 2}
LAYER_KIND = {"conv2d": 0, "depthwise_conv2d": 1, "avg_pool": 2, "global_avg_pool": 2, "dense": 3, "softmax": 4}

STATUS_NAMES = {0: "OK", 1: "INVALID_ARG", 2: "SHAPE", 3: "UNSUPPORTED", 4: "CUDA", 5: "TIMEOUT", 6: "OOM"}

EXPORTS = [
    "tfjsb_init", "tfjsb_shutdown", "tfjsb_set_math", "tfjsb_last_error", "tfjsb_check_device_status",
    "tfjsb_launch_count", "tfjsb_window_out_shape", "tfjsb_matmul", "tfjsb_batch_matmul", "tfjsb_max_pool", "tfjsb_binary", "tfjsb_matmul_static_scratch", "tfjsb_conv2d", "tfjsb_depthwise_conv2d",
    "tfjsb_avg_pool", "tfjsb_softmax", "tfjsb_bias_act", "tfjsb_model_create", "tfjsb_model_destroy",
    "tfjsb_model_output_shape", "tfjsb_model_launches_per_run", "tfjsb_run_model", "tfjsb_run_model_host",
    "tfjsb_run_model_host_async", "tfjsb_model_host_wait",
    "tfjsb_model_set_keep_all", "tfjsb_model_set_graph", "tfjsb_model_set_fusion", "tfjsb_model_layer_output", "tfjsb_model_profile",
    "tfjsb_matmul_bf16", "tfjsb_model_layer_output_f32", "tfjsb_model_layer_shape", "tfjsb_model_layer_kernel",
    "tfjsb_reserve_scratch", "tfjsb_conv2d_backprop_input", "tfjsb_conv2d_backprop_filter",
    "tfjsb_depthwise_conv2d_backprop_input", "tfjsb_depthwise_conv2d_backprop_filter", "tfjsb_act_backprop",
    "tfjsb_bias_backprop",
]


class TfjsbError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"tfjsb status {STATUS_NAMES.get(status, status)}: {message}")
        self.status = status
        self.status_name = STATUS_NAMES.get(status, str(status))


class Tensor(ctypes.Structure):
    _fields_ = [("data", ctypes.c_void_p), ("rank", ctypes.c_int32), ("dims", ctypes.c_int64 * 4)]


class LayerDesc(ctypes.Structure):
    _fields_ = [
        ("kind", ctypes.c_int32),
        ("filter_hw", ctypes.c_int32 * 2),
        ("strides", ctypes.c_int32 * 2),
        ("dilations", ctypes.c_int32 * 2),
        ("pad", ctypes.c_int32),
        ("act", ctypes.c_int32),
        ("out_channels", ctypes.c_int32),
        ("filter", ctypes.c_void_p),
        ("bias", ctypes.c_void_p),
    ]


def _load_library() -> ctypes.CDLL:
    # TFJSB_LIBRARY points at an already built libtfjsb.so (e.g. an instrumented build); otherwise the
    # library is (re)built in-tree when its sources are newer
    path = os.environ.get("TFJSB_LIBRARY") or _build.build()
    lib = ctypes.CDLL(path)
    vp, i32, i64 = ctypes.c_void_p, ctypes.c_int, ctypes.c_int64
    tp = ctypes.POINTER(Tensor)
    ip = ctypes.POINTER(ctypes.c_int)
    lib.tfjsb_init.argtypes = [i32, ctypes.POINTER(vp)]
    lib.tfjsb_shutdown.argtypes = [vp]
    lib.tfjsb_set_math.argtypes = [vp, i32]
    lib.tfjsb_last_error.argtypes = [vp]
    lib.tfjsb_last_error.restype = ctypes.c_char_p
    lib.tfjsb_check_device_status.argtypes = [vp, vp]
    lib.tfjsb_launch_count.argtypes = [vp]
    lib.tfjsb_launch_count.restype = i64
    lib.tfjsb_window_out_shape.argtypes = [i64, i32, i32, i32, i32, ctypes.POINTER(i64), ip, ip]
    lib.tfjsb_matmul.argtypes = [vp, tp, tp, i32, i32, tp, vp]
    lib.tfjsb_matmul_static_scratch.argtypes = [vp, tp, tp, i32, i32, tp, vp]
    lib.tfjsb_batch_matmul.argtypes = [vp, tp, tp, i32, i32, tp, vp]
    lib.tfjsb_max_pool.argtypes = [vp, tp, ip, ip, i32, tp, vp]
    lib.tfjsb_binary.argtypes = [vp, i32, tp, tp, tp, vp]
    lib.tfjsb_conv2d.argtypes = [vp, tp, tp, ip, i32, ip, tp, i32, tp, vp]
    lib.tfjsb_depthwise_conv2d.argtypes = [vp, tp, tp, ip, i32, ip, tp, i32, tp, vp]
    lib.tfjsb_avg_pool.argtypes = [vp, tp, ip, ip, i32, tp, vp]
    lib.tfjsb_softmax.argtypes = [vp, tp, tp, vp]
    lib.tfjsb_bias_act.argtypes = [vp, tp, tp, i32, tp, vp]
    lib.tfjsb_model_create.argtypes = [vp, ctypes.POINTER(LayerDesc), i32, ctypes.POINTER(i64), ctypes.POINTER(vp)]
    lib.tfjsb_model_destroy.argtypes = [vp]
    lib.tfjsb_model_output_shape.argtypes = [vp, ctypes.POINTER(ctypes.c_int32), ctypes.POINTER(i64)]
    lib.tfjsb_model_launches_per_run.argtypes = [vp]
    lib.tfjsb_model_launches_per_run.restype = ctypes.c_int32
    lib.tfjsb_run_model.argtypes = [vp, tp, tp, vp]
    lib.tfjsb_run_model_host.argtypes = [vp, vp, vp, vp]
    lib.tfjsb_run_model_host_async.argtypes = [vp, vp, vp, vp]
    lib.tfjsb_model_host_wait.argtypes = [vp]
    lib.tfjsb_model_set_keep_all.argtypes = [vp, i32]
    lib.tfjsb_model_set_graph.argtypes = [vp, i32]
    lib.tfjsb_model_set_fusion.argtypes = [vp, i32]
    lib.tfjsb_model_layer_output.argtypes = [vp, i32, tp]
    lib.tfjsb_model_profile.argtypes = [vp, tp, tp, i32, ctypes.POINTER(ctypes.c_float), vp]
    lib.tfjsb_matmul_bf16.argtypes = [vp, vp, vp, vp, i32, vp, i32, i64, i64, i64, vp]
    lib.tfjsb_model_layer_output_f32.argtypes = [vp, i32, vp, vp]
    lib.tfjsb_model_layer_shape.argtypes = [vp, i32, ctypes.POINTER(ctypes.c_int32), ctypes.POINTER(ctypes.c_int64)]
    lib.tfjsb_model_layer_kernel.argtypes = [vp, i32, ctypes.c_char_p, ctypes.c_int32]
    lib.tfjsb_reserve_scratch.argtypes = [vp, i64]
    for name in ("tfjsb_conv2d_backprop_input", "tfjsb_conv2d_backprop_filter", "tfjsb_depthwise_conv2d_backprop_input",
                 "tfjsb_depthwise_conv2d_backprop_filter"):
        getattr(lib, name).argtypes = [vp, tp, tp, ip, i32, ip, tp, vp]
    lib.tfjsb_act_backprop.argtypes = [vp, tp, tp, i32, tp, vp]
    lib.tfjsb_bias_backprop.argtypes = [vp, tp, tp, vp]
    return lib


lib = _load_library()


def window_out_shape(size: int, k: int, stride: int, dilation: int, pad: str):
    """(out, pad_before, pad_after) of one spatial dimension (host arithmetic in the library)."""
    out, before, after = ctypes.c_int64(), ctypes.c_int(), ctypes.c_int()
    rc = lib.tfjsb_window_out_shape(size, k, stride, dilation, PAD[pad], ctypes.byref(out), ctypes.byref(before),
                                    ctypes.byref(after))
    if rc:
        raise TfjsbError(rc, f"no output for in={size} k={k} stride={stride} dilation={dilation} pad={pad}")
    return out.value, before.value, after.value


def _desc(t) -> Tensor:
    """tfjsb_tensor over a contiguous fp32 CUDA torch tensor (rank 1..4)."""
    import torch

    if not isinstance(t, torch.Tensor) or not t.is_cuda or t.dtype != torch.float32 or not t.is_contiguous():
        raise TypeError("expected a contiguous fp32 CUDA tensor")
    d = Tensor()
    d.data = t.data_ptr()
    d.rank = t.dim()
    for i, s in enumerate(t.shape):
        d.dims[i] = s
    return d


def _stream() -> int:
    import torch

    return torch.cuda.current_stream().cuda_stream


def _int2(v) -> ctypes.Array:
    return (ctypes.c_int * 2)(int(v[0]), int(v[1]))


class Context:
    """A tfjsb context on one CUDA device."""

    def __init__(self, device: int = 0, math: str = "tf32"):
        import torch

        if not torch.cuda.is_available():
            raise RuntimeError("tfjsb needs a CUDA device; there is no CPU fallback")
        torch.cuda.set_device(device)
        torch.cuda.init()
        self.device = device
        self._h = ctypes.c_void_p()
        rc = lib.tfjsb_init(device, ctypes.byref(self._h))
        if rc:
            raise TfjsbError(rc, "tfjsb_init failed (needs a compute-capability 10.x device)")
        self.set_math(math)

    # -- plumbing
    def _check(self, rc: int):
        if rc:
            raise TfjsbError(rc, lib.tfjsb_last_error(self._h).decode())

    def close(self):
        if self._h:
            self._check(lib.tfjsb_shutdown(self._h))
            self._h = ctypes.c_void_p()

    def set_math(self, math: str):
        self._check(lib.tfjsb_set_math(self._h, MATH[math]))
        self.math = math

    def check_device_status(self):
        self._check(lib.tfjsb_check_device_status(self._h, _stream()))

    @property
    def launch_count(self) -> int:
        return lib.tfjsb_launch_count(self._h)

    def _empty(self, shape):
        import torch

        return torch.empty(tuple(int(s) for s in shape), dtype=torch.float32, device=f"cuda:{self.device}")

    # -- ops
    def matmul(self, a, b, transpose_a: bool = False, transpose_b: bool = False, out=None):
        M = a.shape[1] if transpose_a else a.shape[0]
        N = b.shape[0] if transpose_b else b.shape[1]
        out = self._empty((M, N)) if out is None else out
        self._check(lib.tfjsb_matmul(self._h, _desc(a), _desc(b), int(transpose_a), int(transpose_b), _desc(out),
                                     _stream()))
        return out

    def matmul_bf16(self, a, bt, bias=None, act="none", out_dtype=None, out=None):
        """act(a . bt^T + bias) on bfloat16 storage: a [M,K] and bt [N,K] bfloat16 CUDA tensors, bias fp32 [N]
        or None, result bfloat16 (default) or fp32; products exact, sums fp32 on the tensor cores."""
        import torch

        for t in (a, bt):
            if not t.is_cuda or t.dtype != torch.bfloat16 or not t.is_contiguous() or t.dim() != 2:
                raise TypeError("expected contiguous rank-2 bfloat16 CUDA tensors")
        if a.shape[1] != bt.shape[1]:
            raise ValueError("a [M,K] and bt [N,K] must agree in K")
        M, K, N = a.shape[0], a.shape[1], bt.shape[0]
        if out is None:
            out = torch.empty((M, N), dtype=out_dtype or torch.bfloat16, device=a.device)
        if out.dtype not in (torch.bfloat16, torch.float32) or tuple(out.shape) != (M, N) or not out.is_contiguous():
            raise TypeError("out must be a contiguous [M,N] bfloat16 or fp32 tensor")
        if bias is not None and (bias.dtype != torch.float32 or tuple(bias.shape) != (N,) or not bias.is_contiguous()):
            raise TypeError("bias must be a contiguous fp32 vector of length N")
        self._check(lib.tfjsb_matmul_bf16(self._h, a.data_ptr(), bt.data_ptr(), None if bias is None else bias.data_ptr(),
                                          ACT[act], out.data_ptr(), int(out.dtype == torch.bfloat16), M, N, K, _stream()))
        return out

    def matmul_static_scratch(self, a, b, transpose_a: bool = False, transpose_b: bool = False, out=None):
        """matmul for callers that must not allocate device memory inside the call: operands are
        transposed into a fixed 16 MiB array in the library instead of cudaMalloc'ed scratch.
        Pass `out` (the binding would otherwise allocate it); problems whose operands to transpose
        exceed 4 Mi floats are rejected.  Calls share the array: keep them on one stream."""
        M = a.shape[1] if transpose_a else a.shape[0]
        N = b.shape[0] if transpose_b else b.shape[1]
        out = self._empty((M, N)) if out is None else out
        self._check(lib.tfjsb_matmul_static_scratch(self._h, _desc(a), _desc(b), int(transpose_a),
                                                    int(transpose_b), _desc(out), _stream()))
        return out

    def _conv_out(self, x, fh, fw, strides, pad, dilations, channels):
        ho, _, _ = window_out_shape(x.shape[1], fh, strides[0], dilations[0], pad)
        wo, _, _ = window_out_shape(x.shape[2], fw, strides[1], dilations[1], pad)
        return self._empty((x.shape[0], ho, wo, channels))

    def conv2d(self, x, filter, strides=(1, 1), pad="same", dilations=(1, 1), bias=None, act="none", out=None):
        if out is None:
            out = self._conv_out(x, filter.shape[0], filter.shape[1], strides, pad, dilations, filter.shape[3])
        self._check(lib.tfjsb_conv2d(self._h, _desc(x), _desc(filter), _int2(strides), PAD[pad], _int2(dilations),
                                     None if bias is None else _desc(bias), ACT[act], _desc(out), _stream()))
        return out

    def depthwise_conv2d(self, x, filter, strides=(1, 1), pad="same", dilations=(1, 1), bias=None, act="none",
                         out=None):
        if out is None:
            out = self._conv_out(x, filter.shape[0], filter.shape[1], strides, pad, dilations,
                                 filter.shape[2] * filter.shape[3])
        self._check(lib.tfjsb_depthwise_conv2d(self._h, _desc(x), _desc(filter), _int2(strides), PAD[pad],
                                               _int2(dilations), None if bias is None else _desc(bias), ACT[act],
                                               _desc(out), _stream()))
        return out

    def avg_pool(self, x, filter_size, strides, pad="valid", out=None):
        if out is None:
            out = self._conv_out(x, filter_size[0], filter_size[1], strides, pad, (1, 1), x.shape[3])
        self._check(lib.tfjsb_avg_pool(self._h, _desc(x), _int2(filter_size), _int2(strides), PAD[pad], _desc(out),
                                       _stream()))
        return out

    def max_pool(self, x, filter_size, strides, pad="valid", out=None):
        if out is None:
            out = self._conv_out(x, filter_size[0], filter_size[1], strides, pad, (1, 1), x.shape[3])
        self._check(lib.tfjsb_max_pool(self._h, _desc(x), _int2(filter_size), _int2(strides), PAD[pad], _desc(out),
                                       _stream()))
        return out

    def binary(self, op: str, a, b, out=None):
        """a op b elementwise, op in 'add' / 'sub' / 'mul'; b has a's shape or is a vector of a's last dimension."""
        out = self._empty(a.shape) if out is None else out
        self._check(lib.tfjsb_binary(self._h, BINARY_OP[op], _desc(a), _desc(b), _desc(out), _stream()))
        return out

    def batch_matmul(self, a, b, transpose_a: bool = False, transpose_b: bool = False, out=None):
        M = a.shape[2] if transpose_a else a.shape[1]
        N = b.shape[1] if transpose_b else b.shape[2]
        out = self._empty((a.shape[0], M, N)) if out is None else out
        self._check(lib.tfjsb_batch_matmul(self._h, _desc(a), _desc(b), int(transpose_a), int(transpose_b), _desc(out),
                                           _stream()))
        return out

    def softmax(self, logits, out=None):
        out = self._empty(logits.shape) if out is None else out
        self._check(lib.tfjsb_softmax(self._h, _desc(logits), _desc(out), _stream()))
        return out

    def bias_act(self, x, bias=None, act="none", out=None):
        out = self._empty(x.shape) if out is None else out
        self._check(lib.tfjsb_bias_act(self._h, _desc(x), None if bias is None else _desc(bias), ACT[act],
                                       _desc(out), _stream()))
        return out

    def reserve_scratch(self, nbytes: int):
        self._check(lib.tfjsb_reserve_scratch(self._h, int(nbytes)))

    # -- gradients (geometry arguments are the forward call's)
    def conv2d_backprop_input(self, x_shape, filter, dy, strides=(1, 1), pad="same", dilations=(1, 1), out=None):
        out = self._empty(x_shape) if out is None else out
        self._check(lib.tfjsb_conv2d_backprop_input(self._h, _desc(dy), _desc(filter), _int2(strides), PAD[pad],
                                                    _int2(dilations), _desc(out), _stream()))
        return out

    def conv2d_backprop_filter(self, x, filter_shape, dy, strides=(1, 1), pad="same", dilations=(1, 1), out=None):
        out = self._empty(filter_shape) if out is None else out
        self._check(lib.tfjsb_conv2d_backprop_filter(self._h, _desc(x), _desc(dy), _int2(strides), PAD[pad],
                                                     _int2(dilations), _desc(out), _stream()))
        return out

    def depthwise_conv2d_backprop_input(self, x_shape, filter, dy, strides=(1, 1), pad="same", dilations=(1, 1), out=None):
        out = self._empty(x_shape) if out is None else out
        self._check(lib.tfjsb_depthwise_conv2d_backprop_input(self._h, _desc(dy), _desc(filter), _int2(strides), PAD[pad],
                                                              _int2(dilations), _desc(out), _stream()))
        return out

    def depthwise_conv2d_backprop_filter(self, x, filter_shape, dy, strides=(1, 1), pad="same", dilations=(1, 1), out=None):
        out = self._empty(filter_shape) if out is None else out
        self._check(lib.tfjsb_depthwise_conv2d_backprop_filter(self._h, _desc(x), _desc(dy), _int2(strides), PAD[pad],
                                                               _int2(dilations), _desc(out), _stream()))
        return out

    def act_backprop(self, y, dy, act="none", out=None):
        out = self._empty(y.shape) if out is None else out
        self._check(lib.tfjsb_act_backprop(self._h, _desc(y), _desc(dy), ACT[act], _desc(out), _stream()))
        return out

    def bias_backprop(self, dz, out=None):
        out = self._empty((dz.shape[-1],)) if out is None else out
        self._check(lib.tfjsb_bias_backprop(self._h, _desc(dz), _desc(out), _stream()))
        return out

    def model(self, layers: Sequence, input_shape) -> "Model":
        return Model(self, layers, input_shape)


class Model:
    """Executor for a straight-line layer list (records with kind / filter_hw / strides / dilations /
    pad / act / out_channels / filter / bias, filters and biases as host numpy fp32 arrays)."""

    def __init__(self, ctx: Context, layers: Sequence, input_shape):
        import numpy as np

        self.ctx = ctx
        self.n_layers = len(layers)
        self.layer_names = [getattr(l, "name", "") or l.kind for l in layers]
        descs = (LayerDesc * len(layers))()
        keep = []  # host arrays must outlive the create call
        for d, layer in zip(descs, layers):
            d.kind = LAYER_KIND[layer.kind]
            fh, fw = (0, 0) if layer.kind == "global_avg_pool" else layer.filter_hw
            d.filter_hw[0], d.filter_hw[1] = fh, fw
            d.strides[0], d.strides[1] = layer.strides
            d.dilations[0], d.dilations[1] = layer.dilations
            d.pad = PAD[layer.pad]
            d.act = ACT[layer.act]
            d.out_channels = layer.out_channels
            for field in ("filter", "bias"):
                arr = getattr(layer, field, None)
                if arr is not None:
                    arr = np.ascontiguousarray(arr, dtype=np.float32)
                    keep.append(arr)
                    setattr(d, field, arr.ctypes.data)
        dims = (ctypes.c_int64 * 4)(*[int(s) for s in input_shape])
        self._h = ctypes.c_void_p()
        ctx._check(lib.tfjsb_model_create(ctx._h, descs, len(layers), dims, ctypes.byref(self._h)))
        self.input_shape = tuple(int(s) for s in input_shape)
        rank = ctypes.c_int32()
        odims = (ctypes.c_int64 * 4)()
        ctx._check(lib.tfjsb_model_output_shape(self._h, ctypes.byref(rank), odims))
        self.output_shape = tuple(odims[i] for i in range(rank.value))

    @property
    def launches_per_run(self) -> int:
        """Kernels one run launches in the current mode (fused blocks count once)."""
        return int(lib.tfjsb_model_launches_per_run(self._h))

    def close(self):
        if self._h:
            self.ctx._check(lib.tfjsb_model_destroy(self._h))
            self._h = ctypes.c_void_p()

    def run(self, x, out=None):
        """Enqueue one forward pass on the current stream; device tensors in and out."""
        out = self.ctx._empty(self.output_shape) if out is None else out
        self.ctx._check(lib.tfjsb_run_model(self._h, _desc(x), _desc(out), _stream()))
        return out

    def run_host(self, host_in, host_out):
        """Forward pass from/to host memory (torch CPU tensors, ideally pinned); blocks until done."""
        if host_in.is_cuda or host_out.is_cuda or not host_in.is_contiguous() or not host_out.is_contiguous():
            raise TypeError("run_host takes contiguous CPU tensors")
        if tuple(host_in.shape) != self.input_shape or tuple(host_out.shape) != self.output_shape:
            raise ValueError("host tensors must have the model's input / output shapes")
        self.ctx._check(lib.tfjsb_run_model_host(self._h, host_in.data_ptr(), host_out.data_ptr(), _stream()))
        return host_out

    def run_host_async(self, host_in, host_out):
        """Enqueue a forward pass from/to host memory and return at once; up to two may be outstanding
        (the copy of one overlaps the computation of the one before).  Keep both tensors alive and
        untouched until host_wait() returns."""
        if host_in.is_cuda or host_out.is_cuda or not host_in.is_contiguous() or not host_out.is_contiguous():
            raise TypeError("run_host_async takes contiguous CPU tensors")
        if tuple(host_in.shape) != self.input_shape or tuple(host_out.shape) != self.output_shape:
            raise ValueError("host tensors must have the model's input / output shapes")
        self.ctx._check(lib.tfjsb_run_model_host_async(self._h, host_in.data_ptr(), host_out.data_ptr(), _stream()))

    def host_wait(self):
        """Block until every run_host_async() call has delivered its output."""
        self.ctx._check(lib.tfjsb_model_host_wait(self._h))

    def set_keep_all(self, keep_all: bool):
        self.ctx._check(lib.tfjsb_model_set_keep_all(self._h, int(keep_all)))

    def set_fusion(self, mode: str):
        """'off', 'auto' (default) or 'always': run depthwise + pointwise pairs as one fused kernel."""
        self.ctx._check(lib.tfjsb_model_set_fusion(self._h, {"off": 0, "auto": 1, "always": 2}[mode]))

    def set_graph(self, use_graph: bool):
        """Replay runs as a CUDA graph captured inside the library (run once without it first)."""
        self.ctx._check(lib.tfjsb_model_set_graph(self._h, int(use_graph)))

    def layer_output(self, layer: int):
        """Copy of the output of layer `layer` left by the last run (use set_keep_all(True) first)."""
        import torch

        view = Tensor()
        self.ctx._check(lib.tfjsb_model_layer_output(self._h, layer, ctypes.byref(view)))
        shape = tuple(int(view.dims[i]) for i in range(view.rank))

        class _View:  # device memory owned by the model, described for torch's array-interface import
            __cuda_array_interface__ = {"shape": shape, "typestr": "<f4", "data": (int(view.data), False),
                                        "version": 3, "strides": None}

        torch.cuda.current_stream().synchronize()
        return torch.as_tensor(_View(), device=f"cuda:{self.ctx.device}").clone()

    def layer_output_f32(self, layer: int):
        """fp32 copy of the output of layer `layer` whatever its storage format (bfloat16 layers are
        widened on the device); use set_keep_all(True) before the run."""
        rank = ctypes.c_int32()
        dims = (ctypes.c_int64 * 4)()
        self.ctx._check(lib.tfjsb_model_layer_shape(self._h, layer, ctypes.byref(rank), dims))
        out = self.ctx._empty(tuple(int(dims[i]) for i in range(rank.value)))
        self.ctx._check(lib.tfjsb_model_layer_output_f32(self._h, layer, out.data_ptr(), _stream()))
        return out

    def layer_kernels(self):
        """Name of the kernel that runs each layer in the current mode (after at least one run)."""
        names = []
        buf = ctypes.create_string_buffer(96)
        for i in range(self.n_layers):
            self.ctx._check(lib.tfjsb_model_layer_kernel(self._h, i, buf, len(buf)))
            names.append(buf.value.decode())
        return names

    def profile(self, x, out=None, reps: int = 10):
        """Mean device milliseconds per layer over `reps` runs (event pair around every layer)."""
        out = self.ctx._empty(self.output_shape) if out is None else out
        ms = (ctypes.c_float * self.n_layers)()
        self.ctx._check(lib.tfjsb_model_profile(self._h, _desc(x), _desc(out), reps, ms, _stream()))
        return [float(v) for v in ms]

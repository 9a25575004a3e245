#!/usr/bin/env python
"""Benchmark: MobileNet v1 1.0 224x224 images/s through the CUDA library (one pass = one batch).

    python bench.py [--gpus N] [--steps K] [--warmup W]         # this library
    python bench.py --impl reference [--steps K] [--warmup W]   # the CPU oracle, as it stands

One JSON line on stdout (rank 0).  Workload: the batch-128 throughput configuration
(input [128,224,224,3] fp32, seeded synthetic weights and images); the batch-1 latency of the
same model is reported alongside as `batch1`.  With N > 1 every rank runs an independent replica
of the same batch (weak scaling, no collective on the data path); time is the max over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "MobileNet v1 1.0 224 images/sec, batch 128"
UNIT = "images/s"
BATCH = 128
WORKLOAD = "configs[4]: MobileNet v1 alpha=1.0, input [128,224,224,3] fp32, BN folded, seeded He-normal weights"


# --------------------------------------------------------------------------------- peaks
# NVIDIA's published per-GPU figures for B200 (DGX B200 datasheet: 64 TB/s of HBM3e bandwidth and
# 18 PFLOP/s of TF32 with 2:4 sparsity over eight GPUs, i.e. 8 TB/s and 1.125 PFLOP/s dense each; bf16 is
# twice the TF32 rate).  Every fraction is reported against the measured peak and against these.
STATED_PEAKS = {"hbm_gbs": 8000.0, "tf32_tflops": 1125.0, "bf16_tflops": 2250.0,
                "source": "NVIDIA DGX B200 datasheet, per GPU, dense"}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            p = json.load(fh)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


# --------------------------------------------------------------------------------- clocks
class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU through NVML while the timed region runs."""

    REASONS = {
        0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap",
        0x80: "hw_power_brake_slowdown",
    }

    def __init__(self, torch_device: int, period_s: float = 0.02):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self.period = period_s
        self._stop = threading.Event()
        self._thread = None
        self._handle = None
        try:
            import pynvml
            import torch

            pynvml.nvmlInit()
            self._nvml = pynvml
            handle = None
            try:
                uuid = str(torch.cuda.get_device_properties(torch_device).uuid)
                handle = pynvml.nvmlDeviceGetHandleByUUID(("GPU-" + uuid) if not uuid.startswith("GPU-") else uuid)
            except Exception:
                visible = os.environ.get("CUDA_VISIBLE_DEVICES")
                index = torch_device
                if visible and all(v.strip().isdigit() for v in visible.split(",")):
                    index = int(visible.split(",")[torch_device])
                handle = pynvml.nvmlDeviceGetHandleByIndex(index)
            self._handle = handle
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(handle, pynvml.NVML_CLOCK_SM))
        except Exception:
            self._handle = None

    def _loop(self):
        nv = self._nvml
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self._handle, nv.NVML_CLOCK_SM)))
                try:
                    bits = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self._handle))
                except Exception:
                    bits = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._handle))
                for bit, name in self.REASONS.items():
                    if bits & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            self._stop.wait(self.period)

    def start(self):
        if self._handle is not None:
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()

    def stop(self):
        if self._thread is not None:
            self._stop.set()
            self._thread.join()
        return {"sm_mhz": statistics.median(self.samples) if self.samples else None, "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


# --------------------------------------------------------------------------------- roofline bookkeeping
def layer_work(layers, in_shape, window_out_shape):
    """Algorithmic flops and bytes of every layer (each tensor read or written exactly once, fp32).
    `kernel` holds the op class here; the benchmark replaces it by the name of the kernel the library
    ran for the layer."""
    n, h, w, c = in_shape
    rows = []
    for layer in layers:
        kind = layer.kind
        if kind in ("conv2d", "depthwise_conv2d"):
            fh, fw = layer.filter_hw
            ho, _, _ = window_out_shape(h, fh, layer.strides[0], layer.dilations[0], layer.pad)
            wo, _, _ = window_out_shape(w, fw, layer.strides[1], layer.dilations[1], layer.pad)
            if kind == "conv2d":
                co = layer.out_channels
                flops = 2 * n * ho * wo * co * fh * fw * c
                weights = fh * fw * c * co
                kernel = "pointwise_conv2d" if (fh, fw) == (1, 1) and layer.strides == (1, 1) else "conv2d"
            else:
                co = c * layer.out_channels
                flops = 2 * n * ho * wo * co * fh * fw
                weights = fh * fw * co
                kernel = "depthwise_conv2d"
            nbytes = 4 * (n * h * w * c + weights + co + n * ho * wo * co)
            rows.append(dict(name=layer.name, kernel=kernel, flops=flops, bytes=nbytes, units=n * ho * wo * co))
            h, w, c = ho, wo, co
        elif kind == "global_avg_pool":
            rows.append(dict(name=layer.name, kernel="avg_pool", flops=n * h * w * c, bytes=4 * (n * h * w * c + n * c),
                             units=n * c))
            h = w = 1
        elif kind == "dense":
            k, co = h * w * c, layer.out_channels
            rows.append(dict(name=layer.name, kernel="dense", flops=2 * n * k * co,
                             bytes=4 * (n * k + k * co + co + n * co), units=n * co))
            h, w, c = 1, 1, co
        elif kind == "softmax":
            rows.append(dict(name=layer.name, kernel="softmax", flops=5 * n * c, bytes=8 * n * c, units=n * c))
    return rows


def narrow_layer_work(layers, in_shape, window_out_shape):
    """Algorithmic flops and bytes of every layer in the narrow-storage mode: filters and every layer output
    are 2 bytes per value, except the model input, biases, and the dense and softmax outputs (4 bytes)."""
    n, h, w, c = in_shape
    rows = []
    in_size = 4  # the model input is fp32
    last = len(layers) - 1
    for i, layer in enumerate(layers):
        kind = layer.kind
        out_size = 4 if (kind in ("dense", "softmax") or i == last) else 2
        if kind in ("conv2d", "depthwise_conv2d"):
            fh, fw = layer.filter_hw
            ho, _, _ = window_out_shape(h, fh, layer.strides[0], layer.dilations[0], layer.pad)
            wo, _, _ = window_out_shape(w, fw, layer.strides[1], layer.dilations[1], layer.pad)
            if kind == "conv2d":
                co = layer.out_channels
                flops, weights = 2 * n * ho * wo * co * fh * fw * c, fh * fw * c * co
                tensor = (fh, fw) == (1, 1) and layer.strides == (1, 1)
            else:
                co = c * layer.out_channels
                flops, weights, tensor = 2 * n * ho * wo * co * fh * fw, fh * fw * co, False
            nbytes = in_size * n * h * w * c + 2 * weights + 4 * co + out_size * n * ho * wo * co
            h, w, c = ho, wo, co
        elif kind == "global_avg_pool":
            flops, nbytes, tensor = n * h * w * c, in_size * n * h * w * c + out_size * n * c, False
            h = w = 1
        elif kind == "dense":
            k, co = h * w * c, layer.out_channels
            flops, nbytes, tensor = 2 * n * k * co, in_size * n * k + 2 * k * co + 4 * co + out_size * n * co, True
            h, w, c = 1, 1, co
        else:  # softmax
            flops, nbytes, tensor = 5 * n * c, (in_size + out_size) * n * c, False
        rows.append(dict(name=layer.name, flops=flops, bytes=nbytes, tensor=tensor))
        in_size = out_size
    return rows


FUSED_INTO_PREVIOUS = "(in the previous layer's kernel)"
TENSOR_CORE_KERNELS = ("gemm_tf32", "gemm_bf16", "gemm_pair", "dwpw_fused")


def label_and_merge(rows, ms, kernels):
    """Labels every row with the kernel the library reports for the layer and folds a layer that ran inside
    its predecessor's kernel (a fused depthwise + pointwise pair) into that row: the fused kernel reads the
    depthwise input and writes the pointwise output, the intermediate tensor is never in HBM."""
    out_rows, out_ms = [], []
    for row, t, kernel in zip(rows, ms, kernels):
        if kernel == FUSED_INTO_PREVIOUS and out_rows:
            prev = out_rows[-1]
            inter = 4 * prev["units"]  # the first layer's output = this layer's input, counted once in each row
            out_rows[-1] = dict(name=prev["name"] + "+" + row["name"], kernel=prev["kernel"], flops=prev["flops"] + row["flops"],
                                bytes=prev["bytes"] + row["bytes"] - 2 * inter, units=row["units"])
            out_ms[-1] += t
        else:
            out_rows.append(dict(row, kernel=kernel))
            out_ms.append(t)
    return out_rows, out_ms


def roofline_rows(rows, ms, peaks, fp32_tflops):
    """Per row: the slower of its flops at the compute peak and its bytes at the HBM copy rate.  The per-layer
    times come from event pairs in a short profile at full clocks, so the tensor peak is the burst figure
    (measured bf16 / 2: dense TF32 is nominally half of dense bf16); the fraction against the sustained
    figure and against the published peaks is given beside it."""
    tf32_burst = peaks["bf16_tflops"] / 2.0
    tf32_sustained = peaks["bf16_tflops_sustained"] / 2.0
    out = []
    for row, t_ms in zip(rows, ms):
        on_tensor_cores = any(k in row["kernel"] for k in TENSOR_CORE_KERNELS)
        t = t_ms * 1e-3

        def roof(tensor_tflops, hbm_gbs):
            t_compute = row["flops"] / ((tensor_tflops if on_tensor_cores else fp32_tflops) * 1e12)
            return t_compute, row["bytes"] / (hbm_gbs * 1e9)

        t_compute, t_hbm = roof(tf32_burst, peaks["hbm_gbs"])
        bound = "tensor" if (on_tensor_cores and t_compute > t_hbm) else ("alu" if t_compute > t_hbm else "hbm")
        t_roof = max(t_compute, t_hbm)
        out.append(dict(row, ms=t_ms, bound=bound, roofline_us=t_roof * 1e6, frac=t_roof / t if t > 0 else None,
                        frac_sustained=max(roof(tf32_sustained, peaks["hbm_gbs"])) / t if t > 0 else None,
                        frac_stated=max(roof(STATED_PEAKS["tf32_tflops"], STATED_PEAKS["hbm_gbs"])) / t if t > 0 else None,
                        gbs=row["bytes"] / t / 1e9 if t > 0 else None,
                        tflops=row["flops"] / t / 1e12 if t > 0 else None))
    return out


# --------------------------------------------------------------------------------- reference arm (CPU oracle)
def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    import numpy as np

    import oracle
    import seeded_inputs as si

    cores = os.cpu_count() or 1
    oracle.set_threads(cores)
    images = args.reference_images
    x, layers = si.config_mobilenet(1.0, 224, images, seed=si.CONFIG_SEEDS["mobilenet_100_224_b128"])
    for _ in range(args.warmup):
        oracle.run_model(layers, x)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        out = oracle.run_model(layers, x)
    dt = time.perf_counter() - t0
    assert np.all(np.isfinite(out))
    value = images * args.steps / dt
    sample = f"{images} of the {BATCH} images of the batch per step (images are independent), all {cores} host threads"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64 accumulate, f32 storage", "data": "synthetic",
        "config": {"workload": WORKLOAD, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.get_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)
    return 0


def cpu_baseline_leg(target_seconds: float = 15.0):
    """The oracle as it stands on the host's threads: a bounded sample of the batch on all threads (the
    headline baseline), one image on one thread and on all threads (best of 3), and configs 1 and 2."""
    import oracle
    import seeded_inputs as si

    def best_of(fn, n=3):
        best = float("inf")
        for _ in range(n):
            t0 = time.perf_counter()
            fn()
            best = min(best, time.perf_counter() - t0)
        return best

    cores = os.cpu_count() or 1
    seed = si.CONFIG_SEEDS["mobilenet_100_224_b128"]
    x1, layers = si.config_mobilenet(1.0, 224, 1, seed=seed)
    oracle.set_threads(cores)
    oracle.run_model(layers, x1)  # first-touch / build
    one_all = best_of(lambda: oracle.run_model(layers, x1))
    oracle.set_threads(1)
    one_single = best_of(lambda: oracle.run_model(layers, x1), 2)
    oracle.set_threads(cores)
    images = int(max(2, min(BATCH, target_seconds / max(one_all, 1e-3))))
    x, layers = si.config_mobilenet(1.0, 224, images, seed=seed)
    t0 = time.perf_counter()
    oracle.run_model(layers, x)
    dt = time.perf_counter() - t0
    a, b = si.config_matmul()
    matmul_s = best_of(lambda: oracle.matmul(a, b))
    xb, block = si.config_separable_block()
    block_s = best_of(lambda: oracle.run_model(block, xb))
    flops_per_image = 2 * 568740352
    return {"value": images / dt, "unit": UNIT, "cores": oracle.get_threads(), "kind": "oracle",
            "sample": f"first {images} of the {BATCH} images of one batch, one pass, {dt:.1f} s of CPU time on all host threads",
            "gflops": images * flops_per_image / dt / 1e9,
            "one_image": {"single_thread_ms": one_single * 1e3, "all_threads_ms": one_all * 1e3, "threads": cores,
                          "single_thread_gflops": flops_per_image / one_single / 1e9, "how": "best of 2 / best of 3"},
            "matmul_512": {"ms": matmul_s * 1e3, "gflops": 2 * 512 ** 3 / matmul_s / 1e9, "threads": cores},
            "separable_block_112x112x32_64": {"ms": block_s * 1e3, "threads": cores}}


# --------------------------------------------------------------------------------- this library
def run_ours(args):
    import numpy as np
    import torch

    import paper_1901_05350_b200 as tfjsb
    import seeded_inputs as si
    from paper_1901_05350_b200 import replicas

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    distributed = world > 1
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the op path has no CPU fallback")

    # the CPU baseline uses a thread pool of its own; run it before the first GPU call
    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu_baseline = cpu_baseline_leg()

    torch.cuda.set_device(local_rank)
    if distributed:
        import torch.distributed as dist

        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    peaks = load_peaks()
    ctx = tfjsb.Context(local_rank)
    props = torch.cuda.get_device_properties(local_rank)

    x_host, layers = si.config_mobilenet(1.0, 224, BATCH, seed=si.CONFIG_SEEDS["mobilenet_100_224_b128"])
    model = ctx.model(layers, x_host.shape)
    x = torch.from_numpy(x_host).cuda()
    out = torch.empty(model.output_shape, device="cuda")
    stream = torch.cuda.current_stream()

    def barrier():
        if distributed:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- device-resident throughput: one pass = one replay of the library's CUDA graph of the 27 launches
    # (tfjsb_model_set_graph; the same kernels in the same order, programmatic dependent launch between them)
    model.run(x, out=out)  # launch by launch once: function attributes are set outside a capture
    model.set_graph(True)
    for _ in range(max(args.warmup, 3)):
        model.run(x, out=out)
    barrier()
    sampler = ClockSampler(local_rank)
    sampler.start()
    launches0 = ctx.launch_count
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    start.record(stream)
    for _ in range(args.steps):
        model.run(x, out=out)
    stop.record(stream)
    barrier()
    launches = ctx.launch_count - launches0
    clocks = sampler.stop()
    model.set_graph(False)
    ctx.check_device_status()
    elapsed_ms = replicas.max_over_ranks(start.elapsed_time(stop), device="cuda")
    value = world * BATCH * args.steps / (elapsed_ms * 1e-3)

    # ---- end to end: pinned host input in, probabilities back to the host, every step.  The library's
    # asynchronous host call keeps two steps in flight (two sets of device staging buffers), so the
    # 77 MB input copy of step i+1 overlaps the computation of step i; every step still copies its own
    # input in and its own result out, and the last result is waited for inside the timed region.
    hins = [torch.from_numpy(x_host).pin_memory() for _ in range(2)]
    houts = [torch.empty(model.output_shape).pin_memory() for _ in range(2)]
    e2e_steps = max(3, min(args.steps, 50))
    for i in range(4):
        model.run_host_async(hins[i % 2], houts[i % 2])
    model.host_wait()
    barrier()
    start.record(stream)
    for i in range(e2e_steps):
        model.run_host_async(hins[i % 2], houts[i % 2])
    model.host_wait()
    stop.record(stream)
    barrier()
    e2e_ms = replicas.max_over_ranks(start.elapsed_time(stop), device="cuda")
    # the same with one step at a time (the blocking call): the latency-oriented figure
    start.record(stream)
    for i in range(e2e_steps):
        model.run_host(hins[i % 2], houts[i % 2])
    stop.record(stream)
    barrier()
    e2e_blocking_ms = replicas.max_over_ranks(start.elapsed_time(stop), device="cuda")
    assert torch.equal(houts[0], houts[1])
    e2e = {"value": world * BATCH * e2e_steps / (e2e_ms * 1e-3), "unit": UNIT,
           "h2d_bytes_per_step": int(hins[0].numel() * 4), "d2h_bytes_per_step": int(houts[0].numel() * 4), "steps": e2e_steps,
           "api": "tfjsb_run_model_host_async + tfjsb_model_host_wait, two steps in flight",
           "blocking_api_value": world * BATCH * e2e_steps / (e2e_blocking_ms * 1e-3)}

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
        "ms_per_step": elapsed_ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32 storage and accumulation; tf32 tensor-core multiplies in the GEMM-shaped layers",
        "data": "synthetic",
        "config": {"workload": WORKLOAD, "batch_per_gpu": BATCH, "math": "tf32",
                   "l2": "inputs larger than L2: a pass streams ~5 GB of activations, the largest tensors are 411 MB",
                   "replicas": world, "graph_replay": True},
        "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches),
    }

    if rank == 0:
        # ---- per-layer device times (event pair around every layer), roofline per op and for the dominant kernel
        reps = max(5, min(50, args.steps))
        ms = model.profile(x, out=out, reps=reps)
        fp32_tflops = props.multi_processor_count * 128 * 2 * (clocks["sm_max_mhz"] or 1965) * 1e6 / 1e12
        work, ms = label_and_merge(layer_work(layers, x_host.shape, tfjsb.window_out_shape), ms, model.layer_kernels())
        rows = roofline_rows(work, ms, peaks, fp32_tflops)
        by_kernel = {}
        for r in rows:
            k = by_kernel.setdefault(r["kernel"], dict(ms=0.0, launches=0))
            k["ms"] += r["ms"]
            k["launches"] += 1
        total_ms = sum(r["ms"] for r in rows)
        dominant = max(by_kernel, key=lambda k: by_kernel[k]["ms"])
        dom_rows = [r for r in rows if r["kernel"] == dominant]
        # the dominant kernel's launches that share its majority bound
        bound_ms = {}
        for r in dom_rows:
            bound_ms[r["bound"]] = bound_ms.get(r["bound"], 0.0) + r["ms"]
        bound = max(bound_ms, key=bound_ms.get)
        sel = [r for r in dom_rows if r["bound"] == bound]
        sel_s = sum(r["ms"] for r in sel) * 1e-3
        if bound == "hbm":
            achieved, unit = sum(r["bytes"] for r in sel) / sel_s / 1e9, "GB/s"
            peak, peak_sustained, peak_stated = peaks["hbm_gbs"], peaks["hbm_gbs"], STATED_PEAKS["hbm_gbs"]
            peak_source = peaks["source"] + " HBM copy bandwidth"
        elif bound == "tensor":
            achieved, unit = sum(r["flops"] for r in sel) / sel_s / 1e12, "TFLOP/s"
            peak, peak_sustained, peak_stated = (peaks["bf16_tflops"] / 2.0, peaks["bf16_tflops_sustained"] / 2.0,
                                                 STATED_PEAKS["tf32_tflops"])
            peak_source = peaks["source"] + " bf16 burst / 2 (nominal TF32:bf16 ratio; the layers are timed in a short burst)"
        else:
            achieved, unit = sum(r["flops"] for r in sel) / sel_s / 1e12, "TFLOP/s"
            peak = peak_sustained = peak_stated = fp32_tflops
            peak_source = "derived: SMs x 128 lanes x 2 x max SM clock"
        line["roofline"] = {
            "bound": bound, "achieved": achieved, "peak": peak, "unit": unit, "frac": achieved / peak,
            "traffic": traffic_of(dominant, sel),
            "algorithmic": int(sum(r["bytes"] for r in sel)) if bound == "hbm" else int(sum(r["flops"] for r in sel)),
            "kernel": dominant, "launches": [r["name"] for r in sel],
            "us_per_launch": [round(r["ms"] * 1e3, 2) for r in sel],
            "share_of_step": by_kernel[dominant]["ms"] / total_ms,
            "peak_source": peak_source,
            "frac_of_sustained_peak": achieved / peak_sustained, "frac_of_stated_peak": achieved / peak_stated,
            "stated_peak": peak_stated, "stated_peak_source": STATED_PEAKS["source"],
            "sm_mhz_during_timed_region": clocks["sm_mhz"],
            "how": "algorithmic bytes (or flops) of the listed launches / their summed CUDA-event durations, per pass; "
                   "kernel names come from the library (tfjsb_model_layer_kernel); traffic = ncu DRAM read+write bytes "
                   "per pass for the same launches, from a one-pass capture at the same batch (null: kernel changed since)",
        }
        line["roofline_step"] = {"sum_roofline_us": sum(r["roofline_us"] for r in rows), "sum_measured_us": total_ms * 1e3,
                                 "frac": sum(r["roofline_us"] for r in rows) / (total_ms * 1e3),
                                 "step_us": elapsed_ms / args.steps * 1e3,
                                 "frac_of_step": sum(r["roofline_us"] for r in rows) / (elapsed_ms / args.steps * 1e3)}
        line["per_kernel"] = {k: dict(v, share=v["ms"] / total_ms) for k, v in by_kernel.items()}
        line["per_op"] = [dict(name=r["name"], kernel=r["kernel"], us=round(r["ms"] * 1e3, 2), bound=r["bound"],
                               roofline_us=round(r["roofline_us"], 2), frac=round(r["frac"], 3),
                               frac_sustained=round(r["frac_sustained"], 3), frac_stated=round(r["frac_stated"], 3),
                               gbs=round(r["gbs"], 1), tflops=round(r["tflops"], 2)) for r in rows]

        # ---- batch-1 latency of the same model (the paper's Table 1 protocol: one inference, averaged over 100 runs)
        if world == 1:
            def timed_runs(fn, n=100, warm=10):
                """CUDA-event time of each of n calls of fn (each call enqueues on `stream`), in ms."""
                for _ in range(warm):
                    fn()
                torch.cuda.synchronize()
                evs = [torch.cuda.Event(enable_timing=True) for _ in range(n + 1)]
                evs[0].record(stream)
                for k in range(n):
                    fn()
                    evs[k + 1].record(stream)
                torch.cuda.synchronize()
                each = [evs[k].elapsed_time(evs[k + 1]) for k in range(n)]
                return {"mean_ms": evs[0].elapsed_time(evs[n]) / n, "median_ms": statistics.median(each), "min_ms": min(each)}

            x1h, _ = si.config_mobilenet(1.0, 224, 1, seed=si.CONFIG_SEEDS["mobilenet_100_224"])
            m1 = ctx.model(layers, x1h.shape)
            x1 = torch.from_numpy(x1h).cuda()
            o1 = torch.empty(m1.output_shape, device="cuda")
            plain = timed_runs(lambda: m1.run(x1, out=o1))
            m1.set_graph(True)
            graph = timed_runs(lambda: m1.run(x1, out=o1))
            ctx.check_device_status()
            b1_work = layer_work(layers, x1h.shape, tfjsb.window_out_shape)
            b1_roof_us = sum(max(r["bytes"] / (peaks["hbm_gbs"] * 1e9), r["flops"] / (peaks["bf16_tflops"] / 2 * 1e12))
                             for r in b1_work) * 1e6
            best = min(plain["mean_ms"], graph["mean_ms"])
            line["batch1"] = {"metric": "MobileNet v1 1.0 224 images/sec, batch 1", "value": 1e3 / best, "unit": UNIT,
                              "ms_per_inference_stream": plain["mean_ms"], "ms_per_inference_graph_replay": graph["mean_ms"],
                              "stream": plain, "graph_replay": graph, "launches_per_inference": m1.launches_per_run,
                              "roofline_us": b1_roof_us, "frac": b1_roof_us / (best * 1e3),
                              "note": "all weights and activations are L2-resident at batch 1; bound by each kernel's "
                                      "own critical path, not by bandwidth or arithmetic"}
            m1.close()
            # ---- the two single-op configurations (512^3 matMul; depthwise + pointwise block on 112x112x32), each
            # under graph replay beside its roofline time: both are far below one kernel's fixed latency
            a_h, b_h = si.config_matmul()
            a_d, b_d = torch.from_numpy(a_h).cuda(), torch.from_numpy(b_h).cuda()
            c_d = torch.empty((a_h.shape[0], b_h.shape[1]), device="cuda")
            ctx.matmul(a_d, b_d, out=c_d)  # scratch for the transposed operand is allocated here
            torch.cuda.synchronize()
            mm_stream = timed_runs(lambda: ctx.matmul(a_d, b_d, out=c_d))
            side = torch.cuda.Stream()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=side):
                ctx.matmul(a_d, b_d, out=c_d)
            mm_graph = timed_runs(lambda: g.replay())
            M = K = N = a_h.shape[0]
            mm_bytes, mm_flops = 4 * (M * K + K * N + M * N), 2 * M * K * N
            xb_h, block = si.config_separable_block()
            mb = ctx.model(block, xb_h.shape)
            xb = torch.from_numpy(xb_h).cuda()
            ob = torch.empty(mb.output_shape, device="cuda")
            blk_stream = timed_runs(lambda: mb.run(xb, out=ob))
            mb.set_graph(True)
            blk_graph = timed_runs(lambda: mb.run(xb, out=ob))
            blk_work = layer_work(block, xb_h.shape, tfjsb.window_out_shape)
            blk_kernels = mb.layer_kernels()
            ctx.check_device_status()
            mb.close()
            line["single_op_configs"] = {
                "matmul_512": {"stream": mm_stream, "graph_replay": mm_graph,
                               "roofline_us": max(mm_bytes / (peaks["hbm_gbs"] * 1e9), mm_flops / (peaks["bf16_tflops"] / 2 * 1e12)) * 1e6,
                               "tflops_graph_replay": mm_flops / (mm_graph["mean_ms"] * 1e-3) / 1e12,
                               "note": "includes the transpose of b into K-contiguous scratch (a second launch)"},
                "separable_block_112x112x32_64": {
                    "stream": blk_stream, "graph_replay": blk_graph, "kernels": blk_kernels,
                    "roofline_us": sum(max(r["bytes"] / (peaks["hbm_gbs"] * 1e9), r["flops"] / (peaks["bf16_tflops"] / 2 * 1e12))
                                       for r in blk_work) * 1e6},
                "note": "latency-bound: time per call under graph replay next to the roofline time of the same work"}
            # ---- the same model and batch in the narrow-storage mode (bfloat16 in memory, fp32 sums): a second
            # number beside the headline, never in place of it (the headline's storage format is fp32)
            ctx.set_math("bf16")
            try:
                mn = ctx.model(layers, x_host.shape)
            finally:
                ctx.set_math("tf32")
            on = torch.empty(mn.output_shape, device="cuda")
            for _ in range(5):
                mn.run(x, out=on)
            torch.cuda.synchronize()
            n_steps = max(20, min(200, args.steps))
            start.record(stream)
            for _ in range(n_steps):
                mn.run(x, out=on)
            stop.record(stream)
            torch.cuda.synchronize()
            ctx.check_device_status()
            narrow_ms = start.elapsed_time(stop) / n_steps
            layer_us = [round(v * 1e3, 2) for v in mn.profile(x, out=on, reps=10)]
            # end to end in the same mode: the host buffers stay fp32 (the first layer rounds as it reads)
            for i in range(4):
                mn.run_host_async(hins[i % 2], houts[i % 2])
            mn.host_wait()
            torch.cuda.synchronize()
            start.record(stream)
            for i in range(e2e_steps):
                mn.run_host_async(hins[i % 2], houts[i % 2])
            mn.host_wait()
            stop.record(stream)
            torch.cuda.synchronize()
            narrow_e2e_ms = start.elapsed_time(stop) / e2e_steps
            agree = float((on.argmax(-1) == out.argmax(-1)).float().mean())
            n_rows = narrow_layer_work(layers, x_host.shape, tfjsb.window_out_shape)
            n_roof = [max(r["bytes"] / (peaks["hbm_gbs"] * 1e9),
                          r["flops"] / (peaks["bf16_tflops_sustained"] * 1e12) if r["tensor"] else 0.0) * 1e6 for r in n_rows]
            line["narrow_storage"] = {
                "metric": METRIC + ", bfloat16 storage", "value": BATCH / (narrow_ms * 1e-3), "unit": UNIT,
                "ms_per_step": narrow_ms, "steps": n_steps,
                "e2e_value": BATCH / (narrow_e2e_ms * 1e-3),
                "dtype": "bf16 storage of filters and activations, exact products, f32 sums; model input and output f32",
                "top1_agreement_with_f32_storage": agree,
                "per_layer_us": dict(zip(mn.layer_names, layer_us)),
                "per_layer_roofline_us": dict(zip(mn.layer_names, [round(v, 2) for v in n_roof])),
                "roofline_step": {"sum_roofline_us": sum(n_roof), "sum_measured_us": sum(layer_us),
                                  "frac": sum(n_roof) / sum(layer_us),
                                  "how": "per layer the slower of its bytes (2-byte filters and activations, 4-byte "
                                         "input, biases, logits) at the measured HBM copy rate and, for the GEMM-shaped "
                                         "layers, its flops at the measured sustained bf16 rate"},
            }
            mn.close()
        if cpu_baseline is not None:
            line["cpu_baseline"] = cpu_baseline
        print(json.dumps(line), flush=True)

    model.close()
    ctx.close()
    if distributed:
        dist.barrier()
        dist.destroy_process_group()
    return 0


# DRAM bytes (read + write) per image of one launch, from a one-pass ncu capture (two DRAM byte counters and the
# duration, nothing saved or restored) of the same kernels on the same layers at batch 128, divided by 128.
# Reads are cold and equal the layer's input; writes are counted when L2 evicts them, so layers whose output is
# smaller than L2 under-count their writes.  Keyed by (kernel, launch name); an entry is dropped when its kernel changes.
TRAFFIC_BYTES_PER_IMAGE = {
    ("dwpw_fused_kernel<false>", "dw1+pw1"): 4340584, ("dwpw_fused_kernel<false>", "dw3+pw3"): 2808422,
    ("dwpw_fused_kernel<false>", "dw5+pw5"): 1182998,
    ("depthwise3x3_tma_kernel", "dw2"): 3846712, ("depthwise3x3_tma_kernel", "dw4"): 1830648,
    ("depthwise3x3_tma_kernel", "dw6"): 843598, ("depthwise3x3_tma_kernel", "dw7"): 431010,
    ("depthwise3x3_tma_kernel", "dw8"): 432776, ("depthwise3x3_tma_kernel", "dw9"): 432746,
    ("depthwise3x3_tma_kernel", "dw10"): 432158, ("depthwise3x3_tma_kernel", "dw11"): 432582,
    ("depthwise3x3_tma_kernel", "dw12"): 401734, ("depthwise3x3_tma_kernel", "dw13"): 201166,
}


def traffic_of(kernel, rows):
    vals = [TRAFFIC_BYTES_PER_IMAGE.get((kernel, r["name"])) for r in rows]
    return None if (not vals or any(v is None for v in vals)) else int(sum(vals) * BATCH)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=500)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--reference-images", type=int, default=8,
                    help="reference arm: images of the batch the oracle processes per step")
    ap.add_argument("--no-cpu-baseline", action="store_true", help="skip the oracle timing leg")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())

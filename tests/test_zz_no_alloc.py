"""The allocation-free matMul entry point against the ordinary one.

tfjsb_matmul_static_scratch exists for callers that cannot call cudaMalloc where they call the
library (a real-time loop that may not block on the allocator, a service with a device-memory
budget fixed at start-up): it transposes operands into a fixed array inside the library instead
of allocated scratch.  It runs the same kernels on the same data as tfjsb_matmul, so its output
must be bit-identical, call after call, although the array still holds the previous call's
operands.  This file is collected last so that a run that stops at the first failure has already
run every other test.
"""
import numpy as np
import pytest

import seeded_inputs as si
from helpers import dev, host, rel_fro, same_bits

pytestmark = pytest.mark.gpu


def test_static_scratch_matmul_matches_matmul_on_two_calls_in_a_row(ctx, oracle):
    import torch

    cases = [
        # M, K, N, transpose_a, transpose_b: the second call is smaller, leaving stale data behind it
        (512, 512, 512, False, False),
        (260, 96, 132, True, False),
    ]
    for M, K, N, ta, tb in cases:
        a = si.uniform(901, 0, (K, M) if ta else (M, K), -1, 1)
        b = si.uniform(901, 1, (N, K) if tb else (K, N), -1, 1)
        ad, bd = dev(a), dev(b)
        out = torch.empty(M, N, device="cuda")
        ctx.matmul_static_scratch(ad, bd, ta, tb, out=out)
        ctx.check_device_status()
        got = host(out)
        assert same_bits(got, host(ctx.matmul(ad, bd, ta, tb)))
        assert rel_fro(got, oracle.matmul(a, b, ta, tb)) <= 5e-3
    # the first problem's shape again, with new values, straight after a different problem:
    # whatever the array still holds must not leak into the result
    M, K, N, ta, tb = cases[0]
    a = si.uniform(902, 0, (M, K), -1, 1)
    b = si.uniform(902, 1, (K, N), -1, 1)
    out = torch.empty(M, N, device="cuda")
    ctx.matmul_static_scratch(dev(a), dev(b), ta, tb, out=out)
    assert same_bits(host(out), host(ctx.matmul(dev(a), dev(b), ta, tb)))
    ctx.check_device_status()


def test_static_scratch_matmul_takes_no_device_memory(ctx):
    """Free device memory as the driver reports it (not torch's allocator, which the library does not use)
    is the same before and after a call that has to transpose both operands.  One call comes first so that
    the kernels' code is resident: loading it is a one-time cost of the library, not of the call."""
    import torch

    a = dev(si.uniform(903, 0, (96, 260), -1, 1))    # stored [K, M]: transposed
    b = dev(si.uniform(903, 1, (96, 132), -1, 1))    # stored [K, N]: transposed
    out = torch.empty(260, 132, device="cuda")
    ctx.matmul_static_scratch(a, b, True, False, out=out)
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    ctx.matmul_static_scratch(a, b, True, False, out=out)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before
    ctx.check_device_status()


def test_static_scratch_matmul_rejects_problems_beyond_its_array(ctx, tfjsb):
    import torch

    before = ctx.launch_count
    a = torch.zeros(64, 4096, device="cuda")
    b = torch.zeros(4096, 2048, device="cuda")  # 8 Mi floats to transpose: twice the array
    with pytest.raises(tfjsb.TfjsbError) as err:
        ctx.matmul_static_scratch(a, b, out=torch.empty(64, 2048, device="cuda"))
    assert err.value.status_name == "UNSUPPORTED"
    assert "static scratch" in str(err.value)
    assert ctx.launch_count == before
    # operands that are already K-contiguous need no scratch, whatever their size
    bt = torch.zeros(2048, 4096, device="cuda")
    ctx.matmul_static_scratch(a, bt, False, True, out=torch.empty(64, 2048, device="cuda"))
    ctx.check_device_status()

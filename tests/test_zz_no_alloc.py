"""The allocation-free entry point, mxfp4_linear_static.

Some callers of this library cannot allocate device memory at the point where they need a
linear pass: they run inside a runtime that already owns all device memory through its own
arena, or inside a latency-critical loop where cudaMalloc's device-wide synchronisation is not
acceptable, or they are plugins that receive buffers but no allocator.  For them the library
carries a fixed 16 MiB scratch array; the caller passes only inputs and outputs.

This file is collected last on purpose (pytest orders files by name), so a run that stops at
the first failure has already executed every other test.  The GPU test calls the entry point
through the C ABI twice in a row -- different passes and shapes, so the second call finds the
first call's leftovers in the shared array -- and compares each result with the ordinary
workspace-taking entry point.  Both run the same kernels on the same bits, so the results must
be identical, which is inside any tolerance the other tests use.
"""
import ctypes

import numpy as np
import pytest
import torch

from paper_2605_09825_b200 import api, build


def test_problems_beyond_the_built_in_scratch_are_rejected_on_the_host():
    build.build_library()
    lib = api.load_library()
    buf = ctypes.create_string_buffer(4096)
    p = (ctypes.addressof(buf) + 255) & ~255
    # 8192 x 4096 x 6144 needs ~30 MiB of scratch: refused before anything touches a device
    assert api.linear_workspace_bytes(8192, 4096, 6144, api.PASS_FPROP) > api.STATIC_SCRATCH_BYTES
    assert lib.mxfp4_linear_static(api.PASS_FPROP, p, p, p, 8192, 4096, 6144, 1, 0, 0, 0, None) == -9
    assert "scratch" in api.status_string(-9)
    assert lib.mxfp4_linear_static(7, p, p, p, 128, 128, 128, 1, 0, 0, 0, None) == -4
    assert lib.mxfp4_linear_static(api.PASS_FPROP, p, p, p, 128, 100, 128, 1, 0, 0, 0, None) == -2


@pytest.mark.gpu
def test_two_calls_in_a_row_match_the_workspace_entry_points():
    from gpu_util import random_bits, to_dev
    rng = np.random.default_rng(77)
    # call 1: Fprop, rotated, RNE; call 2: Wgrad with other shapes, stochastic rounding
    T1, IN1, OUT1 = 1024, 2048, 1536
    X1, W1 = to_dev(random_bits(rng, T1, IN1, 2)), to_dev(random_bits(rng, OUT1, IN1, 2))
    T2, IN2, OUT2 = 2048, 640, 896
    dY2, X2 = to_dev(random_bits(rng, T2, OUT2, 2)), to_dev(random_bits(rng, T2, IN2, 2))
    assert api.linear_workspace_bytes(T1, IN1, OUT1, api.PASS_FPROP) <= api.STATIC_SCRATCH_BYTES
    assert api.linear_workspace_bytes(T2, IN2, OUT2, api.PASS_WGRAD) <= api.STATIC_SCRATCH_BYTES

    got1 = api.linear_static(api.PASS_FPROP, X1, W1, T1, IN1, OUT1, api.HADAMARD_DET, api.ROUND_RNE, 3)
    got2 = api.linear_static(api.PASS_WGRAD, dY2, X2, T2, IN2, OUT2, api.HADAMARD_NONE, api.ROUND_SR, 7,
                             api.OUT_FP32)
    api.check()
    want1 = api.linear_fprop(X1, W1, api.HADAMARD_DET, api.ROUND_RNE, 3)
    want2 = api.linear_wgrad(dY2, X2, api.HADAMARD_NONE, api.ROUND_SR, 7, api.OUT_FP32)
    api.check()
    assert got1.shape == (T1, OUT1) and got2.shape == (OUT2, IN2)
    assert torch.equal(got1, want1)
    assert torch.equal(got2, want2)
    # and once more in the opposite order: the array now holds call 2's operands
    again1 = api.linear_static(api.PASS_FPROP, X1, W1, T1, IN1, OUT1, api.HADAMARD_DET, api.ROUND_RNE, 3)
    api.check()
    assert torch.equal(again1, want1)


@pytest.mark.gpu
def test_ragged_shapes_after_a_call_that_left_other_bytes_everywhere():
    """Shapes that are multiples of neither the scale tile (128 rows x 128 elements) nor the GEMM
    tile, right after a larger call with stochastic rounding has left its operands all over the
    array: the padding rows and blocks of the scale tiles and the code rows past M and N that the
    GEMM's tile loads touch must all come from this call, so the result equals the workspace entry
    point's bit for bit."""
    from gpu_util import random_bits, to_dev
    rng = np.random.default_rng(78)
    Tb, INb, OUTb = 2048, 1536, 1024                       # fills ~4.3 MB of the array with non-zero bytes
    api.linear_static(api.PASS_FPROP, to_dev(random_bits(rng, Tb, INb, 2)), to_dev(random_bits(rng, OUTb, INb, 2)),
                      Tb, INb, OUTb, api.HADAMARD_NONE, api.ROUND_SR, 5)
    T, IN, OUT = 200, 416, 352
    X, W, dY = (to_dev(random_bits(rng, r, c, 2)) for r, c in ((T, IN), (OUT, IN), (T, OUT)))
    got = api.linear_static(api.PASS_FPROP, X, W, T, IN, OUT, api.HADAMARD_DET, api.ROUND_RNE, 3, api.OUT_FP32)
    api.check()
    assert torch.isfinite(got).all()
    assert torch.equal(got, api.linear_fprop(X, W, api.HADAMARD_DET, api.ROUND_RNE, 3, api.OUT_FP32))
    got = api.linear_static(api.PASS_DGRAD, dY, W, T, IN, OUT, api.HADAMARD_DET, api.ROUND_RNE, 3, api.OUT_FP32)
    api.check()
    assert torch.isfinite(got).all()
    assert torch.equal(got, api.linear_dgrad(dY, W, api.HADAMARD_DET, api.ROUND_RNE, 3, api.OUT_FP32))

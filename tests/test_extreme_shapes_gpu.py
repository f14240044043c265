"""Shapes at the far ends of what the kernels index: one dimension in the millions with the
others at their minimum, for the quantizers (both orientations, the dual-axis kernel) and for the
GEMM.  Everything is compared with the CPU oracle element by element -- the oracle finishes these
in seconds because the long dimension is the only large one.  (The largest element COUNTS, beyond
2^31 per tensor, are covered by the full-size tests.)"""
import numpy as np
import pytest
import torch

import oracle
from gpu_util import assert_gemm_close, gpu_quantize, random_bits, to_dev
from paper_2605_09825_b200 import api

pytestmark = pytest.mark.gpu

LONG = (1 << 20) + 96          # not a multiple of the 128-wide tiles


def _dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


@pytest.mark.parametrize("rows,cols", [(LONG, 32), (32, LONG)])
@pytest.mark.parametrize("axis", [0, 1])
@pytest.mark.parametrize("hmode,rnd", [(api.HADAMARD_DET, api.ROUND_RNE), (api.HADAMARD_NONE, api.ROUND_SR)])
def test_quantize_one_long_dimension(rows, cols, axis, hmode, rnd):
    rng = np.random.default_rng(rows % 1000 + axis)
    bits = random_bits(rng, rows, cols)
    want_codes, want_scales = oracle.quantize(bits, axis, hmode, rnd, 7, 1)
    codes, scales, _ = gpu_quantize(bits, axis, hmode, rnd, 7, 1)
    assert np.array_equal(scales, want_scales)
    assert np.array_equal(codes, want_codes)


@pytest.mark.parametrize("rows,cols", [(LONG, 32), (32, LONG)])
def test_dual_quantize_one_long_dimension(rows, cols):
    rng = np.random.default_rng(cols % 1000)
    bits = random_bits(rng, rows, cols)
    (cr, sr), (cc, sc) = api.quantize_dual(to_dev(bits), api.HADAMARD_DET, api.ROUND_RNE, 0)
    api.check()
    for axis, codes, raw in ((1, cr, sr), (0, cc, sc)):
        outer, K = (rows, cols) if axis == 1 else (cols, rows)
        want_codes, want_scales = oracle.quantize(bits, axis, api.HADAMARD_DET, api.ROUND_RNE, 0, 0)
        assert np.array_equal(oracle.scales_from_tiled(raw.cpu().numpy(), outer, K // 32), want_scales)
        assert np.array_equal(codes.cpu().numpy(), want_codes)


@pytest.mark.parametrize("M,N,K,out_dtype", [(LONG, 8, 32, api.OUT_BF16), (LONG, 4, 32, api.OUT_FP32),
                                            (8, LONG, 32, api.OUT_BF16)])
def test_gemm_one_long_dimension(M, N, K, out_dtype):
    rng = np.random.default_rng(M % 1000 + N)
    ac = rng.integers(0, 256, (M, K // 2), dtype=np.uint8)
    bc = rng.integers(0, 256, (N, K // 2), dtype=np.uint8)
    asc = rng.integers(120, 134, (M, K // 32), dtype=np.uint8)
    bsc = rng.integers(120, 134, (N, K // 32), dtype=np.uint8)
    out = api.gemm(_dev(ac), _dev(oracle.scales_to_tiled(asc)), _dev(bc), _dev(oracle.scales_to_tiled(bsc)), 0.5,
                   out_dtype)
    api.check()
    ref, S = oracle.gemm(ac, asc, bc, bsc, alpha=0.5)
    assert_gemm_close(out.float().cpu().numpy(), ref, S, out_dtype == api.OUT_BF16, f"{M}x{N}x{K}")


@pytest.mark.parametrize("K,same_sign", [(LONG - 64, False), (LONG - 64, True), (28672, True), (28672, False)])
def test_gemm_long_k_and_what_fp32_accumulation_costs(K, same_sign):
    """The tensor cores add each K = 64 partial product into the fp32 accumulator in TMEM with
    truncation, not round-to-nearest.  A sum of n = K / 64 steps is therefore off, towards zero,
    by up to one ulp of the running sum per step: at most n * 2^-24 * sum|products| for
    magnitudes spread evenly along K (the running sum of magnitudes grows linearly), and that
    much only when all products have one sign.  Measured here: 0.3 * n * 2^-24 * sum|products|
    for same-sign products (1.0e-5 at K = 28672, 3.0e-4 at K = 2^20), 1.2e-6 at K = 28672 and
    1.0e-5 at K = 2^20 for products of mixed sign (every benchmark configuration; any rotated
    operand).  So 1e-5 * sum|products| holds on mixed-sign data up to K of about a million and on
    same-sign data up to K of about 28 000; beyond, the bound the arithmetic gives applies."""
    M = N = 40
    rng = np.random.default_rng(5 + K % 7)
    ac = rng.integers(0, 256, (M, K // 2), dtype=np.uint8)
    bc = rng.integers(0, 256, (N, K // 2), dtype=np.uint8)
    if same_sign:
        ac &= 0x77
        bc &= 0x77
    asc = rng.integers(120, 134, (M, K // 32), dtype=np.uint8)
    bsc = rng.integers(120, 134, (N, K // 32), dtype=np.uint8)
    out = api.gemm(_dev(ac), _dev(oracle.scales_to_tiled(asc)), _dev(bc), _dev(oracle.scales_to_tiled(bsc)), 1.0,
                   api.OUT_FP32)
    api.check()
    ref, S = oracle.gemm(ac, asc, bc, bsc, alpha=1.0)
    err = out.cpu().numpy().astype(np.float64) - ref
    n = (K + 63) // 64
    assert (np.abs(err) <= n * 2.0 ** -24 * S).all()
    if same_sign:
        assert (err <= 0).all()                        # every sum is positive: truncation only lowers it
        assert (np.abs(err) <= 0.5 * n * 2.0 ** -24 * S).all()
    elif K <= 28672:
        assert (np.abs(err) <= 1e-5 * S).all()         # the stated tolerance, with room: mixed signs
        assert (np.abs(err) <= 3e-6 * S).all()

"""The 8-bit passes of the precision ladder (MXFP8) on the GPU vs the CPU oracle, through the
C ABI: codes and scales bit-exact, GEMM within the fp32-accumulation tolerance."""
import numpy as np
import pytest
import torch

import oracle
from gpu_util import assert_gemm_close, random_bits, to_dev
from paper_2605_09825_b200 import api, synth

pytestmark = pytest.mark.gpu


def _mixed_bits(rng, rows, cols):
    x = rng.standard_normal((rows, cols)).astype(np.float32)
    x *= np.exp2(rng.integers(-10, 6, size=(rows, cols))).astype(np.float32)   # reaches the sub-normal codes
    u = x.view(np.uint32)
    return ((u + 0x7FFF + ((u >> 16) & 1)) >> 16).astype(np.uint16)


def _check_quant(bits, axis, layout=api.SCALES_TILED):
    codes, scales = api.quantize_fp8(to_dev(bits), axis, layout)
    api.check()
    wc, ws = oracle.quantize_mxfp8(bits, axis)
    outer, nt = ws.shape
    raw = scales.cpu().numpy()
    got_s = oracle.scales_from_tiled(raw, outer, nt) if layout == api.SCALES_TILED else raw.reshape(outer, nt)
    assert np.array_equal(got_s, ws)
    bad = np.argwhere(codes.cpu().numpy() != wc)
    assert bad.size == 0, f"{len(bad)} codes differ, first at {bad[:4].tolist()}"


@pytest.mark.parametrize("axis", [1, 0])
@pytest.mark.parametrize("rows,cols", [(32, 32), (1, 64), (96, 160), (300, 416), (1000, 1184), (520, 2048)])
def test_quantize_ragged_shapes(rows, cols, axis):
    if axis == 0 and (rows % 32 or cols % 8):
        pytest.skip("column-wise blocks need rows % 32 == 0 and cols % 8 == 0")
    _check_quant(_mixed_bits(np.random.default_rng(rows + cols), rows, cols), axis)


def test_quantize_every_bf16_magnitude_and_both_signs():
    """All 2^16 bf16 patterns except NaN/inf, each in a block whose maximum fixes the scale, so the
    hardware conversion meets every rounding case of the format (ties, sub-normals, saturation)."""
    pats = np.arange(1 << 16, dtype=np.uint16)
    pats = pats[(pats & 0x7F80) != 0x7F80]
    n = (len(pats) + 30) // 31
    bits = np.zeros((n, 32), dtype=np.uint16)
    bits[:, 0] = 0x43E8                                   # 464.0: block maximum, fixes scale 2^0 and saturates
    flat = np.zeros(n * 31, dtype=np.uint16)
    flat[:len(pats)] = pats
    bits[:, 1:] = flat.reshape(n, 31)
    # keep only patterns not above the block maximum (larger ones would move the scale)
    big = (bits[:, 1:] & 0x7FFF) > 0x43E8
    bits[:, 1:][big] = 0
    _check_quant(bits, 1, api.SCALES_CANONICAL)


def test_quantize_canonical_layout_and_strided_source():
    rng = np.random.default_rng(5)
    _check_quant(_mixed_bits(rng, 288, 352), 0, api.SCALES_CANONICAL)
    full = _mixed_bits(rng, 200, 512)
    view = to_dev(full)[:, 64:64 + 256]
    codes, scales = api.quantize_fp8(view, 1)
    api.check()
    wc, ws = oracle.quantize_mxfp8(np.ascontiguousarray(full[:, 64:64 + 256]), 1)
    assert np.array_equal(codes.cpu().numpy(), wc)
    assert np.array_equal(oracle.scales_from_tiled(scales.cpu().numpy(), 200, 8), ws)


@pytest.mark.parametrize("M,N,K", [(128, 192, 128), (256, 384, 512), (300, 200, 96), (520, 1000, 1184), (64, 8, 32)])
@pytest.mark.parametrize("out_dtype", [api.OUT_FP32, api.OUT_BF16])
def test_gemm_random_codes(M, N, K, out_dtype):
    rng = np.random.default_rng(M + N + K)
    a_codes = rng.integers(0, 256, (M, K)).astype(np.uint8)
    b_codes = rng.integers(0, 256, (N, K)).astype(np.uint8)
    a_codes[(a_codes & 0x7F) == 0x7F] = 0x41
    b_codes[(b_codes & 0x7F) == 0x7F] = 0xC1
    a_scales = rng.integers(118, 132, (M, K // 32)).astype(np.uint8)
    b_scales = rng.integers(118, 132, (N, K // 32)).astype(np.uint8)
    dev = lambda x: torch.from_numpy(x).cuda()
    out = api.gemm_fp8(dev(a_codes), dev(oracle.scales_to_tiled(a_scales)), dev(b_codes),
                       dev(oracle.scales_to_tiled(b_scales)), 0.25, out_dtype)
    api.check()
    ref, S = oracle.gemm_mxfp8(a_codes, a_scales, b_codes, b_scales, alpha=0.25)
    assert_gemm_close(out.float().cpu().numpy(), ref, S, out_dtype == api.OUT_BF16, f"fp8 gemm {M}x{N}x{K}")


@pytest.mark.parametrize("pass_", [0, 1, 2])
def test_linear_pass_at_8_bits_matches_the_oracle(pass_):
    rng = np.random.default_rng(40 + pass_)
    T, in_f, out_f = 416, 288, 672
    X, W, dY = random_bits(rng, T, in_f, 3), random_bits(rng, out_f, in_f, 2), random_bits(rng, T, out_f, 4)
    a, b = ((X, W), (dY, W), (dY, X))[pass_]
    out = api.linear_pass(pass_, api.PRECISION_MXFP8, to_dev(a), to_dev(b), out_dtype=api.OUT_FP32)
    api.check()
    ref, S = oracle.linear_pass_mxfp8(pass_, a, b)
    assert_gemm_close(out.cpu().numpy(), ref, S, False, f"8-bit pass {pass_}")


def test_linear_pass_at_4_bits_is_the_per_pass_entry_point():
    rng = np.random.default_rng(50)
    X, W = to_dev(random_bits(rng, 256, 512)), to_dev(random_bits(rng, 384, 512))
    a = api.linear_pass(api.PASS_FPROP, api.PRECISION_MXFP4, X, W, 1, 0, 3)
    assert torch.equal(a, api.linear_fprop(X, W, 1, 0, 3))
    with pytest.raises(api.Mxfp4Error) as exc:
        api.linear_pass(api.PASS_FPROP, 3, X, W)
    assert exc.value.status == -4


def test_8_bit_pass_is_closer_to_the_exact_product_than_the_4_bit_pass():
    """The ladder's premise: an FP8 pass carries less quantization error than an MXFP4 pass."""
    t = synth.linear_tensors("o", 512, 4)
    X, W = to_dev(t["X"]), to_dev(t["W"])
    ref = X.double() @ W.double().t()
    snr = lambda got: 10 * np.log10(ref.pow(2).sum().item() / (got.double() - ref).pow(2).sum().item())
    s8 = snr(api.linear_pass(api.PASS_FPROP, api.PRECISION_MXFP8, X, W, out_dtype=api.OUT_FP32))
    s4 = snr(api.linear_pass(api.PASS_FPROP, api.PRECISION_MXFP4, X, W, 1, 0, 0, out_dtype=api.OUT_FP32))
    api.check()
    assert s8 > s4 + 10.0, (s8, s4)

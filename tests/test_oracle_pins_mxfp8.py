"""Pins for the 8-bit (MXFP8: E4M3 elements, E8M0 block scales) part of the oracle: the format's
published bit layout via torch's float8_e4m3fn (a library routine), closed forms in exact
rational arithmetic, hand-worked blocks, numpy matmul.  No GPU needed."""
from fractions import Fraction

import numpy as np
import torch

import oracle
from conftest import read_golden_lines
from test_oracle_pins import bf16_bits, bf16_fraction, floor_log2


def _grid():
    """The 127 finite magnitudes straight from the definition: sub-normals m * 2^-9, normals
    (1 + m/8) * 2^(e-7) up to 448."""
    g = [Fraction(m, 8) * Fraction(1, 64) for m in range(8)]
    for e in range(1, 16):
        for m in range(8):
            if e == 15 and m == 7:
                continue
            g.append((1 + Fraction(m, 8)) * Fraction(2) ** (e - 7))
    return g


GRID8 = _grid()


def _random_bits(rng, rows, cols, spread=6):
    x = rng.standard_normal((rows, cols)) * np.exp2(rng.integers(-spread, spread, (rows, cols)))
    return (x.astype(np.float32).view(np.uint32) >> 16).astype(np.uint16)


def test_decode_matches_the_definition_and_torch():
    codes = torch.arange(256, dtype=torch.uint8)
    lib = codes.view(torch.float8_e4m3fn).double().numpy()
    assert len(GRID8) == 127 and GRID8[-1] == 448
    for c in range(256):
        if c & 0x7F == 0x7F:
            assert np.isnan(lib[c])
            continue
        want = GRID8[c & 0x7F] * (-1 if c & 0x80 else 1)
        assert Fraction(oracle.e4m3_decode(c)) == want
        assert oracle.e4m3_decode(c) == lib[c]
    assert np.signbit(oracle.e4m3_decode(0x80))


def test_encode_matches_torch_round_to_nearest_even_inside_the_range():
    rng = np.random.default_rng(61)
    x = (rng.standard_normal(200000) * np.exp2(rng.integers(-12, 9, 200000))).astype(np.float32)
    x = x[np.abs(x) < 464.0]                           # torch has no saturation: beyond that it gives NaN
    want = torch.from_numpy(x).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    got = np.array([oracle.e4m3_encode(float(v)) for v in x], dtype=np.uint8)
    assert (got == want).all()


def test_encode_is_the_nearest_grid_point_ties_to_even_and_saturates():
    # every bf16 pattern up to 2^10 in magnitude, against the argmin of the exact distance
    for p in range(0, 0x4480):                         # 0 .. 1024.0
        x = bf16_fraction(p)
        want = min(range(127), key=lambda c: (abs(x - GRID8[c]), c % 2))
        if x >= 448:
            want = 126
        f = float(np.array([p << 16], dtype=np.uint32).view(np.float32)[0])
        assert oracle.e4m3_encode(f) == want, (hex(p), want)
        assert oracle.e4m3_encode(-f) == (want | 0x80)
    # the ties themselves: midpoints of neighbouring grid points go to the even code
    for c in range(126):
        mid = (GRID8[c] + GRID8[c + 1]) / 2
        f = float(mid)
        assert Fraction(f) == mid                      # representable in fp32
        assert oracle.e4m3_encode(f) == (c if c % 2 == 0 else c + 1)
    for big in (448.0, 463.9, 464.0, 480.0, 511.9, 1e30):
        assert oracle.e4m3_encode(big) == 0x7E and oracle.e4m3_encode(-big) == 0xFE


def test_hand_worked_block():
    """The block worked by hand in tests/golden/worked_blocks_32x32_and_mxfp8.txt."""
    g = [ln.split() for ln in read_golden_lines("worked_blocks_32x32_and_mxfp8.txt") if ln.startswith("mxfp8_block")][0]
    vals = [3.0, 1.0, -0.75, 2.0 ** -15, 2.0 ** -17] + [0.0] * 27
    bits = np.array([[bf16_bits(v) for v in vals]], dtype=np.uint16)
    codes, scales = oracle.quantize_mxfp8(bits, 1)
    assert scales[0, 0] == int(g[1])
    assert codes[0, :5].tolist() == [int(x, 16) for x in g[2:7]]
    assert (codes[0, 5:] == 0).all()


def test_scale_rule_and_saturation_band():
    """The scaled block maximum lies in [256, 512); above 448 it saturates to 448 (the 8-bit
    counterpart of the 4-bit format's (6, 8) band)."""
    rng = np.random.default_rng(67)
    bits = _random_bits(rng, 64, 96)
    codes, scales = oracle.quantize_mxfp8(bits, 1)
    x = (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    for o in range(64):
        for t in range(3):
            blk = x[o, 32 * t:32 * t + 32]
            amax = Fraction(float(np.abs(blk).max()))
            byte = int(scales[o, t])
            assert byte == max(0, min(254, floor_log2(amax) - 8 + 127))
            scaled = amax / Fraction(2) ** (byte - 127)
            assert 256 <= scaled < 512
            j = int(np.abs(blk).argmax())
            top = codes[o, 32 * t + j] & 0x7F
            assert 0x78 <= top <= 0x7E                 # exponent field 15
            if scaled >= 448:
                assert top == 0x7E
    zero = np.zeros((1, 32), dtype=np.uint16)
    c, s = oracle.quantize_mxfp8(zero, 1)
    assert s[0, 0] == 0 and (c == 0).all()


def test_requantizing_the_dequantized_block_is_idempotent_and_error_is_bounded():
    rng = np.random.default_rng(71)
    bits = _random_bits(rng, 32, 64, spread=2)
    codes, scales = oracle.quantize_mxfp8(bits, 1)
    x = (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    dec = np.array([oracle.e4m3_decode(int(c)) for c in codes.ravel()]).reshape(codes.shape)
    scale = np.exp2(np.repeat(scales.astype(np.float64), 32, axis=1) - 127)
    deq = dec * scale
    mag = np.abs(x) / scale
    # relative error <= 2^-4 for normal results, absolute <= 2^-10 (half a sub-normal step) below
    ok = np.where(mag >= 2.0 ** -6, np.abs(x - deq) <= np.abs(x) * 2.0 ** -4 + 1e-300,
                  np.abs(x - deq) <= 2.0 ** -10 * scale)
    assert ok[mag < 448].all()
    # dequantized values are bf16-representable here (4 significant bits), so feed them back
    back = (deq.astype(np.float32).view(np.uint32) >> 16).astype(np.uint16)
    assert ((back.astype(np.uint32) << 16).view(np.float32) == deq.astype(np.float32)).all()
    codes2, scales2 = oracle.quantize_mxfp8(back, 1)
    same_scale = scales2 == scales
    assert same_scale.mean() > 0.9
    rep = np.repeat(same_scale, 32, axis=1)
    assert (codes2[rep] == codes[rep]).all()


def test_axis0_equals_axis1_on_the_transposed_source():
    rng = np.random.default_rng(73)
    src = _random_bits(rng, 96, 80)
    a = oracle.quantize_mxfp8(src, 0)
    b = oracle.quantize_mxfp8(np.ascontiguousarray(src.T), 1)
    assert a[0].shape == (80, 96) and a[1].shape == (80, 3)
    assert (a[0] == b[0]).all() and (a[1] == b[1]).all()


def test_gemm_against_numpy_matmul_with_torch_decode():
    rng = np.random.default_rng(79)
    M, N, K = 24, 40, 96
    a_codes = rng.integers(0, 256, (M, K)).astype(np.uint8)
    b_codes = rng.integers(0, 256, (N, K)).astype(np.uint8)
    a_codes[(a_codes & 0x7F) == 0x7F] = 0x3A           # no NaN codes
    b_codes[(b_codes & 0x7F) == 0x7F] = 0xB1
    a_scales = rng.integers(120, 134, (M, K // 32)).astype(np.uint8)
    b_scales = rng.integers(120, 134, (N, K // 32)).astype(np.uint8)
    dec = lambda c: torch.from_numpy(c).view(torch.float8_e4m3fn).double().numpy()
    A = dec(a_codes) * np.exp2(np.repeat(a_scales.astype(np.float64), 32, axis=1) - 127)
    B = dec(b_codes) * np.exp2(np.repeat(b_scales.astype(np.float64), 32, axis=1) - 127)
    ref, S = oracle.gemm_mxfp8(a_codes, a_scales, b_codes, b_scales, alpha=0.5)
    assert np.allclose(ref, 0.5 * A @ B.T, rtol=1e-13, atol=0)
    assert np.allclose(S, 0.5 * np.abs(A) @ np.abs(B).T, rtol=1e-13, atol=0)
    rows = np.array([3, 0, 23])
    ref2, _ = oracle.gemm_mxfp8(a_codes, a_scales, b_codes, b_scales, alpha=0.5, rows=rows)
    assert (ref2 == ref[rows]).all()
    # a transposed-operand mistake would show here: one-hot A picks single elements of B
    a1 = np.zeros((1, K), dtype=np.uint8); a1[0, 37] = 0x38     # 1.0 at k = 37
    s1 = np.full((1, K // 32), 127, dtype=np.uint8)
    r, _ = oracle.gemm_mxfp8(a1, s1, b_codes, b_scales)
    assert np.array_equal(r[0], B[:, 37])


def test_linear_passes_use_the_operand_orientation_of_the_4_bit_path():
    """On operands that are exactly representable in E4M3 under their block scale the 8-bit pass
    is the exact product, whichever orientation it quantizes along."""
    rng = np.random.default_rng(83)
    T, in_f, out_f = 64, 96, 32
    mk = lambda r, c: np.vectorize(bf16_bits)(rng.integers(-8, 9, (r, c)).astype(np.float64) / 4).astype(np.uint16)
    X, W, dY = mk(T, in_f), mk(out_f, in_f), mk(T, out_f)
    f = lambda b: (b.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    ref, _ = oracle.linear_pass_mxfp8(0, X, W)
    assert np.array_equal(ref, f(X) @ f(W).T)
    ref, _ = oracle.linear_pass_mxfp8(1, dY, W)
    assert np.array_equal(ref, f(dY) @ f(W))
    ref, _ = oracle.linear_pass_mxfp8(2, dY, X)
    assert np.array_equal(ref, f(dY).T @ f(X))

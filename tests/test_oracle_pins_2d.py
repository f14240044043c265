"""Pins for the oracle's 32 x 32 block strategy (Appendix D): transpose invariance, a region
worked by hand, exact brute force in rational arithmetic, and its relation to the (separately
pinned) 1 x 32 quantizer.  No GPU needed."""
from fractions import Fraction

import numpy as np

import oracle
from conftest import read_golden_lines
from test_oracle_pins import (GRID, bf16_bits, bf16_fraction, expected_scale_byte, nearest_code, unpack)


def _random_bits(rng, rows, cols, spread=6):
    """bf16 patterns with magnitudes spread over several binades, both signs."""
    x = rng.standard_normal((rows, cols)) * np.exp2(rng.integers(-spread, spread, (rows, cols)))
    return (x.astype(np.float32).view(np.uint32) >> 16).astype(np.uint16)


def _nibbles(codes):
    out = np.empty((codes.shape[0], codes.shape[1] * 2), dtype=np.uint8)
    out[:, 0::2] = codes & 0xF
    out[:, 1::2] = codes >> 4
    return out


def test_2d_blocks_are_transpose_invariant_without_rotation():
    """Quantizing X along its rows and X along its columns gives the same code for every element
    and the same scale for every 32 x 32 region -- the property the strategy is named for."""
    rng = np.random.default_rng(41)
    src = _random_bits(rng, 96, 160)
    c1, s1 = oracle.quantize(src, 1, 0, 0, block2d=True)      # operand = X      [96 x 160]
    c0, s0 = oracle.quantize(src, 0, 0, 0, block2d=True)      # operand = X^T    [160 x 96]
    assert (_nibbles(c0) == _nibbles(c1).T).all()
    # region (R, C) of X: scale entries s1[32R + i][C] and s0[32C + j][R] all hold the same byte
    for R in range(3):
        for C in range(5):
            blk1 = s1[32 * R:32 * R + 32, C]
            blk0 = s0[32 * C:32 * C + 32, R]
            assert len(set(blk1.tolist()) | set(blk0.tolist())) == 1
    # ... which 1 x 32 blocks do not have
    d1, _ = oracle.quantize(src, 1, 0, 0)
    d0, _ = oracle.quantize(src, 0, 0, 0)
    assert (_nibbles(d0) != _nibbles(d1).T).any()


def test_hand_worked_region_with_one_outlier():
    """The region worked by hand in tests/golden/worked_blocks_32x32_and_mxfp8.txt: 32 x 32 of ones
    with one 48."""
    g = [ln.split() for ln in read_golden_lines("worked_blocks_32x32_and_mxfp8.txt") if ln.startswith("region32x32")][0]
    byte2d, code48, code1_2d, byte1d, code1_1d = (int(x) for x in g[1:])
    vals = np.full((32, 32), bf16_bits(1.0), dtype=np.uint16)
    vals[5, 9] = bf16_bits(48.0)
    codes, scales = oracle.quantize(vals, 1, 0, 0, block2d=True)
    assert (scales == byte2d).all()
    nib = _nibbles(codes)
    assert nib[5, 9] == code48
    nib[5, 9] = code1_2d
    assert (nib == code1_2d).all()
    codes1, scales1 = oracle.quantize(vals, 1, 0, 0)
    assert scales1[5, 0] == byte2d and (np.delete(scales1[:, 0], 5) == byte1d).all()
    assert (np.delete(_nibbles(codes1), 5, axis=0) == code1_1d).all()


def test_brute_force_in_rational_arithmetic_with_a_ragged_last_region():
    """Every region's scale and every element's code recomputed from the definition with exact
    fractions (no rotation, RNE): scale = 2^(floor(log2 max|x|) - 2) over the region, code =
    nearest grid point to x / scale (even code on ties, saturating at 6), sign kept."""
    rng = np.random.default_rng(43)
    for axis in (1, 0):
        # outer = 72 = 2 full regions + one of 8 rows, K = 64, either way round
        src = _random_bits(rng, 72, 64, spread=3) if axis == 1 else _random_bits(rng, 64, 72, spread=3)
        codes, scales = oracle.quantize(src, axis, 0, 0, block2d=True)
        view = src if axis == 1 else src.T
        outer, K = view.shape
        nib = _nibbles(codes)
        for g0 in range(0, outer, 32):
            g1 = min(g0 + 32, outer)
            for t in range(K // 32):
                vals = [[bf16_fraction(int(p)) for p in view[o, 32 * t:32 * t + 32]] for o in range(g0, g1)]
                byte = expected_scale_byte(max(abs(x) for row in vals for x in row))
                assert (scales[g0:g1, t] == byte).all()
                scale = Fraction(2) ** (byte - 127)
                for o in range(g0, g1):
                    for j, x in enumerate(vals[o - g0]):
                        want = nearest_code(min(abs(x) / scale, Fraction(6)))
                        sign = 8 if (int(view[o, 32 * t + j]) & 0x8000) else 0
                        assert nib[o, 32 * t + j] == (sign | want)


def test_region_scale_is_the_largest_row_scale_for_every_rotation_mode():
    """The scale byte grows with the block maximum, so a region's byte is the largest of the
    per-row bytes the 1 x 32 quantizer (pinned elsewhere) gives its rows; rows that already had
    that byte keep their codes, under RNE and -- same element indices, same random bits --
    under stochastic rounding."""
    rng = np.random.default_rng(47)
    src = _random_bits(rng, 96, 104)                      # axis 0: outer = 104 = 3 regions + 8 rows
    for mode in range(5):
        for rnd in (0, 1):
            for axis in (1, 0):
                if axis == 1:
                    s = np.ascontiguousarray(src[:, :96])
                else:
                    s = src
                c2, s2 = oracle.quantize(s, axis, mode, rnd, seed=5, tag=1, block2d=True)
                c1, s1 = oracle.quantize(s, axis, mode, rnd, seed=5, tag=1)
                outer = s1.shape[0]
                same_rows = 0
                for g0 in range(0, outer, 32):
                    g1 = min(g0 + 32, outer)
                    assert (s2[g0:g1] == s1[g0:g1].max(axis=0, keepdims=True)).all()
                    for o in range(g0, g1):
                        for t in range(s1.shape[1]):
                            if s1[o, t] == s2[o, t]:
                                same_rows += 1
                                assert (c2[o, 16 * t:16 * t + 16] == c1[o, 16 * t:16 * t + 16]).all()
                assert same_rows > 0


def test_2d_error_bound_and_dequantized_values():
    """Every element of a region lies within half a grid gap (times the region's scale) of its
    reconstruction; the region maximum maps into [4, 8), so only values in (6, 8) saturate."""
    rng = np.random.default_rng(53)
    src = _random_bits(rng, 64, 64, spread=2)
    codes, scales = oracle.quantize(src, 1, 0, 0, block2d=True)
    deq = oracle.dequantize(codes, scales)
    x = (src.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    scale = np.exp2(np.repeat(scales.astype(np.float64), 32, axis=1) - 127)
    mag = np.abs(x) / scale
    assert mag.max() < 8.0
    # grid gaps: 0.5 below 2, 1 from 2 to 4, 2 from 4 to 6; above 6 the value saturates (error < 2)
    bound = np.where(mag <= 2, 0.25, np.where(mag <= 4, 0.5, np.where(mag <= 6, 1.0, 2.0))) * scale
    assert (np.abs(x - deq) <= bound).all()

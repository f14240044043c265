"""Pins for the CPU oracle: every check here compares the oracle with something other than
itself -- hand-derived worked tiles, the generator's published known answers, closed forms
evaluated in exact rational arithmetic, library routines (scipy's Hadamard matrix, numpy's
matmul), invariants of the mathematics.  No GPU needed.
"""
from fractions import Fraction

import numpy as np
import pytest
import scipy.linalg

import oracle
from conftest import read_golden_lines

GRID = [Fraction(0), Fraction(1, 2), Fraction(1), Fraction(3, 2), Fraction(2), Fraction(3),
        Fraction(4), Fraction(6)]


# ----------------------------------------------------------------------------- helpers
def bf16_bits(x):
    """Exact bf16 pattern of a value known to be representable."""
    f = np.float32(x)
    u = int(np.array([f], dtype=np.float32).view(np.uint32)[0])
    assert u & 0xFFFF == 0, f"{x} is not a bf16 value"
    return np.uint16(u >> 16)


def bits_row(values):
    return np.array([[bf16_bits(v) for v in values]], dtype=np.uint16)


def bf16_fraction(p):
    """Exact rational value of a finite bf16 bit pattern."""
    sign = -1 if p & 0x8000 else 1
    e = (p >> 7) & 0xFF
    m = p & 0x7F
    assert e != 0xFF
    if e == 0:
        return sign * Fraction(m, 1 << 7) * Fraction(1, 1 << 126)
    return sign * (1 + Fraction(m, 1 << 7)) * (Fraction(2) ** (e - 127))


def floor_log2(q):
    """floor(log2 q) for a positive Fraction, by integer arithmetic only."""
    e = q.numerator.bit_length() - q.denominator.bit_length()
    if Fraction(2) ** e > q:
        e -= 1
    assert Fraction(2) ** e <= q < Fraction(2) ** (e + 1)
    return e


def expected_scale_byte(amax):
    """2^(floor(log2 amax) - 2) as an E8M0 byte, clamped; zero / sub-normal amax -> 0."""
    if amax < Fraction(1, 1 << 126):
        return 0
    return max(0, min(254, floor_log2(amax) - 2 + 127))


def nearest_code(a):
    """E2M1 magnitude code nearest to a >= 0: argmin of the exact distance, even code on ties."""
    return min(range(8), key=lambda c: (abs(a - GRID[c]), c % 2))


def unpack(codes_row):
    out = []
    for b in codes_row:
        out += [int(b) & 0xF, int(b) >> 4]
    return out


def quant_tile(values, **kw):
    codes, scales = oracle.quantize(bits_row(values), 1, **kw)
    return unpack(codes[0]), int(scales[0, 0])


# ----------------------------------------------------------------------------- P1 decode
def test_decode_table_is_the_e2m1_grid():
    codes = np.array([[(2 * i) | ((2 * i + 1) << 4) for i in range(8)] + [0] * 8], dtype=np.uint8)
    scales = np.array([[127]], dtype=np.uint8)
    deq = oracle.dequantize(codes, scales)[0, :16]
    want = [0, .5, 1, 1.5, 2, 3, 4, 6, -0., -.5, -1, -1.5, -2, -3, -4, -6]
    assert deq.tolist() == want
    assert np.signbit(deq[8])
    # the scale is a pure power of two: byte b multiplies by 2^(b-127)
    for b in (0, 1, 126, 128, 200, 254):
        d = oracle.dequantize(codes, np.array([[b]], dtype=np.uint8))[0, 7]
        assert d == 6.0 * 2.0 ** (b - 127)


# ----------------------------------------------------------------------------- P2 rounding
@pytest.mark.parametrize("tie,down,up", [(0.25, 0, 1), (0.75, 1, 2), (1.25, 2, 3), (1.75, 3, 4),
                                         (2.5, 4, 5), (3.5, 5, 6), (5.0, 6, 7)])
def test_rne_ties_go_to_the_even_code(tie, down, up):
    even = down if down % 2 == 0 else up
    t = np.float32(tie)
    tb = int(bf16_bits(t))
    below = np.array([tb - 1], dtype=np.uint16).astype(np.uint32) << 16
    above = np.array([tb + 1], dtype=np.uint16).astype(np.uint32) << 16
    below, above = below.view(np.float32)[0], above.view(np.float32)[0]
    # element 0 = 6.0 fixes the scale at 2^0; then tie, its bf16 neighbours, and negatives
    vals = [6.0, t, below, above, -t, -below, -above] + [0.0] * 25
    codes, byte = quant_tile(vals)
    assert byte == 127
    assert codes[:7] == [7, even, down, up, 8 | even, 8 | down, 8 | up]


def test_saturation_above_six():
    codes, byte = quant_tile([4.0, 6.0, 7.0, 7.9375, -7.5] + [0.0] * 27)
    assert byte == 127 and codes[:5] == [6, 7, 7, 7, 0xF]


# ----------------------------------------------------------------------------- P3 scale rule
@pytest.mark.parametrize("x,byte,code", [
    (1.0, 125, 0x6), (4.0, 127, 0x6), (6.0, 127, 0x7), (7.0, 127, 0x7), (3.984375, 126, 0x7),
    (0.0, 0, 0x0), (-1.0, 125, 0xE), (2.0 ** -10, 115, 0x6), (3.0 * 2.0 ** 20, 146, 0x7 - 1 + 0),
])
def test_scale_rule_spot_values(x, byte, code):
    # single non-zero element: scale = 2^(floor(log2|x|) - 2), so x/scale lands in [4, 8)
    if x == 3.0 * 2.0 ** 20:
        code = 0x7  # 3*2^20 / 2^19 = 6
    codes, b = quant_tile([x] + [0.0] * 31)
    assert (b, codes[0]) == (byte, code)
    assert codes[1:] == [0] * 31


def test_scale_rule_extremes():
    big = np.array([[0x7F7F] + [0] * 31], dtype=np.uint16)       # largest finite bf16
    codes, scales = oracle.quantize(big, 1)
    assert int(scales[0, 0]) == 252 and unpack(codes[0])[0] == 0x7
    tiny = np.array([[0x0001] + [0] * 31], dtype=np.uint16)      # smallest bf16 subnormal
    codes, scales = oracle.quantize(tiny, 1)
    assert int(scales[0, 0]) == 0 and unpack(codes[0])[0] == 0x0
    negzero = np.array([[0x8000] * 32], dtype=np.uint16)         # all -0: zero block keeps signs
    codes, scales = oracle.quantize(negzero, 1)
    assert int(scales[0, 0]) == 0 and unpack(codes[0]) == [8] * 32


# ----------------------------------------------------------------------------- P5 exhaustive
def test_every_bf16_pattern_as_single_nonzero_element():
    pats = [p for p in range(1 << 16) if ((p >> 7) & 0xFF) != 0xFF]
    src = np.zeros((len(pats), 32), dtype=np.uint16)
    pos = np.array([p % 32 for p in pats])
    src[np.arange(len(pats)), pos] = np.array(pats, dtype=np.uint16)
    codes, scales = oracle.quantize(src, 1)
    for i, p in enumerate(pats):
        x = bf16_fraction(p)
        byte = expected_scale_byte(abs(x))
        mag = nearest_code(abs(x) / Fraction(2) ** (byte - 127))
        want = ((p >> 15) << 3) | mag
        got = unpack(codes[i])
        assert int(scales[i, 0]) == byte, hex(p)
        assert got[pos[i]] == want, hex(p)
        assert sum(got) == want, hex(p)


def test_every_bf16_pattern_below_a_fixed_block_maximum():
    # element 1 = 1024 pins the scale at 2^8 while element 0 sweeps the whole sub-amax range
    pats = [p for p in range(1 << 16)
            if ((p >> 7) & 0xFF) != 0xFF and abs(bf16_fraction(p)) < 2048]
    src = np.zeros((len(pats), 32), dtype=np.uint16)
    src[:, 0] = np.array(pats, dtype=np.uint16)
    src[:, 1] = bf16_bits(1024.0)
    codes, scales = oracle.quantize(src, 1)
    assert (scales[:, 0] == 135).all()
    for i, p in enumerate(pats):
        mag = nearest_code(abs(bf16_fraction(p)) / 256)
        assert unpack(codes[i])[0] == (((p >> 15) << 3) | mag), hex(p)
        assert unpack(codes[i])[1] == 0x6


# ----------------------------------------------------------------------------- P4 / P6
def _random_bits(rng, rows, cols, spread=8):
    x = rng.standard_normal((rows, cols)).astype(np.float32)
    x *= np.exp2(rng.integers(-spread, spread, size=(rows, 1))).astype(np.float32)
    u = x.view(np.uint32)
    return ((u + 0x7FFF + ((u >> 16) & 1)) >> 16).astype(np.uint16)


def test_requantizing_the_dequantized_tile_is_idempotent():
    rng = np.random.default_rng(11)
    src = _random_bits(rng, 64, 256)
    codes, scales = oracle.quantize(src, 1)
    deq = oracle.dequantize(codes, scales).astype(np.float32)   # grid * 2^e is exact in bf16
    bits = (deq.view(np.uint32) >> 16).astype(np.uint16)
    assert ((deq.view(np.uint32) & 0xFFFF) == 0).all()
    codes2, scales2 = oracle.quantize(bits, 1)
    assert (codes2 == codes).all() and (scales2 == scales).all()


def test_rne_error_bound_and_block_maximum_lands_in_4_to_8():
    rng = np.random.default_rng(12)
    src = _random_bits(rng, 128, 512)
    x = (src.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    codes, scales = oracle.quantize(src, 1)
    deq = oracle.dequantize(codes, scales)
    scale = np.repeat(np.exp2(scales.astype(np.float64) - 127), 32, axis=1)
    s = np.abs(x) / scale
    amax_scaled = s.reshape(128, -1, 32).max(axis=2)
    assert (amax_scaled >= 4).all() and (amax_scaled < 8).all()
    bound = np.where(s < 2, 0.25, np.where(s < 4, 0.5, 1.0)) * scale
    unclipped = s <= 6
    assert (np.abs(x - deq)[unclipped] <= bound[unclipped]).all()
    assert (np.abs(deq)[~unclipped] == 6 * scale[~unclipped]).all()


# ----------------------------------------------------------------------------- P7 / P8 Hadamard
def test_fwht_matches_the_sylvester_matrix():
    H = scipy.linalg.hadamard(32).astype(np.float64)
    assert (H @ H.T == 32 * np.eye(32)).all()
    for j in range(32):
        e = np.zeros(32, dtype=np.float32)
        e[j] = 1
        assert (oracle.fwht32(e) == H[:, j]).all()
        assert H[3, j] == (-1) ** bin(3 & j).count("1")
    rng = np.random.default_rng(5)
    for _ in range(20):
        v = rng.integers(-64, 64, 32).astype(np.float32)
        hv = oracle.fwht32(v)
        assert (hv == H @ v).all()
        assert (oracle.fwht32(hv) == 32 * v).all()


def test_fwht_rounding_follows_the_fixed_stage_order():
    # with values that do not add exactly in fp32 the result depends on the association;
    # recompute the five stages with numpy fp32 vector ops (a different formulation: whole
    # stages as strided array slices) and demand identical bits
    rng = np.random.default_rng(6)
    for _ in range(50):
        v = (rng.standard_normal(32) * np.exp2(rng.integers(-20, 20, 32))).astype(np.float32)
        w = v.copy()
        for h in (1, 2, 4, 8, 16):
            w = w.reshape(-1, 2, h)
            w = np.stack([w[:, 0, :] + w[:, 1, :], w[:, 0, :] - w[:, 1, :]], axis=1).reshape(32)
        assert (oracle.fwht32(v).view(np.uint32) == w.view(np.uint32)).all()


def test_rotation_leaves_the_exact_inner_product_unchanged():
    rng = np.random.default_rng(7)
    for seed in (0, 7):
        m = oracle.sign_mask(seed)
        d = np.array([-1.0 if (m >> j) & 1 else 1.0 for j in range(32)], dtype=np.float32)
        for _ in range(20):
            a = rng.integers(-32, 32, 32).astype(np.float32)
            b = rng.integers(-32, 32, 32).astype(np.float32)
            assert float(oracle.fwht32(a) @ oracle.fwht32(b)) == 32 * float(a @ b)
            assert float(oracle.fwht32(a * d) @ oracle.fwht32(b * d)) == 32 * float(a @ b)


# ----------------------------------------------------------------------------- P9 / P10 worked tiles
def _worked():
    out = {}
    for ln in read_golden_lines("worked_tiles.txt"):
        f = ln.split()
        out[f[0]] = (int(f[1]), [int(c, 16) for c in f[2:]])
    return out


def test_worked_tiles():
    w = _worked()
    ramp = [j - 15.5 for j in range(32)]
    outlier = [1.0] * 32
    outlier[5] = 50.0
    assert quant_tile(ramp) == (w["ramp"][1], w["ramp"][0])
    assert quant_tile(ramp, hadamard_mode=1) == (w["ramp_h32"][1], w["ramp_h32"][0])
    assert quant_tile(outlier) == (w["outlier"][1], w["outlier"][0])
    assert quant_tile(outlier, hadamard_mode=1) == (w["outlier_h32"][1], w["outlier_h32"][0])


def test_worked_tiles_16_point_variant():
    w = _worked()
    ramp = [j - 15.5 for j in range(32)]
    outlier = [1.0] * 32
    outlier[5] = 50.0
    assert quant_tile(ramp, hadamard_mode=3) == (w["ramp_h16"][1], w["ramp_h16"][0])
    assert quant_tile(outlier, hadamard_mode=3) == (w["outlier_h16"][1], w["outlier_h16"][0])


def test_fwht16_matches_the_sylvester_matrix_per_half():
    H = scipy.linalg.hadamard(16).astype(np.float64)
    rng = np.random.default_rng(15)
    for _ in range(20):
        v = rng.integers(-64, 64, 32).astype(np.float32)
        hv = oracle.fwht16x2(v)
        assert (hv[:16] == H @ v[:16]).all() and (hv[16:] == H @ v[16:]).all()
        assert (oracle.fwht16x2(hv) == 16 * v).all()
    a = rng.integers(-32, 32, 32).astype(np.float32)
    b = rng.integers(-32, 32, 32).astype(np.float32)
    assert float(oracle.fwht16x2(a) @ oracle.fwht16x2(b)) == 16 * float(a @ b)
    # the 16-point butterfly is the first four stages of the 32-point one: bits must agree
    # with a numpy strided-stage formulation on values that do not add exactly
    for _ in range(20):
        v = (rng.standard_normal(32) * np.exp2(rng.integers(-20, 20, 32))).astype(np.float32)
        w = v.copy()
        for h in (1, 2, 4, 8):
            w = w.reshape(-1, 2, h)
            w = np.stack([w[:, 0, :] + w[:, 1, :], w[:, 0, :] - w[:, 1, :]], axis=1).reshape(32)
        assert (oracle.fwht16x2(v).view(np.uint32) == w.view(np.uint32)).all()


def test_randomized_16_point_is_sign_flip_then_rotation():
    rng = np.random.default_rng(18)
    src = _random_bits(rng, 16, 128)
    for seed in (0, 7):
        m = oracle.sign_mask(seed) & 0xFFFF
        flip = np.array([0x8000 if (m >> (j % 16)) & 1 else 0 for j in range(128)], dtype=np.uint16)
        a = oracle.quantize(src, 1, hadamard_mode=4, seed=seed)
        b = oracle.quantize(src ^ flip[None, :], 1, hadamard_mode=3)
        assert (a[0] == b[0]).all() and (a[1] == b[1]).all()


def test_rotation_disperses_the_outlier():
    outlier = np.ones(32)
    outlier[5] = 50.0
    H = scipy.linalg.hadamard(32).astype(np.float64)
    c0, s0 = oracle.quantize(bits_row(outlier), 1)
    c1, s1 = oracle.quantize(bits_row(outlier), 1, hadamard_mode=1)
    err0 = ((oracle.dequantize(c0, s0)[0] - outlier) ** 2).sum()
    err1 = ((H @ oracle.dequantize(c1, s1)[0] / 32 - outlier) ** 2).sum()
    assert err0 == 35.0 and err1 == 8.0


def test_randomized_rotation_is_sign_flip_then_rotation():
    rng = np.random.default_rng(8)
    src = _random_bits(rng, 16, 128)
    for seed in (0, 7):
        m = oracle.sign_mask(seed)
        flip = np.array([0x8000 if (m >> (j % 32)) & 1 else 0 for j in range(128)], dtype=np.uint16)
        a = oracle.quantize(src, 1, hadamard_mode=2, seed=seed)
        b = oracle.quantize(src ^ flip[None, :], 1, hadamard_mode=1)
        assert (a[0] == b[0]).all() and (a[1] == b[1]).all()


# ----------------------------------------------------------------------------- P11 Philox
def test_philox_known_answers():
    for ln in read_golden_lines("philox4x32_10_kat.txt"):
        w = [int(x, 16) for x in ln.split()]
        assert oracle.philox4x32_10(w[0:4], w[4:6]).tolist() == w[6:10]


def test_philox_counter_and_key_words_are_not_interchangeable():
    base = oracle.philox4x32_10([1, 2, 3, 4], [5, 6]).tolist()
    assert oracle.philox4x32_10([2, 1, 3, 4], [5, 6]).tolist() != base
    assert oracle.philox4x32_10([1, 2, 3, 4], [6, 5]).tolist() != base


# ----------------------------------------------------------------------------- P12 / P13 SR
def _sr_golden():
    g = {}
    for ln in read_golden_lines("sr_worked_tile.txt"):
        k, *v = ln.split()
        g[k] = v
    return g


def test_sr_worked_tile_and_sign_masks():
    g = _sr_golden()
    assert oracle.philox4x32_10([0, 0, 0, 0], [7, 0])[0] == int(g["first_philox_word"][0], 16)
    vals = [4.0] + [1.25] * 31
    codes, scales = oracle.quantize(bits_row(vals), 1, rounding=1, seed=7, tag=0)
    assert int(scales[0, 0]) == 127
    assert unpack(codes[0]) == [int(c, 16) for c in g["codes"]]
    assert [f"{b:02x}" for b in codes[0]] == g["packed"]
    assert oracle.sign_mask(7) == int(g["sign_mask_seed7"][0], 16)
    assert oracle.sign_mask(0) == int(g["sign_mask_seed0"][0], 16)


def test_sr_comparison_is_strict_at_equality():
    """u = (u8 + 1/2)/256 equal to frac stays down.  The random byte comes from the generator's
    published first vector, the expected codes from the hand derivation in the golden file."""
    g = _sr_golden()
    kat = [int(x, 16) for x in read_golden_lines("philox4x32_10_kat.txt")[0].split()]
    assert kat[:6] == [0] * 6
    u8 = (kat[6] >> 16) & 0xFF                       # element 2: byte 2 of word 0
    assert u8 == int(g["strict_u8_element2"][0], 16) == 39
    for n in (78, 79, 80):
        assert Fraction(n, 512) == Fraction(n, 1024) / Fraction(1, 2)          # frac between 0 and 0.5
        want = 1 if Fraction(2 * u8 + 1, 512) < Fraction(n, 512) else 0
        assert want == int(g[f"strict_n{n}_code"][0])
        vals = [4.0, 0.0, n / 1024] + [0.0] * 29
        codes, scales = oracle.quantize(bits_row(vals), 1, rounding=1, seed=0, tag=0)
        got = unpack(codes[0])
        assert int(scales[0, 0]) == 127 and got[0] == 6 and got[2] == want, (n, got[:4])
        assert all(c == 0 for i, c in enumerate(got) if i not in (0, 2))


def test_sr_is_unbiased_and_never_moves_grid_points():
    # row o of a [rows x 32] matrix uses element indices 32*o .. 32*o+31: fresh bits per row
    rows = 1 << 15
    for val, lo, hi in ((1.125, 1.0, 1.5), (2.25, 2.0, 3.0), (0.125, 0.0, 0.5), (5.5, 4.0, 6.0)):
        tile = [4.0] + [val] * 15 + [-val] * 16
        src = np.repeat(bits_row(tile), rows, axis=0)
        codes, scales = oracle.quantize(src, 1, rounding=1, seed=123, tag=1)
        deq = oracle.dequantize(codes, scales)
        assert set(np.unique(np.abs(deq[:, 1:]))) <= {lo, hi}
        step = hi - lo
        n = rows * 15
        sigma = step * 0.5 / np.sqrt(n)
        assert abs(deq[:, 1:16].mean() - val) <= step / 512 + 5 * sigma
        assert abs(deq[:, 16:].mean() + val) <= step / 512 + 5 * sigma
        assert (deq[:, 0] == 4.0).all()
    # clipping stays deterministic, exact grid points stay put
    tile = [7.5, 6.0, 3.0, 0.5, 0.0, -1.5] + [0.0] * 26
    src = np.repeat(bits_row(tile), 256, axis=0)
    codes, scales = oracle.quantize(src, 1, rounding=1, seed=9)
    deq = oracle.dequantize(codes, scales)
    assert (deq[:, :6] == np.array([6.0, 6.0, 3.0, 0.5, 0.0, -1.5])).all()


def test_sr_streams_differ_by_seed_and_operand_tag():
    rng = np.random.default_rng(3)
    src = _random_bits(rng, 32, 256)
    a = oracle.quantize(src, 1, rounding=1, seed=7, tag=0)[0]
    assert (oracle.quantize(src, 1, rounding=1, seed=7, tag=0)[0] == a).all()
    assert (oracle.quantize(src, 1, rounding=1, seed=8, tag=0)[0] != a).any()
    assert (oracle.quantize(src, 1, rounding=1, seed=7, tag=1)[0] != a).any()
    # SR only ever picks one of the two neighbours RNE chooses between
    r = oracle.quantize(src, 1)[0]
    lo_r, lo_a = (r & 7).astype(int), (a & 7).astype(int)
    assert (np.abs(lo_r - lo_a) <= 1).all()


# ----------------------------------------------------------------------------- P14 GEMM
def _decode_np(codes, scales):
    """Independent dequantiser: table lookup + numpy exp2 (not the C routine)."""
    table = np.array([0, .5, 1, 1.5, 2, 3, 4, 6, -0., -.5, -1, -1.5, -2, -3, -4, -6])
    lo, hi = codes & 0xF, codes >> 4
    vals = np.stack([table[lo], table[hi]], axis=-1).reshape(codes.shape[0], -1)
    return vals * np.repeat(np.exp2(scales.astype(np.float64) - 127), 32, axis=1)


def test_gemm_against_numpy_matmul_on_random_codes():
    rng = np.random.default_rng(21)
    M, N, K = 37, 29, 96
    ac = rng.integers(0, 256, (M, K // 2), dtype=np.uint8)
    bc = rng.integers(0, 256, (N, K // 2), dtype=np.uint8)
    asc = rng.integers(110, 140, (M, K // 32), dtype=np.uint8)
    bsc = rng.integers(110, 140, (N, K // 32), dtype=np.uint8)
    A, B = _decode_np(ac, asc), _decode_np(bc, bsc)
    assert (oracle.dequantize(ac, asc) == A).all()
    ref, S = oracle.gemm(ac, asc, bc, bsc, alpha=0.25)
    want = 0.25 * (A @ B.T)
    wantS = 0.25 * (np.abs(A) @ np.abs(B).T)
    assert np.allclose(ref, want, rtol=1e-13, atol=0)
    assert np.allclose(S, wantS, rtol=1e-13, atol=0)
    rows = [5, 0, 36]
    sub, subS = oracle.gemm(ac, asc, bc, bsc, alpha=0.25, rows=rows)
    assert (sub == ref[rows]).all() and (subS == S[rows]).all()


def test_gemm_scale_indexing_with_one_hot_operands():
    # one non-zero code and one non-unit scale at a time: catches swapped scale indices
    M, N, K = 3, 4, 128
    for (m, n, k) in ((0, 0, 0), (2, 3, 127), (1, 2, 33), (2, 0, 64)):
        ac = np.zeros((M, K // 2), np.uint8)
        bc = np.zeros((N, K // 2), np.uint8)
        asc = np.full((M, K // 32), 127, np.uint8)
        bsc = np.full((N, K // 32), 127, np.uint8)
        ac[m, k // 2] = 0x2 << (4 * (k % 2))      # +1.0
        bc[n, k // 2] = 0xB << (4 * (k % 2))      # -1.5
        asc[m, k // 32] = 130                     # x8
        bsc[n, k // 32] = 125                     # x1/4
        ref, S = oracle.gemm(ac, asc, bc, bsc)
        want = np.zeros((M, N))
        want[m, n] = -1.5 * 8 * 0.25
        assert (ref == want).all() and (S == np.abs(want)).all()


def test_quantize_then_gemm_is_exact_for_on_grid_operands():
    rng = np.random.default_rng(22)
    grid = np.array([0, .5, 1, 1.5, 2, 3, 4, 6])
    M, N, K = 16, 24, 64

    def on_grid(rows):
        v = grid[rng.integers(0, 8, (rows, K))] * rng.choice([-1.0, 1.0], (rows, K))
        v[:, ::32] = 4.0                               # block maximum in [4, 8): scale is 2^e
        v *= np.exp2(rng.integers(-6, 6, (rows, K // 32))).repeat(32, axis=1)
        return v

    a, b = on_grid(M), on_grid(N)
    qa = oracle.quantize(np.array([[bf16_bits(x) for x in r] for r in a], dtype=np.uint16), 1)
    qb = oracle.quantize(np.array([[bf16_bits(x) for x in r] for r in b], dtype=np.uint16), 1)
    ref, _ = oracle.gemm(*qa, *qb)
    assert (ref == a @ b.T).all()


def test_linear_passes_follow_the_cancellation_identities():
    # operands made of small integers with every 32-block maximum a power of two times [4,8)
    # are not generally on the grid after rotation, so compare with a wide tolerance here;
    # the point is the axis convention of each pass (Appendix C), not the quantisation error
    rng = np.random.default_rng(23)
    T, IN, OUT = 64, 96, 128
    X = rng.standard_normal((T, IN)).astype(np.float32)
    W = rng.standard_normal((OUT, IN)).astype(np.float32)
    dY = rng.standard_normal((T, OUT)).astype(np.float32)
    tob = lambda x: ((x.view(np.uint32) + 0x7FFF + ((x.view(np.uint32) >> 16) & 1)) >> 16).astype(np.uint16)
    tof = lambda b: (b.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    Xb, Wb, dYb = tob(X), tob(W), tob(dY)
    for mode in (0, 1, 2, 3, 4):
        y, _ = oracle.linear_fprop(Xb, Wb, hadamard_mode=mode, seed=7)
        dx, _ = oracle.linear_dgrad(dYb, Wb, hadamard_mode=mode, seed=7)
        dw, _ = oracle.linear_wgrad(dYb, Xb, hadamard_mode=mode, seed=7)
        for got, want in ((y, tof(Xb) @ tof(Wb).T), (dx, tof(dYb) @ tof(Wb)),
                          (dw, tof(dYb).T @ tof(Xb))):
            assert got.shape == want.shape
            rel = np.linalg.norm(got - want) / np.linalg.norm(want)
            assert rel < 0.2, (mode, rel)


# ----------------------------------------------------------------------------- P15 axis
def test_axis0_equals_axis1_on_the_transposed_source():
    rng = np.random.default_rng(31)
    src = _random_bits(rng, 96, 80)        # K = rows = 96 for axis 0
    for mode, rnd in ((0, 0), (1, 0), (2, 0), (0, 1), (1, 1), (3, 0), (4, 1)):
        a = oracle.quantize(src, 0, mode, rnd, seed=7, tag=1)
        b = oracle.quantize(np.ascontiguousarray(src.T), 1, mode, rnd, seed=7, tag=1)
        assert a[0].shape == (80, 48) and a[1].shape == (80, 3)
        assert (a[0] == b[0]).all() and (a[1] == b[1]).all()


# ----------------------------------------------------------------------------- scale tiling
def test_tiled_scale_layout_is_a_permutation_with_the_documented_offsets():
    outer, nt = 300, 10
    n = oracle.tiled_scale_bytes(outer, nt)
    assert n == 3 * 3 * 512
    seen = set()
    for o in range(outer):
        for t in range(nt):
            seen.add(oracle.scale_offset_tiled(o, t, nt))
    assert len(seen) == outer * nt and max(seen) < n
    # documented offsets: row 0 -> 0; row 1 -> +16; row 32 -> +4; block 1 -> +1;
    # block 4 -> next 512-byte tile; row 128 -> next row of tiles
    assert oracle.scale_offset_tiled(1, 0, nt) == 16
    assert oracle.scale_offset_tiled(32, 0, nt) == 4
    assert oracle.scale_offset_tiled(0, 1, nt) == 1
    assert oracle.scale_offset_tiled(0, 4, nt) == 512
    assert oracle.scale_offset_tiled(128, 0, nt) == 3 * 512
    sc = np.random.default_rng(1).integers(0, 255, (outer, nt), dtype=np.uint8)
    assert (oracle.scales_from_tiled(oracle.scales_to_tiled(sc), outer, nt) == sc).all()


def test_bad_arguments_are_rejected():
    src = np.zeros((4, 48), dtype=np.uint16)          # K = 48 is not a multiple of 32
    with pytest.raises(ValueError):
        oracle.quantize(src, 1)
    with pytest.raises(ValueError):
        oracle.quantize(np.zeros((4, 64), dtype=np.uint16), 1, hadamard_mode=5)

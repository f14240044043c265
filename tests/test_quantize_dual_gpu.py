"""One-read dual-axis quantize and the 32 x 32 block strategy (Appendix D) on the GPU vs the
CPU oracle: codes and scales bit-exact, through the C ABI."""
import numpy as np
import pytest

import oracle
from gpu_util import random_bits, to_dev
from paper_2605_09825_b200 import api, synth

pytestmark = pytest.mark.gpu

VARIANTS = [(0, 0), (1, 0), (2, 0), (3, 0), (4, 0), (0, 1), (1, 1), (2, 1), (3, 1), (4, 1)]


def _mixed_bits(rng, rows, cols):
    """Magnitudes spread element by element, so the rows of a region disagree on their scale."""
    x = rng.standard_normal((rows, cols)).astype(np.float32)
    x *= np.exp2(rng.integers(-5, 5, size=(rows, cols))).astype(np.float32)
    u = x.view(np.uint32)
    return ((u + 0x7FFF + ((u >> 16) & 1)) >> 16).astype(np.uint16)


def _assert_operand(codes, scales_raw, want_codes, want_scales, layout=api.SCALES_TILED, what=""):
    outer, nt = want_scales.shape
    got_c = codes.cpu().numpy()
    raw = scales_raw.cpu().numpy()
    got_s = oracle.scales_from_tiled(raw, outer, nt) if layout == api.SCALES_TILED else raw.reshape(outer, nt)
    bad = np.argwhere(got_s != want_scales)
    assert bad.size == 0, f"{what}: {len(bad)} scales differ, first at {bad[:4].tolist()}"
    bad = np.argwhere(got_c != want_codes)
    assert bad.size == 0, f"{what}: {len(bad)} code bytes differ, first at {bad[:4].tolist()}"


@pytest.mark.parametrize("hmode,rnd", VARIANTS)
@pytest.mark.parametrize("block_shape", [api.BLOCK_1X32, api.BLOCK_32X32])
@pytest.mark.parametrize("rows,cols", [(32, 32), (160, 416), (1056, 672), (384, 2144)])
def test_dual_matches_the_oracle_in_both_orientations(rows, cols, block_shape, hmode, rnd):
    rng = np.random.default_rng(rows * 31 + cols)
    bits = _mixed_bits(rng, rows, cols)
    (cr, sr), (cc, sc) = api.quantize_dual(to_dev(bits), hmode, rnd, seed=9, tags=(2, 3), block_shape=block_shape)
    api.check()
    b2d = block_shape == api.BLOCK_32X32
    _assert_operand(cr, sr, *oracle.quantize(bits, 1, hmode, rnd, 9, 2, block2d=b2d), what="row-wise")
    _assert_operand(cc, sc, *oracle.quantize(bits, 0, hmode, rnd, 9, 3, block2d=b2d), what="column-wise")


@pytest.mark.parametrize("hmode,rnd", VARIANTS)
@pytest.mark.parametrize("axis", [1, 0])
@pytest.mark.parametrize("rows,cols", [(32, 32), (96, 160), (300, 416), (1000, 1184)])
def test_single_axis_2d_blocks_match_the_oracle(rows, cols, axis, hmode, rnd):
    if axis == 0 and (rows % 32 or cols % 8):
        pytest.skip("column-wise blocks need rows % 32 == 0 and cols % 8 == 0")
    rng = np.random.default_rng(rows * 17 + cols)
    bits = _mixed_bits(rng, rows, cols)
    codes, scales = api.quantize(to_dev(bits), axis, hmode, rnd, 4, 1, block_shape=api.BLOCK_32X32)
    api.check()
    _assert_operand(codes, scales, *oracle.quantize(bits, axis, hmode, rnd, 4, 1, block2d=True))


def test_2d_blocks_differ_from_1d_on_these_inputs():
    """Guards the two tests above against inputs on which both strategies would agree."""
    rng = np.random.default_rng(3)
    bits = _mixed_bits(rng, 96, 160)
    a = oracle.quantize(bits, 1, 1, 0, block2d=True)
    b = oracle.quantize(bits, 1, 1, 0)
    assert (a[1] != b[1]).any() and (a[0] != b[0]).any()


def test_dual_on_layer_shaped_tensors_and_canonical_scales():
    t = synth.config1()
    for name in ("X", "W"):
        bits = t[name]
        if bits.shape[0] % 32 or bits.shape[1] % 32:
            continue
        (cr, sr), (cc, sc) = api.quantize_dual(to_dev(bits), 1, 0, 7, scale_layout=api.SCALES_CANONICAL)
        api.check()
        _assert_operand(cr, sr, *oracle.quantize(bits, 1, 1, 0, 7, 0), layout=api.SCALES_CANONICAL)
        _assert_operand(cc, sc, *oracle.quantize(bits, 0, 1, 0, 7, 1), layout=api.SCALES_CANONICAL)


def test_dual_strided_source_and_padding_bytes():
    rng = np.random.default_rng(23)
    full = random_bits(rng, 160, 512)
    view = to_dev(full)[:, 64:64 + 288]                       # ld = 512, cols = 288
    (cr, sr), (cc, sc) = api.quantize_dual(view, 2, 1, 5)
    api.check()
    sub = np.ascontiguousarray(full[:, 64:64 + 288])
    _assert_operand(cr, sr, *oracle.quantize(sub, 1, 2, 1, 5, 0))
    _assert_operand(cc, sc, *oracle.quantize(sub, 0, 2, 1, 5, 1))
    # padding rows / blocks of both tiled scale buffers hold 0
    for raw, outer, K in ((sr.cpu().numpy(), 160, 288), (sc.cpu().numpy(), 288, 160)):
        used = np.zeros(raw.size, dtype=bool)
        o = np.arange(outer)[:, None]
        tt = np.arange(K // 32)[None, :]
        off = ((o // 128) * ((K // 32 + 3) // 4) + tt // 4) * 512 + (o % 32) * 16 + ((o % 128) // 32) * 4 + tt % 4
        used[off] = True
        assert (raw[~used] == 0).all()


def test_dual_feeds_the_gemm():
    """Dgrad from dual outputs: dX = dY W with dY row-wise and W column-wise, against the oracle."""
    rng = np.random.default_rng(29)
    dY, W = random_bits(rng, 256, 384, 2), random_bits(rng, 384, 512, 2)
    (dyc, dys), _ = api.quantize_dual(to_dev(dY), 1, 0, 0, tags=(0, 9))
    _, (wc, ws) = api.quantize_dual(to_dev(W), 1, 0, 0, tags=(9, 1))
    out = api.gemm(dyc, dys, wc, ws, 1.0 / 32, api.OUT_FP32)
    api.check()
    ref, S = oracle.linear_dgrad(dY, W, 1, 0, 0)
    got = out.cpu().numpy().astype(np.float64)
    assert (np.abs(got - ref) <= 1e-5 * S + 1e-38).all()


def test_dual_rejects_bad_arguments():
    rng = np.random.default_rng(1)
    with pytest.raises(api.Mxfp4Error) as exc:
        api.quantize_dual(to_dev(random_bits(rng, 48, 64)))
    assert exc.value.status == -2
    with pytest.raises(api.Mxfp4Error) as exc:
        api.quantize_dual(to_dev(random_bits(rng, 64, 64)), block_shape=2)
    assert exc.value.status == -4


def test_dual_special_values_in_both_orientations():
    """Every finite bf16 pattern as the only non-zero element of its row-wise block AND of its
    column-wise block (so no rotation overflows), plus a region of negative zeros: sub-normal block
    maxima, the scale clamp, signed zeros and saturation reach both paths of the kernel."""
    pats = np.array([p for p in range(1 << 16) if ((p >> 7) & 0xFF) != 0xFF], dtype=np.uint16)
    rows, cols = 8192 + 32, 256
    bits = np.zeros((rows, cols), dtype=np.uint16)
    k = np.arange(len(pats))
    r, cb = k // 8, k % 8                                    # one pattern per (row, 32-column block) ...
    bits[r, cb * 32 + r % 32] = pats                         # ... and per (32-row group, column)
    bits[-32:, :] = 0x8000                                   # a region of negative zeros
    for hmode, rnd in ((0, 0), (1, 0), (3, 1), (2, 0)):
        (cr, sr), (cc, sc) = api.quantize_dual(to_dev(bits), hmode, rnd, 5)
        api.check()
        _assert_operand(cr, sr, *oracle.quantize(bits, 1, hmode, rnd, 5, 0), what=f"row-wise mode {hmode}")
        _assert_operand(cc, sc, *oracle.quantize(bits, 0, hmode, rnd, 5, 1), what=f"column-wise mode {hmode}")


def test_dual_canary_bytes_around_all_four_outputs():
    import torch
    rng = np.random.default_rng(31)
    rows, cols = 224, 160
    src = to_dev(random_bits(rng, rows, cols))
    pad = 4096
    sizes = (api.codes_bytes(rows, cols), api.scales_bytes(rows, cols), api.codes_bytes(cols, rows),
             api.scales_bytes(cols, rows))
    bufs = [torch.full((n + 2 * pad,), 0xA5, dtype=torch.uint8, device="cuda") for n in sizes]
    view = lambda b, n: b[pad:pad + n]
    api.quantize_dual(src, 1, 0, 0,
                      out_row=(view(bufs[0], sizes[0]).view(rows, cols // 2), view(bufs[1], sizes[1])),
                      out_col=(view(bufs[2], sizes[2]).view(cols, rows // 2), view(bufs[3], sizes[3])))
    api.check()
    for b, n in zip(bufs, sizes):
        assert (b[:pad] == 0xA5).all() and (b[pad + n:] == 0xA5).all()


def test_dual_is_reproducible_run_to_run():
    t = synth.config1()
    a = api.quantize_dual(to_dev(t["X"]), 2, 1, 7)
    b = api.quantize_dual(to_dev(t["X"]), 2, 1, 7)
    api.check()
    import torch
    for (x0, x1), (y0, y1) in zip(a, b):
        assert torch.equal(x0, y0) and torch.equal(x1, y1)


@pytest.mark.parametrize("pass_", [0, 1, 2])
def test_passes_with_32x32_blocks(pass_):
    """mxfp4_linear_pass with 32 x 32 blocks: bit-identical to quantize_2d + gemm, and within
    tolerance of the oracle's 2D quantization followed by its fp64 GEMM."""
    import torch
    from gpu_util import assert_gemm_close
    rng = np.random.default_rng(60 + pass_)
    T, in_f, out_f = 416, 288, 672
    X, W, dY = _mixed_bits(rng, T, in_f), _mixed_bits(rng, out_f, in_f), _mixed_bits(rng, T, out_f)
    a, b = ((X, W), (dY, W), (dY, X))[pass_]
    axes = ((1, 1), (1, 0), (0, 0))[pass_]
    out = api.linear_pass(pass_, api.PRECISION_MXFP4_32X32, to_dev(a), to_dev(b), 1, 0, 3, api.OUT_FP32)
    qa = api.quantize(to_dev(a), axes[0], 1, 0, 3, 0, block_shape=api.BLOCK_32X32)
    qb = api.quantize(to_dev(b), axes[1], 1, 0, 3, 1, block_shape=api.BLOCK_32X32)
    assert torch.equal(out, api.gemm(*qa, *qb, 1.0 / 32, api.OUT_FP32))
    api.check()
    oa = oracle.quantize(a, axes[0], 1, 0, 3, 0, block2d=True)
    ob = oracle.quantize(b, axes[1], 1, 0, 3, 1, block2d=True)
    ref, S = oracle.gemm(*oa, *ob, alpha=1.0 / 32)
    assert_gemm_close(out.cpu().numpy(), ref, S, False, f"32x32 pass {pass_}")

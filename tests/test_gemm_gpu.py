"""CUDA block-scaled GEMM and the fused linear passes vs the CPU oracle, through the C ABI.

Tolerance (stated by the benchmark spec for fp32 outputs): |out - ref| <= 1e-5 * sum|products|; bf16
outputs add half a bf16 ulp of the reference.  Products of E2M1 values and power-of-two scales
are exact, so only the fp32 accumulation order differs from the fp64 reference.
"""
import numpy as np
import pytest
import torch

import oracle
from gpu_util import assert_gemm_close, random_bits, to_dev
from paper_2605_09825_b200 import api, synth

pytestmark = pytest.mark.gpu


def _dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def _run_gemm(ac, asc, bc, bsc, alpha, out_dtype):
    out = api.gemm(_dev(ac), _dev(oracle.scales_to_tiled(asc)), _dev(bc), _dev(oracle.scales_to_tiled(bsc)),
                   alpha, out_dtype)
    api.check()
    return out.float().cpu().numpy()


def _random_operands(rng, M, N, K, lo=118, hi=136):
    ac = rng.integers(0, 256, (M, K // 2), dtype=np.uint8)
    bc = rng.integers(0, 256, (N, K // 2), dtype=np.uint8)
    asc = rng.integers(lo, hi, (M, K // 32), dtype=np.uint8)
    bsc = rng.integers(lo, hi, (N, K // 32), dtype=np.uint8)
    return ac, asc, bc, bsc


def test_all_ones_counts_k():
    M, N, K = 128, 256, 256
    ac = np.full((M, K // 2), 0x22, np.uint8)
    bc = np.full((N, K // 2), 0x22, np.uint8)
    asc = np.full((M, K // 32), 127, np.uint8)
    bsc = np.full((N, K // 32), 127, np.uint8)
    out = _run_gemm(ac, asc, bc, bsc, 1.0, api.OUT_FP32)
    assert (out == K).all()


def test_scale_indexing_by_row_and_block():
    # unit codes; every (row, block) of A and B carries its own exponent, so any mix-up of
    # rows, 32-row groups, blocks or operands changes the result
    M, N, K = 256, 512, 512
    ac = np.full((M, K // 2), 0x22, np.uint8)
    bc = np.full((N, K // 2), 0x22, np.uint8)
    rng = np.random.default_rng(3)
    asc = rng.integers(120, 134, (M, K // 32), dtype=np.uint8)
    bsc = rng.integers(120, 134, (N, K // 32), dtype=np.uint8)
    out = _run_gemm(ac, asc, bc, bsc, 1.0, api.OUT_FP32)
    ref, S = oracle.gemm(ac, asc, bc, bsc)
    assert_gemm_close(out, ref, S, False, "scale indexing")


def test_one_hot_codes_locate_every_k():
    M, N, K = 128, 256, 512
    rng = np.random.default_rng(4)
    ac = np.zeros((M, K // 2), np.uint8)
    bc = np.full((N, K // 2), 0x22, np.uint8)
    ks = rng.integers(0, K, M)
    ac[np.arange(M), ks // 2] = np.where(ks % 2 == 0, 0x06, 0x60).astype(np.uint8)   # 4.0 at k
    # B holds a different value per k so that the product names the k that was hit
    vals = rng.integers(1, 8, (N, K)).astype(np.uint8)
    bc = (vals[:, 0::2] | (vals[:, 1::2] << 4)).astype(np.uint8)
    asc = np.full((M, K // 32), 127, np.uint8)
    bsc = np.full((N, K // 32), 127, np.uint8)
    out = _run_gemm(ac, asc, bc, bsc, 1.0, api.OUT_FP32)
    ref, _ = oracle.gemm(ac, asc, bc, bsc)
    assert (out == ref).all()


@pytest.mark.parametrize("M,N,K", [(128, 256, 256), (256, 256, 512), (384, 768, 1024), (200, 328, 416),
                                   (1, 8, 32), (129, 264, 96), (520, 1000, 2080)])
@pytest.mark.parametrize("out_dtype", [api.OUT_FP32, api.OUT_BF16])
def test_random_operands_full_compare(M, N, K, out_dtype):
    rng = np.random.default_rng(M * 31 + N * 7 + K)
    ac, asc, bc, bsc = _random_operands(rng, M, N, K)
    out = _run_gemm(ac, asc, bc, bsc, 0.03125, out_dtype)
    ref, S = oracle.gemm(ac, asc, bc, bsc, alpha=0.03125)
    assert_gemm_close(out, ref, S, out_dtype == api.OUT_BF16, f"gemm {M}x{N}x{K}")


def test_bf16_output_is_the_rounded_fp32_output():
    rng = np.random.default_rng(9)
    ac, asc, bc, bsc = _random_operands(rng, 256, 512, 512)
    f = _run_gemm(ac, asc, bc, bsc, 1.0, api.OUT_FP32)
    b = _run_gemm(ac, asc, bc, bsc, 1.0, api.OUT_BF16)
    assert (torch.from_numpy(f).to(torch.bfloat16).float().numpy() == b).all()


def test_gemm_is_deterministic_and_respects_ld_out():
    rng = np.random.default_rng(10)
    M, N, K = 256, 264, 512
    ac, asc, bc, bsc = _random_operands(rng, M, N, K)
    args = (_dev(ac), _dev(oracle.scales_to_tiled(asc)), _dev(bc), _dev(oracle.scales_to_tiled(bsc)))
    big = torch.full((M, 512), 777.0, dtype=torch.float32, device="cuda")
    api.gemm(*args, 1.0, api.OUT_FP32, out=big[:, :N])
    once = api.gemm(*args, 1.0, api.OUT_FP32)
    api.check()
    assert (big[:, :N] == once).all() and (big[:, N:] == 777.0).all()


def test_config1_fprop_full_output():
    t = synth.config1()
    X, W = to_dev(t["X"]), to_dev(t["W"])
    for hmode in (0, 1, 2, 3, 4):
        y = api.linear_fprop(X, W, hmode, 0, 7, api.OUT_FP32)
        api.check()
        ref, S = oracle.linear_fprop(t["X"], t["W"], hmode, 0, 7)
        assert_gemm_close(y.cpu().numpy(), ref, S, False, f"config 1 fprop mode {hmode}")


@pytest.mark.parametrize("hmode,rnd", [(0, 0), (1, 0), (2, 0), (0, 1), (3, 0), (4, 1)])
def test_three_passes_small_layer(hmode, rnd):
    rng = np.random.default_rng(40 + hmode)
    T, IN, OUT = 384, 512, 320
    Xb, Wb, dYb = random_bits(rng, T, IN, 2), random_bits(rng, OUT, IN, 2), random_bits(rng, T, OUT, 2)
    X, W, dY = to_dev(Xb), to_dev(Wb), to_dev(dYb)
    for out_dtype in (api.OUT_FP32, api.OUT_BF16):
        bf = out_dtype == api.OUT_BF16
        y = api.linear_fprop(X, W, hmode, rnd, 7, out_dtype)
        dx = api.linear_dgrad(dY, W, hmode, rnd, 7, out_dtype)
        dw = api.linear_wgrad(dY, X, hmode, rnd, 7, out_dtype)
        api.check()
        assert_gemm_close(y.float().cpu().numpy(), *oracle.linear_fprop(Xb, Wb, hmode, rnd, 7), bf, "fprop")
        assert_gemm_close(dx.float().cpu().numpy(), *oracle.linear_dgrad(dYb, Wb, hmode, rnd, 7), bf, "dgrad")
        assert_gemm_close(dw.float().cpu().numpy(), *oracle.linear_wgrad(dYb, Xb, hmode, rnd, 7), bf, "wgrad")


def test_host_buffer_entry_point_matches_device_entry_point():
    rng = np.random.default_rng(50)
    T, IN, OUT = 256, 256, 384
    Xb, Wb = random_bits(rng, T, IN, 2), random_bits(rng, OUT, IN, 2)
    Xh = torch.from_numpy(Xb.view(np.int16)).view(torch.bfloat16).pin_memory()
    Wh = torch.from_numpy(Wb.view(np.int16)).view(torch.bfloat16).pin_memory()
    Yh = torch.empty((T, OUT), dtype=torch.bfloat16).pin_memory()
    dX, dW_, dY = (torch.empty_like(Xh, device="cuda"), torch.empty_like(Wh, device="cuda"),
                   torch.empty((T, OUT), dtype=torch.bfloat16, device="cuda"))
    ws = torch.empty(api.linear_workspace_bytes(T, IN, OUT, api.PASS_FPROP), dtype=torch.uint8, device="cuda")
    api.linear_host(api.PASS_FPROP, Xh, Wh, Yh, T, IN, OUT, dX, dW_, dY, ws)
    want = api.linear_fprop(to_dev(Xb), to_dev(Wb))
    api.check()
    assert (Yh.cuda() == want).all()


def test_an_expired_bounded_wait_is_reported_and_the_context_stays_usable():
    api.check()                                       # clean slate
    api.selftest_wait_timeout()
    with pytest.raises(api.Mxfp4Error) as err:
        api.check()
    assert err.value.status == -7
    api.check()                                       # the status was cleared by the read
    # and the device still computes correctly afterwards
    test_all_ones_counts_k()


@pytest.mark.parametrize("M,N,K,ld,out_dtype", [(130, 100, 32, 104, api.OUT_BF16), (257, 50, 160, 52, api.OUT_FP32),
                                                (64, 385, 64, 392, api.OUT_BF16), (300, 769, 288, 776, api.OUT_FP32),
                                                (33, 3, 32, 4, api.OUT_FP32), (40, 7, 64, 8, api.OUT_BF16),
                                                (129, 391, 96, 392, api.OUT_FP32)])
def test_ragged_n_with_padded_leading_dimension(M, N, K, ld, out_dtype):
    # N is not a multiple of the 16-byte store granule (8 bf16 / 4 fp32), down to N smaller than one granule; the columns between N and ld must stay untouched
    rng = np.random.default_rng(M + N + K)
    ac, asc, bc, bsc = _random_operands(rng, M, N, K)
    dt = torch.bfloat16 if out_dtype == api.OUT_BF16 else torch.float32
    big = torch.full((M, ld), 7.0, dtype=dt, device="cuda")
    api.gemm(_dev(ac), _dev(oracle.scales_to_tiled(asc)), _dev(bc), _dev(oracle.scales_to_tiled(bsc)), 0.5,
             out_dtype, out=big[:, :N])
    api.check()
    ref, S = oracle.gemm(ac, asc, bc, bsc, alpha=0.5)
    assert_gemm_close(big[:, :N].float().cpu().numpy(), ref, S, out_dtype == api.OUT_BF16, "ragged N")
    assert (big[:, N:] == 7.0).all()


def test_scale_bytes_of_rows_that_do_not_exist_never_reach_an_output():
    """The tiled scale buffers hold whole tiles of 128 rows; what stands in the rows past M (or N)
    belongs to accumulator rows (columns) that are never stored.  With 0xFF -- the E8M0 NaN -- in
    all of them the result is the same and finite."""
    rng = np.random.default_rng(77)
    M, N, K = 200, 304, 256
    ac, asc, bc, bsc = _random_operands(rng, M, N, K)
    ref, S = oracle.gemm(ac, asc, bc, bsc, alpha=1.0)
    a_pad = np.full((256, K // 32), 0xFF, dtype=np.uint8)
    b_pad = np.full((384, K // 32), 0xFF, dtype=np.uint8)
    a_pad[:M], b_pad[:N] = asc, bsc
    a_t, b_t = oracle.scales_to_tiled(a_pad), oracle.scales_to_tiled(b_pad)
    assert a_t.size == api.scales_bytes(M, K, api.SCALES_TILED) and b_t.size == api.scales_bytes(N, K, api.SCALES_TILED)
    for out_dtype in (api.OUT_FP32, api.OUT_BF16):
        out = api.gemm(_dev(ac), _dev(a_t), _dev(bc), _dev(b_t), 1.0, out_dtype)
        api.check()
        got = out.float().cpu().numpy()
        assert np.isfinite(got).all()
        assert_gemm_close(got, ref, S, out_dtype == api.OUT_BF16, "0xFF in the padding rows")


def test_plain_stream_order_launches_still_work():
    """MXFP4_PDL=0 turns the programmatic-dependent-launch attribute off; same results."""
    import os
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    res = subprocess.run([sys.executable, "-c", "import __graft_entry__ as g; g.smoke()"], cwd=root,
                         env=dict(os.environ, MXFP4_PDL="0"), capture_output=True, text=True, timeout=600)
    assert res.returncode == 0, res.stdout + res.stderr


def test_mma_rate_probe_runs_and_reports_its_flops():
    """The diagnostic that measures the tensor pipe's own ceiling: a short launch completes, leaves
    the status word clean and reports 2 * 256 * 192 * 64 * 8 flops per iteration and CTA pair."""
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    for rnd in (False, True):
        fl = api.probe_mma_rate(200, rnd)
        api.check()
        assert fl == 2.0 * 256 * 192 * 64 * 8 * 200 * (sms // 2)
    with pytest.raises(api.Mxfp4Error):
        api.probe_mma_rate(0, True)


@pytest.mark.parametrize("M,N", [(2344, 900), (2344, 1900), (1300, 1900)])
def test_band_order_with_a_ragged_last_band(M, N):
    """K = 65536 makes a 256-row tile of A 8 MB and a 384-row tile of B 12 MB, so the tile order
    works in bands, along whichever axis the host estimates fewer HBM reads for: (2344, 900) one band
    of all three tile columns, tile column fastest; (2344, 1900) bands of 2, 2 and 1 tile columns (the
    last one narrow, the last tile column ragged); (1300, 1900) bands of 4 and 2 tile ROWS (the last
    tile row ragged).  Whole output against the fp64 checker on the same codes and scales, sampled
    rows of every band against the CPU oracle."""
    import gemm_checker
    rng = np.random.default_rng(65536 + M + N)
    K = 65536
    ac, asc, bc, bsc = _random_operands(rng, M, N, K, lo=122, hi=132)
    out = api.gemm(_dev(ac), _dev(oracle.scales_to_tiled(asc)), _dev(bc), _dev(oracle.scales_to_tiled(bsc)),
                   0.03125, api.OUT_FP32)
    api.check()
    rows = np.array([r for r in (0, 255, 256, 1023, 1024, 1279, 1280, 1299, 1500, 2047, 2048, 2303, 2304, 2343) if r < M])
    ref, S = oracle.gemm(ac, asc, bc, bsc, alpha=0.03125, rows=rows)
    assert_gemm_close(out[torch.from_numpy(rows).cuda()].cpu().numpy(), ref, S, False, "band order, sampled rows")
    _, _, _, cref, cS = gemm_checker.check(ac[rows], asc[rows], bc, bsc, 0.03125, None, want_ref=True)
    assert np.all(np.abs(cref.cpu().numpy() - ref) <= 1e-12 * S + 1e-300)
    n_bad, first, worst, _, _ = gemm_checker.check(ac, asc, bc, bsc, 0.03125, out)
    assert n_bad == 0 and worst <= 1.0, (n_bad, first // N, first % N, worst)

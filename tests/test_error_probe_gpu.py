"""Quantization-error probe: its figures equal the ones computed from the CPU oracle, and the
orderings that the paper states qualitatively (stochastic rounding carries more quantization
error than round-to-nearest when Wgrad is quantized; the rotation lowers the error on
heavy-tailed operands) hold for this library's kernels on the synthetic stand-in operands."""
import numpy as np
import pytest

import oracle
from paper_2605_09825_b200 import error_probe, synth

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("pass_name", ["wgrad", "fprop"])
def test_error_orderings(pass_name):
    snr = error_probe.run(pass_name, tokens=1024, linear="down")["snr_db"]
    snr8 = snr.pop("mxfp8")
    assert snr8 > max(snr.values()) + 10.0, (snr8, snr)          # three more mantissa bits: ~18 dB
    assert all(8.0 < v < 25.0 for v in snr.values()), snr       # 4-bit elements: ~12-16 dB
    assert snr["none_32x32"] <= snr["none"] + 0.05, snr          # a shared scale can only be coarser
    assert snr["det_h32_32x32"] <= snr["det_h32"] + 0.05, snr
    assert snr["sr"] < snr["none"] - 1.5, snr                   # SR doubles the error variance or so
    assert snr["sr_det_h32"] < snr["det_h32"] - 1.5, snr
    assert snr["det_h32"] > snr["none"] + 0.3, snr              # rotation spreads the outliers
    assert snr["det_h16"] > snr["none"] + 0.3, snr
    assert abs(snr["rand_h32"] - snr["det_h32"]) < 0.3, snr     # sign flips do not change the MSE much


def _snr_db(got, ref):
    err = float(((got - ref) ** 2).sum())
    return 10.0 * np.log10(float((ref ** 2).sum()) / err)


@pytest.mark.parametrize("pass_name", ["wgrad", "fprop", "dgrad"])
def test_probe_snr_equals_the_oracles(pass_name):
    """The probe's figure for every variant against the same figure computed from the CPU oracle:
    oracle-quantized operands multiplied in fp64, measured against the exact fp64 product (numpy)
    of the same bf16 inputs.  The quantized operands are bit-identical on both sides, so only the
    fp32 accumulation of the GEMM separates the two: 0.05 dB is generous."""
    tokens, linear, seed = 256, "o", 7
    t = synth.linear_tensors(linear, tokens, 4)
    f64 = lambda bits: synth.bf16_bits_to_f32(bits).astype(np.float64)
    X, W, dY = f64(t["X"]), f64(t["W"]), f64(t["dY"])
    pass_id = {"fprop": 0, "dgrad": 1, "wgrad": 2}[pass_name]
    a_bits, b_bits = ((t["X"], t["W"]), (t["dY"], t["W"]), (t["dY"], t["X"]))[pass_id]
    exact = (X @ W.T, dY @ W, dY.T @ X)[pass_id]
    ofn = (oracle.linear_fprop, oracle.linear_dgrad, oracle.linear_wgrad)[pass_id]
    ax_a, ax_b = ((1, 1), (1, 0), (0, 0))[pass_id]
    want = {}
    for name, hmode, rnd in error_probe.VARIANTS:
        want[name] = _snr_db(ofn(a_bits, b_bits, hmode, rnd, seed)[0], exact)
    for name, hmode, alpha in (("none_32x32", 0, 1.0), ("det_h32_32x32", 1, 1.0 / 32)):
        qa = oracle.quantize(a_bits, ax_a, hmode, 0, seed, 0, block2d=True)
        qb = oracle.quantize(b_bits, ax_b, hmode, 0, seed, 1, block2d=True)
        want[name] = _snr_db(oracle.gemm(*qa, *qb, alpha=alpha)[0], exact)
    want["mxfp8"] = _snr_db(oracle.linear_pass_mxfp8(pass_id, a_bits, b_bits)[0], exact)
    got = error_probe.run(pass_name, tokens=tokens, linear=linear, seed=seed)["snr_db"]
    assert set(got) == set(want)
    for name in want:
        assert abs(got[name] - want[name]) < 0.05, (pass_name, name, got[name], want[name])

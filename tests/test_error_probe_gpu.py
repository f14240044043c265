"""Quantization-error probe: orderings that the paper states qualitatively (stochastic rounding
carries more quantization error than round-to-nearest when Wgrad is quantized; the rotation
lowers the error on heavy-tailed operands) hold for this library's kernels on the synthetic
stand-in operands."""
import pytest

from paper_2605_09825_b200 import error_probe

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

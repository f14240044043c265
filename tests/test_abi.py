"""The C-ABI library builds, loads and exports every symbol the header declares; argument
errors are reported on the host before any device work.  No GPU needed."""
import ctypes
import os
import re

import pytest

from paper_2605_09825_b200 import api, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build_library()
    return api.load_library()


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "mxfp4.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(mxfp4_[a-z0-9_]+)\s*\(", text)))


def test_header_symbols_are_exported(lib):
    names = _declared_symbols()
    assert set(names) == set(api.EXPORTS)
    for n in names:
        assert hasattr(lib, n), n


def test_version_and_status_strings(lib):
    assert api.version() >= 100
    assert api.status_string(0) == "ok"
    for code in range(-8, 0):
        assert api.status_string(code) not in ("ok", "unknown status")


def test_size_helpers(lib):
    assert api.codes_bytes(256, 512) == 256 * 256
    assert api.scales_bytes(256, 512, api.SCALES_CANONICAL) == 256 * 16
    assert api.scales_bytes(256, 512, api.SCALES_TILED) == 2 * 4 * 512
    assert api.scales_bytes(300, 160, api.SCALES_TILED) == 3 * 2 * 512   # padded to whole tiles
    assert api.codes_bytes(4, 48) == 0 and api.scales_bytes(4, 48, 1) == 0
    assert api.scales_bytes(4, 64, 7) == 0
    # fprop at T=256, in=512, out=256: two operands of 256 x 512
    want = 2 * (256 * 256 + 2 * 4 * 512)
    assert api.linear_workspace_bytes(256, 512, 256, api.PASS_FPROP) == want
    assert api.linear_workspace_bytes(256, 512, 256, 5) == 0


def test_argument_errors_come_back_as_status_codes(lib):
    buf = ctypes.create_string_buffer(1 << 16)
    base = ctypes.addressof(buf)
    p = (base + 15) & ~15
    q = lib.mxfp4_quantize
    assert q(None, 32, 32, 32, 1, 0, 0, 0, 0, p, p, 0, None) == -1            # NULL
    assert q(p, 32, 32, 32, 2, 0, 0, 0, 0, p, p, 0, None) == -4               # axis
    assert q(p, 32, 32, 32, 1, 5, 0, 0, 0, p, p, 0, None) == -4               # hadamard mode
    assert q(p, 32, 32, 32, 1, 0, 2, 0, 0, p, p, 0, None) == -4               # rounding
    assert q(p, 32, 32, 32, 1, 0, 0, 0, 0, p, p, 9, None) == -4               # layout
    assert q(p, 32, 48, 48, 1, 0, 0, 0, 0, p, p, 0, None) == -2               # K % 32
    assert q(p, 48, 32, 32, 0, 0, 0, 0, 0, p, p, 0, None) == -2               # K = rows % 32
    assert q(p, 32, 64, 32, 1, 0, 0, 0, 0, p, p, 0, None) == -2               # ld < cols
    assert q(p + 2, 32, 32, 32, 1, 0, 0, 0, 0, p, p, 0, None) == -3           # alignment
    assert q(p, 32, 32, 36, 1, 0, 0, 0, 0, p, p, 0, None) == -3               # ld % 8
    g = lib.mxfp4_gemm
    assert g(None, p, p, p, 128, 128, 128, 1.0, p, 0, 128, None, 0, None) == -1
    assert g(p, p, p, p, 128, 128, 100, 1.0, p, 0, 128, None, 0, None) == -2
    assert g(p, p, p, p, 128, 128, 128, 1.0, p, 3, 128, None, 0, None) == -4
    assert g(p, p, p, p, 128, 128, 128, 1.0, p, 0, 64, None, 0, None) == -2   # ld_out < N
    assert g(p, p, p, p, 128, 100, 128, 1.0, p, 0, 100, None, 0, None) == -3  # ld_out * 2 % 16
    f = lib.mxfp4_linear_fprop
    assert f(p, p, p, 128, 128, 128, 1, 0, 0, 0, None, 0, None) == -5         # no workspace
    assert f(p, p, p, 128, 100, 128, 1, 0, 0, 0, p, 1 << 15, None) == -2      # in % 32
    assert f(None, p, p, 128, 128, 128, 1, 0, 0, 0, p, 1 << 15, None) == -1


def test_output_errors_are_found_before_the_quantize_launch(lib):
    """What the GEMM at the end of a fused pass would reject (output dtype, output alignment) and
    what the second tensor of a layer call would trip over are reported by checks that run before
    the first launch or copy: they come back even on a machine without a GPU."""
    buf = ctypes.create_string_buffer(1 << 17)
    p = (ctypes.addressof(buf) + 255) & ~255
    ws = 1 << 16
    f = lib.mxfp4_linear_fprop
    assert f(p, p, p, 128, 128, 128, 1, 0, 0, 7, p, ws, None) == -4            # out_dtype
    assert f(p, p, p + 4, 128, 128, 128, 1, 0, 0, 0, p, ws, None) == -3        # out alignment
    assert f(p, p + 2, p, 128, 128, 128, 1, 0, 0, 0, p, ws, None) == -3        # second operand alignment
    h = lib.mxfp4_linear_host
    assert h(0, p, p, p, 128, 128, 128, 1, 0, 0, 9, p, p, p, p, ws, None) == -4
    assert h(0, p, p, p, 128, 128, 128, 1, 0, 0, 0, p, p + 8, p, p, ws, None) == -3
    assert h(0, p, p, p, 128, 128, 128, 1, 0, 0, 0, p, p, p, p, 16, None) == -5
    fw = lib.mxfp4_linear_forward
    big = 1 << 16
    assert fw(p, p + 2, p, 64, 64, 64, 1, 0, 0, 0, p, big, p, big, None) == -3  # W misaligned
    assert fw(p, p, p, 64, 64, 64, 1, 0, 0, 5, p, big, p, big, None) == -4      # out_dtype
    bw = lib.mxfp4_linear_backward
    assert bw(p, p, p + 6, 64, 64, 64, 1, 0, 0, 0, 0, p, big, p, big, None) == -3
    assert bw(p, p, p, 64, 64, 64, 1, 0, 0, 0, 3, p, big, p, big, None) == -4


def test_empty_and_oversized_shapes_are_shape_errors(lib):
    """Zero-sized tensors and sizes past the kernels' 32-bit tile arithmetic (a dimension of 2^31 or
    more, more than 2^30 tiles, 2^31 or more tile K-steps) are refused on the host, before the
    device is looked at."""
    buf = ctypes.create_string_buffer(1 << 12)
    p = (ctypes.addressof(buf) + 255) & ~255
    big = 0x7FFFFFE0                                    # the largest multiple of 32 below 2^31
    q, g, d = lib.mxfp4_quantize, lib.mxfp4_gemm, lib.mxfp4_quantize_dual
    for axis in (0, 1):
        assert q(p, 0, 32, 32, axis, 0, 0, 0, 0, p, p, 1, None) == -2
        assert q(p, 32, 0, 0, axis, 0, 0, 0, 0, p, p, 1, None) == -2
        assert q(p, 1 << 31, 32, 32, axis, 0, 0, 0, 0, p, p, 1, None) == -2
        assert q(p, 32, 1 << 31, 1 << 31, axis, 0, 0, 0, 0, p, p, 1, None) == -2
        assert q(p, big, big, big, axis, 0, 0, 0, 0, p, p, 1, None) == -2            # 2^48 tiles
    assert d(p, 0, 32, 32, 1, 0, 0, 0, 1, 0, p, p, p, p, 1, None) == -2
    assert d(p, big, big, big, 1, 0, 0, 0, 1, 0, p, p, p, p, 1, None) == -2
    assert g(p, p, p, p, 0, 128, 128, 1.0, p, 0, 128, None, 0, None) == -2
    assert g(p, p, p, p, 128, 0, 128, 1.0, p, 0, 128, None, 0, None) == -2
    assert g(p, p, p, p, 128, 128, 0, 1.0, p, 0, 128, None, 0, None) == -2
    assert g(p, p, p, p, 1 << 31, 128, 128, 1.0, p, 0, 128, None, 0, None) == -2
    assert g(p, p, p, p, big, big, 32, 1.0, p, 0, big, None, 0, None) == -2          # 2^45 tiles
    assert g(p, p, p, p, 1 << 20, 1 << 20, 1 << 30, 1.0, p, 0, 1 << 20, None, 0, None) == -2   # tiles x K-steps
    f = lib.mxfp4_linear_fprop
    assert f(p, p, p, 0, 128, 128, 1, 0, 0, 0, p, 1 << 15, None) == -2
    assert f(p, p, p, big, big, big, 1, 0, 0, 0, p, 1 << 15, None) == -2
    fw = lib.mxfp4_linear_forward
    assert fw(p, p, p, 0, 64, 64, 1, 0, 0, 0, p, 1 << 16, p, 1 << 16, None) == -2
    assert fw(p, p, p, big, big, big, 1, 0, 0, 0, p, 1 << 16, p, 1 << 16, None) == -2

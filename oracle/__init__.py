"""CPU oracle for the MXFP4 quantize + block-scaled GEMM path (test infrastructure only).

This package wraps ``mxfp4_oracle.c`` (plain C, fp32 exactly where the method fixes fp32,
fp64 for the GEMM) with numpy in / numpy out functions.  It imports nothing from the CUDA
package and the CUDA package imports nothing from here.  Only tests, the smoke check and
the benchmark's CPU-baseline leg may use it.

bf16 tensors are passed as ``uint16`` arrays holding the raw bit patterns.

Passages followed: Appendix A.1 Eq. (1) (micro-scaling), Appendix A.2 (Hadamard rotation,
random sign flips), Appendix C (which axis each operand of Fprop / Dgrad / Wgrad is rotated
and quantized along), Appendix D (row-wise and column-wise 32-blocks).
Stochastic rounding: parity unpinned against the paper (it gives no definition).

``mxfp8_oracle.c`` holds the 8-bit passes of the precision ladder (Table 1): the paper names the
format only as "FP8"; the reading taken is MXFP8 (E4M3 elements, the same E8M0 block scale).
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "mxfp4_oracle.c")
_SRC8 = os.path.join(_HERE, "mxfp8_oracle.c")      # the 8-bit passes of the precision ladder
_LIB = os.path.join(_HERE, "libmxfp4_oracle.so")

HADAMARD_NONE, HADAMARD_DET, HADAMARD_RAND, HADAMARD_DET16, HADAMARD_RAND16 = 0, 1, 2, 3, 4
ROUND_RNE, ROUND_SR = 0, 1


def build(force: bool = False) -> str:
    """Compile the C oracle into ``libmxfp4_oracle.so`` next to its source (gcc, OpenMP)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < max(os.path.getmtime(_SRC),
                                                                         os.path.getmtime(_SRC8)):
        tmp = _LIB + f".tmp{os.getpid()}"
        cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off",
               "-o", tmp, _SRC, _SRC8, "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is not None:
        return _lib
    lib = ctypes.CDLL(build())
    u8p = ctypes.POINTER(ctypes.c_uint8)
    i64 = ctypes.c_int64
    lib.oracle_philox4x32_10.argtypes = [ctypes.POINTER(ctypes.c_uint32)] * 3
    lib.oracle_philox4x32_10.restype = None
    lib.oracle_sign_mask.argtypes = [ctypes.c_uint64]
    lib.oracle_sign_mask.restype = ctypes.c_uint32
    lib.oracle_fwht32.argtypes = [ctypes.POINTER(ctypes.c_float)]
    lib.oracle_fwht32.restype = None
    lib.oracle_fwht16x2.argtypes = [ctypes.POINTER(ctypes.c_float)]
    lib.oracle_fwht16x2.restype = None
    lib.oracle_quantize.argtypes = [ctypes.POINTER(ctypes.c_uint16), i64, i64, i64, ctypes.c_int,
                                    ctypes.c_int, ctypes.c_int, ctypes.c_uint64, ctypes.c_uint32,
                                    u8p, u8p]
    lib.oracle_quantize.restype = ctypes.c_int
    lib.oracle_quantize_2d.argtypes = lib.oracle_quantize.argtypes
    lib.oracle_quantize_2d.restype = ctypes.c_int
    lib.oracle_e4m3_decode.argtypes, lib.oracle_e4m3_decode.restype = [ctypes.c_uint8], ctypes.c_double
    lib.oracle_e4m3_encode.argtypes, lib.oracle_e4m3_encode.restype = [ctypes.c_float], ctypes.c_uint8
    lib.oracle_quantize_mxfp8.argtypes = [ctypes.POINTER(ctypes.c_uint16), i64, i64, i64, ctypes.c_int, u8p, u8p]
    lib.oracle_quantize_mxfp8.restype = ctypes.c_int
    lib.oracle_gemm_rows_mxfp8.argtypes = [u8p, u8p, u8p, u8p, i64, i64, i64, ctypes.c_double,
                                           ctypes.POINTER(ctypes.c_int64), i64,
                                           ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_double)]
    lib.oracle_gemm_rows_mxfp8.restype = ctypes.c_int
    lib.oracle_scale_offset_tiled.argtypes = [i64, i64, i64]
    lib.oracle_scale_offset_tiled.restype = i64
    lib.oracle_dequantize.argtypes = [u8p, u8p, i64, i64, ctypes.POINTER(ctypes.c_double)]
    lib.oracle_dequantize.restype = ctypes.c_int
    lib.oracle_gemm_rows.argtypes = [u8p, u8p, u8p, u8p, i64, i64, i64, ctypes.c_double,
                                     ctypes.POINTER(i64), i64, ctypes.POINTER(ctypes.c_double),
                                     ctypes.POINTER(ctypes.c_double)]
    lib.oracle_gemm_rows.restype = ctypes.c_int
    lib.oracle_num_threads.argtypes = []
    lib.oracle_num_threads.restype = ctypes.c_int
    _lib = lib
    return lib


def _ptr(a: np.ndarray, ctype):
    return a.ctypes.data_as(ctypes.POINTER(ctype))


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def philox4x32_10(ctr, key) -> np.ndarray:
    """Four 32-bit outputs of Philox4x32-10 for a 4-word counter and a 2-word key."""
    c = np.asarray(ctr, dtype=np.uint32).copy()
    k = np.asarray(key, dtype=np.uint32).copy()
    assert c.shape == (4,) and k.shape == (2,)
    out = np.zeros(4, dtype=np.uint32)
    _load().oracle_philox4x32_10(_ptr(c, ctypes.c_uint32), _ptr(k, ctypes.c_uint32),
                                 _ptr(out, ctypes.c_uint32))
    return out


def sign_mask(seed: int) -> int:
    """32-bit sign mask of the randomized rotation for ``seed`` (Appendix A.2)."""
    return int(_load().oracle_sign_mask(ctypes.c_uint64(seed)))


def fwht32(v) -> np.ndarray:
    """Unnormalised 32-point Walsh-Hadamard transform in fp32, fixed butterfly order."""
    a = np.ascontiguousarray(v, dtype=np.float32).copy()
    assert a.shape == (32,)
    _load().oracle_fwht32(_ptr(a, ctypes.c_float))
    return a


def fwht16x2(v) -> np.ndarray:
    """Two unnormalised 16-point Walsh-Hadamard transforms, one per half of a 32-vector."""
    a = np.ascontiguousarray(v, dtype=np.float32).copy()
    assert a.shape == (32,)
    _load().oracle_fwht16x2(_ptr(a, ctypes.c_float))
    return a


def quantize(src_bits: np.ndarray, axis: int = 1, hadamard_mode: int = 0, rounding: int = 0,
             seed: int = 0, tag: int = 0, block2d: bool = False):
    """MXFP4-quantize a [rows x cols] bf16 matrix (uint16 bit patterns).

    Returns ``(codes [outer x K/2] uint8, scales [outer x K/32] uint8)`` for the operand view
    (axis=1: outer=rows, K=cols; axis=0: outer=cols, K=rows -- the transposed operand).
    ``block2d`` selects the 32 x 32 block strategy of Appendix D (one scale per 32 operand rows
    x 32 elements, replicated into every row's scale entry) instead of 1 x 32 blocks.
    """
    assert src_bits.dtype == np.uint16 and src_bits.ndim == 2
    src = np.ascontiguousarray(src_bits)
    rows, cols = src.shape
    outer, K = (rows, cols) if axis == 1 else (cols, rows)
    codes = np.empty((outer, K // 2), dtype=np.uint8)
    scales = np.empty((outer, K // 32), dtype=np.uint8)
    fn = _load().oracle_quantize_2d if block2d else _load().oracle_quantize
    rc = fn(_ptr(src, ctypes.c_uint16), rows, cols, cols, axis, hadamard_mode,
            rounding, ctypes.c_uint64(seed), ctypes.c_uint32(tag),
            _ptr(codes, ctypes.c_uint8), _ptr(scales, ctypes.c_uint8))
    if rc != 0:
        raise ValueError(f"oracle_quantize rejected its arguments (rc={rc})")
    return codes, scales


def scale_offset_tiled(o: int, t: int, nt: int) -> int:
    return int(_load().oracle_scale_offset_tiled(o, t, nt))


def tiled_scale_bytes(outer: int, nt: int) -> int:
    """Size of the tiled scale buffer: whole 128-row x 4-block tiles of 512 bytes."""
    return ((outer + 127) // 128) * ((nt + 3) // 4) * 512


def scales_from_tiled(buf: np.ndarray, outer: int, nt: int) -> np.ndarray:
    """Undo the 128x4 tiling: gather canonical [outer x nt] scales out of a tiled buffer."""
    buf = np.asarray(buf, dtype=np.uint8).reshape(-1)
    assert buf.size >= tiled_scale_bytes(outer, nt)
    o = np.arange(outer, dtype=np.int64)[:, None]
    t = np.arange(nt, dtype=np.int64)[None, :]
    tiles_k = (nt + 3) // 4
    off = ((o // 128) * tiles_k + (t // 4)) * 512 + (o % 32) * 16 + ((o % 128) // 32) * 4 + (t % 4)
    # the vectorised index above restates oracle_scale_offset_tiled; spot-check it against C
    for oo, tt in ((0, 0), (outer - 1, nt - 1), (outer // 2, nt // 2)):
        assert off[oo, tt] == scale_offset_tiled(oo, tt, nt)
    return buf[off]


def scales_to_tiled(scales: np.ndarray, pad: int = 0) -> np.ndarray:
    """Canonical [outer x nt] scales -> tiled buffer (padding bytes = ``pad``)."""
    outer, nt = scales.shape
    out = np.full(tiled_scale_bytes(outer, nt), pad, dtype=np.uint8)
    o = np.arange(outer, dtype=np.int64)[:, None]
    t = np.arange(nt, dtype=np.int64)[None, :]
    tiles_k = (nt + 3) // 4
    off = ((o // 128) * tiles_k + (t // 4)) * 512 + (o % 32) * 16 + ((o % 128) // 32) * 4 + (t % 4)
    out[off] = scales
    return out


def dequantize(codes: np.ndarray, scales: np.ndarray) -> np.ndarray:
    """Eq. (1): grid[code] * 2^(scale-127) as float64 [outer x K]."""
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    scales = np.ascontiguousarray(scales, dtype=np.uint8)
    outer, kh = codes.shape
    K = kh * 2
    assert scales.shape == (outer, K // 32)
    out = np.empty((outer, K), dtype=np.float64)
    rc = _load().oracle_dequantize(_ptr(codes, ctypes.c_uint8), _ptr(scales, ctypes.c_uint8),
                                   outer, K, _ptr(out, ctypes.c_double))
    if rc != 0:
        raise ValueError("oracle_dequantize rejected its arguments")
    return out


def gemm(a_codes, a_scales, b_codes, b_scales, alpha: float = 1.0, rows=None):
    """fp64 block-scaled product ``alpha * deq(A) @ deq(B).T`` and the tolerance base S.

    ``rows`` (optional) restricts the output to those rows of A.  Returns ``(ref, S)`` of
    shape [len(rows) or M, N].
    """
    a_codes = np.ascontiguousarray(a_codes, dtype=np.uint8)
    b_codes = np.ascontiguousarray(b_codes, dtype=np.uint8)
    a_scales = np.ascontiguousarray(a_scales, dtype=np.uint8)
    b_scales = np.ascontiguousarray(b_scales, dtype=np.uint8)
    M, kh = a_codes.shape
    N, kh2 = b_codes.shape
    assert kh == kh2
    K = 2 * kh
    assert a_scales.shape == (M, K // 32) and b_scales.shape == (N, K // 32)
    if rows is None:
        rows_arr, rp, nrows = None, None, M
    else:
        rows_arr = np.ascontiguousarray(rows, dtype=np.int64)
        rp, nrows = _ptr(rows_arr, ctypes.c_int64), int(rows_arr.size)
    ref = np.empty((nrows, N), dtype=np.float64)
    S = np.empty((nrows, N), dtype=np.float64)
    rc = _load().oracle_gemm_rows(_ptr(a_codes, ctypes.c_uint8), _ptr(a_scales, ctypes.c_uint8),
                                  _ptr(b_codes, ctypes.c_uint8), _ptr(b_scales, ctypes.c_uint8),
                                  M, N, K, float(alpha), rp, nrows, _ptr(ref, ctypes.c_double),
                                  _ptr(S, ctypes.c_double))
    if rc != 0:
        raise ValueError(f"oracle_gemm_rows failed (rc={rc})")
    return ref, S


def _alpha(hadamard_mode: int) -> float:
    # H H^T = n I for the +-1 matrix of order n: the product of two rotated operands carries n
    return {0: 1.0, 1: 1.0 / 32.0, 2: 1.0 / 32.0, 3: 1.0 / 16.0, 4: 1.0 / 16.0}[hadamard_mode]


def linear_fprop(X, W, hadamard_mode=1, rounding=0, seed=0, rows=None):
    """Y = X W^T (Appendix C, forward): both operands rotated/quantized along ``in``."""
    a = quantize(X, 1, hadamard_mode, rounding, seed, 0)
    b = quantize(W, 1, hadamard_mode, rounding, seed, 1)
    return gemm(*a, *b, alpha=_alpha(hadamard_mode), rows=rows)


def linear_dgrad(dY, W, hadamard_mode=1, rounding=0, seed=0, rows=None):
    """dX = dY W (Appendix C, Dgrad): dY along ``out``; W column-wise (operand W^T)."""
    a = quantize(dY, 1, hadamard_mode, rounding, seed, 0)
    b = quantize(W, 0, hadamard_mode, rounding, seed, 1)
    return gemm(*a, *b, alpha=_alpha(hadamard_mode), rows=rows)


def linear_wgrad(dY, X, hadamard_mode=1, rounding=0, seed=0, rows=None):
    """dW = dY^T X (Appendix C, Wgrad): both operands quantized along the token axis."""
    a = quantize(dY, 0, hadamard_mode, rounding, seed, 0)
    b = quantize(X, 0, hadamard_mode, rounding, seed, 1)
    return gemm(*a, *b, alpha=_alpha(hadamard_mode), rows=rows)


# ----------------------------------------------------------------------------- 8-bit passes
def e4m3_decode(code: int) -> float:
    return float(_load().oracle_e4m3_decode(int(code)))


def e4m3_encode(x: float) -> int:
    return int(_load().oracle_e4m3_encode(ctypes.c_float(x)))


def quantize_mxfp8(src_bits: np.ndarray, axis: int = 1):
    """MXFP8 (E4M3 elements, E8M0 scale per 32 along K) of a [rows x cols] bf16 matrix.

    Returns ``(codes [outer x K] uint8, scales [outer x K/32] uint8)`` for the operand view of
    :func:`quantize`.  Round-to-nearest-even, saturating; no rotation.
    """
    assert src_bits.dtype == np.uint16 and src_bits.ndim == 2
    src = np.ascontiguousarray(src_bits)
    rows, cols = src.shape
    outer, K = (rows, cols) if axis == 1 else (cols, rows)
    codes = np.empty((outer, K), dtype=np.uint8)
    scales = np.empty((outer, K // 32), dtype=np.uint8)
    rc = _load().oracle_quantize_mxfp8(_ptr(src, ctypes.c_uint16), rows, cols, cols, axis,
                                       _ptr(codes, ctypes.c_uint8), _ptr(scales, ctypes.c_uint8))
    if rc != 0:
        raise ValueError(f"oracle_quantize_mxfp8 rejected its arguments (rc={rc})")
    return codes, scales


def gemm_mxfp8(a_codes, a_scales, b_codes, b_scales, alpha: float = 1.0, rows=None):
    """fp64 block-scaled product of E4M3 operands and the tolerance base S (see :func:`gemm`)."""
    a_codes = np.ascontiguousarray(a_codes, dtype=np.uint8)
    b_codes = np.ascontiguousarray(b_codes, dtype=np.uint8)
    a_scales = np.ascontiguousarray(a_scales, dtype=np.uint8)
    b_scales = np.ascontiguousarray(b_scales, dtype=np.uint8)
    M, K = a_codes.shape
    N, K2 = b_codes.shape
    assert K == K2 and a_scales.shape == (M, K // 32) and b_scales.shape == (N, K // 32)
    if rows is None:
        rows_arr, rp, nrows = None, None, M
    else:
        rows_arr = np.ascontiguousarray(rows, dtype=np.int64)
        rp, nrows = _ptr(rows_arr, ctypes.c_int64), int(rows_arr.size)
    ref = np.empty((nrows, N), dtype=np.float64)
    S = np.empty((nrows, N), dtype=np.float64)
    rc = _load().oracle_gemm_rows_mxfp8(_ptr(a_codes, ctypes.c_uint8), _ptr(a_scales, ctypes.c_uint8),
                                        _ptr(b_codes, ctypes.c_uint8), _ptr(b_scales, ctypes.c_uint8),
                                        M, N, K, float(alpha), rp, nrows, _ptr(ref, ctypes.c_double),
                                        _ptr(S, ctypes.c_double))
    if rc != 0:
        raise ValueError(f"oracle_gemm_rows_mxfp8 failed (rc={rc})")
    return ref, S


def linear_pass_mxfp8(pass_: int, a_bits, b_bits, rows=None):
    """One pass of a linear layer left in 8 bits (Table 1): operand orientation as Appendix C,
    (a, b) = (X, W) / (dY, W) / (dY, X) for pass 0 / 1 / 2."""
    axes = ((1, 1), (1, 0), (0, 0))[pass_]
    a = quantize_mxfp8(a_bits, axes[0])
    b = quantize_mxfp8(b_bits, axes[1])
    return gemm_mxfp8(*a, *b, rows=rows)

"""Thin ctypes binding over ``libmxfp4.so`` (the C ABI declared in ``include/mxfp4.h``).

Argument marshalling only: torch provides device memory and the current CUDA stream; every
step of the path runs inside the library's kernels.  There is no CPU or PyTorch fallback:
if the shared library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os

import torch

from . import build as _build

HADAMARD_NONE, HADAMARD_DET, HADAMARD_RAND, HADAMARD_DET16, HADAMARD_RAND16 = 0, 1, 2, 3, 4
ROUND_RNE, ROUND_SR = 0, 1
SCALES_CANONICAL, SCALES_TILED = 0, 1
BLOCK_1X32, BLOCK_32X32 = 0, 1
OUT_BF16, OUT_FP32 = 0, 1
LAYER_SAVED, LAYER_FORWARD, LAYER_BACKWARD = 0, 1, 2
PRECISION_MXFP4, PRECISION_MXFP8, PRECISION_MXFP4_32X32 = 0, 1, 2
PASS_FPROP, PASS_DGRAD, PASS_WGRAD = 0, 1, 2
AXIS_ROWS, AXIS_COLS = 0, 1

EXPORTS = (
    "mxfp4_version", "mxfp4_status_string", "mxfp4_codes_bytes", "mxfp4_scales_bytes",
    "mxfp4_quantize", "mxfp4_quantize_2d", "mxfp4_quantize_dual", "mxfp4_quantize_pair", "mxfp4_gemm", "mxfp4_linear_workspace_bytes", "mxfp4_linear_fprop",
    "mxfp4_linear_dgrad", "mxfp4_linear_wgrad", "mxfp4_linear_layer_bytes", "mxfp4_linear_forward",
    "mxfp4_linear_backward", "mxfp4_linear_layer_host", "mxfp4_linear_layer_host_drain", "mxfp4_quantize_fp8", "mxfp4_gemm_fp8",
    "mxfp4_linear_pass_workspace_bytes", "mxfp4_linear_pass", "mxfp4_linear_host", "mxfp4_linear_static",
    "mxfp4_check", "mxfp4_selftest_wait_timeout", "mxfp4_bounds_checked", "mxfp4_selftest_bounds",
    "mxfp4_probe_mma_rate",
)
STATIC_SCRATCH_BYTES = 16 * 1024 * 1024


class QuantDesc(ctypes.Structure):
    """``mxfp4_quant_desc``: one tensor of an ``mxfp4_quantize_pair`` call."""
    _fields_ = [("src_bf16", ctypes.c_void_p), ("rows", ctypes.c_int64), ("cols", ctypes.c_int64),
                ("ld_src", ctypes.c_int64), ("axis", ctypes.c_int32), ("operand_tag", ctypes.c_uint32),
                ("codes", ctypes.c_void_p), ("scales", ctypes.c_void_p)]


class Mxfp4Error(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        super().__init__(f"{what} failed: {status} ({status_string(status)})")


_lib = None


def library_path() -> str:
    """Path of the shared library; ``MXFP4_LIBRARY`` overrides the in-tree build."""
    return os.environ.get("MXFP4_LIBRARY") or _build.LIB_PATH


def load_library() -> ctypes.CDLL:
    """Load ``libmxfp4.so`` (must have been built in-tree); raises if it is missing."""
    global _lib
    if _lib is not None:
        return _lib
    path = library_path()
    if not os.path.exists(path):
        raise FileNotFoundError(
            f"{path} not found: build it with `python -m paper_2605_09825_b200.build` "
            "(there is no fallback path)")
    lib = ctypes.CDLL(path)
    vp, i64, u64, u32, ci, sz = (ctypes.c_void_p, ctypes.c_int64, ctypes.c_uint64, ctypes.c_uint32,
                                 ctypes.c_int, ctypes.c_size_t)
    lib.mxfp4_version.argtypes, lib.mxfp4_version.restype = [], ci
    lib.mxfp4_status_string.argtypes, lib.mxfp4_status_string.restype = [ci], ctypes.c_char_p
    lib.mxfp4_codes_bytes.argtypes, lib.mxfp4_codes_bytes.restype = [i64, i64], sz
    lib.mxfp4_scales_bytes.argtypes, lib.mxfp4_scales_bytes.restype = [i64, i64, ci], sz
    lib.mxfp4_quantize.argtypes = [vp, i64, i64, i64, ci, ci, ci, u64, u32, vp, vp, ci, vp]
    lib.mxfp4_quantize.restype = ci
    lib.mxfp4_quantize_2d.argtypes = lib.mxfp4_quantize.argtypes
    lib.mxfp4_quantize_2d.restype = ci
    lib.mxfp4_quantize_dual.argtypes = [vp, i64, i64, i64, ci, ci, u64, u32, u32, ci, vp, vp, vp, vp, ci, vp]
    lib.mxfp4_quantize_dual.restype = ci
    lib.mxfp4_quantize_pair.argtypes = [ctypes.POINTER(QuantDesc), ctypes.POINTER(QuantDesc), ci, ci, u64, ci, vp]
    lib.mxfp4_quantize_pair.restype = ci
    lib.mxfp4_gemm.argtypes = [vp, vp, vp, vp, i64, i64, i64, ctypes.c_float, vp, ci, i64, vp, sz, vp]
    lib.mxfp4_gemm.restype = ci
    lib.mxfp4_linear_workspace_bytes.argtypes = [i64, i64, i64, ci]
    lib.mxfp4_linear_workspace_bytes.restype = sz
    for name in ("mxfp4_linear_fprop", "mxfp4_linear_dgrad", "mxfp4_linear_wgrad"):
        fn = getattr(lib, name)
        fn.argtypes = [vp, vp, vp, i64, i64, i64, ci, ci, u64, ci, vp, sz, vp]
        fn.restype = ci
    lib.mxfp4_quantize_fp8.argtypes, lib.mxfp4_quantize_fp8.restype = [vp, i64, i64, i64, ci, vp, vp, ci, vp], ci
    lib.mxfp4_gemm_fp8.argtypes = [vp, vp, vp, vp, i64, i64, i64, ctypes.c_float, vp, ci, i64, vp]
    lib.mxfp4_gemm_fp8.restype = ci
    lib.mxfp4_linear_pass_workspace_bytes.argtypes = [i64, i64, i64, ci, ci]
    lib.mxfp4_linear_pass_workspace_bytes.restype = sz
    lib.mxfp4_linear_pass.argtypes = [ci, ci, vp, vp, vp, i64, i64, i64, ci, ci, u64, ci, vp, sz, vp]
    lib.mxfp4_linear_pass.restype = ci
    lib.mxfp4_linear_layer_bytes.argtypes, lib.mxfp4_linear_layer_bytes.restype = [i64, i64, i64, ci], sz
    lib.mxfp4_linear_forward.argtypes = [vp, vp, vp, i64, i64, i64, ci, ci, u64, ci, vp, sz, vp, sz, vp]
    lib.mxfp4_linear_forward.restype = ci
    lib.mxfp4_linear_backward.argtypes = [vp, vp, vp, i64, i64, i64, ci, ci, u64, ci, ci, vp, sz, vp, sz, vp]
    lib.mxfp4_linear_backward.restype = ci
    lib.mxfp4_linear_layer_host.argtypes = [vp] * 6 + [i64, i64, i64, ci, ci, u64, ci, ci, ci] + [vp] * 6 + \
        [vp, sz, vp, sz, vp, ci]
    lib.mxfp4_linear_layer_host.restype = ci
    lib.mxfp4_linear_layer_host_drain.argtypes, lib.mxfp4_linear_layer_host_drain.restype = [vp], ci
    lib.mxfp4_linear_host.argtypes = [ci, vp, vp, vp, i64, i64, i64, ci, ci, u64, ci, vp, vp, vp, vp,
                                      sz, vp]
    lib.mxfp4_linear_host.restype = ci
    lib.mxfp4_linear_static.argtypes = [ci, vp, vp, vp, i64, i64, i64, ci, ci, u64, ci, vp]
    lib.mxfp4_linear_static.restype = ci
    lib.mxfp4_check.argtypes, lib.mxfp4_check.restype = [vp], ci
    lib.mxfp4_selftest_wait_timeout.argtypes, lib.mxfp4_selftest_wait_timeout.restype = [vp], ci
    lib.mxfp4_selftest_bounds.argtypes, lib.mxfp4_selftest_bounds.restype = [vp], ci
    lib.mxfp4_bounds_checked.argtypes, lib.mxfp4_bounds_checked.restype = [], ci
    lib.mxfp4_probe_mma_rate.argtypes = [ci, ci, vp, ctypes.POINTER(ctypes.c_double)]
    lib.mxfp4_probe_mma_rate.restype = ci
    _lib = lib
    return lib


def version() -> int:
    return int(load_library().mxfp4_version())


def status_string(status: int) -> str:
    return load_library().mxfp4_status_string(int(status)).decode()


def codes_bytes(outer: int, K: int) -> int:
    return int(load_library().mxfp4_codes_bytes(outer, K))


def scales_bytes(outer: int, K: int, scale_layout: int = SCALES_TILED) -> int:
    return int(load_library().mxfp4_scales_bytes(outer, K, scale_layout))


def linear_workspace_bytes(T: int, in_features: int, out_features: int, pass_: int) -> int:
    return int(load_library().mxfp4_linear_workspace_bytes(T, in_features, out_features, pass_))


def _stream() -> int:
    return int(torch.cuda.current_stream().cuda_stream)


def _dev_ptr(t: torch.Tensor) -> int:
    if not t.is_cuda:
        raise ValueError("expected a CUDA tensor")
    return int(t.data_ptr())


def _raise(rc: int, what: str):
    if rc != 0:
        raise Mxfp4Error(rc, what)


def quantize(src: torch.Tensor, axis: int = AXIS_COLS, hadamard_mode: int = HADAMARD_NONE,
             rounding: int = ROUND_RNE, seed: int = 0, operand_tag: int = 0,
             scale_layout: int = SCALES_TILED, codes: torch.Tensor | None = None,
             scales: torch.Tensor | None = None, block_shape: int = 0):
    """``mxfp4_quantize`` (``block_shape`` BLOCK_1X32) or ``mxfp4_quantize_2d`` (BLOCK_32X32) on a
    2-D bf16 CUDA tensor (rows may be strided: ``ld = stride(0)``).

    Returns ``(codes uint8 [outer, K/2], scales uint8 [scales_bytes])``; output tensors are
    allocated with torch unless passed in.
    """
    if src.dtype != torch.bfloat16 or src.dim() != 2 or src.stride(1) != 1:
        raise ValueError("src must be a 2-D bf16 tensor with contiguous rows")
    rows, cols = src.shape
    outer, K = (rows, cols) if axis == AXIS_COLS else (cols, rows)
    lib = load_library()
    if K % 32 != 0 or K <= 0 or outer <= 0:
        _raise(-2, "mxfp4_quantize")
    if codes is None:
        codes = torch.empty((outer, K // 2), dtype=torch.uint8, device=src.device)
    if scales is None:
        scales = torch.empty(scales_bytes(outer, K, scale_layout), dtype=torch.uint8, device=src.device)
    ld = src.stride(0) if rows > 1 else cols   # a single row's stride is arbitrary in torch
    fn = lib.mxfp4_quantize_2d if block_shape == BLOCK_32X32 else lib.mxfp4_quantize
    rc = fn(_dev_ptr(src), rows, cols, ld, axis, hadamard_mode, rounding,
            ctypes.c_uint64(seed), ctypes.c_uint32(operand_tag), _dev_ptr(codes),
            _dev_ptr(scales), scale_layout, _stream())
    _raise(rc, "mxfp4_quantize")
    return codes, scales


def quantize_dual(src: torch.Tensor, hadamard_mode: int = HADAMARD_NONE, rounding: int = ROUND_RNE,
                  seed: int = 0, tags=(0, 1), block_shape: int = 0, scale_layout: int = SCALES_TILED,
                  out_row=None, out_col=None):
    """``mxfp4_quantize_dual``: row-wise and column-wise operands of ``src`` from one read.

    Returns ``((codes [rows, cols/2], scales), (codes [cols, rows/2], scales))``; ``out_row`` /
    ``out_col`` are optional ``(codes, scales)`` tensors to write into.
    """
    if src.dtype != torch.bfloat16 or src.dim() != 2 or src.stride(1) != 1:
        raise ValueError("src must be a 2-D bf16 tensor with contiguous rows")
    rows, cols = src.shape
    lib = load_library()
    if rows % 32 != 0 or cols % 32 != 0 or rows <= 0 or cols <= 0:
        _raise(-2, "mxfp4_quantize_dual")
    cr, sr = out_row if out_row is not None else (
        torch.empty((rows, cols // 2), dtype=torch.uint8, device=src.device),
        torch.empty(scales_bytes(rows, cols, scale_layout), dtype=torch.uint8, device=src.device))
    cc, sc = out_col if out_col is not None else (
        torch.empty((cols, rows // 2), dtype=torch.uint8, device=src.device),
        torch.empty(scales_bytes(cols, rows, scale_layout), dtype=torch.uint8, device=src.device))
    rc = lib.mxfp4_quantize_dual(_dev_ptr(src), rows, cols, src.stride(0), hadamard_mode, rounding,
                                 ctypes.c_uint64(seed), ctypes.c_uint32(tags[0]), ctypes.c_uint32(tags[1]),
                                 block_shape, _dev_ptr(cr), _dev_ptr(sr), _dev_ptr(cc), _dev_ptr(sc),
                                 scale_layout, _stream())
    _raise(rc, "mxfp4_quantize_dual")
    return (cr, sr), (cc, sc)


def _quant_desc(src, axis, tag, scale_layout, codes, scales):
    if src.dtype != torch.bfloat16 or src.dim() != 2 or src.stride(1) != 1:
        raise ValueError("src must be a 2-D bf16 tensor with contiguous rows")
    rows, cols = src.shape
    outer, K = (rows, cols) if axis == AXIS_COLS else (cols, rows)
    if K % 32 != 0 or K <= 0 or outer <= 0:
        _raise(-2, "mxfp4_quantize_pair")
    if codes is None:
        codes = torch.empty((outer, K // 2), dtype=torch.uint8, device=src.device)
    if scales is None:
        scales = torch.empty(scales_bytes(outer, K, scale_layout), dtype=torch.uint8, device=src.device)
    ld = src.stride(0) if rows > 1 else cols
    return QuantDesc(_dev_ptr(src), rows, cols, ld, axis, tag, _dev_ptr(codes), _dev_ptr(scales)), codes, scales


def quantize_pair(src_a: torch.Tensor, axis_a: int, src_b: torch.Tensor, axis_b: int,
                  hadamard_mode: int = HADAMARD_NONE, rounding: int = ROUND_RNE, seed: int = 0,
                  tags=(0, 1), scale_layout: int = SCALES_TILED, out_a=None, out_b=None):
    """``mxfp4_quantize_pair``: both tensors through one launch.

    ``out_a`` / ``out_b`` are optional ``(codes, scales)`` tensors.  Returns
    ``((codes_a, scales_a), (codes_b, scales_b))``.
    """
    lib = load_library()
    ca, sa = out_a if out_a is not None else (None, None)
    cb, sb = out_b if out_b is not None else (None, None)
    da, ca, sa = _quant_desc(src_a, axis_a, tags[0], scale_layout, ca, sa)
    db, cb, sb = _quant_desc(src_b, axis_b, tags[1], scale_layout, cb, sb)
    rc = lib.mxfp4_quantize_pair(ctypes.byref(da), ctypes.byref(db), hadamard_mode, rounding,
                                 ctypes.c_uint64(seed), scale_layout, _stream())
    _raise(rc, "mxfp4_quantize_pair")
    return (ca, sa), (cb, sb)


def gemm(a_codes: torch.Tensor, a_scales: torch.Tensor, b_codes: torch.Tensor, b_scales: torch.Tensor,
         alpha: float = 1.0, out_dtype: int = OUT_BF16, out: torch.Tensor | None = None):
    """``mxfp4_gemm``: ``alpha * A B^T`` from packed codes [M, K/2], [N, K/2] and tiled scales."""
    M, kh = a_codes.shape
    N, kh2 = b_codes.shape
    if kh != kh2:
        raise ValueError("A and B disagree on K")
    K = 2 * kh
    if out is None:
        out = torch.empty((M, N), dtype=torch.bfloat16 if out_dtype == OUT_BF16 else torch.float32,
                          device=a_codes.device)
    rc = load_library().mxfp4_gemm(_dev_ptr(a_codes), _dev_ptr(a_scales), _dev_ptr(b_codes),
                                   _dev_ptr(b_scales), M, N, K, ctypes.c_float(alpha), _dev_ptr(out),
                                   out_dtype, out.stride(0), None, 0, _stream())
    _raise(rc, "mxfp4_gemm")
    return out


def _linear(name: str, pass_: int, a: torch.Tensor, b: torch.Tensor, T: int, in_f: int, out_f: int,
            out_shape, hadamard_mode, rounding, seed, out_dtype, workspace, out):
    for t in (a, b):
        if t.dtype != torch.bfloat16 or not t.is_contiguous():
            raise ValueError("inputs must be contiguous bf16 tensors")
    need = linear_workspace_bytes(T, in_f, out_f, pass_)
    if workspace is None:
        workspace = torch.empty(max(need, 1), dtype=torch.uint8, device=a.device)
    if out is None:
        out = torch.empty(out_shape, dtype=torch.bfloat16 if out_dtype == OUT_BF16 else torch.float32,
                          device=a.device)
    fn = getattr(load_library(), name)
    rc = fn(_dev_ptr(a), _dev_ptr(b), _dev_ptr(out), T, in_f, out_f, hadamard_mode, rounding,
            ctypes.c_uint64(seed), out_dtype, _dev_ptr(workspace), workspace.numel(), _stream())
    _raise(rc, name)
    return out


def linear_fprop(X, W, hadamard_mode=HADAMARD_DET, rounding=ROUND_RNE, seed=0, out_dtype=OUT_BF16,
                 workspace=None, out=None):
    """Y [T, out] = X [T, in] W[out, in]^T through ``mxfp4_linear_fprop``."""
    T, in_f = X.shape
    out_f = W.shape[0]
    return _linear("mxfp4_linear_fprop", PASS_FPROP, X, W, T, in_f, out_f, (T, out_f), hadamard_mode,
                   rounding, seed, out_dtype, workspace, out)


def linear_dgrad(dY, W, hadamard_mode=HADAMARD_DET, rounding=ROUND_RNE, seed=0, out_dtype=OUT_BF16,
                 workspace=None, out=None):
    """dX [T, in] = dY [T, out] W [out, in] through ``mxfp4_linear_dgrad``."""
    T, out_f = dY.shape
    in_f = W.shape[1]
    return _linear("mxfp4_linear_dgrad", PASS_DGRAD, dY, W, T, in_f, out_f, (T, in_f), hadamard_mode,
                   rounding, seed, out_dtype, workspace, out)


def linear_wgrad(dY, X, hadamard_mode=HADAMARD_DET, rounding=ROUND_RNE, seed=0, out_dtype=OUT_BF16,
                 workspace=None, out=None):
    """dW [out, in] = dY [T, out]^T X [T, in] through ``mxfp4_linear_wgrad``."""
    T, out_f = dY.shape
    in_f = X.shape[1]
    return _linear("mxfp4_linear_wgrad", PASS_WGRAD, dY, X, T, in_f, out_f, (out_f, in_f),
                   hadamard_mode, rounding, seed, out_dtype, workspace, out)


def quantize_fp8(src: torch.Tensor, axis: int = AXIS_COLS, scale_layout: int = SCALES_TILED, codes=None,
                 scales=None):
    """``mxfp4_quantize_fp8``: MXFP8 (E4M3 + E8M0 per 32) operand of a 2-D bf16 CUDA tensor.
    Returns ``(codes uint8 [outer, K], scales uint8 [scales_bytes])``."""
    if src.dtype != torch.bfloat16 or src.dim() != 2 or src.stride(1) != 1:
        raise ValueError("src must be a 2-D bf16 tensor with contiguous rows")
    rows, cols = src.shape
    outer, K = (rows, cols) if axis == AXIS_COLS else (cols, rows)
    lib = load_library()
    if K % 32 != 0 or K <= 0 or outer <= 0:
        _raise(-2, "mxfp4_quantize_fp8")
    if codes is None:
        codes = torch.empty((outer, K), dtype=torch.uint8, device=src.device)
    if scales is None:
        scales = torch.empty(scales_bytes(outer, K, scale_layout), dtype=torch.uint8, device=src.device)
    ld = src.stride(0) if rows > 1 else cols
    rc = lib.mxfp4_quantize_fp8(_dev_ptr(src), rows, cols, ld, axis, _dev_ptr(codes), _dev_ptr(scales),
                                scale_layout, _stream())
    _raise(rc, "mxfp4_quantize_fp8")
    return codes, scales


def gemm_fp8(a_codes, a_scales, b_codes, b_scales, alpha: float = 1.0, out_dtype: int = OUT_BF16, out=None):
    """``mxfp4_gemm_fp8``: ``alpha * A B^T`` from E4M3 codes [M, K], [N, K] and tiled scales."""
    M, K = a_codes.shape
    N, K2 = b_codes.shape
    if K != K2:
        raise ValueError("A and B disagree on K")
    out = _out_tensor((M, N), out_dtype, a_codes.device, out)
    rc = load_library().mxfp4_gemm_fp8(_dev_ptr(a_codes), _dev_ptr(a_scales), _dev_ptr(b_codes), _dev_ptr(b_scales),
                                       M, N, K, ctypes.c_float(alpha), _dev_ptr(out), out_dtype, out.stride(0),
                                       _stream())
    _raise(rc, "mxfp4_gemm_fp8")
    return out


def linear_pass(pass_: int, precision: int, a, b, hadamard_mode=HADAMARD_DET, rounding=ROUND_RNE, seed=0,
                out_dtype=OUT_BF16, workspace=None, out=None):
    """``mxfp4_linear_pass``: one pass at MXFP4 or MXFP8; (a, b) = (X, W) / (dY, W) / (dY, X)."""
    for t in (a, b):
        if t.dtype != torch.bfloat16 or not t.is_contiguous():
            raise ValueError("inputs must be contiguous bf16 tensors")
    if pass_ == PASS_FPROP:
        T, in_f, out_f, shape = a.shape[0], a.shape[1], b.shape[0], (a.shape[0], b.shape[0])
    elif pass_ == PASS_DGRAD:
        T, out_f, in_f, shape = a.shape[0], a.shape[1], b.shape[1], (a.shape[0], b.shape[1])
    else:
        T, out_f, in_f, shape = a.shape[0], a.shape[1], b.shape[1], (a.shape[1], b.shape[1])
    lib = load_library()
    if workspace is None:
        need = int(lib.mxfp4_linear_pass_workspace_bytes(T, in_f, out_f, pass_, precision))
        workspace = torch.empty(max(need, 1), dtype=torch.uint8, device=a.device)
    out = _out_tensor(shape, out_dtype, a.device, out)
    rc = lib.mxfp4_linear_pass(pass_, precision, _dev_ptr(a), _dev_ptr(b), _dev_ptr(out), T, in_f, out_f,
                               hadamard_mode, rounding, ctypes.c_uint64(seed), out_dtype, _dev_ptr(workspace),
                               workspace.numel(), _stream())
    _raise(rc, "mxfp4_linear_pass")
    return out


def linear_layer_bytes(T: int, in_f: int, out_f: int, which: int) -> int:
    return int(load_library().mxfp4_linear_layer_bytes(T, in_f, out_f, which))


def _out_tensor(shape, out_dtype, device, out):
    if out is not None:
        return out
    return torch.empty(shape, dtype=torch.bfloat16 if out_dtype == OUT_BF16 else torch.float32, device=device)


def linear_forward(X, W, hadamard_mode=HADAMARD_DET, rounding=ROUND_RNE, seed=0, out_dtype=OUT_BF16,
                   saved=None, workspace=None, out=None):
    """``mxfp4_linear_forward``: Y = X W^T with X and W each read once.  Returns ``(Y, saved)``;
    ``saved`` (uint8) holds the column-wise operands ``linear_backward`` needs."""
    for t in (X, W):
        if t.dtype != torch.bfloat16 or not t.is_contiguous():
            raise ValueError("inputs must be contiguous bf16 tensors")
    T, in_f = X.shape
    out_f = W.shape[0]
    if saved is None:
        saved = torch.empty(max(linear_layer_bytes(T, in_f, out_f, LAYER_SAVED), 1), dtype=torch.uint8, device=X.device)
    if workspace is None:
        workspace = torch.empty(max(linear_layer_bytes(T, in_f, out_f, LAYER_FORWARD), 1), dtype=torch.uint8,
                                device=X.device)
    out = _out_tensor((T, out_f), out_dtype, X.device, out)
    rc = load_library().mxfp4_linear_forward(_dev_ptr(X), _dev_ptr(W), _dev_ptr(out), T, in_f, out_f, hadamard_mode,
                                             rounding, ctypes.c_uint64(seed), out_dtype, _dev_ptr(saved),
                                             saved.numel(), _dev_ptr(workspace), workspace.numel(), _stream())
    _raise(rc, "mxfp4_linear_forward")
    return out, saved


def linear_backward(dY, saved, in_f: int, hadamard_mode=HADAMARD_DET, rounding=ROUND_RNE, seed=0,
                    dx_dtype=OUT_BF16, dw_dtype=OUT_BF16, workspace=None, dX=None, dW=None):
    """``mxfp4_linear_backward``: ``(dX, dW)`` from dY and what ``linear_forward`` saved."""
    if dY.dtype != torch.bfloat16 or not dY.is_contiguous():
        raise ValueError("dY must be a contiguous bf16 tensor")
    T, out_f = dY.shape
    if workspace is None:
        workspace = torch.empty(max(linear_layer_bytes(T, in_f, out_f, LAYER_BACKWARD), 1), dtype=torch.uint8,
                                device=dY.device)
    dX = _out_tensor((T, in_f), dx_dtype, dY.device, dX)
    dW = _out_tensor((out_f, in_f), dw_dtype, dY.device, dW)
    rc = load_library().mxfp4_linear_backward(_dev_ptr(dY), _dev_ptr(dX), _dev_ptr(dW), T, in_f, out_f, hadamard_mode,
                                              rounding, ctypes.c_uint64(seed), dx_dtype, dw_dtype, _dev_ptr(saved),
                                              saved.numel(), _dev_ptr(workspace), workspace.numel(), _stream())
    _raise(rc, "mxfp4_linear_backward")
    return dX, dW


def linear_layer_host(X_host, W_host, dY_host, Y_host, dX_host, dW_host, dev: dict, saved, workspace,
                      hadamard_mode=HADAMARD_DET, rounding=ROUND_RNE, seed=0, y_dtype=OUT_BF16,
                      dx_dtype=OUT_BF16, dw_dtype=OUT_BF16, drain=True):
    """``mxfp4_linear_layer_host``: forward + backward of one linear from host (ideally pinned)
    tensors into host tensors; ``dev`` maps "x", "w", "dy", "y", "dx", "dw" to device staging."""
    T, in_f = X_host.shape
    out_f = W_host.shape[0]
    rc = load_library().mxfp4_linear_layer_host(
        X_host.data_ptr(), W_host.data_ptr(), dY_host.data_ptr(), Y_host.data_ptr(), dX_host.data_ptr(),
        dW_host.data_ptr(), T, in_f, out_f, hadamard_mode, rounding, ctypes.c_uint64(seed), y_dtype, dx_dtype,
        dw_dtype, _dev_ptr(dev["x"]), _dev_ptr(dev["w"]), _dev_ptr(dev["dy"]), _dev_ptr(dev["y"]),
        _dev_ptr(dev["dx"]), _dev_ptr(dev["dw"]), _dev_ptr(saved), saved.numel(), _dev_ptr(workspace),
        workspace.numel(), _stream(), 1 if drain else 0)
    _raise(rc, "mxfp4_linear_layer_host")


def linear_layer_host_drain():
    """Wait for every undrained ``linear_layer_host`` call on the current stream."""
    _raise(load_library().mxfp4_linear_layer_host_drain(_stream()), "mxfp4_linear_layer_host_drain")


def linear_host(pass_: int, a_host: torch.Tensor, b_host: torch.Tensor, out_host: torch.Tensor, T: int,
                in_f: int, out_f: int, dev_a, dev_b, dev_out, workspace, hadamard_mode=HADAMARD_DET,
                rounding=ROUND_RNE, seed=0, out_dtype=OUT_BF16):
    """``mxfp4_linear_host``: host (ideally pinned) inputs/outputs, copies inside the call."""
    for t in (a_host, b_host, out_host):
        if t.is_cuda:
            raise ValueError("host tensors expected")
    rc = load_library().mxfp4_linear_host(
        pass_, a_host.data_ptr(), b_host.data_ptr(), out_host.data_ptr(), T, in_f, out_f,
        hadamard_mode, rounding, ctypes.c_uint64(seed), out_dtype, _dev_ptr(dev_a), _dev_ptr(dev_b),
        _dev_ptr(dev_out), _dev_ptr(workspace), workspace.numel(), _stream())
    _raise(rc, "mxfp4_linear_host")
    return out_host


def linear_static(pass_: int, a: torch.Tensor, b: torch.Tensor, T: int, in_f: int, out_f: int,
                  hadamard_mode=HADAMARD_DET, rounding=ROUND_RNE, seed=0, out_dtype=OUT_BF16,
                  out: torch.Tensor | None = None):
    """``mxfp4_linear_static``: a fused pass whose scratch is the library's built-in array.

    For callers that may not allocate device memory: the caller provides inputs and (here,
    optionally) the output; the library allocates nothing.  Problems whose scratch need exceeds
    ``STATIC_SCRATCH_BYTES`` are rejected with status -9.  Calls share one array per device, so
    overlapping calls on different streams race; the first call on a device should come before
    any stream capture.
    """
    for t in (a, b):
        if t.dtype != torch.bfloat16 or not t.is_contiguous():
            raise ValueError("inputs must be contiguous bf16 tensors")
    shape = {PASS_FPROP: (T, out_f), PASS_DGRAD: (T, in_f), PASS_WGRAD: (out_f, in_f)}[pass_]
    if out is None:
        out = torch.empty(shape, dtype=torch.bfloat16 if out_dtype == OUT_BF16 else torch.float32,
                          device=a.device)
    rc = load_library().mxfp4_linear_static(pass_, _dev_ptr(a), _dev_ptr(b), _dev_ptr(out), T, in_f, out_f,
                                            hadamard_mode, rounding, ctypes.c_uint64(seed), out_dtype,
                                            _stream())
    _raise(rc, "mxfp4_linear_static")
    return out


def probe_mma_rate(iterations: int = 10000, random_operands: bool = True) -> float:
    """``mxfp4_probe_mma_rate``: enqueue one launch of the shared-memory-resident MMA loop on the
    current stream; returns the floating-point operations it performs (time it with CUDA events)."""
    fl = ctypes.c_double(0.0)
    _raise(load_library().mxfp4_probe_mma_rate(iterations, int(random_operands), _stream(), ctypes.byref(fl)),
           "mxfp4_probe_mma_rate")
    return fl.value


def bounds_checked() -> bool:
    """True when the loaded library is the bounds-checking debug build (``-DMXFP4_BOUNDS``)."""
    return bool(load_library().mxfp4_bounds_checked())


def selftest_bounds() -> None:
    """``mxfp4_selftest_bounds``: the next :func:`check` raises with status -10 (and clears it)."""
    _raise(load_library().mxfp4_selftest_bounds(_stream()), "mxfp4_selftest_bounds")


def selftest_wait_timeout() -> None:
    """Enqueue the bounded-wait self-test; the next :func:`check` raises with status -7."""
    _raise(load_library().mxfp4_selftest_wait_timeout(_stream()), "mxfp4_selftest_wait_timeout")


def check() -> None:
    """Synchronise the current stream and raise if a kernel recorded a device-side error."""
    _raise(load_library().mxfp4_check(_stream()), "mxfp4_check")

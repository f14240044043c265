"""fp64 CUDA checker of whole GEMM outputs (test infrastructure; see mx_gemm_check.cu).

Built in-tree with nvcc on first use (or by ``__graft_entry__.build()``); loaded with ctypes.
"""
from __future__ import annotations

import ctypes
import os
import struct
import subprocess

import numpy as np
import torch

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "mx_gemm_check.cu")
LIB = os.path.join(HERE, "libmx_gemm_check.so")
_lib = None


def build(force: bool = False) -> str:
    if not force and os.path.exists(LIB) and os.path.getmtime(LIB) >= os.path.getmtime(SRC):
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    tmp = LIB + f".tmp{os.getpid()}"
    cmd = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "-lineinfo", "-shared",
           "-Xcompiler", "-fPIC", "-o", tmp, SRC]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed building the GEMM checker:\n" + res.stdout + res.stderr)
    os.replace(tmp, LIB)
    return LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        vp, ll, dbl, ci = ctypes.c_void_p, ctypes.c_longlong, ctypes.c_double, ctypes.c_int
        lib.mxcheck_gemm.argtypes = [vp, vp, vp, vp, ll, ll, ll, dbl, vp, ci, ll, dbl, dbl, vp, vp, vp]
        lib.mxcheck_gemm.restype = ci
        _lib = lib
    return _lib


def _dev_u8(a) -> torch.Tensor:
    if isinstance(a, torch.Tensor):
        return a.contiguous()
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.uint8)).cuda()


def check(a_codes, a_scales, b_codes, b_scales, alpha: float, out: torch.Tensor | None, rel_tol: float = 1e-5,
          want_ref: bool = False):
    """Run the checker.  Operands: uint8 arrays (numpy or CUDA tensors), scales canonical [rows x K/32].

    Returns ``(n_bad, first_bad_index, worst_ratio, ref, S)``; ref / S are CUDA float64 tensors when
    ``want_ref`` (else None).  ``out`` (bf16 or fp32 CUDA tensor [M x N], any row stride) may be None."""
    ac, asc, bc, bsc = _dev_u8(a_codes), _dev_u8(a_scales), _dev_u8(b_codes), _dev_u8(b_scales)
    M, kh = ac.shape
    N = bc.shape[0]
    K = 2 * kh
    assert bc.shape[1] == kh and tuple(asc.shape) == (M, K // 32) and tuple(bsc.shape) == (N, K // 32)
    ref = s = None
    if want_ref:
        ref = torch.empty((M, N), dtype=torch.float64, device="cuda")
        s = torch.empty((M, N), dtype=torch.float64, device="cuda")
    is_bf16, ld, optr = 0, N, None
    if out is not None:
        assert out.is_cuda and tuple(out.shape) == (M, N) and out.stride(1) == 1
        assert out.dtype in (torch.bfloat16, torch.float32)
        is_bf16, ld, optr = int(out.dtype == torch.bfloat16), out.stride(0), out.data_ptr()
    verdict = (ctypes.c_ulonglong * 3)()
    torch.cuda.synchronize()
    rc = _load().mxcheck_gemm(ac.data_ptr(), asc.data_ptr(), bc.data_ptr(), bsc.data_ptr(), M, N, K, float(alpha), optr,
                              is_bf16, ld, rel_tol, 2.0 ** -8 if is_bf16 else 0.0,
                              ref.data_ptr() if want_ref else None, s.data_ptr() if want_ref else None, verdict)
    if rc != 0:
        raise RuntimeError(f"mxcheck_gemm failed: {rc}")
    worst = struct.unpack("d", struct.pack("Q", verdict[2]))[0]
    return int(verdict[0]), int(verdict[1]), worst, ref, s

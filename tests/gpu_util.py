"""Shared helpers of the GPU parity tests (marshalling only)."""
import numpy as np
import torch

import oracle
from paper_2605_09825_b200 import api


def to_dev(bits: np.ndarray) -> torch.Tensor:
    """uint16 bf16 bit patterns -> bf16 CUDA tensor holding the same bits."""
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def random_bits(rng, rows, cols, spread=6):
    x = rng.standard_normal((rows, cols)).astype(np.float32)
    x *= np.exp2(rng.integers(-spread, spread, size=(rows, 1))).astype(np.float32)
    u = x.view(np.uint32)
    return ((u + 0x7FFF + ((u >> 16) & 1)) >> 16).astype(np.uint16)


def gpu_quantize(bits, axis, hmode, rounding, seed=0, tag=0, layout=api.SCALES_TILED):
    """Run the CUDA quantizer; return (codes, canonical scales, raw scale buffer) as numpy."""
    src = to_dev(bits)
    codes, scales = api.quantize(src, axis, hmode, rounding, seed, tag, layout)
    api.check()
    rows, cols = bits.shape
    outer, K = (rows, cols) if axis == 1 else (cols, rows)
    raw = scales.cpu().numpy()
    canon = oracle.scales_from_tiled(raw, outer, K // 32) if layout == api.SCALES_TILED \
        else raw.reshape(outer, K // 32)
    return codes.cpu().numpy(), canon, raw


def assert_gemm_close(out, ref, S, bf16: bool, what=""):
    """|out - ref| <= 1e-5 * S (+ half a bf16 ulp of ref for bf16 outputs), element by element."""
    out = np.asarray(out, dtype=np.float64)
    tol = 1e-5 * S + (2.0 ** -8 * np.abs(ref) if bf16 else 0.0)
    # denormal-range outputs can differ by one fp32 ulp of the smallest normal
    tol = tol + 1e-38
    # written so that a NaN or an infinity in `out` fails (a NaN compares false either way round)
    bad = ~(np.abs(out - ref) <= tol)
    if bad.any():
        idx = np.argwhere(bad)[:8]
        msg = [f"{what}: {bad.sum()} of {bad.size} elements out of tolerance"]
        for i, j in idx:
            msg.append(f"  [{i},{j}] got {out[i, j]!r} want {ref[i, j]!r} S {S[i, j]!r}")
        raise AssertionError("\n".join(msg))

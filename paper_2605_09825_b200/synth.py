"""Seeded synthetic inputs shaped like Llama-3.1-8B linear layers.

This module holds input generation only -- none of the method's arithmetic -- so that the
CPU oracle's tests and the CUDA path's tests can feed both sides the very same bits.
Tensors are returned as ``uint16`` numpy arrays holding bf16 bit patterns (fp32 values
rounded to bf16 with round-to-nearest-even).

The paper trains Llama-3.1-8B on C4; neither the dataset nor trained weights are needed
for kernel work, so seeded tensors with the layer shapes and heavy-tailed / outlier-bearing
distributions stand in for activations, weights and gradients:

  config 1  tiny Fprop      X,W [256x512]            N(0,1), 0.1 % of positions x50, seed 0
  config 2  QKV Fprop       X [8192x4096] N(0,1) with 8 outlier channels x20; W [6144x4096] N(0,0.02^2)
  config 3  gate+up         X, W [28672x4096] as config 2; dY [8192x28672] Student-t(3)*1e-3
  config 4  down Wgrad      dY [8192x4096] Student-t(3)*1e-3; X [8192x14336] |N(0,1)|*N(0,1)
  config 5  layer stack     T=16384 tokens; QKV, O, gate+up, down linears; same recipes

Large tensors are generated in row chunks, each chunk from its own child seed, so results do
not depend on the number of worker threads.
"""
from __future__ import annotations

from concurrent.futures import ThreadPoolExecutor
import os

import numpy as np

_CHUNK_ROWS = 256


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (nearest, ties to even) and return the 16-bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounded = u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def _chunked(rows: int, cols: int, seed_words, fill) -> np.ndarray:
    """Fill a [rows x cols] bf16-bits array chunk by chunk; ``fill(rng, r0, n) -> float32 [n x cols]``."""
    out = np.empty((rows, cols), dtype=np.uint16)
    starts = list(range(0, rows, _CHUNK_ROWS))

    def work(ci):
        r0 = starts[ci]
        n = min(_CHUNK_ROWS, rows - r0)
        rng = np.random.Generator(np.random.PCG64(np.random.SeedSequence(list(seed_words) + [ci])))
        out[r0:r0 + n] = f32_to_bf16_bits(fill(rng, r0, n))

    workers = min(len(starts), max(1, os.cpu_count() or 1))
    if workers <= 1:
        for ci in range(len(starts)):
            work(ci)
    else:
        with ThreadPoolExecutor(max_workers=workers) as ex:
            list(ex.map(work, range(len(starts))))
    return out


def normal(rows: int, cols: int, seed: int, tensor_id: int, std: float = 1.0) -> np.ndarray:
    return _chunked(rows, cols, [seed, tensor_id],
                    lambda rng, r0, n: rng.standard_normal((n, cols), dtype=np.float32) * np.float32(std))


def normal_outlier_positions(rows: int, cols: int, seed: int, tensor_id: int, frac: float = 1e-3,
                             factor: float = 50.0) -> np.ndarray:
    """N(0,1) with a seeded ``frac`` of positions multiplied by ``factor``."""
    def fill(rng, r0, n):
        x = rng.standard_normal((n, cols), dtype=np.float32)
        hit = rng.random((n, cols), dtype=np.float32) < np.float32(frac)
        x[hit] *= np.float32(factor)
        return x
    return _chunked(rows, cols, [seed, tensor_id], fill)


def normal_outlier_channels(rows: int, cols: int, seed: int, tensor_id: int, n_channels: int = 8,
                            factor: float = 20.0) -> np.ndarray:
    """N(0,1) activations with ``n_channels`` seeded columns multiplied by ``factor``."""
    rng0 = np.random.Generator(np.random.PCG64(np.random.SeedSequence([seed, tensor_id, 0xC0FFEE])))
    chans = rng0.choice(cols, size=n_channels, replace=False)

    def fill(rng, r0, n):
        x = rng.standard_normal((n, cols), dtype=np.float32)
        x[:, chans] *= np.float32(factor)
        return x
    return _chunked(rows, cols, [seed, tensor_id], fill)


def student_t(rows: int, cols: int, seed: int, tensor_id: int, nu: float = 3.0,
              scale: float = 1e-3) -> np.ndarray:
    """Heavy-tailed gradients: Student-t(nu) * scale."""
    return _chunked(rows, cols, [seed, tensor_id],
                    lambda rng, r0, n: (rng.standard_t(nu, (n, cols)) * scale).astype(np.float32))


def swiglu_like(rows: int, cols: int, seed: int, tensor_id: int) -> np.ndarray:
    """Post-SwiGLU-like activations: |N(0,1)| * N(0,1)."""
    def fill(rng, r0, n):
        a = np.abs(rng.standard_normal((n, cols), dtype=np.float32))
        return a * rng.standard_normal((n, cols), dtype=np.float32)
    return _chunked(rows, cols, [seed, tensor_id], fill)


# (out, in) of the four linears of one Llama-3.1-8B layer
LLAMA8B_LINEARS = {
    "qkv": (6144, 4096),       # 32 q heads + 2 x 8 kv heads, 128 wide
    "o": (4096, 4096),
    "gate_up": (28672, 4096),  # gate and up concatenated
    "down": (4096, 14336),
}


def linear_tensors(name: str, tokens: int, seed: int, which=("X", "W", "dY")) -> dict:
    """X [T x in], W [out x in], dY [T x out] of one named linear at ``tokens`` tokens."""
    out_f, in_f = LLAMA8B_LINEARS[name]
    tid = {"qkv": 10, "o": 20, "gate_up": 30, "down": 40}[name]
    t = {}
    if "X" in which:
        if name == "down":
            t["X"] = swiglu_like(tokens, in_f, seed, tid + 1)
        else:
            t["X"] = normal_outlier_channels(tokens, in_f, seed, tid + 1)
    if "W" in which:
        t["W"] = normal(out_f, in_f, seed, tid + 2, std=0.02)
    if "dY" in which:
        t["dY"] = student_t(tokens, out_f, seed, tid + 3)
    return t


def config1() -> dict:
    """Tiny Fprop: M=256, N=256, K=512, seed 0."""
    return {"X": normal_outlier_positions(256, 512, 0, 1), "W": normal_outlier_positions(256, 512, 0, 2)}


def config2(tokens: int = 8192) -> dict:
    """QKV projection Fprop (data seed 2)."""
    return linear_tensors("qkv", tokens, 2, ("X", "W"))


def config3(tokens: int = 8192) -> dict:
    """MLP gate+up Fprop and Dgrad (data seed 3)."""
    return linear_tensors("gate_up", tokens, 3, ("X", "W", "dY"))


def config4(tokens: int = 8192) -> dict:
    """down_proj Wgrad (data seed 4; the rounding / sign-mask seed of its variants is 7)."""
    return linear_tensors("down", tokens, 4, ("X", "dY"))


def config5(tokens: int = 16384) -> dict:
    """Full layer linear stack at ``tokens`` tokens (data seed 5): {name: {X, W, dY}}."""
    return {name: linear_tensors(name, tokens, 5) for name in LLAMA8B_LINEARS}

"""Quantization-error probe for the MXFP4 linear passes (needs a B200).

The paper's first key observation is qualitative: with the weight-gradient GEMM quantized,
stochastic rounding and randomized rotations carry more quantization error than the
deterministic rotation.  This probe puts numbers on that for the library's own kernels, on the
synthetic operands that stand in for the paper's gradients and activations: it runs one pass
(Wgrad by default) through the fused MXFP4 path for every stabiliser variant and reports the
signal-to-noise ratio of the result against an fp64 product of the same bf16 inputs.

    python -m paper_2605_09825_b200.error_probe [--pass wgrad|fprop|dgrad] [--tokens 4096]

The fp64 reference is ``torch.matmul`` in float64 (a library routine used as the yardstick of
this measurement only; it is not part of the product path).  Prints one JSON line.
"""
from __future__ import annotations

import argparse
import json

import numpy as np
import torch

from . import api, synth

VARIANTS = [
    ("none", api.HADAMARD_NONE, api.ROUND_RNE),
    ("det_h32", api.HADAMARD_DET, api.ROUND_RNE),
    ("det_h16", api.HADAMARD_DET16, api.ROUND_RNE),
    ("rand_h32", api.HADAMARD_RAND, api.ROUND_RNE),
    ("rand_h16", api.HADAMARD_RAND16, api.ROUND_RNE),
    ("sr", api.HADAMARD_NONE, api.ROUND_SR),
    ("sr_det_h32", api.HADAMARD_DET, api.ROUND_SR),
]


def _dev(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


def snr_db(got: torch.Tensor, ref: torch.Tensor) -> float:
    err = (got.double() - ref).pow(2).sum().item()
    sig = ref.pow(2).sum().item()
    return float("inf") if err == 0 else 10.0 * float(np.log10(sig / err))


def run(pass_name: str = "wgrad", tokens: int = 4096, linear: str = "down", seed: int = 7) -> dict:
    t = synth.linear_tensors(linear, tokens, 4)
    X, W, dY = _dev(t["X"]), _dev(t["W"]), _dev(t["dY"])
    if pass_name == "fprop":
        fn, a, b, ref = api.linear_fprop, X, W, X.double() @ W.double().t()
    elif pass_name == "dgrad":
        fn, a, b, ref = api.linear_dgrad, dY, W, dY.double() @ W.double()
    else:
        fn, a, b, ref = api.linear_wgrad, dY, X, dY.double().t() @ X.double()
    out = {}
    for name, hmode, rnd in VARIANTS:
        got = fn(a, b, hmode, rnd, seed, api.OUT_FP32)
        api.check()
        out[name] = round(snr_db(got, ref), 3)
    # the 32 x 32 block strategy (Appendix D) and the 8-bit format of the ladder's other passes,
    # from explicit quantize + GEMM calls (operand orientation per pass as in the wrappers)
    pass_id = {"fprop": api.PASS_FPROP, "dgrad": api.PASS_DGRAD, "wgrad": api.PASS_WGRAD}[pass_name]
    ax_a, ax_b = ((1, 1), (1, 0), (0, 0))[pass_id]
    for name, hmode, alpha in (("none_32x32", api.HADAMARD_NONE, 1.0), ("det_h32_32x32", api.HADAMARD_DET, 1.0 / 32)):
        qa = api.quantize(a, ax_a, hmode, api.ROUND_RNE, seed, 0, block_shape=api.BLOCK_32X32)
        qb = api.quantize(b, ax_b, hmode, api.ROUND_RNE, seed, 1, block_shape=api.BLOCK_32X32)
        out[name] = round(snr_db(api.gemm(*qa, *qb, alpha, api.OUT_FP32), ref), 3)
    out["mxfp8"] = round(snr_db(api.linear_pass(pass_id, api.PRECISION_MXFP8, a, b, out_dtype=api.OUT_FP32), ref), 3)
    api.check()
    return {"pass": pass_name, "linear": linear, "tokens": tokens, "seed": seed, "snr_db": out,
            "inputs": "synthetic: dY Student-t(3)*1e-3, X |N|*N (down) or N(0,1)+outlier channels, W N(0,0.02^2)"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--pass", dest="pass_name", default="wgrad", choices=["fprop", "dgrad", "wgrad"])
    ap.add_argument("--tokens", type=int, default=4096)
    ap.add_argument("--linear", default="down", choices=sorted(synth.LLAMA8B_LINEARS))
    args = ap.parse_args()
    print(json.dumps(run(args.pass_name, args.tokens, args.linear)))


if __name__ == "__main__":
    main()

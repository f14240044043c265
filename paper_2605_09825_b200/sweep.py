"""Per-kernel throughput sweeps on the benchmark configurations (needs a B200).

    python -m paper_2605_09825_b200.sweep quantize [--config 4] [--reps 50]
    python -m paper_2605_09825_b200.sweep gemm     [--reps 50]
    python -m paper_2605_09825_b200.sweep fused    [--reps 50]

``quantize``: every variant of the quantizer -- row-wise and column-wise, each rotation mode, RNE
and stochastic rounding, the dual-axis kernel, 32 x 32 blocks, the 8-bit format -- on the largest
tensor of a configuration, as GB/s of algorithmic traffic (2.53125 B/element single-axis, 3.0625
dual-axis, 3.03125 eight-bit) and as a fraction of the measured copy bandwidth.
``gemm``: the block-scaled GEMM alone on the shapes of configurations 2-5, as TFLOP/s and as a
fraction of the nominal dense FP4 rate; ``fused``: the same shapes through the per-pass entry
points, quantization included.

Timing: CUDA events around single launches, 20 warm-up launches, then ``--reps`` timed ones with
a 256 MB buffer rewritten before each (so operands come from HBM, not L2); median and best are
reported.  Inputs are the seeded synthetic tensors of ``synth`` (never zeros).  One JSON line per
case.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics

import numpy as np
import torch

from . import api, synth

HMODES = {"none": api.HADAMARD_NONE, "h32": api.HADAMARD_DET, "rh32": api.HADAMARD_RAND,
          "h16": api.HADAMARD_DET16, "rh16": api.HADAMARD_RAND16}
NOMINAL_FP4_TFLOPS = 9000.0


def _peaks():
    path = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


def _dev(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


class Timer:
    def __init__(self, reps: int):
        self.reps = reps
        self.flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")

    def __call__(self, fn):
        for _ in range(20):
            fn()
        times = []
        for r in range(self.reps):
            self.flush.fill_(r & 0xFF)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            fn()
            e1.record()
            torch.cuda.synchronize()
            times.append(e0.elapsed_time(e1) * 1e3)
        return statistics.median(times), min(times)


def sweep_quantize(config: int, reps: int):
    hbm, src = _peaks()
    tensors = {2: ("X", synth.config2), 3: ("dY", synth.config3), 4: ("X", synth.config4)}
    name, gen = tensors[config]
    x = _dev(gen()[name])
    rows, cols = x.shape
    n = rows * cols
    timer = Timer(reps)
    buf = {1: (torch.empty((rows, cols // 2), dtype=torch.uint8, device="cuda"),
               torch.empty(api.scales_bytes(rows, cols), dtype=torch.uint8, device="cuda")),
           0: (torch.empty((cols, rows // 2), dtype=torch.uint8, device="cuda"),
               torch.empty(api.scales_bytes(cols, rows), dtype=torch.uint8, device="cuda"))}

    def emit(case, med, best, bytes_per_el):
        print(json.dumps({"sweep": "quantize", "config": config, "tensor": f"{name} {rows}x{cols}", "case": case,
                          "us_median": round(med, 2), "us_best": round(best, 2), "bytes_per_element": bytes_per_el,
                          "gbs_median": round(n * bytes_per_el / med / 1e3, 1),
                          "frac_of_copy_bandwidth": round(n * bytes_per_el / med / 1e3 / hbm, 3),
                          "frac_of_nominal_8tbs": round(n * bytes_per_el / med / 1e3 / 8000.0, 3),
                          "copy_bandwidth_gbs": hbm, "copy_bandwidth_source": src}), flush=True)

    for hname, hmode in HMODES.items():
        for rname, rnd in (("rne", api.ROUND_RNE), ("sr", api.ROUND_SR)):
            for axis in (1, 0):
                c, s = buf[axis]
                med, best = timer(lambda: api.quantize(x, axis, hmode, rnd, 7, 0, codes=c, scales=s))
                emit(f"{'row' if axis else 'col'}-wise {hname} {rname}", med, best, 2.53125)
        med, best = timer(lambda: api.quantize_dual(x, hmode, api.ROUND_RNE, 7, out_row=buf[1], out_col=buf[0]))
        emit(f"dual-axis {hname} rne", med, best, 3.0625)
    med, best = timer(lambda: api.quantize_dual(x, api.HADAMARD_DET, api.ROUND_RNE, 7, block_shape=api.BLOCK_32X32,
                                                out_row=buf[1], out_col=buf[0]))
    emit("dual-axis h32 rne 32x32 blocks", med, best, 3.0625)
    c8 = torch.empty((rows, cols), dtype=torch.uint8, device="cuda")
    med, best = timer(lambda: api.quantize_fp8(x, 1, codes=c8, scales=buf[1][1]))
    emit("row-wise mxfp8", med, best, 3.03125)
    api.check()


GEMM_CASES = [("config 2 QKV Fprop", "qkv", 0, 8192), ("config 3 gate+up Fprop", "gate_up", 0, 8192),
              ("config 3 gate+up Dgrad", "gate_up", 1, 8192), ("config 4 down Wgrad", "down", 2, 8192)] + \
             [(f"config 5 {n} {p}", n, i, 16384) for n in ("qkv", "o", "gate_up", "down")
              for i, p in enumerate(("Fprop", "Dgrad", "Wgrad"))]


def _operands(linear: str, pass_: int, tokens: int):
    t = synth.linear_tensors(linear, tokens, 5)
    a = _dev(t["X"] if pass_ == 0 else t["dY"])
    b = _dev(t["X"] if pass_ == 2 else t["W"])
    out_f, in_f = synth.LLAMA8B_LINEARS[linear]
    mnk = ((tokens, out_f, in_f), (tokens, in_f, out_f), (out_f, in_f, tokens))[pass_]
    return a, b, mnk


def sweep_gemm(reps: int, fused: bool):
    timer = Timer(reps)
    for label, linear, pass_, tokens in GEMM_CASES:
        a, b, (M, N, K) = _operands(linear, pass_, tokens)
        out = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
        if fused:
            ws = torch.empty(api.linear_workspace_bytes(tokens, *reversed(synth.LLAMA8B_LINEARS[linear]), pass_),
                             dtype=torch.uint8, device="cuda")
            fn = (api.linear_fprop, api.linear_dgrad, api.linear_wgrad)[pass_]
            med, best = timer(lambda: fn(a, b, api.HADAMARD_DET, api.ROUND_RNE, 0, api.OUT_BF16, workspace=ws, out=out))
        else:
            ax_a, ax_b = ((1, 1), (1, 0), (0, 0))[pass_]
            (ac, a_s), (bc, b_s) = api.quantize_pair(a, ax_a, b, ax_b, api.HADAMARD_DET, api.ROUND_RNE, 0)
            med, best = timer(lambda: api.gemm(ac, a_s, bc, b_s, 1.0 / 32, api.OUT_BF16, out=out))
        fl = 2.0 * M * N * K
        print(json.dumps({"sweep": "fused" if fused else "gemm", "case": label, "M": M, "N": N, "K": K,
                          "us_median": round(med, 2), "us_best": round(best, 2),
                          "tflops_median": round(fl / med / 1e6, 1),
                          "frac_of_nominal_fp4_peak": round(fl / med / 1e6 / NOMINAL_FP4_TFLOPS, 3)}), flush=True)
        del a, b, out
    api.check()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("what", choices=["quantize", "gemm", "fused"])
    ap.add_argument("--config", type=int, default=4, choices=[2, 3, 4])
    ap.add_argument("--reps", type=int, default=50)
    args = ap.parse_args()
    if not torch.cuda.is_available():
        raise SystemExit("the sweeps need a CUDA device")
    if args.what == "quantize":
        sweep_quantize(args.config, args.reps)
    else:
        sweep_gemm(args.reps, args.what == "fused")


if __name__ == "__main__":
    main()

#!/usr/bin/env python
"""Benchmark of the MXFP4 linear-layer hot path on B200.

One "step" is one pass of the whole hot path -- Hadamard + quantize of both operands and the
block-scaled GEMM, for Fprop, Dgrad and Wgrad of every linear of the workload -- over one batch
of seeded synthetic tensors shaped like Llama-3.1-8B layers.  The default workload is the full
layer linear stack at 16384 tokens (4 linears x 3 passes = 12 GEMMs), the one configuration that
exercises every step of the path; ``--workload qkv|gate_up|down`` selects the single-linear
configurations.  ``--schedule layer`` (default) runs each linear as forward + backward with every
tensor read once by the dual-axis quantize (3 quantize + 3 GEMM launches per linear);
``--schedule per_pass`` runs the three per-pass entry points (one two-tensor quantize launch + one
GEMM launch each).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload W] [--schedule S]
                    [--impl ours|reference]

Prints ONE JSON line.  ``value`` is whole-job TFLOP/s (2*M*N*K per GEMM, quantize time
included) with inputs resident in HBM; ``e2e`` is the same metric through the host-buffer
entry point with the host<->device copies inside the timed region; ``roofline`` describes the
dominant kernel (the GEMM) from per-launch CUDA-event timings taken in this run;
``cpu_baseline`` times the CPU oracle on a bounded sample of the same workload.
With ``--impl reference`` the CPU oracle itself is the timed arm.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time
import zlib

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

METRIC = "MXFP4 linear-layer TFLOP/s incl. Hadamard+quantize (Fprop+Dgrad+Wgrad)"
UNIT = "TFLOP/s"

WORKLOADS = {
    # name: (tokens, [linear names])
    "layer_stack": (16384, ["qkv", "o", "gate_up", "down"]),
    "qkv": (8192, ["qkv"]),
    "gate_up": (8192, ["gate_up"]),
    "down": (8192, ["down"]),
}


HADAMARD = {"none": (0, "no rotation"), "h32": (1, "deterministic H32"), "rh32": (2, "randomized H32"),
            "h16": (3, "deterministic H16"), "rh16": (4, "randomized H16")}


def workload_label(name: str, tokens: int, hadamard: str = "h32") -> str:
    rot = HADAMARD[hadamard][1]
    if name == "layer_stack":
        return ("Llama-3.1-8B layer linear stack (QKV, O, gate+up, down) x (Fprop, Dgrad, Wgrad), "
                f"{tokens} tokens, {rot}, RNE")
    return f"Llama-3.1-8B {name} linear x (Fprop, Dgrad, Wgrad), {tokens} tokens, {rot}, RNE"


def pass_dims(pass_: int, T: int, in_f: int, out_f: int):
    if pass_ == 0:
        return T, out_f, in_f
    if pass_ == 1:
        return T, in_f, out_f
    return out_f, in_f, T


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0,
            "source": "fallback"}


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-i", str(self.index), "-lms", "20"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for ln in self.proc.stdout:
            self.lines.append((time.time(), ln.strip()))

    def stop(self, t_begin=None, t_end=None):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]

        def parse(lines):
            mhz, mx, watts, reasons = [], None, [], set()
            for _, ln in lines:
                f = [x.strip() for x in ln.split(",")]
                if len(f) < 8:
                    continue
                try:
                    mhz.append(float(f[1]))
                    mx = float(f[2])
                    watts.append(float(f[3]))
                except ValueError:
                    continue
                for n, v in zip(names, f[4:8]):
                    if v.lower().startswith("active"):
                        reasons.add(n)
            return mhz, mx, watts, reasons

        inside = [x for x in self.lines
                  if t_begin is None or (t_begin <= x[0] <= (t_end or x[0]) + 0.05)]
        window = "timed region"
        if not inside:            # region shorter than one sampling period: use the whole run
            inside, window = self.lines, "whole run (timed region shorter than a sample)"
        mhz, mx, watts, reasons = parse(inside)
        return {"sm_mhz": statistics.median(mhz) if mhz else None, "sm_max_mhz": mx,
                "power_w_max": max(watts) if watts else None, "reasons": sorted(reasons),
                "samples": len(mhz), "window": window}


def aggregate_over_ranks(elapsed_ms: float, world: int) -> float:
    """Max of the per-rank device times (all ranks run the same work: weak scaling replicas)."""
    import torch
    import torch.distributed as dist
    if world <= 1 or not dist.is_initialized():
        return elapsed_ms
    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([elapsed_ms], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sweep_quantize_variants(dev_in, peaks, api, reps: int = 10):
    """GB/s of every quantizer variant -- {no rotation, deterministic H32, randomized H32} x {RNE,
    stochastic rounding} x {row-wise, column-wise, dual-axis}, plus the 16-point rotation with RNE
    for its ratio to the 32-point one -- on the activations of config 2
    (X 8192 x 4096), the gradient of config 3 (dY 8192 x 28672) and the activations of config 4
    (X 8192 x 14336): the first 8192 tokens of this step's tensors, which follow those recipes.
    Single launches, CUDA events, a 256 MB buffer rewritten before each so that nothing comes from
    L2; median of `reps` after 3 warm-ups.  Algorithmic bytes: 2.53125 per element single-axis,
    3.0625 dual-axis."""
    import torch
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    tensors = {"config 2 X 8192x4096": dev_in["qkv"]["X"][:8192],
               "config 3 dY 8192x28672": dev_in["gate_up"]["dY"][:8192],
               "config 4 X 8192x14336": dev_in["down"]["X"][:8192]}
    hbm = peaks["hbm_gbs"]
    out = {"unit": "GB/s of algorithmic bytes", "peak": hbm, "peak_source": peaks["source"] + " copy bandwidth",
           "timing": f"single launches, L2 rewritten before each, median of {reps}", "cases": {}}

    def timed(fn):
        ts = []
        for r in range(3 + reps):
            flush.fill_(r & 0xFF)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            fn()
            e1.record()
            torch.cuda.synchronize()
            if r >= 3:
                ts.append(e0.elapsed_time(e1))
        return statistics.median(ts)

    for tname, x in tensors.items():
        rows, cols = x.shape
        n = rows * cols
        buf = {1: (torch.empty((rows, cols // 2), dtype=torch.uint8, device="cuda"),
                   torch.empty(api.scales_bytes(rows, cols), dtype=torch.uint8, device="cuda")),
               0: (torch.empty((cols, rows // 2), dtype=torch.uint8, device="cuda"),
                   torch.empty(api.scales_bytes(cols, rows), dtype=torch.uint8, device="cuda"))}
        table = {}
        for hname, hmode in (("none", api.HADAMARD_NONE), ("h32", api.HADAMARD_DET), ("rh32", api.HADAMARD_RAND),
                             ("h16", api.HADAMARD_DET16)):
            for rname, rnd in (("rne", api.ROUND_RNE), ("sr", api.ROUND_SR)):
                if hname == "h16" and rname == "sr":
                    continue          # the 16-point variant is listed for its H16 : H32 ratio only
                for axis, aname in ((1, "row"), (0, "col")):
                    c, sc = buf[axis]
                    ms = timed(lambda: api.quantize(x, axis, hmode, rnd, 7, 0, codes=c, scales=sc))
                    gbs = n * 2.53125 / (ms * 1e-3) / 1e9
                    table[f"{aname} {hname} {rname}"] = {"us": round(ms * 1e3, 1), "gbs": round(gbs, 1),
                                                         "frac": round(gbs / hbm, 3)}
                ms = timed(lambda: api.quantize_dual(x, hmode, rnd, 7, out_row=buf[1], out_col=buf[0]))
                gbs = n * 3.0625 / (ms * 1e-3) / 1e9
                table[f"dual {hname} {rname}"] = {"us": round(ms * 1e3, 1), "gbs": round(gbs, 1),
                                                  "frac": round(gbs / hbm, 3)}
        # the paper's one kernel-level number is the H16 : H32 throughput ratio (1.08 on its hardware)
        table["h16_to_h32_ratio"] = {ax: round(table[f"{ax} h16 rne"]["gbs"] / table[f"{ax} h32 rne"]["gbs"], 3)
                                     for ax in ("row", "col", "dual")}
        out["cases"][tname] = table
        del buf
    del flush
    api.check()
    return out


# --------------------------------------------------------------------------- oracle arm
def oracle_sample(steps: int, warmup: int):
    """Time the CPU oracle on a bounded sample: the QKV Fprop restricted to 2048 tokens."""
    import oracle
    from paper_2605_09825_b200 import synth
    tokens = 2048
    t = synth.linear_tensors("qkv", tokens, 2, ("X", "W"))
    flops = 2.0 * tokens * 6144 * 4096
    times = []
    for i in range(warmup + steps):
        t0 = time.perf_counter()
        oracle.linear_fprop(t["X"], t["W"], 1, 0, 0)
        dt = time.perf_counter() - t0
        if i >= warmup:
            times.append(dt)
    mean = sum(times) / len(times)
    return {"value": flops / mean / 1e12, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
            "sample": f"QKV Fprop (quantize X [{tokens}x4096] and W [6144x4096] with H32, fp64 GEMM) "
                      f"restricted to {tokens} tokens; {len(times)} runs, mean {mean:.2f} s"}, mean


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    steps = max(1, min(args.steps, 3))
    warm = min(args.warmup, 1)
    base, mean = oracle_sample(steps, warm)
    tokens, _ = WORKLOADS[args.workload]
    line = {
        "impl": "reference", "metric": METRIC, "value": base["value"], "unit": UNIT,
        "n_gpus": args.gpus, "steps": steps, "warmup": warm, "ms_per_step": mean * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "e2m1 x e2m1 -> f64",
        "data": "synthetic", "config": {"workload": workload_label(args.workload, tokens, args.hadamard),
                                        "note": "CPU oracle on a bounded sample of this workload"},
        "cpu_baseline": base,
        "e2e": {"value": base["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# --------------------------------------------------------------------------- CUDA arm
def run_ours(args):
    import torch
    from paper_2605_09825_b200 import api, synth

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback for the product path")
    torch.cuda.set_device(local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    api.load_library()
    peaks = load_peaks()
    tokens, names = WORKLOADS[args.workload]
    hmode, rnd, seed = HADAMARD[args.hadamard][0], api.ROUND_RNE, 0
    alpha = {0: 1.0, 1: 1.0 / 32, 2: 1.0 / 32, 3: 1.0 / 16, 4: 1.0 / 16}[hmode]

    # ---- inputs: seeded synthetic, generated on the host, then resident in HBM
    host, dev_in = {}, {}
    checksums = {}
    for n in names:
        t = synth.linear_tensors(n, tokens, 5)
        if rank == 0 and not args.no_checksums:
            checksums[n] = {k: f"{zlib.crc32(memoryview(np.ascontiguousarray(v)).cast('B')):08x}" for k, v in t.items()}
        host[n] = {k: torch.from_numpy(v.view(np.int16)).view(torch.bfloat16) for k, v in t.items()}
        dev_in[n] = {k: v.cuda() for k, v in host[n].items()}
    dims = {n: synth.LLAMA8B_LINEARS[n] for n in names}   # (out, in)
    max_out = max(max(tokens * o, tokens * i, o * i) for o, i in dims.values())
    out_buf = torch.empty(max_out, dtype=torch.bfloat16, device="cuda")
    lib = api.load_library()
    # precision ladder (Table 1): the passes named in --mxfp4-passes run MXFP4, the others MXFP8
    fp4_passes = {"fprop": 0, "dgrad": 1, "wgrad": 2}
    chosen = [x for x in args.mxfp4_passes.split(",") if x and x != "none"]
    if any(x not in fp4_passes for x in chosen):
        raise SystemExit("--mxfp4-passes takes a comma-separated subset of fprop,dgrad,wgrad (or 'none')")
    precision = [api.PRECISION_MXFP4 if name in chosen else api.PRECISION_MXFP8 for name in ("fprop", "dgrad", "wgrad")]
    ladder = any(pr == api.PRECISION_MXFP8 for pr in precision)
    if ladder:
        args.schedule = "per_pass"          # the layer-level calls are MXFP4 throughout
        args.no_e2e = args.no_configs = True  # the host-buffer call and the single-pass configs are MXFP4 only
    ws_bytes = max(int(lib.mxfp4_linear_pass_workspace_bytes(tokens, i, o, p, precision[p]))
                   for o, i in dims.values() for p in range(3))
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")
    stream = torch.cuda.current_stream()
    sptr = int(stream.cuda_stream)

    passes = []   # (linear, pass, a, b, M, N, K)
    for n in names:
        o, i = dims[n]
        d = dev_in[n]
        passes.append((n, 0, d["X"], d["W"]) + pass_dims(0, tokens, i, o))
        passes.append((n, 1, d["dY"], d["W"]) + pass_dims(1, tokens, i, o))
        passes.append((n, 2, d["dY"], d["X"]) + pass_dims(2, tokens, i, o))
    flops_per_step = sum(2.0 * M * N * K for (_, _, _, _, M, N, K) in passes)
    fused = [lib.mxfp4_linear_fprop, lib.mxfp4_linear_dgrad, lib.mxfp4_linear_wgrad]
    layer = args.schedule == "layer"
    if layer:
        saved_bytes = max(api.linear_layer_bytes(tokens, i, o, api.LAYER_SAVED) for o, i in dims.values())
        lws_bytes = max(api.linear_layer_bytes(tokens, i, o, w) for o, i in dims.values()
                        for w in (api.LAYER_FORWARD, api.LAYER_BACKWARD))
        saved = torch.empty(saved_bytes, dtype=torch.uint8, device="cuda")
        lws = torch.empty(lws_bytes, dtype=torch.uint8, device="cuda")
        out_buf2 = torch.empty(max_out, dtype=torch.bfloat16, device="cuda")

    def step_per_pass():
        for (n, p, a, b, M, N, K) in passes:
            o, i = dims[n]
            rc = lib.mxfp4_linear_pass(p, precision[p], a.data_ptr(), b.data_ptr(), out_buf.data_ptr(), tokens, i, o,
                                       hmode, rnd, seed, api.OUT_BF16, ws.data_ptr(), ws_bytes, sptr)
            if rc != 0:
                raise api.Mxfp4Error(rc, "fused linear pass")

    def step_layer():
        # forward then backward of each linear: X, W and dY are each read once
        for n in names:
            o, i = dims[n]
            d = dev_in[n]
            rc = lib.mxfp4_linear_forward(d["X"].data_ptr(), d["W"].data_ptr(), out_buf.data_ptr(), tokens, i, o,
                                          hmode, rnd, seed, api.OUT_BF16, saved.data_ptr(), saved_bytes,
                                          lws.data_ptr(), lws_bytes, sptr)
            if rc != 0:
                raise api.Mxfp4Error(rc, "mxfp4_linear_forward")
            rc = lib.mxfp4_linear_backward(d["dY"].data_ptr(), out_buf.data_ptr(), out_buf2.data_ptr(), tokens, i, o,
                                           hmode, rnd, seed, api.OUT_BF16, api.OUT_BF16, saved.data_ptr(),
                                           saved_bytes, lws.data_ptr(), lws_bytes, sptr)
            if rc != 0:
                raise api.Mxfp4Error(rc, "mxfp4_linear_backward")

    step = step_layer if layer else step_per_pass

    def sync_all():
        torch.cuda.synchronize()
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
            torch.cuda.synchronize()

    sampler = ClockSampler(local_rank)
    sampler.start()
    for _ in range(max(args.warmup, 3)):
        step()
    api.check()

    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sync_all()
    t_begin = time.time()
    e0.record(stream)
    for _ in range(args.steps):
        step()
    e1.record(stream)
    sync_all()
    t_end = time.time()
    elapsed_ms = aggregate_over_ranks(e0.elapsed_time(e1), world)
    api.check()

    # ---- the same step, decomposed, with CUDA events around every launch (roofline inputs)
    q_bytes_per_element = 3.0625 if layer else 2.53125

    def a_b_axes(p):
        return ((1, 1), (1, 0), (0, 0))[p]

    gemm_ms = gemm_flops = quant_ms = quant_bytes = 0.0
    n_quant = 0
    gemm_times = {}         # per launch of the step, label -> (flops, [ms per repetition])
    quant_times = {}        # per quantize launch of the step, index -> (bytes, [ms per repetition])
    r256 = lambda v: (v + 255) // 256 * 256
    n_dec = max(2, args.decomposed_reps + 1)          # the first decomposed pass is a warm-up

    def operand_views(buf, off, outer, K):
        """(codes, scales, next offset) inside a byte buffer, as the library lays operands out."""
        c = buf[off: off + outer * K // 2].view(outer, K // 2)
        off += r256(outer * K // 2)
        sb = api.scales_bytes(outer, K)
        return c, buf[off: off + sb], off + r256(sb)

    for rep in range(n_dec):
        evs = []
        fp8_evs = []
        if layer:
            for n in names:
                o, i = dims[n]
                d = dev_in[n]
                T = tokens
                xr_c, xr_s, off = operand_views(lws, 0, T, i)
                wr_c, wr_s, _ = operand_views(lws, off, o, i)
                xt_c, xt_s, off = operand_views(saved, 0, i, T)
                wt_c, wt_s, _ = operand_views(saved, off, i, o)
                ev = [torch.cuda.Event(enable_timing=True) for _ in range(8)]
                ev[0].record(stream)
                api.quantize_dual(d["X"], hmode, rnd, seed, tags=(0, 1), out_row=(xr_c, xr_s), out_col=(xt_c, xt_s))
                ev[1].record(stream)
                api.quantize_dual(d["W"], hmode, rnd, seed, tags=(1, 1), out_row=(wr_c, wr_s), out_col=(wt_c, wt_s))
                ev[2].record(stream)
                api.gemm(xr_c, xr_s, wr_c, wr_s, alpha, api.OUT_BF16, out=out_buf[: T * o].view(T, o))
                ev[3].record(stream)
                dy_c, dy_s, off = operand_views(lws, 0, T, o)
                dyt_c, dyt_s, _ = operand_views(lws, off, o, T)
                ev[4].record(stream)
                api.quantize_dual(d["dY"], hmode, rnd, seed, tags=(0, 0), out_row=(dy_c, dy_s), out_col=(dyt_c, dyt_s))
                ev[5].record(stream)
                api.gemm(dy_c, dy_s, wt_c, wt_s, alpha, api.OUT_BF16, out=out_buf[: T * i].view(T, i))
                ev[6].record(stream)
                api.gemm(dyt_c, dyt_s, xt_c, xt_s, alpha, api.OUT_BF16, out=out_buf2[: o * i].view(o, i))
                ev[7].record(stream)
                evs.append(([(ev[0], ev[1], T * i), (ev[1], ev[2], o * i), (ev[4], ev[5], T * o)],
                            [(ev[2], ev[3], 2.0 * T * o * i, f"{n} fprop {T}x{o}x{i}"),
                             (ev[5], ev[6], 2.0 * T * o * i, f"{n} dgrad {T}x{i}x{o}"),
                             (ev[6], ev[7], 2.0 * T * o * i, f"{n} wgrad {o}x{i}x{T}")]))
        else:
            for (n, p, a, b, M, N, K) in passes:
                ax_a, ax_b = a_b_axes(p)
                if precision[p] == api.PRECISION_MXFP8:
                    # 8-bit pass: timed as a whole (its kernels are not the roofline's subject)
                    ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
                    ev[0].record(stream)
                    lib.mxfp4_linear_pass(p, precision[p], a.data_ptr(), b.data_ptr(), out_buf.data_ptr(), tokens,
                                          dims[n][1], dims[n][0], hmode, rnd, seed, api.OUT_BF16, ws.data_ptr(),
                                          ws_bytes, sptr)
                    ev[1].record(stream)
                    fp8_evs.append((ev[0], ev[1], 2.0 * M * N * K))
                    continue
                ac, a_s, off = operand_views(ws, 0, M, K)
                bc, b_s, _ = operand_views(ws, off, N, K)
                ev = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
                ev[0].record(stream)
                api.quantize_pair(a, ax_a, b, ax_b, hmode, rnd, seed, tags=(0, 1), out_a=(ac, a_s), out_b=(bc, b_s))
                ev[1].record(stream)
                api.gemm(ac, a_s, bc, b_s, alpha, api.OUT_BF16, out=out_buf[: M * N].view(M, N))
                ev[2].record(stream)
                evs.append(([(ev[0], ev[1], (M + N) * K)],
                            [(ev[1], ev[2], 2.0 * M * N * K, f"{n} {('fprop', 'dgrad', 'wgrad')[p]} {M}x{N}x{K}")]))
        torch.cuda.synchronize()
        if rep == 0:
            continue   # first decomposed pass is a warm-up
        qi = 0
        for qs, gs in evs:
            for a0, a1, elems in qs:
                quant_times.setdefault(qi, (elems * q_bytes_per_element, []))[1].append(a0.elapsed_time(a1))
                qi += 1
            for a0, a1, fl, label in gs:
                gemm_times.setdefault(label, (fl, []))[1].append(a0.elapsed_time(a1))
    # medians over the repetitions, per launch; the step's totals are sums of those medians
    gemm_by_shape = {}
    for label, (fl, ts) in gemm_times.items():
        med = statistics.median(ts)
        gemm_ms += med
        gemm_flops += fl
        gemm_by_shape[label] = round(fl / (med * 1e-3) / 1e12, 1)
    for _, (nbytes, ts) in quant_times.items():
        quant_ms += statistics.median(ts)
        quant_bytes += nbytes
        n_quant += 1
    clocks = sampler.stop(t_begin, t_end)
    api.check()

    # ---- the step's twelve GEMMs alone, back to back without events between them (operands quantized
    # once beforehand, each linear in buffers of its own): the per-launch events of the decomposed leg
    # keep a launch's set-up from overlapping its predecessor's tail, so that leg understates the GEMMs
    gemm_b2b = None
    quant_b2b_ms = None
    if layer and not ladder:
        gops = []
        for n in names:
            o, i = dims[n]
            d = dev_in[n]
            (xr, xs), (xt, xts) = api.quantize_dual(d["X"], hmode, rnd, seed, tags=(0, 1))
            (wr, ws_), (wt, wts) = api.quantize_dual(d["W"], hmode, rnd, seed, tags=(1, 1))
            (dyr, dys), (dyt, dyts) = api.quantize_dual(d["dY"], hmode, rnd, seed, tags=(0, 0))
            gops.append(((xr, xs, wr, ws_, out_buf[: tokens * o].view(tokens, o)),
                         (dyr, dys, wt, wts, out_buf[: tokens * i].view(tokens, i)),
                         (dyt, dyts, xt, xts, out_buf2[: o * i].view(o, i))))

        qbufs = []          # every tensor's quantize outputs (row-wise, column-wise), reused by the quantize loop below
        for n in names:
            d = dev_in[n]
            for k_, tg in (("X", (0, 1)), ("W", (1, 1)), ("dY", (0, 0))):
                t_ = d[k_]
                r_, c_ = t_.shape
                qbufs.append((t_, tg,
                              (torch.empty((r_, c_ // 2), dtype=torch.uint8, device="cuda"),
                               torch.empty(api.scales_bytes(r_, c_), dtype=torch.uint8, device="cuda")),
                              (torch.empty((c_, r_ // 2), dtype=torch.uint8, device="cuda"),
                               torch.empty(api.scales_bytes(c_, r_), dtype=torch.uint8, device="cuda"))))

        def quant_loop():
            for t_, tg, orow, ocol in qbufs:
                api.quantize_dual(t_, hmode, rnd, seed, tags=tg, out_row=orow, out_col=ocol)

        for _ in range(3):
            quant_loop()
        torch.cuda.synchronize()
        q0, q1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        q0.record(stream)
        for _ in range(args.steps):
            quant_loop()
        q1.record(stream)
        torch.cuda.synchronize()
        quant_b2b_ms = q0.elapsed_time(q1) / args.steps
        del qbufs

        def gemm_loop():
            for trio in gops:
                for (ac_, as_, bc_, bs_, o_) in trio:
                    api.gemm(ac_, as_, bc_, bs_, alpha, api.OUT_BF16, out=o_)

        for _ in range(3):
            gemm_loop()
        torch.cuda.synchronize()
        g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        g0.record(stream)
        for _ in range(args.steps):
            gemm_loop()
        g1.record(stream)
        torch.cuda.synchronize()
        b2b_ms = g0.elapsed_time(g1) / args.steps
        gemm_b2b = {"ms_per_step": b2b_ms, "tflops": flops_per_step / (b2b_ms * 1e-3) / 1e12,
                    "note": f"the 12 GEMM launches of a step back to back, {args.steps} repetitions, one event pair around all"}
        del gops
        api.check()

    # ---- every quantizer variant on the config-2/3/4 tensors (single launches, L2 rewritten before each)
    quantize_variants = None
    if args.workload == "layer_stack" and not args.no_variants and not ladder:
        quantize_variants = sweep_quantize_variants(dev_in, peaks, api)

    # ---- the single-pass configurations (8192 tokens), fused call, L2 flushed between repetitions
    per_config = {}
    if args.workload == "layer_stack" and not args.no_configs:
        flush = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device="cuda")
        T8 = 8192
        cases = [("config 2: QKV Fprop", "qkv", 0), ("config 3: gate+up Fprop", "gate_up", 0),
                 ("config 3: gate+up Dgrad", "gate_up", 1), ("config 4: down Wgrad", "down", 2)]
        for label, n, pss in cases:
            o, i = dims[n]
            d = dev_in[n]
            a_t = (d["X"] if pss == 0 else d["dY"])[:T8]
            b_t = d["X"][:T8] if pss == 2 else d["W"]
            M, N, K = pass_dims(pss, T8, i, o)
            times = []
            for rep in range(8):
                flush.zero_()
                c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                c0.record(stream)
                rc = fused[pss](a_t.data_ptr(), b_t.data_ptr(), out_buf.data_ptr(), T8, i, o, hmode, rnd, seed,
                                api.OUT_BF16, ws.data_ptr(), ws_bytes, sptr)
                c1.record(stream)
                if rc != 0:
                    raise api.Mxfp4Error(rc, "fused linear pass")
                torch.cuda.synchronize()
                if rep >= 3:
                    times.append(c0.elapsed_time(c1))
            ms = statistics.median(times)
            tf = 2.0 * M * N * K / (ms * 1e-3) / 1e12
            per_config[label] = {"M": M, "N": N, "K": K, "ms": ms, "tflops_incl_quantize": tf,
                                 "frac_of_nominal_fp4_peak": tf / 9000.0,
                                 "state": "per-pass entry point, L2 flushed, measured right after the step loop "
                                          "(SM clock still power-capped; a cold GPU runs these 15-25 % faster)"}
        del flush
        api.check()

    # ---- ceiling of the tensor pipe itself on this device, in this run: the GEMM's own pair MMAs on
    # operands that stay in shared memory (no loads, no epilogue), constant and random operand bits
    mma_only = None
    if not args.no_mma_probe:
        def mma_rate(random_operands, launches):
            time.sleep(1.0)                   # let the clocks recover from the previous leg
            api.probe_mma_rate(10000, random_operands)
            torch.cuda.synchronize()
            m0, m1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            m0.record(stream)
            fl = 0.0
            for _ in range(launches):
                fl += api.probe_mma_rate(10000, random_operands)
            m1.record(stream)
            torch.cuda.synchronize()
            return fl / (m0.elapsed_time(m1) * 1e-3) / 1e12
        mma_only = {"constant_operands_tflops": mma_rate(False, 10), "random_operands_burst_tflops": mma_rate(True, 5),
                    "random_operands_sustained_tflops": mma_rate(True, 60),   # each after a second of idling
                    "note": "mxfp4_probe_mma_rate: 256x192x64 pair MMAs, eight per iteration as in one K-step of the "
                            "GEMM, operands resident in shared memory; 10 / 5 / 60 launches of ~5 ms; with random "
                            "operand bits the tensor pipe alone reaches the power limit"}
        api.check()

    # ---- the GEMM kernel's own steady state: 148 tiles of K = 65536 (tile switches, epilogue and partial
    # waves negligible) on quantized-activation-like codes (or constant ones: --steady-state-codes const).
    # With constant codes this loop runs at ~8.1 PFLOP/s (91 % of the MMA-only rate): in cycles the K loop
    # is close to the tensor pipe; with codes that toggle it is the power limit that holds it lower.
    steady_state = None
    if not args.no_mma_probe and not ladder:
        time.sleep(1.0)                       # let the clocks recover from the previous leg
        Ms, Ns, Ks = 1024, 37 * 384, 65536
        gen = torch.Generator(device="cuda").manual_seed(11)

        def like_codes(rows):
            if args.steady_state_codes == "const":
                return torch.full((rows, Ks // 2), 0x22, dtype=torch.uint8, device="cuda")
            mag = torch.clamp((torch.randn(rows, Ks, device="cuda", generator=gen).abs() * 2.0).round(), 0, 7).to(torch.uint8)
            sgn = (torch.rand(rows, Ks, device="cuda", generator=gen) < 0.5).to(torch.uint8) << 3
            c = mag | sgn
            return (c[:, 0::2] | (c[:, 1::2] << 4)).contiguous()

        a_c, b_c = like_codes(Ms), like_codes(Ns)
        a_s = torch.randint(124, 130, (api.scales_bytes(Ms, Ks),), dtype=torch.uint8, device="cuda", generator=gen)
        b_s = torch.randint(124, 130, (api.scales_bytes(Ns, Ks),), dtype=torch.uint8, device="cuda", generator=gen)
        o_s = torch.empty((Ms, Ns), dtype=torch.bfloat16, device="cuda")
        for _ in range(3):
            api.gemm(a_c, a_s, b_c, b_s, 1.0, api.OUT_BF16, out=o_s)
        torch.cuda.synchronize()

        def rate(launches):
            s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            s0.record(stream)
            for _ in range(launches):
                api.gemm(a_c, a_s, b_c, b_s, 1.0, api.OUT_BF16, out=o_s)
            s1.record(stream)
            torch.cuda.synchronize()
            return 2.0 * Ms * Ns * Ks * launches / (s0.elapsed_time(s1) * 1e-3) / 1e12

        burst, sustained = rate(20), rate(300)          # ~6 ms, then ~0.1 s
        del a_c, b_c, a_s, b_s, o_s
        # bytes between L2 and the SMs per K-step of a CTA pair: codes 2 x (16 + 24) KB + scale tiles 2 x (1 + 3) KB
        pair_kstep_bytes = 2 * (16384 + 24576) + 2 * (1024 + 3072)
        step_bytes = 0.0
        for (_, _, _, _, M, N, K) in passes:
            tiles = ((M + 255) // 256) * ((N + 383) // 384)
            step_bytes += tiles * ((K + 255) // 256) * pair_kstep_bytes + M * N * 2     # operand feed + bf16 output
        steady_state = {"codes": args.steady_state_codes, "burst_tflops": burst, "sustained_tflops": sustained,
                        "l2_sm_bytes_per_step": step_bytes,
                        "note": "gemm_mxf4_pair_kernel on 1024 x 14208 x 65536 (148 tiles, one long K loop each): 20 launches, "
                                "then 300 (0.1 s).  Same kernel, no tile switch, no epilogue to speak of: what is lost "
                                "against the MMA-only ceiling is operand movement (cycles and, with toggling codes, power)"}
        api.check()

    fp8_info = None
    if ladder:
        f8_ms = sum(a0.elapsed_time(a1) for a0, a1, _ in fp8_evs)
        f8_fl = sum(fl for _, _, fl in fp8_evs)
        fp8_info = {"passes": len(fp8_evs), "tflops_incl_quantize": f8_fl / (f8_ms * 1e-3) / 1e12,
                    "format": "MXFP8 (E4M3 elements, E8M0 scale per 32), no rotation"}
    n_gemm = max(1, len(passes) - len(fp8_evs))
    if gemm_ms == 0.0:                      # all passes in 8 bits: nothing for the MXFP4 roofline
        gemm_ms, gemm_flops, quant_ms, quant_bytes, n_quant = 1.0, 0.0, 1.0, 0.0, 1
    # Peak for the contraction: the measured cuBLAS bf16 rate x the nominal FP4 : bf16 ratio (9 : 2.25).
    # The timed region lasts a fraction of a second, so the BURST figure is the one that applies;
    # the sustained figure (seconds under the power cap) and the nominal 9 PFLOP/s are given beside it.
    fp4_peak = 4.0 * peaks["bf16_tflops"]
    fp4_peak_sustained = 4.0 * peaks["bf16_tflops_sustained"]
    # `achieved` comes from the decomposed step: the same launches in the same order as the timed step,
    # interleaved with the quantize launches, a CUDA event between consecutive launches (median of the
    # repetitions per launch).  The back-to-back loops (no events, GEMMs only) are reported beside it.
    gemm_tflops = gemm_flops / (gemm_ms * 1e-3) / 1e12
    gemm_ms_used = gemm_ms
    gemm_timing = f"median of {n_dec - 1} repetitions per launch inside the decomposed step, CUDA events on the launching stream"
    sm_mhz = clocks.get("sm_mhz") or 0.0
    sm_count = torch.cuda.get_device_properties(local_rank).multi_processor_count
    # tensor-pipe issue ceiling at the clock sampled during the timed region: a 256 x 192 x 64 pair
    # MMA takes 96 cycles on two SMs = 32768 flop per clock per SM
    pipe_peak = 32768.0 * sm_count * sm_mhz * 1e6 / 1e12 if sm_mhz else None
    step_tflops = flops_per_step / (elapsed_ms / args.steps * 1e-3) / 1e12
    roofline = {
        "kernel": "gemm_mxf4_pair_kernel", "bound": "tensor", "achieved": gemm_tflops, "peak": fp4_peak,
        "unit": "TFLOP/s", "frac": gemm_tflops / fp4_peak,
        "peak_source": f"4 x burst cuBLAS bf16 ({peaks['source']}: {peaks['bf16_tflops']:.1f}); the timed region is "
                       f"{elapsed_ms * 1e-3:.2f} s, so the burst figure applies",
        "frac_of_4x_sustained_bf16": gemm_tflops / fp4_peak_sustained, "peak_4x_sustained_bf16": fp4_peak_sustained,
        "frac_of_nominal_fp4": gemm_tflops / 9000.0, "peak_nominal_fp4": 9000.0,
        "frac_of_tensor_pipe_at_sampled_clock": (gemm_tflops / pipe_peak) if pipe_peak else None,
        "tensor_pipe_peak_at_sampled_clock": pipe_peak, "sampled_sm_mhz": sm_mhz or None,
        # ncu, dram__bytes_read.sum + dram__bytes_write.sum per launch (profiles/).  Full layer stack at
        # 16384 tokens: mean of the step's 12 launches, one-pass capture of the bench's own launches
        # (4.86 GB per step; operands + outputs are 4.16 GB: the long-K GEMMs re-read the streamed panel once
        # per band of the tile order, and ncu flushes the caches before each launch, which a running step does
        # not).  Other workloads: one captured 8192 x 6144 x 4096 launch, not scaled.
        "traffic": 405.1e6 if (args.workload == "layer_stack" and layer and not ladder) else 78.6e6,
        "traffic_note": ("mean over the step's 12 launches of dram__bytes_read.sum + dram__bytes_write.sum, one-pass ncu "
                         "capture of this command's launches (algorithmic operand + output bytes: 346.8e6 per launch)"
                         if (args.workload == "layer_stack" and layer and not ladder) else
                         "dram__bytes_read.sum + dram__bytes_write.sum of one captured 8192x6144x4096 launch "
                         "(algorithmic bytes of that launch 130.1e6); not scaled to the shapes of this step"),
        "flops_per_launch": gemm_flops / n_gemm, "avg_launch_ms": gemm_ms_used / n_gemm,
        "launch_timing": gemm_timing,
        "tflops_by_launch": gemm_by_shape,
        "tflops_by_launch_timing": f"median of {n_dec - 1} repetitions per launch, an event between consecutive launches",
        "gemms_back_to_back": gemm_b2b,
        "mma_only_ceiling": mma_only,
        "frac_of_mma_only_random_sustained": (gemm_tflops / mma_only["random_operands_sustained_tflops"]) if mma_only else None,
        "kernel_steady_state": (dict(steady_state, frac_of_burst=gemm_tflops / steady_state["burst_tflops"],
                                     frac_of_sustained=gemm_tflops / steady_state["sustained_tflops"],
                                     l2_sm_tbs_in_step=steady_state["l2_sm_bytes_per_step"] / (gemm_ms_used * 1e-3) / 1e12)
                                if steady_state else None),
        "fused_path": {"tflops": step_tflops, "frac_of_nominal_fp4": step_tflops / 9000.0,
                       "frac_of_4x_burst_bf16": step_tflops / fp4_peak,
                       "frac_of_4x_sustained_bf16": step_tflops / fp4_peak_sustained,
                       "note": "the whole step (quantize + GEMM launches) against the same peaks; target 0.60 of nominal"},
        "decomposed": {"gemm_ms": gemm_ms, "quantize_ms": quant_ms, "sum_ms": gemm_ms + quant_ms,
                       "ms_per_step": elapsed_ms / args.steps,
                       "note": "sum of per-launch medians with an event between launches; the events keep a "
                               "launch's set-up from overlapping the previous launch's tail (programmatic "
                               "dependent launch), so the sum exceeds the step time by a few per cent"},
    }
    quant_gbs = quant_bytes / (quant_ms * 1e-3) / 1e9
    # ncu, single-axis kernel on a 117.4 M-element tensor: 234.9 MB read + 45.4 MB written = 2.39 B
    # per element (reads = source bytes exactly; part of the output is still in L2 when the kernel
    # ends); the dual-axis kernel reads the same 2 B and writes twice the codes.  Traffic is
    # proportional to elements, so it is scaled to the mean launch.
    traffic_per_element = 2.39 + (0.39 if layer else 0.0)
    quantize_info = {"kernel": "quantize_dual_kernel" if layer else "quantize_kernel", "bound": "hbm",
                     "achieved": quant_gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                     "frac": quant_gbs / peaks["hbm_gbs"], "bytes_per_element": q_bytes_per_element,
                     "avg_launch_ms": quant_ms / n_quant, "launches_per_step": n_quant,
                     "traffic": traffic_per_element * quant_bytes / q_bytes_per_element / n_quant}
    if quant_b2b_ms:
        # the step's 12 quantize launches back to back (no GEMMs, no events between launches): the kernel's own
        # pipelined rate at the clock it gets when nothing else throttles the device (reported beside `achieved`)
        b2b_gbs = quant_bytes / (quant_b2b_ms * 1e-3) / 1e9
        quantize_info["back_to_back"] = {"ms_per_step": quant_b2b_ms, "gbs": b2b_gbs, "frac": b2b_gbs / peaks["hbm_gbs"],
                                         "note": f"the step's {n_quant} quantize launches back to back (no GEMMs between them), "
                                                 f"{args.steps} repetitions, one CUDA-event pair around all of them"}
    if gemm_b2b:
        # what is left of the (event-free) step after the GEMMs' own back-to-back time: the quantize
        # launches as they run inside the step, without the measurement events between launches
        q_ms = elapsed_ms / args.steps - gemm_b2b["ms_per_step"]
        if q_ms > 0:
            q_gbs = quant_bytes / (q_ms * 1e-3) / 1e9
            quantize_info["in_step_estimate"] = {"ms_per_step": q_ms, "gbs": q_gbs, "frac": q_gbs / peaks["hbm_gbs"],
                                                 "note": "step time minus the 12 GEMMs' back-to-back time"}
    if layer:
        # the same quantized operands cost two single-axis launches (5.0625 B/element) in the per-pass
        # schedule: this launch's rate in those terms, for comparison with that schedule's figure
        quantize_info["as_two_single_axis_passes_gbs"] = quant_gbs * 5.0625 / 3.0625

    # ---- end to end: host buffers in, host buffer out, copies inside the timed region
    e2e = None
    if not args.no_e2e:
        pin = {n: {k: v.pin_memory() for k, v in host[n].items()} for n in names}
        out_host = torch.empty(max_out, dtype=torch.bfloat16).pin_memory()
        stage_a = torch.empty(max(tokens * max(o, i) for o, i in dims.values()), dtype=torch.bfloat16, device="cuda")
        stage_b = torch.empty(max(max(tokens * i, o * i) for o, i in dims.values()), dtype=torch.bfloat16, device="cuda")
        h2d = d2h = 0
        for (n, p, a, b, M, N, K) in passes:
            h2d += (a.numel() + b.numel()) * 2
            d2h += M * N * 2

        def e2e_step_per_pass():
            for (n, p, a, b, M, N, K) in passes:
                o, i = dims[n]
                ah = pin[n]["X" if p == 0 else "dY"]
                bh = pin[n]["X" if p == 2 else "W"]
                rc = lib.mxfp4_linear_host(p, ah.data_ptr(), bh.data_ptr(), out_host.data_ptr(), tokens, i, o,
                                           hmode, rnd, seed, api.OUT_BF16, stage_a.data_ptr(), stage_b.data_ptr(),
                                           out_buf.data_ptr(), ws.data_ptr(), ws_bytes, sptr)
                if rc != 0:
                    raise api.Mxfp4Error(rc, "mxfp4_linear_host")

        if layer:
            # one host-buffer call per linear: X, W, dY cross the bus once, Y, dX, dW come back
            h2d = sum(t.numel() * 2 for n in names for t in pin[n].values())
            del stage_a, stage_b
            big = lambda f: max(f(o, i) for o, i in dims.values())
            stg = {"x": torch.empty(big(lambda o, i: tokens * i), dtype=torch.bfloat16, device="cuda"),
                   "w": torch.empty(big(lambda o, i: o * i), dtype=torch.bfloat16, device="cuda"),
                   "dy": torch.empty(big(lambda o, i: tokens * o), dtype=torch.bfloat16, device="cuda"),
                   "y": out_buf, "dx": out_buf2,
                   "dw": torch.empty(big(lambda o, i: o * i), dtype=torch.bfloat16, device="cuda")}
            # every linear's results land in host buffers of their own (nothing is overwritten)
            host_out = {n: {"y": torch.empty(tokens * o, dtype=torch.bfloat16).pin_memory(),
                            "dx": torch.empty(tokens * i, dtype=torch.bfloat16).pin_memory(),
                            "dw": torch.empty(o * i, dtype=torch.bfloat16).pin_memory()}
                        for n, (o, i) in dims.items()}

        def e2e_step_layer():
            for n in names:
                o, i = dims[n]
                h = pin[n]
                rc = lib.mxfp4_linear_layer_host(
                    h["X"].data_ptr(), h["W"].data_ptr(), h["dY"].data_ptr(), host_out[n]["y"].data_ptr(),
                    host_out[n]["dx"].data_ptr(), host_out[n]["dw"].data_ptr(), tokens, i, o, hmode, rnd, seed,
                    api.OUT_BF16, api.OUT_BF16, api.OUT_BF16, stg["x"].data_ptr(), stg["w"].data_ptr(),
                    stg["dy"].data_ptr(), stg["y"].data_ptr(), stg["dx"].data_ptr(), stg["dw"].data_ptr(),
                    saved.data_ptr(), saved_bytes, lws.data_ptr(), lws_bytes, sptr, 0)
                if rc != 0:
                    raise api.Mxfp4Error(rc, "mxfp4_linear_layer_host")
            rc = lib.mxfp4_linear_layer_host_drain(sptr)      # all results of the step are in host memory
            if rc != 0:
                raise api.Mxfp4Error(rc, "mxfp4_linear_layer_host_drain")

        e2e_step = e2e_step_layer if layer else e2e_step_per_pass

        e2e_step()
        n_e2e = max(1, min(args.steps, 6))
        sync_all()
        t0 = time.perf_counter()
        for _ in range(n_e2e):
            e2e_step()
        sync_all()
        e2e_ms = aggregate_over_ranks((time.perf_counter() - t0) * 1e3, world)
        # what the bus itself gives with both directions busy: plain pinned copies of 1 GiB each way
        # at the same time on two streams (the end-to-end step moves h2d and d2h bytes concurrently)
        bus = None
        try:
            nb = 1 << 30
            hb_in, hb_out = torch.empty(nb, dtype=torch.uint8).pin_memory(), torch.empty(nb, dtype=torch.uint8).pin_memory()
            db_in, db_out = torch.empty(nb, dtype=torch.uint8, device="cuda"), torch.empty(nb, dtype=torch.uint8, device="cuda")
            s_up, s_down = torch.cuda.Stream(), torch.cuda.Stream()
            best = 0.0
            for rep in range(3):
                torch.cuda.synchronize()
                tb = time.perf_counter()
                with torch.cuda.stream(s_up):
                    db_in.copy_(hb_in, non_blocking=True)
                with torch.cuda.stream(s_down):
                    hb_out.copy_(db_out, non_blocking=True)
                torch.cuda.synchronize()
                best = max(best, nb / (time.perf_counter() - tb) / 1e9)
            bus = best
            del hb_in, hb_out, db_in, db_out
        except Exception:
            bus = None
        e2e_gbs = max(h2d, d2h) / (e2e_ms / n_e2e * 1e-3) / 1e9
        e2e = {"value": world * flops_per_step * n_e2e / (e2e_ms * 1e-3) / 1e12, "unit": UNIT,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": n_e2e,
               "ms_per_step": e2e_ms / n_e2e,
               "bus": {"bound": "pcie", "achieved_gbs_each_way": e2e_gbs, "peak_gbs_each_way": bus,
                       "frac": (e2e_gbs / bus) if bus else None,
                       "peak_source": "measured in this run: 1 GiB pinned copies, both directions at once"},
               "note": ("mxfp4_linear_layer_host per linear: pinned X, W, dY copied in once each, Y, dX, dW "
                        "copied out to their own host buffers, copies overlapped with each other, with the kernels and "
                        "across the linears of a step, drained once per step"
                        if layer else
                        "mxfp4_linear_host per pass: pinned host inputs copied in, result copied out, "
                        "stream drained each call")}

    # ---- context: cuBLAS bf16 and FP8 on the same GEMM shapes (not the target)
    context = {}
    if not args.no_context:
        try:
            def time_fn(fn, reps=3):
                fn()
                torch.cuda.synchronize()
                a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a0.record()
                for _ in range(reps):
                    fn()
                a1.record()
                torch.cuda.synchronize()
                return a0.elapsed_time(a1) / reps
            bf_ms = f8_ms = 0.0
            for (n, p, a, b, M, N, K) in passes:
                A = torch.randn(M, K, device="cuda", dtype=torch.bfloat16)
                B = torch.randn(N, K, device="cuda", dtype=torch.bfloat16)
                bf_ms += time_fn(lambda: torch.matmul(A, B.t()))
                A8, B8 = A.to(torch.float8_e4m3fn), B.to(torch.float8_e4m3fn)
                one = torch.ones((), device="cuda", dtype=torch.float32)
                f8_ms += time_fn(lambda: torch._scaled_mm(A8, B8.t(), scale_a=one, scale_b=one,
                                                          out_dtype=torch.bfloat16))
                del A, B, A8, B8
            context = {"cublas_bf16_tflops": flops_per_step / (bf_ms * 1e-3) / 1e12,
                       "cublas_fp8_tflops": flops_per_step / (f8_ms * 1e-3) / 1e12,
                       "note": "GEMMs only (no quantize/cast time), same 12 shapes"}
        except Exception as exc:   # context only
            context = {"error": repr(exc)[:200]}

    if world > 1:
        import torch.distributed as dist
        dist.barrier()
        dist.destroy_process_group()
    if rank != 0:
        return
    cpu_base = None
    if world == 1 and not args.no_cpu_baseline:
        cpu_base, _ = oracle_sample(2, 1)   # about 15 s of host time

    ms_per_step = elapsed_ms / args.steps
    line = {
        "metric": METRIC, "value": world * flops_per_step / (ms_per_step * 1e-3) / 1e12, "unit": UNIT,
        "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "e2m1 (mxfp4) x e2m1, f32 accumulate",
        "data": "synthetic",
        "config": {"workload": workload_label(args.workload, tokens, args.hadamard), "passes_per_step": len(passes),
                   "mxfp4_passes": chosen if chosen else "none (all passes MXFP8)",
                   "schedule": ("layer: forward + backward per linear, each of X, W, dY read once by the dual-axis "
                                "quantize" if layer else "per pass: both operands of each pass quantized from bf16"),
                   "flops_per_step": flops_per_step, "out_dtype": "bf16",
                   "input_crc32": checksums,
                   "l2": "inputs larger than L2 (several GB per step), no flush needed",
                   "parallelism": "replicas only" if world > 1 else "single GPU"},
        "roofline": roofline, "quantize": quantize_info, "quantize_variants": quantize_variants,
        "mxfp8_passes": fp8_info,
        "frac_of_nominal_fp4_peak": world and (flops_per_step / (ms_per_step * 1e-3) / 1e12) / 9000.0,
        "cpu_baseline": cpu_base, "e2e": e2e, "gpu_launches": 2 * len(passes) * args.steps,   # per linear: 3 quantize + 3 GEMM (layer) or 3 x (1 + 1)
        "clocks": clocks, "context": context, "per_config": per_config,
    }
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--no-checksums", action="store_true", help="skip the CRC-32 of the input tensors")
    ap.add_argument("--mxfp4-passes", default="fprop,dgrad,wgrad",
                    help="precision ladder: comma-separated passes that run MXFP4 (the rest run MXFP8); 'none' or '' "
                         "for the all-8-bit baseline; anything but all three implies --schedule per_pass")
    ap.add_argument("--schedule", default="layer", choices=["layer", "per_pass"],
                    help="layer: mxfp4_linear_forward/backward (each tensor read once); per_pass: the three "
                         "per-pass entry points")
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="layer_stack", choices=sorted(WORKLOADS))
    ap.add_argument("--hadamard", default="h32", choices=sorted(HADAMARD))
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-context", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-configs", action="store_true")
    ap.add_argument("--no-variants", action="store_true", help="skip the per-variant quantize table")
    ap.add_argument("--no-mma-probe", action="store_true", help="skip the shared-memory-resident MMA ceiling")
    ap.add_argument("--steady-state-codes", default="like", choices=["like", "const"],
                    help="operand codes of the GEMM steady-state leg: quantized-activation-like (default) or constant")
    ap.add_argument("--decomposed-reps", type=int, default=20,
                    help="repetitions of the per-launch timed step (medians feed the roofline)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()

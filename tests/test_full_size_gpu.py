"""Parity at the benchmark's full sizes, in the launch configuration bench.py times (fused
passes, bf16 outputs, deterministic H32 + RNE and the config-4 variants): quantized operands
bit-exact against the oracle on whole tensors; GEMM outputs checked twice --
  * against the CPU oracle on sampled rows it computes one by one, all columns of each: one
    seeded row out of EVERY 128-row slab of the output plus the slab-edge rows, so every
    256 x 384 tile of the persistent grid, every wave of it and both CTAs of every pair meet
    the oracle;
  * EVERY element against a slow fp64 CUDA checker (tests/gemm_checker: one thread per output,
    integer products, fp64 sums, nothing shared with the library) that multiplies the ORACLE's
    quantized operands and is itself first held against the oracle on those sampled rows."""
import numpy as np
import pytest
import torch

import gemm_checker
import oracle
from gpu_util import assert_gemm_close, to_dev
from paper_2605_09825_b200 import api, synth

pytestmark = pytest.mark.gpu


def _rows(M, seed, stride=128):
    """Edge rows plus one seeded row in every `stride`-row slab of M (the last slab may be short)."""
    rng = np.random.default_rng(seed)
    fixed = [0, 1, 31, 32, 127, 128, M - 129, M - 128, M - 1]
    starts = np.arange(0, M, stride)
    per_slab = starts + rng.integers(0, np.minimum(stride, M - starts))
    return np.unique(np.concatenate([np.array(fixed), per_slab])).astype(np.int64)


ALPHA = {0: 1.0, 1: 1.0 / 32, 2: 1.0 / 32, 3: 1.0 / 16, 4: 1.0 / 16}     # exact factor that undoes H H^T = n I
AXES = ((1, 1), (1, 0), (0, 0))                                          # operand orientation per pass (Appendix C)


def _check_output(out, pass_, a_bits, b_bits, hmode, rnd, seed, what, rows_seed):
    """`out` (CUDA tensor, whole GEMM result of the product path) against the oracle on sampled
    rows and against the fp64 checker on every element."""
    qa = oracle.quantize(a_bits, AXES[pass_][0], hmode, rnd, seed, 0)
    qb = oracle.quantize(b_bits, AXES[pass_][1], hmode, rnd, seed, 1)
    M = out.shape[0]
    rows = _rows(M, rows_seed)
    ref, S = oracle.gemm(*qa, *qb, alpha=ALPHA[hmode], rows=rows)
    bf16 = out.dtype == torch.bfloat16
    got = out[torch.from_numpy(rows).cuda()].float().cpu().numpy()
    assert_gemm_close(got, ref, S, bf16, what)
    # the checker on the same rows of the oracle's operands: must reproduce the oracle (both sum
    # exact block products in fp64; only the order of the last additions may differ)
    _, _, _, cref, cS = gemm_checker.check(qa[0][rows], qa[1][rows], qb[0], qb[1], ALPHA[hmode], None, want_ref=True)
    cref, cS = cref.cpu().numpy(), cS.cpu().numpy()
    assert np.all(np.abs(cref - ref) <= 1e-12 * S + 1e-300), f"{what}: checker differs from the oracle"
    assert np.all(np.abs(cS - S) <= 1e-12 * S + 1e-300), f"{what}: checker's tolerance base differs from the oracle's"
    # every element of the product path's output against the checker
    n_bad, first, worst, _, _ = gemm_checker.check(*qa, *qb, ALPHA[hmode], out)
    assert n_bad == 0, (f"{what}: {n_bad} of {out.numel()} elements out of tolerance, first at "
                        f"[{first // out.shape[1]}, {first % out.shape[1]}], worst error / tolerance {worst:.3g}")
    assert worst <= 1.0


def _check_pass(pass_, a_bits, b_bits, hmode, rnd, seed, what):
    a, b = to_dev(a_bits), to_dev(b_bits)
    fn = (api.linear_fprop, api.linear_dgrad, api.linear_wgrad)[pass_]
    out = fn(a, b, hmode, rnd, seed, api.OUT_BF16)
    api.check()
    del a, b
    _check_output(out, pass_, a_bits, b_bits, hmode, rnd, seed, what, 1234 + pass_)
    del out


def _check_quant(bits, axis, hmode, rnd, seed, tag):
    codes, scales = api.quantize(to_dev(bits), axis, hmode, rnd, seed, tag)
    api.check()
    wc, ws = oracle.quantize(bits, axis, hmode, rnd, seed, tag)
    outer, K = wc.shape[0], wc.shape[1] * 2
    assert (codes.cpu().numpy() == wc).all()
    assert (oracle.scales_from_tiled(scales.cpu().numpy(), outer, K // 32) == ws).all()


def test_config2_qkv_fprop():
    t = synth.config2()
    _check_pass(0, t["X"], t["W"], 1, 0, 0, "config 2 fprop")


def test_config3_gate_up_fprop_and_dgrad():
    t = synth.config3()
    _check_pass(0, t["X"], t["W"], 1, 0, 0, "config 3 fprop")
    _check_pass(1, t["dY"], t["W"], 1, 0, 0, "config 3 dgrad")
    _check_quant(t["dY"], 1, 1, 0, 0, 0)        # the largest operand of the path, row-wise
    _check_quant(t["W"], 0, 1, 0, 0, 1)         # W^T for Dgrad, column-wise


@pytest.mark.parametrize("hmode,rnd", [(1, 0), (2, 0), (0, 1), (3, 0)])
def test_config4_down_wgrad_variants(hmode, rnd):
    t = synth.config4()
    _check_pass(2, t["dY"], t["X"], hmode, rnd, 7, f"config 4 wgrad mode {hmode} rounding {rnd}")
    _check_quant(t["X"], 0, hmode, rnd, 7, 1)   # X^T [14336 x 8192], column-wise, whole tensor


@pytest.mark.parametrize("name", ["qkv", "o", "gate_up", "down"])
def test_config5_layer_stack_16384_tokens(name):
    t = synth.linear_tensors(name, 16384, 5)
    _check_pass(0, t["X"], t["W"], 1, 0, 0, f"config 5 {name} fprop")
    _check_pass(1, t["dY"], t["W"], 1, 0, 0, f"config 5 {name} dgrad")
    _check_pass(2, t["dY"], t["X"], 1, 0, 0, f"config 5 {name} wgrad")


@pytest.mark.parametrize("name", ["qkv", "o", "gate_up", "down"])
def test_config5_layer_schedule_16384_tokens(name):
    """The schedule bench.py times by default: forward + backward per linear, every tensor read
    once by the dual-axis quantize.  Sampled output rows against the oracle; the kept column-wise
    operands (the whole saved buffer) bit-exact for the smallest linear."""
    t = synth.linear_tensors(name, 16384, 5)
    X, W, dY = to_dev(t["X"]), to_dev(t["W"]), to_dev(t["dY"])
    in_f = X.shape[1]
    Y, saved = api.linear_forward(X, W, 1, 0, 0)
    dX, dW = api.linear_backward(dY, saved, in_f, 1, 0, 0)
    api.check()
    for out, pass_, a, b, what in ((Y, 0, t["X"], t["W"], "fprop"), (dX, 1, t["dY"], t["W"], "dgrad"),
                                   (dW, 2, t["dY"], t["X"], "wgrad")):
        _check_output(out, pass_, a, b, 1, 0, 0, f"config 5 {name} layer schedule {what}", 4321)
    if name == "o":
        raw = saved.cpu().numpy()
        r256 = lambda n: (n + 255) // 256 * 256
        off = 0
        for bits in (t["X"], t["W"]):
            wc, ws = oracle.quantize(bits, 0, 1, 0, 0, 1)
            outer, K = wc.shape[0], wc.shape[1] * 2
            assert (raw[off:off + wc.size].reshape(wc.shape) == wc).all()
            off += r256(wc.size)
            sb = api.scales_bytes(outer, K)
            assert (oracle.scales_from_tiled(raw[off:off + sb], outer, K // 32) == ws).all()
            off += r256(sb)


def test_config3_dual_quantize_of_the_largest_tensor():
    """dY of gate+up at 8192 tokens (448 MiB of bf16): both orientations, whole tensors, bit-exact."""
    t = synth.config3()
    (cr, sr), (cc, sc) = api.quantize_dual(to_dev(t["dY"]), 1, 0, 0, tags=(0, 0))
    api.check()
    for codes, scales, axis in ((cr, sr, 1), (cc, sc, 0)):
        wc, ws = oracle.quantize(t["dY"], axis, 1, 0, 0, 0)
        assert (codes.cpu().numpy() == wc).all()
        assert (oracle.scales_from_tiled(scales.cpu().numpy(), wc.shape[0], wc.shape[1] * 2 // 32) == ws).all()


def test_eight_times_the_benchmark_token_count():
    """131072 tokens (1 GiB of bf16 activations, 2^29 elements): index arithmetic beyond the
    benchmark's sizes.  Dual-axis quantize bit-exact on the whole tensor in both orientations,
    Fprop and Wgrad outputs on sampled rows."""
    T, in_f, out_f = 131072, 4096, 1024
    t = synth.linear_tensors("o", T, 6)                  # X [T x 4096], W, dY [T x 4096]
    Xb, Wb, dYb = t["X"], np.ascontiguousarray(t["W"][:out_f]), np.ascontiguousarray(t["dY"][:, :out_f])
    X, W, dY = to_dev(Xb), to_dev(Wb), to_dev(dYb)
    (cr, sr), (cc, sc) = api.quantize_dual(X, 1, 0, 0, tags=(0, 1))
    api.check()
    for codes, scales, axis, tag in ((cr, sr, 1, 0), (cc, sc, 0, 1)):
        wc, ws = oracle.quantize(Xb, axis, 1, 0, 0, tag)
        assert (codes.cpu().numpy() == wc).all()
        assert (oracle.scales_from_tiled(scales.cpu().numpy(), wc.shape[0], wc.shape[1] * 2 // 32) == ws).all()
        del wc, ws
    del cr, sr, cc, sc
    Y, saved = api.linear_forward(X, W, 1, 0, 0)
    dX, dW = api.linear_backward(dY, saved, in_f, 1, 0, 0, api.OUT_BF16, api.OUT_FP32)
    api.check()
    _check_output(Y, 0, Xb, Wb, 1, 0, 0, "fprop at 131072 tokens", 99)
    _check_output(dW, 2, dYb, Xb, 1, 0, 0, "wgrad over 131072 tokens", 98)


@pytest.mark.parametrize("hmode,rnd", [(1, 0), (2, 0), (0, 1)])
def test_config4_dual_quantize_variants(hmode, rnd):
    """Config 4's X [8192 x 14336] (post-SwiGLU-like) through the dual-axis kernel for the three
    variants of that configuration, whole tensor, both orientations, bit-exact."""
    t = synth.config4()
    (cr, sr), (cc, sc) = api.quantize_dual(to_dev(t["X"]), hmode, rnd, 7, tags=(0, 1))
    api.check()
    for codes, scales, axis, tag in ((cr, sr, 1, 0), (cc, sc, 0, 1)):
        wc, ws = oracle.quantize(t["X"], axis, hmode, rnd, 7, tag)
        assert (codes.cpu().numpy() == wc).all()
        assert (oracle.scales_from_tiled(scales.cpu().numpy(), wc.shape[0], wc.shape[1] * 2 // 32) == ws).all()

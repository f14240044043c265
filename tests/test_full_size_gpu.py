"""Parity at the benchmark's full sizes, in the launch configuration bench.py times (fused
passes, bf16 outputs, deterministic H32 + RNE and the config-4 variants): quantized operands
bit-exact against the oracle on whole tensors, GEMM outputs on sampled rows the oracle computes
one by one, all columns of each.  The sample holds one seeded row out of EVERY 128-row slab of
the output plus the slab-edge rows, so every 256 x 384 tile of the persistent grid, every wave
of it and both CTAs of every pair meet the oracle."""
import numpy as np
import pytest
import torch

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


def _check_pass(pass_, a_bits, b_bits, hmode, rnd, seed, what):
    a, b = to_dev(a_bits), to_dev(b_bits)
    fn = (api.linear_fprop, api.linear_dgrad, api.linear_wgrad)[pass_]
    ofn = (oracle.linear_fprop, oracle.linear_dgrad, oracle.linear_wgrad)[pass_]
    out = fn(a, b, hmode, rnd, seed, api.OUT_BF16)
    api.check()
    M = out.shape[0]
    rows = _rows(M, 1234 + pass_)
    ref, S = ofn(a_bits, b_bits, hmode, rnd, seed, rows=rows)
    got = out[torch.from_numpy(rows).cuda()].float().cpu().numpy()
    assert_gemm_close(got, ref, S, True, what)
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
    for out, ofn, a, b, what in ((Y, oracle.linear_fprop, t["X"], t["W"], "fprop"),
                                 (dX, oracle.linear_dgrad, t["dY"], t["W"], "dgrad"),
                                 (dW, oracle.linear_wgrad, t["dY"], t["X"], "wgrad")):
        rows = _rows(out.shape[0], 4321)
        ref, S = ofn(a, b, 1, 0, 0, rows=rows)
        got = out[torch.from_numpy(rows).cuda()].float().cpu().numpy()
        assert_gemm_close(got, ref, S, True, f"config 5 {name} layer schedule {what}")
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
    rows = _rows(T, 99)
    ref, S = oracle.linear_fprop(Xb, Wb, 1, 0, 0, rows=rows)
    assert_gemm_close(Y[torch.from_numpy(rows).cuda()].float().cpu().numpy(), ref, S, True, "fprop at 131072 tokens")
    rows = _rows(out_f, 98)
    ref, S = oracle.linear_wgrad(dYb, Xb, 1, 0, 0, rows=rows)
    assert_gemm_close(dW[torch.from_numpy(rows).cuda()].cpu().numpy(), ref, S, False, "wgrad over 131072 tokens")


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

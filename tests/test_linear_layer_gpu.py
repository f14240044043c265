"""Layer-level forward / backward (each tensor read once) vs the CPU oracle and vs the per-pass
entry points, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
from gpu_util import assert_gemm_close, random_bits, to_dev
from paper_2605_09825_b200 import api, synth

pytestmark = pytest.mark.gpu


def _tensors(T, in_f, out_f, seed):
    rng = np.random.default_rng(seed)
    return random_bits(rng, T, in_f, 3), random_bits(rng, out_f, in_f, 2), random_bits(rng, T, out_f, 4)


@pytest.mark.parametrize("hmode,rnd", [(0, 0), (1, 0), (2, 0), (3, 0), (1, 1), (4, 1)])
@pytest.mark.parametrize("T,in_f,out_f", [(256, 512, 256), (416, 288, 672)])
def test_layer_passes_match_the_oracle(T, in_f, out_f, hmode, rnd):
    X, W, dY = _tensors(T, in_f, out_f, T + in_f)
    Y, saved = api.linear_forward(to_dev(X), to_dev(W), hmode, rnd, 5, api.OUT_FP32)
    dX, dW = api.linear_backward(to_dev(dY), saved, in_f, hmode, rnd, 5, api.OUT_FP32, api.OUT_FP32)
    api.check()
    for got, (ref, S), what in ((Y, oracle.linear_fprop(X, W, hmode, rnd, 5), "Y"),
                                (dX, oracle.linear_dgrad(dY, W, hmode, rnd, 5), "dX"),
                                (dW, oracle.linear_wgrad(dY, X, hmode, rnd, 5), "dW")):
        assert_gemm_close(got.cpu().numpy(), ref, S, bf16=False, what=what)


@pytest.mark.parametrize("hmode,rnd", [(1, 0), (2, 1)])
def test_layer_passes_are_bit_identical_to_the_per_pass_entry_points(hmode, rnd):
    T, in_f, out_f = 1056, 640, 1408
    X, W, dY = (to_dev(b) for b in _tensors(T, in_f, out_f, 77))
    Y, saved = api.linear_forward(X, W, hmode, rnd, 3)
    dX, dW = api.linear_backward(dY, saved, in_f, hmode, rnd, 3, api.OUT_BF16, api.OUT_FP32)
    api.check()
    assert torch.equal(Y, api.linear_fprop(X, W, hmode, rnd, 3))
    assert torch.equal(dX, api.linear_dgrad(dY, W, hmode, rnd, 3))
    assert torch.equal(dW, api.linear_wgrad(dY, X, hmode, rnd, 3, api.OUT_FP32))


def test_saved_buffer_holds_the_column_wise_operands():
    """What backward reads is exactly Q(X^T) then Q(W^T): codes + tiled scales, 256-byte rounded."""
    T, in_f, out_f = 160, 96, 224
    Xb, Wb, _ = _tensors(T, in_f, out_f, 9)
    _, saved = api.linear_forward(to_dev(Xb), to_dev(Wb), 1, 0, 0)
    api.check()
    raw = saved.cpu().numpy()
    r256 = lambda n: (n + 255) // 256 * 256
    off = 0
    for bits, tag, outer, K in ((Xb, 1, in_f, T), (Wb, 1, in_f, out_f)):
        codes, scales = oracle.quantize(bits, 0, 1, 0, 0, tag)
        n = outer * K // 2
        assert np.array_equal(raw[off:off + n].reshape(outer, K // 2), codes)
        off += r256(n)
        sb = api.scales_bytes(outer, K)
        assert np.array_equal(oracle.scales_from_tiled(raw[off:off + sb], outer, K // 32), scales)
        off += r256(sb)
    assert off == api.linear_layer_bytes(T, in_f, out_f, api.LAYER_SAVED)


def test_layer_argument_errors():
    X, W, dY = (to_dev(b) for b in _tensors(64, 64, 64, 1))
    small = torch.empty(256, dtype=torch.uint8, device="cuda")
    with pytest.raises(api.Mxfp4Error) as exc:
        api.linear_forward(X, W, saved=small)
    assert exc.value.status == -5
    _, saved = api.linear_forward(X, W)
    with pytest.raises(api.Mxfp4Error) as exc:
        api.linear_backward(dY, saved, 64, workspace=small)
    assert exc.value.status == -5
    assert api.linear_layer_bytes(48, 64, 64, api.LAYER_SAVED) == 0       # T not a multiple of 32
    assert api.linear_layer_bytes(64, 64, 64, 3) == 0
    bad = to_dev(random_bits(np.random.default_rng(2), 48, 64))
    with pytest.raises(api.Mxfp4Error) as exc:
        api.linear_forward(bad, W, saved=torch.empty(1 << 20, dtype=torch.uint8, device="cuda"),
                           workspace=torch.empty(1 << 20, dtype=torch.uint8, device="cuda"))
    assert exc.value.status == -2


def test_host_buffer_layer_call_matches_the_device_calls():
    T, in_f, out_f = 416, 288, 672
    Xb, Wb, dYb = _tensors(T, in_f, out_f, 13)
    host = [torch.from_numpy(b.view(np.int16)).view(torch.bfloat16).pin_memory() for b in (Xb, Wb, dYb)]
    Yh = torch.empty((T, out_f), dtype=torch.bfloat16).pin_memory()
    dXh = torch.empty((T, in_f), dtype=torch.bfloat16).pin_memory()
    dWh = torch.empty((out_f, in_f), dtype=torch.float32).pin_memory()
    e = lambda shape, dt: torch.empty(shape, dtype=dt, device="cuda")
    dev = {"x": e((T, in_f), torch.bfloat16), "w": e((out_f, in_f), torch.bfloat16), "dy": e((T, out_f), torch.bfloat16),
           "y": e((T, out_f), torch.bfloat16), "dx": e((T, in_f), torch.bfloat16), "dw": e((out_f, in_f), torch.float32)}
    saved = e(api.linear_layer_bytes(T, in_f, out_f, api.LAYER_SAVED), torch.uint8)
    ws = e(max(api.linear_layer_bytes(T, in_f, out_f, w) for w in (api.LAYER_FORWARD, api.LAYER_BACKWARD)), torch.uint8)
    for _ in range(2):                                   # twice: the second call reuses streams and events
        api.linear_layer_host(*host, Yh, dXh, dWh, dev, saved, ws, 1, 0, 3, api.OUT_BF16, api.OUT_BF16, api.OUT_FP32)
        api.check()
        X, W, dY = (h.cuda() for h in host)
        Y, sv = api.linear_forward(X, W, 1, 0, 3)
        dX, dW = api.linear_backward(dY, sv, in_f, 1, 0, 3, api.OUT_BF16, api.OUT_FP32)
        assert torch.equal(Yh, Y.cpu()) and torch.equal(dXh, dX.cpu()) and torch.equal(dWh, dW.cpu())
        Yh.zero_(); dXh.zero_(); dWh.zero_()


def test_undrained_host_calls_overlap_and_keep_their_results():
    """Three layers queued without draining, sharing one set of staging buffers: every layer's
    host outputs must be that layer's results once the drain returns."""
    T, in_f, out_f = 416, 288, 672
    e = lambda shape, dt: torch.empty(shape, dtype=dt, device="cuda")
    dev = {"x": e((T, in_f), torch.bfloat16), "w": e((out_f, in_f), torch.bfloat16), "dy": e((T, out_f), torch.bfloat16),
           "y": e((T, out_f), torch.bfloat16), "dx": e((T, in_f), torch.bfloat16), "dw": e((out_f, in_f), torch.bfloat16)}
    saved = e(api.linear_layer_bytes(T, in_f, out_f, api.LAYER_SAVED), torch.uint8)
    ws = e(max(api.linear_layer_bytes(T, in_f, out_f, w) for w in (api.LAYER_FORWARD, api.LAYER_BACKWARD)), torch.uint8)
    layers = []
    for k in range(3):
        bits = _tensors(T, in_f, out_f, 100 + k)
        host = [torch.from_numpy(b.view(np.int16)).view(torch.bfloat16).pin_memory() for b in bits]
        outs = [torch.zeros(s_, dtype=torch.bfloat16).pin_memory() for s_ in ((T, out_f), (T, in_f), (out_f, in_f))]
        layers.append((host, outs))
    for host, outs in layers:
        api.linear_layer_host(*host, *outs, dev, saved, ws, 1, 0, 3, drain=False)
    api.linear_layer_host_drain()
    api.check()
    for host, outs in layers:
        X, W, dY = (h.cuda() for h in host)
        Y, sv = api.linear_forward(X, W, 1, 0, 3)
        dX, dW = api.linear_backward(dY, sv, in_f, 1, 0, 3)
        assert torch.equal(outs[0], Y.cpu()) and torch.equal(outs[1], dX.cpu()) and torch.equal(outs[2], dW.cpu())

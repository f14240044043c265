"""The fp64 CUDA checker used by the full-size parity tests (tests/gemm_checker): it builds and
exports its entry point (CPU); on a GPU it reproduces the CPU oracle on whole small outputs with
ragged edges, and it finds a single planted error at the right place."""
import ctypes

import numpy as np
import pytest
import torch

import gemm_checker
import oracle


def test_checker_builds_and_exports_its_entry_point():
    lib = ctypes.CDLL(gemm_checker.build())
    assert hasattr(lib, "mxcheck_gemm")


def _operands(rng, M, N, K):
    ac = rng.integers(0, 256, size=(M, K // 2), dtype=np.uint8)
    bc = rng.integers(0, 256, size=(N, K // 2), dtype=np.uint8)
    asc = rng.integers(110, 140, size=(M, K // 32), dtype=np.uint8)
    bsc = rng.integers(110, 140, size=(N, K // 32), dtype=np.uint8)
    return ac, asc, bc, bsc


@pytest.mark.gpu
@pytest.mark.parametrize("M,N,K", [(16, 16, 32), (37, 53, 288), (130, 200, 1056), (1, 7, 64)])
def test_checker_reproduces_the_oracle(M, N, K):
    rng = np.random.default_rng(M * N + K)
    ac, asc, bc, bsc = _operands(rng, M, N, K)
    ref, S = oracle.gemm(ac, asc, bc, bsc, alpha=0.0625)
    _, _, _, cref, cS = gemm_checker.check(ac, asc, bc, bsc, 0.0625, None, want_ref=True)
    assert np.all(np.abs(cref.cpu().numpy() - ref) <= 1e-13 * S)
    assert np.all(np.abs(cS.cpu().numpy() - S) <= 1e-13 * S)


@pytest.mark.gpu
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_checker_finds_one_planted_error(dtype):
    rng = np.random.default_rng(5)
    M, N, K = 70, 90, 160
    ac, asc, bc, bsc = _operands(rng, M, N, K)
    ref, S = oracle.gemm(ac, asc, bc, bsc, alpha=1.0)
    out = torch.from_numpy(ref).cuda().to(dtype)
    n_bad, _, worst, _, _ = gemm_checker.check(ac, asc, bc, bsc, 1.0, out)
    assert n_bad == 0 and worst <= 1.0
    out[41, 17] += (3e-5 * S[41, 17] + 2.0 ** -6 * abs(ref[41, 17]))      # beyond both terms of the tolerance
    n_bad, first, worst, _, _ = gemm_checker.check(ac, asc, bc, bsc, 1.0, out)
    assert n_bad == 1 and first == 41 * N + 17 and worst > 1.0
    out[3, 88] = float("nan")
    n_bad, first, _, _, _ = gemm_checker.check(ac, asc, bc, bsc, 1.0, out)
    assert n_bad == 2 and first == 3 * N + 88

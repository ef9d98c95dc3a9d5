"""Final binarisation of weight rows in the rotated coordinates (Alg. 2, last step) against the CPU oracle.

The GPU rotates in fp32-equivalent arithmetic (error below 1e-6 of a row's largest rotated magnitude), the oracle in
fp64; a sign bit may differ only where the oracle's |X - mu| lies inside that window, and such bits are counted.  The
row shift and the scale are means over K values and must agree to 2e-6 of the row's largest magnitude.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_00422_b200 import inputs as gen

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def bwla():
    from paper_2605_00422_b200 import bwla as b
    return b


def _check(bwla, W_host, W_dev, P1, P2):
    ref = oracle.binarize(W_host, P1, P2)
    ws = torch.zeros(bwla.bwla_binarize_workspace_bytes(W_host.shape[1]), dtype=torch.uint8, device="cuda")
    packed, alpha, mu = bwla.bwla_binarize_rows(W_dev, torch.from_numpy(P1).cuda(), torch.from_numpy(P2).cuda(), workspace=ws)
    assert bwla.bwla_check_status(ws) == 0
    N, K = W_host.shape
    amax = np.abs(ref["X"]).max(axis=1)
    np.testing.assert_array_less(np.abs(mu.cpu().numpy().astype(np.float64) - ref["mu"]), 2e-6 * amax + 1e-30)
    np.testing.assert_array_less(np.abs(alpha.cpu().numpy().astype(np.float64) - ref["alpha"]), 2e-6 * amax + 1e-30)
    got = oracle.unpack_signs(packed.cpu().numpy().view(np.uint32), K)
    want = oracle.unpack_signs(ref["packed"], K)
    differ = got != want
    near_zero = np.abs(ref["X"] - ref["mu"][:, None]) <= 3e-6 * amax[:, None]
    assert not np.any(differ & ~near_zero), f"{np.count_nonzero(differ & ~near_zero)} sign bits differ outside the window"
    print(f"\n[{N} x {K}] sign bits inside the window: {np.count_nonzero(near_zero)}, of them different: {np.count_nonzero(differ)}")
    return packed, alpha, mu


@pytest.mark.parametrize("n1,n2,N", [(32, 32, 70), (64, 80, 300), (86, 128, 64), (160, 160, 40)])
def test_fp32_rows(bwla, n1, n2, N):
    rng = np.random.default_rng([9, n1, n2])
    P1, P2 = gen.orthogonal_f32(n1, rng), gen.orthogonal_f32(n2, rng)
    W = (rng.standard_normal((N, n1 * n2)) * 0.02 + rng.uniform(-0.01, 0.01, (N, 1))).astype(np.float32)
    _check(bwla, W, torch.from_numpy(W).cuda(), P1, P2)


def test_bf16_rows_with_a_row_stride(bwla):
    n1, n2, N = 64, 64, 130
    K = n1 * n2
    rng = np.random.default_rng(4)
    P1, P2 = gen.orthogonal_f32(n1, rng), gen.orthogonal_f32(n2, rng)
    Wb = gen.bf16_bits_from_f32((rng.standard_normal((N, K)) * 0.05).astype(np.float32))
    W = gen.f32_from_bf16_bits(Wb)
    big = torch.zeros(N, K + 64, dtype=torch.bfloat16, device="cuda")
    big[:, :K] = torch.from_numpy(W).cuda().to(torch.bfloat16)
    _check(bwla, W, big[:, :K], P1, P2)


def test_binarised_layer_reproduces_rows_that_are_binary_after_the_rotation(bwla):
    """End to end: W = (mu + c s) R^T is binarised on the GPU and the resulting layer (with mu) applied to x equals W x up
    to the activation quantiser's error."""
    n1, n2, N, M = 32, 32, 128, 16
    K = n1 * n2
    rng = np.random.default_rng(12)
    P1, P2 = gen.orthogonal_f32(n1, rng), gen.orthogonal_f32(n2, rng)
    R = np.kron(P1.astype(np.float64), P2.astype(np.float64))
    s = np.where(rng.random((N, K)) < 0.5, -1.0, 1.0)
    s[:, : K // 2] = -s[:, K // 2:]                                     # balanced rows
    c, m = rng.uniform(0.01, 0.03, N), rng.uniform(-0.002, 0.002, N)
    W = ((m[:, None] + c[:, None] * s) @ R.T).astype(np.float32)
    packed, alpha, mu = _check(bwla, W, torch.from_numpy(W).cuda(), P1, P2)
    np.testing.assert_allclose(alpha.cpu().numpy(), c, rtol=2e-4)
    xb = gen.bf16_bits_from_f32(rng.standard_normal((M, K)).astype(np.float32))
    x = gen.f32_from_bf16_bits(xb).astype(np.float64)
    xd = torch.from_numpy(gen.f32_from_bf16_bits(xb)).cuda().to(torch.bfloat16)
    out = bwla.bwla_w1ax_linear(xd, torch.from_numpy(P1).cuda(), torch.from_numpy(P2).cuda(), 8, packed, alpha, mu=mu)
    want = x @ W.astype(np.float64).T
    got = out.float().cpu().numpy().astype(np.float64)
    assert np.linalg.norm(got - want) / np.linalg.norm(want) < 2e-2

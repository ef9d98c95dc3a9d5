"""W1A16, the weight-only operating point, against the CPU oracle.

The GPU rounds its own fp32 rotation to bf16, the oracle the fp64 one: a rotated value within the rotation error of a
bf16 rounding boundary may round the other way, which moves one of K summands of an output by one bf16 step of that
value (far below the output tolerance).  The output is held to the bounds of the other layer tests: rel-L2 <= 2e-3 and
every element within 1e-2 * rms(y) + 2^-8 * |y|.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_00422_b200 import inputs as gen
from tests import helpers as H

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def bwla():
    from paper_2605_00422_b200 import bwla as b
    return b


def _case(bwla, cfg, shape, M, with_mu=False, sample=None):
    lay = gen.make_layer(cfg, shape, 8, direct_words=True)
    xb = gen.make_activations(cfg, shape, M)
    dl = H.DeviceLayer(lay, bwla)
    mu_h = None
    mu_d = None
    if with_mu:
        mu_h = (np.random.default_rng(3).uniform(-1, 1, shape.N) * 1e-3).astype(np.float32)
        mu_d = torch.from_numpy(mu_h).cuda()
    layer = bwla.Layer(dl.P1, dl.P2, 8, dl.packed, dl.alpha, dl.U, dl.V, mu=mu_d)
    ws = torch.zeros(bwla.bwla_w1a16_workspace_bytes(layer, M), dtype=torch.uint8, device="cuda")
    out = bwla.bwla_layer_w1a16_linear(layer, H.bf16_to_dev(xb), workspace=ws)
    assert bwla.bwla_check_status(ws) == 0
    rows = np.arange(M) if sample is None else sample
    ref = oracle.linear_a16(xb[rows], lay.P1, lay.P2, dl.packed_host, lay.alpha, lay.U, lay.V, mu=mu_h)
    rep = H.check_output(H.bf16_to_host(out[rows]), ref["y"])
    assert rep["rel_l2"] <= 2e-3
    print(f"\n[{shape.name} M={M}] rel L2 {rep['rel_l2']:.2e}, max |err|/rms {rep['max_abs_over_rms']:.3f}")
    return rep


def test_small_layer_with_row_shift(bwla):
    _case(bwla, 0, gen.CONFIG_SHAPES[0][0], 16, with_mu=True)


@pytest.mark.parametrize("idx,M", [(0, 16), (1, 1), (3, 130)])
def test_llama7b_shapes(bwla, idx, M):
    _case(bwla, 1, gen.CONFIG_SHAPES[1][idx], M)


@pytest.mark.parametrize("idx,M", [(1, 8), (3, 64), (6, 8)])
def test_qwen32b_shapes(bwla, idx, M):
    _case(bwla, 2, gen.CONFIG_SHAPES[2][idx], M)


def test_prefill_sized_batch_on_sampled_tokens(bwla):
    M = 2048
    _case(bwla, 2, gen.CONFIG_SHAPES[2][0], M, sample=H.token_sample(M))


@pytest.mark.parametrize("K,N,n1,n2,r,M", [
    (192, 200, 12, 16, 0, 5),         # three k-blocks (an odd number: the last accumulator holds one), ragged rows, no low-rank branch
    (1024, 129, 32, 32, 13, 130),     # one row beyond a tile, a rank that is not a multiple of 8, a ragged second token tile
    (64, 8, 8, 8, 4, 1),              # a single k-block, one token
    (2048, 384, 32, 64, 64, 17),      # the full rank of 64
])
def test_small_and_ragged_shapes(bwla, K, N, n1, n2, r, M):
    sh = gen.small_shape(K, N, n1, n2, r, shape_id=K + N)
    lay = gen.make_layer(0, sh, 8, with_mu=(r == 13))
    xb = gen.make_activations(0, sh, M)
    dl = H.DeviceLayer(lay, bwla)
    layer = bwla.Layer(dl.P1, dl.P2, 8, dl.packed, dl.alpha, dl.U, dl.V, mu=dl.mu)
    ws = torch.zeros(bwla.bwla_w1a16_workspace_bytes(layer, M), dtype=torch.uint8, device="cuda")
    out = torch.full((M, N + 3), 7.0, dtype=torch.bfloat16, device="cuda")       # a row stride that is not a multiple of 8
    bwla.bwla_layer_w1a16_linear(layer, H.bf16_to_dev(xb), out=out[:, :N], workspace=ws)
    assert bwla.bwla_check_status(ws) == 0
    assert torch.all(out[:, N:] == 7.0)                                           # nothing written beyond the rows
    ref = oracle.linear_a16(xb, lay.P1, lay.P2, dl.packed_host, lay.alpha, lay.U, lay.V, mu=lay.mu)
    H.check_output(H.bf16_to_host(out[:, :N].contiguous()), ref["y"])

"""Parity with the CPU oracle at prefill-sized token counts and on the workload shapes the small cases leave out.

The oracle takes seconds per hundred tokens at these sizes, so it runs on a stratified sample of the tokens (tokens
are independent rows): every position inside the first 128-token tile, the whole last tile, and one position of
every tile in between, against all N output rows.  The CUDA path always runs the full problem, in the launch
configuration the benchmark times.  What is compared on the sample:

  * the codes and scales the fused call itself left in its workspace (read back through bwla_workspace_section),
    against the fp64 quantiser of the oracle's rotation, with the near-tie rule of tests/helpers.py;
  * the bf16 outputs against the oracle's fp64 layer output;
  * the int32 accumulators of bwla_w1a_gemm_codes for identical codes, bit-exact against the oracle's integer
    contraction, and the outputs for identical codes within one bf16 step: the sampled tokens are given the oracle's
    codes and scales, the other tokens seeded random codes (they only have to keep every tile of the launch busy).
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
    b.bwla_force_path(b.BWLA_PATH_AUTO)
    return b


def run_sampled_case(bwla, cfg, shape, M, bits, check_acc=True):
    lay = gen.make_layer(cfg, shape, bits, direct_words=True)
    xb = gen.make_activations(cfg, shape, M)
    sample = H.token_sample(M)
    dl = H.DeviceLayer(lay, bwla)
    xd = H.bf16_to_dev(xb)
    ws = bwla.new_workspace(M, shape.K, shape.N, shape.r, bits)
    out = bwla.bwla_w1ax_linear(xd, dl.P1, dl.P2, bits, dl.packed, dl.alpha, dl.U, dl.V, workspace=ws)
    assert bwla.bwla_check_status(ws) == 0
    gpu_codes, gpu_scales = H.fused_call_codes(bwla, ws, M, shape, bits)

    ref = oracle.linear(xb[sample], lay.P1, lay.P2, bits, dl.packed_host, lay.alpha, lay.U, lay.V)
    rep = H.check_codes(gpu_codes[sample].cpu().numpy(), gpu_scales[sample].cpu().numpy(), ref["Y"], bits)
    assert rep["mismatches"] <= max(4, rep["elements"] // 10000)
    slack = H.code_step_slack(gpu_codes[sample].cpu().numpy(), ref, lay.alpha)
    rep.update(H.check_output(H.bf16_to_host(out[sample]), ref["y"], step_slack=slack))
    assert rep["rel_l2"] <= 2e-3

    if check_acc:
        # identical codes in -> identical integer accumulators out
        qmax = (1 << (bits - 1)) - 1
        rng = np.random.default_rng([422, cfg, shape.shape_id, M, bits])
        codes_in = rng.integers(-qmax, qmax + 1, size=(M, shape.K), dtype=np.int8)
        scales_in = np.ones(M, np.float32)
        codes_in[sample] = ref["codes"]
        scales_in[sample] = ref["scales"]
        out2, acc = bwla.bwla_w1a_gemm_codes(torch.from_numpy(codes_in).cuda(), torch.from_numpy(scales_in).cuda(), bits,
                                             dl.packed, dl.alpha, xd, dl.U, dl.V, want_acc=True, workspace=ws)
        assert bwla.bwla_check_status(ws) == 0
        got = acc[sample].cpu().numpy().astype(np.int64)
        wrong = np.argwhere(got != ref["acc"])
        assert wrong.size == 0, (f"{len(wrong)} integer accumulators differ; first (sampled token, row) pairs "
                                 f"{wrong[:8].tolist()}")
        rep2 = H.check_output(H.bf16_to_host(out2[sample]), ref["y"], H.summand_magnitude(ref, lay.alpha))
        assert rep2["max_bf16_steps"] <= 1.0 + 1e-9
    print(f"\n[{shape.name} M={M} b={bits}] sampled tokens {len(sample)}, near ties {rep['near_ties']}, code mismatches "
          f"{rep['mismatches']} of {rep['elements']}, rel L2 {rep['rel_l2']:.2e}, max |err|/rms {rep['max_abs_over_rms']:.3f}, "
          f"elements over the literal 1e-2*rms bound {rep['over_literal_bound']}")
    return rep


# config 2 (Qwen3-32B shapes): index 0 q, 1 k, 2 v, 3 o, 4 gate, 5 up, 6 down
@pytest.mark.parametrize("idx,M", [(4, 2048), (6, 2048), (0, 512), (3, 512), (2, 4096), (5, 64), (1, 1), (4, 1), (6, 1)])
def test_qwen32b_shapes_sampled(bwla, idx, M):
    run_sampled_case(bwla, 2, gen.CONFIG_SHAPES[2][idx], M, 6)


# config 1 (LLaMA-2-7B shapes): index 0 qkv, 1 o, 2 gate_up, 3 down
@pytest.mark.parametrize("idx,M", [(2, 16), (2, 128), (0, 128), (3, 128), (1, 2048), (3, 2048), (2, 1)])
def test_llama7b_shapes_sampled(bwla, idx, M):
    run_sampled_case(bwla, 1, gen.CONFIG_SHAPES[1][idx], M, 6)


# config 3: down_proj with the heavier-tailed activations at every bit width
@pytest.mark.parametrize("bits,M", [(4, 32), (6, 32), (8, 32), (4, 2048), (8, 2048)])
def test_heavy_tails_sampled(bwla, bits, M):
    run_sampled_case(bwla, 3, gen.CONFIG_SHAPES[3][0], M, bits)


def test_tensor_core_path_matches_the_simple_kernel_at_full_size(bwla):
    """Every accumulator of a prefill-sized problem, not a sample: the tensor-core contraction against the
    one-warp-per-row kernel on the device (which the sampled cases above tie to the oracle)."""
    shape, M, bits = gen.CONFIG_SHAPES[2][0], 2048, 6
    lay = gen.make_layer(2, shape, bits, direct_words=True)
    dl = H.DeviceLayer(lay, bwla)
    rng = np.random.default_rng(5)
    codes = torch.from_numpy(rng.integers(-31, 32, size=(M, shape.K), dtype=np.int8)).cuda()
    scales = torch.ones(M, device="cuda")
    ws = bwla.new_workspace(M, shape.K, shape.N, 0, bits)
    assert bwla.bwla_chosen_path(M, shape.K, shape.N, 0, bits) == bwla.BWLA_PATH_I8
    _, acc = bwla.bwla_w1a_gemm_codes(codes, scales, bits, dl.packed, dl.alpha, want_out=False, want_acc=True, workspace=ws)
    bwla.bwla_force_path(bwla.BWLA_PATH_SIMPLE)
    try:
        _, acc2 = bwla.bwla_w1a_gemm_codes(codes, scales, bits, dl.packed, dl.alpha, want_out=False, want_acc=True, workspace=ws)
    finally:
        bwla.bwla_force_path(bwla.BWLA_PATH_AUTO)
    assert bwla.bwla_check_status(ws) == 0
    assert torch.equal(acc, acc2)
    # and a handful of rows against the oracle itself
    rows = [0, 127, 128, 4095, shape.N - 1]
    want = oracle.gemm(codes[:3].cpu().numpy(), dl.packed_host[rows])
    assert np.array_equal(acc[:3][:, rows].cpu().numpy().astype(np.int64), want)

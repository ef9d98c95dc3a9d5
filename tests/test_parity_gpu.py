"""Parity of the CUDA path (called through the C ABI) with the CPU oracle, element by element.

The tolerances are stated in tests/helpers.py.  All inputs are seeded and synthetic.
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


# ------------------------------------------------------------------------------------------------
# pack_signs
# ------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("N,K", [(1, 32), (5, 96), (130, 1024), (33, 11008)])
def test_pack_signs_bit_exact(bwla, N, K):
    rng = np.random.default_rng(N * 7 + K)
    W = rng.standard_normal((N, K)).astype(np.float32)
    W[0, :3] = [0.0, -0.0, np.nan]
    got = H.words_to_host(bwla.bwla_pack_signs(torch.from_numpy(W).cuda()))
    assert np.array_equal(got, oracle.pack_signs(W))
    Wb = gen.bf16_bits_from_f32(W)
    got_b = H.words_to_host(bwla.bwla_pack_signs(H.bf16_to_dev(Wb)))
    assert np.array_equal(got_b, oracle.pack_signs_bf16(Wb))


def test_pack_signs_strided_and_empty(bwla):
    W = torch.randn(7, 128, device="cuda")
    view = W[:, :64]
    got = H.words_to_host(bwla.bwla_pack_signs(view))
    assert np.array_equal(got, oracle.pack_signs(view.cpu().numpy()))
    assert bwla.bwla_pack_signs(torch.empty(0, 64, device="cuda")).shape == (0, 2)


# ------------------------------------------------------------------------------------------------
# rotate + quantise
# ------------------------------------------------------------------------------------------------
ROT_CASES = [
    # (n1, n2, M, bits)
    (32, 32, 16, 6),      # config 0
    (8, 12, 3, 6),        # n2 multiple of 4, tiny
    (4, 8, 5, 4),         # K = 32, a single word
    (32, 3, 2, 8),        # n2 not a multiple of 4: scalar contraction
    (64, 80, 9, 6),       # Qwen3 hidden 5120
    (86, 128, 4, 6),      # LLaMA down_proj, n1 not a multiple of 4
    (64, 128, 4, 8),
    (160, 160, 3, 4),     # largest K (25600)
    (64, 80, 1, 6),       # one token spread over a cluster of CTAs
    (160, 160, 1, 8),
    (86, 128, 2, 6),      # uneven row slabs
    (24, 8, 1, 6),        # slab boundaries must stay on 32-element groups
    (160, 160, 150, 6),   # many tokens of the largest K: clusters that stay and take several tokens each
    (160, 160, 41, 8),
    (128, 40, 2, 6),      # n2 a multiple of 8 but not of 16: only the first contraction on the tensor-core path
    (96, 72, 3, 8),
    (80, 64, 5, 4),       # both contractions on the tensor-core path, slab of 10 rows padded to 16
]


@pytest.mark.parametrize("n1,n2,M,bits", ROT_CASES)
def test_rotate_quant_codes_and_scales(bwla, n1, n2, M, bits):
    K = n1 * n2
    shape = gen.small_shape(K, 32, n1, n2, 0, shape_id=n1 * 1000 + n2)
    lay = gen.make_layer(0, shape, bits)
    xb = gen.make_activations(0, shape, M)
    codes, scales = bwla.bwla_rotate_quant_act(H.bf16_to_dev(xb), H.f32_to_dev(lay.P1), H.f32_to_dev(lay.P2), bits)
    Y = oracle.rotate(xb, lay.P1, lay.P2)
    rep = H.check_codes(codes.cpu().numpy(), scales.cpu().numpy(), Y, bits)
    assert rep["mismatches"] <= max(4, rep["elements"] // 10000)


def test_rotate_quant_heavy_tails_all_bit_widths(bwla):
    # config 3 recipe: Student-t nu = 2.5, 1 % of channels x100
    shape = gen.CONFIG_SHAPES[3][0]
    lay = gen.make_layer(3, shape, 6)
    xb = gen.make_activations(3, shape, 4)
    Y = oracle.rotate(xb, lay.P1, lay.P2)
    xd, P1, P2 = H.bf16_to_dev(xb), H.f32_to_dev(lay.P1), H.f32_to_dev(lay.P2)
    for bits in (4, 6, 8):
        codes, scales = bwla.bwla_rotate_quant_act(xd, P1, P2, bits)
        H.check_codes(codes.cpu().numpy(), scales.cpu().numpy(), Y, bits)


def test_rotate_quant_degenerate_rows_and_strided_input(bwla):
    n1, n2, bits = 8, 8, 6
    x = np.zeros((4, 64), np.float32)
    x[1, 5] = 3.0                                  # a single non-zero entry
    x[2, :] = 1.0                                  # constant row
    x[3, :] = np.linspace(-1, 1, 64)
    xb = gen.bf16_bits_from_f32(x)
    eye = torch.eye(8, device="cuda")
    wide = torch.zeros(4, 128, dtype=torch.bfloat16, device="cuda")
    wide[:, :64] = H.bf16_to_dev(xb)
    codes, scales = bwla.bwla_rotate_quant_act(wide[:, :64], eye, eye, bits)
    Y = oracle.rotate(xb, np.eye(8, dtype=np.float32), np.eye(8, dtype=np.float32))
    H.check_codes(codes.cpu().numpy(), scales.cpu().numpy(), Y, bits)
    assert scales[0].item() == 1.0 and int(codes[0].abs().max()) == 0
    c0, s0 = bwla.bwla_rotate_quant_act(torch.empty(0, 64, dtype=torch.bfloat16, device="cuda"), eye, eye, bits)
    assert c0.shape == (0, 64) and s0.shape == (0,)


# ------------------------------------------------------------------------------------------------
# whole layer and the contraction from given codes
# ------------------------------------------------------------------------------------------------
def _run_layer_case(bwla, cfg, shape, M, bits, with_mu=False, direct_words=False, path=None):
    lay = gen.make_layer(cfg, shape, bits, direct_words=direct_words, with_mu=with_mu)
    xb = gen.make_activations(cfg, shape, M)
    dl = H.DeviceLayer(lay, bwla)
    xd = H.bf16_to_dev(xb)
    if path is not None:
        bwla.bwla_force_path(path)
    try:
        ws = bwla.new_workspace(M, shape.K, shape.N, shape.r, bits)
        out = bwla.bwla_w1ax_linear(xd, dl.P1, dl.P2, bits, dl.packed, dl.alpha, dl.U, dl.V, dl.mu, workspace=ws)
        assert bwla.bwla_check_status(ws) == 0
        ref = oracle.linear(xb, lay.P1, lay.P2, bits, dl.packed_host, lay.alpha, lay.U, lay.V, lay.mu)
        gpu_codes, gpu_scales = H.fused_call_codes(bwla, ws, M, shape, bits)
        H.check_codes(gpu_codes.cpu().numpy(), gpu_scales.cpu().numpy(), ref["Y"], bits)
        rep = H.check_output(H.bf16_to_host(out), ref["y"], step_slack=H.code_step_slack(gpu_codes.cpu().numpy(), ref, lay.alpha, lay.mu))
        # identical codes in -> identical integer accumulators out
        codes = torch.from_numpy(ref["codes"]).cuda()
        scales = torch.from_numpy(ref["scales"]).cuda()
        out2, acc = bwla.bwla_w1a_gemm_codes(codes, scales, bits, dl.packed, dl.alpha, xd, dl.U, dl.V, dl.mu,
                                             want_acc=True, workspace=ws)
        assert bwla.bwla_check_status(ws) == 0
        got_acc = acc.cpu().numpy().astype(np.int64)
        wrong = np.argwhere(got_acc != ref["acc"])
        assert wrong.size == 0, (f"{len(wrong)} integer accumulators differ; first (token, row) pairs {wrong[:8].tolist()}, "
                                 f"row tiles {sorted(set((wrong[:, 1] // 128).tolist()))[:8]}, tokens {sorted(set(wrong[:, 0].tolist()))[:8]}, "
                                 f"differences {(got_acc - ref['acc'])[wrong[:12, 0], wrong[:12, 1]].tolist()}")
        rep2 = H.check_output(H.bf16_to_host(out2), ref["y"], H.summand_magnitude(ref, lay.alpha))
        assert rep2["max_bf16_steps"] <= 1.0 + 1e-9
    finally:
        bwla.bwla_force_path(bwla.BWLA_PATH_AUTO)
    return rep


@pytest.mark.parametrize("M", [3, 16, 130])
def test_output_of_one_layer_feeds_the_next_without_synchronisation(bwla, M):
    """Two calls on one stream, the second reading what the first writes: stream order must hold although the kernels
    are launched with programmatic overlap (a prologue that read x before the preceding kernel had finished would see
    the poison written here, or the previous round's activations)."""
    bits = 6
    shA = gen.small_shape(2048, 1024, 32, 64, 16, shape_id=71)
    shB = gen.small_shape(1024, 384, 32, 32, 16, shape_id=72)
    layA, layB = gen.make_layer(0, shA, bits), gen.make_layer(0, shB, bits)
    dA, dB = H.DeviceLayer(layA, bwla), H.DeviceLayer(layB, bwla)
    wsA = bwla.new_workspace(M, shA.K, shA.N, shA.r, bits)
    wsB = bwla.new_workspace(M, shB.K, shB.N, shB.r, bits)
    y1 = torch.empty((M, shA.N), dtype=torch.bfloat16, device="cuda")
    y2 = torch.empty((M, shB.N), dtype=torch.bfloat16, device="cuda")
    for rnd in range(3):
        xb = gen.make_activations(0, shA, M, layer=rnd)
        xd = H.bf16_to_dev(xb)
        y1.view(torch.int16).fill_(0x7FC0)          # NaN: a premature read cannot go unnoticed
        torch.cuda.synchronize()
        bwla.bwla_w1ax_linear(xd, dA.P1, dA.P2, bits, dA.packed, dA.alpha, dA.U, dA.V, dA.mu, out=y1, workspace=wsA)
        bwla.bwla_w1ax_linear(y1, dB.P1, dB.P2, bits, dB.packed, dB.alpha, dB.U, dB.V, dB.mu, out=y2, workspace=wsB)
        torch.cuda.synchronize()
        assert bwla.bwla_check_status(wsA) == 0 and bwla.bwla_check_status(wsB) == 0
        y1_bits = H.bf16_to_host(y1)
        refA = oracle.linear(xb, layA.P1, layA.P2, bits, dA.packed_host, layA.alpha, layA.U, layA.V, layA.mu)
        H.check_output(y1_bits, refA["y"])
        # the second layer is judged on the activations it was really given
        refB = oracle.linear(y1_bits, layB.P1, layB.P2, bits, dB.packed_host, layB.alpha, layB.U, layB.V, layB.mu)
        H.check_output(H.bf16_to_host(y2), refB["y"])


@pytest.mark.parametrize("N,K,n1,n2", [(5120, 8192, 64, 128), (3328, 5120, 64, 80), (2944, 6144, 64, 96), (2560, 7168, 64, 112)])
def test_few_tokens_odd_k_splits(bwla, N, K, n1, n2):
    """Row-tile counts for which the contraction splits K three, five, six and seven ways (clusters of that size)."""
    shape = gen.small_shape(K, N, n1, n2, 16, shape_id=N + K)
    _run_layer_case(bwla, 0, shape, 16, 6, direct_words=True)
    _run_layer_case(bwla, 0, shape, 5, 8, direct_words=True, with_mu=True)


def test_config0_single_w1a6_linear(bwla):
    rep = _run_layer_case(bwla, 0, gen.CONFIG_SHAPES[0][0], 16, 6)
    assert rep["rel_l2"] <= 2e-3


@pytest.mark.parametrize("K,N,n1,n2,r,M,bits", [
    (96, 40, 8, 12, 4, 3, 6),        # ragged everything
    (32, 1, 4, 8, 0, 1, 8),          # one word, one row, one token, no low-rank branch
    (256, 130, 16, 16, 8, 17, 4),    # N and M straddle tile edges
    (1024, 300, 32, 32, 16, 70, 6),
    (2048, 129, 32, 64, 0, 9, 8),
])
def test_small_and_ragged_shapes(bwla, K, N, n1, n2, r, M, bits):
    _run_layer_case(bwla, 0, gen.small_shape(K, N, n1, n2, r, shape_id=K + N), M, bits)


@pytest.mark.parametrize("K,N,n1,n2,r,M,bits", [
    (96, 40, 8, 12, 4, 3, 6),        # three sign words per row, ragged rows, three tokens in a four-token kernel
    (32, 1, 4, 8, 0, 1, 8),          # one word, one row, one token
    (1024, 300, 32, 32, 16, 4, 4),
    (2048, 129, 32, 64, 0, 2, 8),
    (1056, 77, 32, 33, 8, 2, 6),     # 33 sign words: the second chunk of word positions holds a single word
])
def test_bitplane_path_small_and_ragged_shapes(bwla, K, N, n1, n2, r, M, bits):
    _run_layer_case(bwla, 0, gen.small_shape(K, N, n1, n2, r, shape_id=K + N), M, bits, with_mu=(r == 16),
                    path=bwla.BWLA_PATH_BITPLANE)


@pytest.mark.parametrize("idx,M,bits", [(4, 1, 6), (6, 1, 6), (1, 2, 6), (6, 4, 4), (0, 1, 8), (6, 2, 8)])
def test_bitplane_path_qwen32b_shapes(bwla, idx, M, bits):
    _run_layer_case(bwla, 2, gen.CONFIG_SHAPES[2][idx], M, bits, direct_words=True, path=bwla.BWLA_PATH_BITPLANE)


def test_path_choice_follows_the_measured_table(bwla):
    """The tcgen05 kernel wherever it can run (it was measured faster at every token count on the workload shapes); a few
    tokens of a shape it cannot take go to the bit-plane kernel, more tokens to the simple one."""
    sh = gen.CONFIG_SHAPES[2][4]
    for M in (1, 16, 2048):
        assert bwla.bwla_chosen_path(M, sh.K, sh.N, sh.r, 6) == bwla.BWLA_PATH_I8
    assert bwla.bwla_chosen_path(2, 1056, 77, 8, 6) == bwla.BWLA_PATH_BITPLANE      # K % 128 != 0
    assert bwla.bwla_chosen_path(9, 1056, 77, 8, 6) == bwla.BWLA_PATH_SIMPLE


def test_mu_shift_is_applied(bwla):
    _run_layer_case(bwla, 0, gen.small_shape(512, 96, 16, 32, 8, shape_id=5), 6, 6, with_mu=True)


@pytest.mark.parametrize("idx,M", [(0, 16), (1, 1), (3, 16)])
def test_llama7b_shapes(bwla, idx, M):
    _run_layer_case(bwla, 1, gen.CONFIG_SHAPES[1][idx], M, 6)


@pytest.mark.parametrize("idx,M", [(0, 8), (1, 64), (3, 8), (6, 8)])
def test_qwen32b_shapes(bwla, idx, M):
    _run_layer_case(bwla, 2, gen.CONFIG_SHAPES[2][idx], M, 6, direct_words=True)


def test_blocks_that_split_k_for_the_low_rank_term_give_the_same_bits_every_time(bwla):
    """down_proj at 16 tokens: several blocks share a tile of T = V x, each takes a part of K, and whichever arrives
    last adds the parts in the order of K.  The result must not depend on the order of arrival, and the arrival
    counters in the workspace must be back at zero for the next call."""
    shape = gen.CONFIG_SHAPES[2][6]
    _run_layer_case(bwla, 2, shape, 16, 6, direct_words=True)
    lay = gen.make_layer(2, shape, 6, direct_words=True)
    dl = H.DeviceLayer(lay, bwla)
    xd = H.bf16_to_dev(gen.make_activations(2, shape, 16))
    ws = bwla.new_workspace(16, shape.K, shape.N, shape.r, 6)
    first = None
    for _ in range(8):
        out = bwla.bwla_w1ax_linear(xd, dl.P1, dl.P2, 6, dl.packed, dl.alpha, dl.U, dl.V, dl.mu, workspace=ws)
        bits = H.bf16_to_host(out)
        if first is None:
            first = bits
        assert np.array_equal(bits, first)
    assert bwla.bwla_check_status(ws) == 0
    assert int(ws[:256].view(torch.int32).abs().sum().item()) == 0      # status words, counters included, are zero again


@pytest.mark.parametrize("bits", [4, 6, 8])
def test_bit_width_sweep_down_proj(bwla, bits):
    _run_layer_case(bwla, 3, gen.CONFIG_SHAPES[3][0], 1, bits, direct_words=True)


def test_accumulators_stay_exact_when_the_gpu_was_idle_before_the_call(bwla):
    """A cold start (idle clocks, slow first copies) shifts the relative timing of the weight stream, the expansion and
    the MMAs inside the contraction; the integer accumulators must not depend on it."""
    import time
    shape = gen.CONFIG_SHAPES[1][0]
    lay = gen.make_layer(1, shape, 6)
    xb = gen.make_activations(1, shape, 16)
    dl = H.DeviceLayer(lay, bwla)
    xd = H.bf16_to_dev(xb)
    Y = oracle.rotate(xb, lay.P1, lay.P2)
    q = oracle.quantize(Y, 6, "f64")
    want = oracle.gemm(q["codes"], dl.packed_host)
    codes, scales = torch.from_numpy(q["codes"]).cuda(), torch.from_numpy(q["scales"]).cuda()
    ws = bwla.new_workspace(16, shape.K, shape.N, shape.r, 6)
    for _ in range(6):
        time.sleep(0.3)
        _, acc = bwla.bwla_w1a_gemm_codes(codes, scales, 6, dl.packed, dl.alpha, xd, dl.U, dl.V, want_out=False,
                                          want_acc=True, workspace=ws)
        assert bwla.bwla_check_status(ws) == 0
        assert np.array_equal(acc.cpu().numpy().astype(np.int64), want)


def test_a_set_status_word_is_reported_cleared_and_the_next_call_is_clean(bwla):
    """The device-timeout path without making any wait run long: a bounded wait that gives up sets the workspace
    status word, and a call that finds the word set skips its work.  Here the word is set by the test; the call must
    leave the context usable, bwla_check_status must report and clear the condition, and the next call must match
    the oracle."""
    shape = gen.CONFIG_SHAPES[0][0]
    lay = gen.make_layer(0, shape, 6)
    xb = gen.make_activations(0, shape, 16)
    dl = H.DeviceLayer(lay, bwla)
    xd = H.bf16_to_dev(xb)
    ws = bwla.new_workspace(16, shape.K, shape.N, shape.r, 6)
    ws[:4].view(torch.int32)[0] = 1
    bwla.bwla_w1ax_linear(xd, dl.P1, dl.P2, 6, dl.packed, dl.alpha, dl.U, dl.V, workspace=ws)
    assert bwla.bwla_check_status(ws) == bwla.BWLA_ERR_DEVICE_TIMEOUT
    assert bwla.bwla_check_status(ws) == 0                      # reading it cleared it
    out = bwla.bwla_w1ax_linear(xd, dl.P1, dl.P2, 6, dl.packed, dl.alpha, dl.U, dl.V, workspace=ws)
    assert bwla.bwla_check_status(ws) == 0
    ref = oracle.linear(xb, lay.P1, lay.P2, 6, dl.packed_host, lay.alpha, lay.U, lay.V)
    H.check_output(H.bf16_to_host(out), ref["y"])


def test_accumulator_range_guard_of_the_tensor_core_path(bwla):
    """The tensor core sums -128 * code over the set sign bits; where 128 * K * 2^(b-1) could leave int32 the shape
    must go to the simple kernel."""
    assert bwla.bwla_chosen_path(16, 130944, 1024, 0, 8) == bwla.BWLA_PATH_I8      # 128 * K * 128 < 2^31
    assert bwla.bwla_chosen_path(16, 131072, 1024, 0, 8) == bwla.BWLA_PATH_SIMPLE  # ... = 2^31
    assert bwla.bwla_chosen_path(16, 131072, 1024, 0, 6) == bwla.BWLA_PATH_I8      # 6-bit codes leave room


def test_empty_batch_and_argument_errors(bwla):
    shape = gen.small_shape(64, 16, 8, 8, 0)
    lay = gen.make_layer(0, shape, 6)
    dl = H.DeviceLayer(lay, bwla)
    x0 = torch.empty(0, 64, dtype=torch.bfloat16, device="cuda")
    ws = bwla.new_workspace(1, 64, 16, 0, 6)
    assert bwla.bwla_w1ax_linear(x0, dl.P1, dl.P2, 6, dl.packed, dl.alpha, workspace=ws).shape == (0, 16)
    x = H.bf16_to_dev(gen.make_activations(0, shape, 2))
    with pytest.raises(bwla.BwlaError) as e:
        bwla.bwla_w1ax_linear(x, dl.P1, dl.P2, 5, dl.packed, dl.alpha, workspace=ws)     # bits not in {4,6,8}
    assert e.value.status == bwla.BWLA_ERR_INVALID_ARG
    with pytest.raises(bwla.BwlaError) as e:
        bwla.bwla_w1ax_linear(x, dl.P1, dl.P2[:4, :4].contiguous(), 6, dl.packed, dl.alpha, workspace=ws)  # K != n1*n2
    assert e.value.status == bwla.BWLA_ERR_INVALID_ARG
    with pytest.raises(bwla.BwlaError) as e:
        bwla.bwla_w1ax_linear(x, dl.P1, dl.P2, 6, dl.packed, dl.alpha, workspace=ws[:256])  # workspace too small
    assert e.value.status == bwla.BWLA_ERR_WORKSPACE
    # the context is still healthy
    out = bwla.bwla_w1ax_linear(x, dl.P1, dl.P2, 6, dl.packed, dl.alpha, workspace=bwla.new_workspace(2, 64, 16, 0, 6))
    torch.cuda.synchronize()
    assert out.shape == (2, 16)

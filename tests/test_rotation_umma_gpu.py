"""The tcgen05 rotation + quantiser (reached through prepared layers) against the CPU oracle, in three stages:

  (A) the rotated activations the kernel hands out, against the oracle's fp64 rotation: the error must stay below
      the code window, 1e-6 of the token's full scale (the tensor core adds each group of 16 products into its fp32
      accumulator with truncation, about half an ulp of the running sum per step, so the error grows with n1 + n2:
      2e-7 at 32 x 32, 7e-7 at 160 x 160);
  (B) the oracle's quantiser with the fp32 decision rule, applied to the GPU's own Y, must give the GPU's codes and
      scales exactly: the quantiser itself is then tested bit for bit, whatever the rotation error;
  (C) the GPU codes against the fp64 definition, with the near-tie rule of tests/helpers.py.

And grouped calls (several layers reading one x) against the oracle layer by layer.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_00422_b200 import inputs as gen
from tests import helpers as H
from tests.test_parity_gpu import ROT_CASES

pytestmark = pytest.mark.gpu

# factor sizes the tensor-core kernel takes: n2 a multiple of 8
UMMA_CASES = [c for c in ROT_CASES if c[1] % 8 == 0] + [
    (64, 80, 300, 6),     # more tokens than SMs: CTAs stay and take tokens in turn
    (64, 64, 130, 6),     # LLaMA hidden size
    (86, 128, 160, 6),
    (160, 160, 75, 6),    # clusters of four per token, two tokens per cluster and a ragged tail
    (16, 16, 7, 8),       # a single 16-column chunk
    (192, 8, 3, 6),       # the widest n1, the narrowest n2
    (40, 200, 5, 4),      # two lane tiles of 104 + 96 rows
]


@pytest.fixture(scope="module")
def bwla():
    from paper_2605_00422_b200 import bwla as b
    b.bwla_force_path(b.BWLA_PATH_AUTO)
    b.bwla_force_rotation(b.BWLA_ROT_AUTO)
    return b


def _layer_for_rotation(bwla, lay, shape, bits):
    packed = torch.zeros((8, shape.K // 32), dtype=torch.int32, device="cuda")
    alpha = torch.ones(8, device="cuda")
    return bwla.Layer(H.f32_to_dev(lay.P1), H.f32_to_dev(lay.P2), bits, packed, alpha)


@pytest.mark.parametrize("n1,n2,M,bits", UMMA_CASES)
def test_rotation_stages_a_b_c(bwla, n1, n2, M, bits):
    K = n1 * n2
    shape = gen.small_shape(K, 32, n1, n2, 0, shape_id=n1 * 1000 + n2)
    lay = gen.make_layer(0, shape, bits)
    xb = gen.make_activations(0, shape, M)
    L = _layer_for_rotation(bwla, lay, shape, bits)
    codes, scales, y = bwla.bwla_layer_rotate_quant(L, H.bf16_to_dev(xb), want_y=True)
    torch.cuda.synchronize()
    codes, scales, y = codes.cpu().numpy(), scales.cpu().numpy(), y.cpu().numpy().astype(np.float64)
    Y = oracle.rotate(xb, lay.P1, lay.P2)
    # (A)
    amax = np.abs(Y).max(axis=1, keepdims=True)
    amax[amax == 0] = 1.0
    rel = float((np.abs(y - Y) / amax).max())
    assert rel <= 9e-7, f"rotation error {rel:.2e} of the token's full scale"
    # (B)
    q32 = oracle.quantize(y, bits, "f32")
    assert np.array_equal(q32["codes"], codes)
    assert np.array_equal(q32["scales"], scales)
    # (C)
    rep = H.check_codes(codes, scales, Y, bits)
    assert rep["mismatches"] <= max(4, rep["elements"] // 10000)
    print(f"\n[{n1}x{n2} M={M} b={bits}] rotation error {rel:.2e} of full scale, near ties {rep['near_ties']}, "
          f"mismatches {rep['mismatches']} of {rep['elements']}")


def test_forced_rotation_kernels_agree_with_the_oracle(bwla):
    """Both rotation kernels behind bwla_w1ax_linear on the same problem."""
    shape = gen.CONFIG_SHAPES[2][1]
    lay = gen.make_layer(2, shape, 6, direct_words=True)
    xb = gen.make_activations(2, shape, 24)
    dl = H.DeviceLayer(lay, bwla)
    ref = oracle.linear(xb, lay.P1, lay.P2, 6, dl.packed_host, lay.alpha, lay.U, lay.V)
    try:
        for which in (bwla.BWLA_ROT_SIMT, bwla.BWLA_ROT_UMMA):
            bwla.bwla_force_rotation(which)
            ws = bwla.new_workspace(24, shape.K, shape.N, shape.r, 6)
            out = bwla.bwla_w1ax_linear(H.bf16_to_dev(xb), dl.P1, dl.P2, 6, dl.packed, dl.alpha, dl.U, dl.V, workspace=ws)
            assert bwla.bwla_check_status(ws) == 0
            c, s = H.fused_call_codes(bwla, ws, 24, shape, 6)
            H.check_codes(c.cpu().numpy(), s.cpu().numpy(), ref["Y"], 6)
            H.check_output(H.bf16_to_host(out), ref["y"])
    finally:
        bwla.bwla_force_rotation(bwla.BWLA_ROT_AUTO)


@pytest.mark.parametrize("idxs,M", [((0, 1, 2), 16), ((4, 5), 16), ((4, 5), 1), ((0, 1, 2), 200), ((6,), 16), ((3,), 5)])
def test_grouped_layers_match_the_oracle_layer_by_layer(bwla, idxs, M):
    """q/k/v and gate/up of the Qwen3-32B shapes through bwla_w1ax_linear_group: one x, one rotation launch, every
    layer's output against its own oracle result."""
    bits = 6
    shapes = [gen.CONFIG_SHAPES[2][i] for i in idxs]
    lays = [gen.make_layer(2, sh, bits, direct_words=True) for sh in shapes]
    xb = gen.make_activations(2, shapes[0], M)
    dls = [H.DeviceLayer(l, bwla) for l in lays]
    layers = [bwla.Layer(d.P1, d.P2, bits, d.packed, d.alpha, d.U, d.V) for d in dls]
    ws = bwla.new_group_workspace(layers, M)
    outs = bwla.bwla_w1ax_linear_group(layers, H.bf16_to_dev(xb), workspace=ws)
    assert bwla.bwla_check_status(ws) == 0
    for lay, d, out in zip(lays, dls, outs):
        ref = oracle.linear(xb, lay.P1, lay.P2, bits, d.packed_host, lay.alpha, lay.U, lay.V)
        rep = H.check_output(H.bf16_to_host(out), ref["y"])
        assert rep["rel_l2"] <= 2e-3
    # the same call again on the same workspace gives the same bits
    outs2 = bwla.bwla_w1ax_linear_group(layers, H.bf16_to_dev(xb), workspace=ws)
    assert bwla.bwla_check_status(ws) == 0
    for a, b in zip(outs, outs2):
        assert torch.equal(a.view(torch.int16), b.view(torch.int16))


# ------------------------------------------------------------------------------------------------
# per-token asymmetric quantiser (the paper's stated setting, Sec. 4.1)
# ------------------------------------------------------------------------------------------------
def _check_asym_codes(u, s, z, Y, bits):
    """GPU codes / scales / zero points against the oracle's fp64 definition: what a code stands for, u - z, must agree
    except at flagged near-ties (+-1); where the zero point itself sat on a rounding boundary the two may be shifted
    against each other, which only shows at the clamped ends of the range."""
    ref = oracle.quantize_asym(Y, bits, "f64")
    L = (1 << bits) - 1
    window = oracle.near_tie_window_asym(bits)
    r_gpu = u.astype(np.int32) - z.astype(np.int32)[:, None]
    r_ref = ref["codes"].astype(np.int32) - ref["zeros"].astype(np.int32)[:, None]
    bad = r_gpu != r_ref
    assert np.all(np.abs(r_gpu - r_ref)[bad] == 1), "a code differs from the oracle by more than one step"
    zero_moved = z != ref["zeros"]
    assert np.all(ref["dist_zero"][zero_moved] <= window), "a zero point differs away from a rounding boundary"
    at_clamp = (ref["codes"] == 0) | (ref["codes"] == L) | (u == 0) | (u == L)
    excused = (ref["dist"] <= window) | (zero_moved[:, None] & at_clamp)
    assert not (bad & ~excused).any(), f"{int((bad & ~excused).sum())} code mismatches outside the near-tie window"
    assert np.all(np.abs(s.astype(np.float64) - ref["scales"]) <= 2e-6 * ref["scales"])
    return {"mismatches": int(bad.sum()), "near_ties": int((ref["dist"] <= window).sum()), "zero_moved": int(zero_moved.sum())}


@pytest.mark.parametrize("n1,n2,M,bits", [(32, 32, 16, 6), (64, 80, 9, 6), (64, 80, 200, 8), (86, 128, 4, 4), (160, 160, 5, 6),
                                         (160, 160, 80, 8), (4, 8, 5, 4)])
def test_asymmetric_quantiser_stages_b_and_c(bwla, n1, n2, M, bits):
    K = n1 * n2
    shape = gen.small_shape(K, 32, n1, n2, 0, shape_id=n1 * 1000 + n2)
    lay = gen.make_layer(0, shape, bits)
    xb = gen.make_activations(0, shape, M)
    xb[0] = gen.bf16_bits_from_f32(np.abs(gen.f32_from_bf16_bits(xb[0])))      # a row whose mean is far from zero
    if M > 2:
        xb[2] = 0                                                              # an all-zero row
    L = _layer_for_rotation(bwla, lay, shape, bits)
    u, s, z, y = bwla.bwla_layer_rotate_quant_asym(L, H.bf16_to_dev(xb), want_y=True)
    torch.cuda.synchronize()
    u, s, z, y = u.cpu().numpy(), s.cpu().numpy(), z.cpu().numpy(), y.cpu().numpy().astype(np.float64)
    # (B) the oracle's quantiser with the fp32 decision rule on the GPU's own Y: bit for bit
    q32 = oracle.quantize_asym(y, bits, "f32")
    assert np.array_equal(q32["codes"], u) and np.array_equal(q32["zeros"], z) and np.array_equal(q32["scales"], s)
    # (C) against the fp64 definition on the oracle's rotation
    rep = _check_asym_codes(u, s, z, oracle.rotate(xb, lay.P1, lay.P2), bits)
    print(f"\\n[asym {n1}x{n2} M={M} b={bits}] {rep}")


@pytest.mark.parametrize("idxs,M,bits,path", [((0, 1, 2), 16, 6, None), ((4, 5), 3, 8, None), ((6,), 16, 6, None), ((3,), 130, 6, None),
                                              ((1,), 2, 6, "bitplane"), ((1,), 5, 8, "simple")])
def test_asymmetric_layers_match_the_oracle(bwla, idxs, M, bits, path):
    shapes = [gen.CONFIG_SHAPES[2][i] for i in idxs]
    lays = [gen.make_layer(2, sh, bits, direct_words=True, with_mu=(i == 0)) for i, sh in enumerate(shapes)]
    xb = gen.make_activations(2, shapes[0], M)
    xb[0] = gen.bf16_bits_from_f32(np.abs(gen.f32_from_bf16_bits(xb[0])))
    dls = [H.DeviceLayer(l, bwla) for l in lays]
    layers = [bwla.Layer(d.P1, d.P2, bits, d.packed, d.alpha, d.U, d.V, d.mu, asymmetric=True) for d in dls]
    if path:
        bwla.bwla_force_path({"bitplane": bwla.BWLA_PATH_BITPLANE, "simple": bwla.BWLA_PATH_SIMPLE}[path])
    try:
        ws = bwla.new_group_workspace(layers, M)
        outs = bwla.bwla_w1ax_linear_group(layers, H.bf16_to_dev(xb), workspace=ws)
        assert bwla.bwla_check_status(ws) == 0
    finally:
        bwla.bwla_force_path(bwla.BWLA_PATH_AUTO)
    for lay, d, out in zip(lays, dls, outs):
        ref = oracle.linear_asym(xb, lay.P1, lay.P2, bits, d.packed_host, lay.alpha, lay.U, lay.V, lay.mu)
        # a code one step off at a near-tie moves the token's outputs by (|alpha| + |mu|) * s_t: the standalone entry
        # gives this layer's codes (same kernel, same arithmetic)
        u, s, z, _ = bwla.bwla_layer_rotate_quant_asym(layers[lays.index(lay)], H.bf16_to_dev(xb))
        r_gpu = u.cpu().numpy().astype(np.int32) - z.cpu().numpy().astype(np.int32)[:, None]
        r_ref = ref["codes"].astype(np.int32) - ref["zeros"].astype(np.int32)[:, None]
        flips = np.abs(r_gpu - r_ref).sum(axis=1).astype(np.float64)
        per_row = np.abs(lay.alpha.astype(np.float64)) + (0.0 if lay.mu is None else np.abs(lay.mu.astype(np.float64)))
        slack = flips[:, None] * per_row[None, :] * ref["scales"].astype(np.float64)[:, None]
        rep = H.check_output(H.bf16_to_host(out), ref["y"], step_slack=slack)
        assert rep["rel_l2"] <= 2e-3


def test_group_workspace_needs_only_its_first_256_bytes_zeroed(bwla):
    """The arrival counters of every layer's split sums of T live in the first status block: a workspace that is garbage
    behind its first 256 bytes gives the same outputs as a zero-filled one (K = 25600 and 8192 split K at 16 tokens)."""
    for idxs in ((6,), (3,), (0, 1, 2)):
        shapes = [gen.CONFIG_SHAPES[2][i] for i in idxs]
        lays = [gen.make_layer(2, sh, 6, direct_words=True) for sh in shapes]
        dls = [H.DeviceLayer(l, bwla) for l in lays]
        layers = [bwla.Layer(d.P1, d.P2, 6, d.packed, d.alpha, d.U, d.V) for d in dls]
        x = H.bf16_to_dev(gen.make_activations(2, shapes[0], 16))
        clean = bwla.new_group_workspace(layers, 16)
        outs_a = bwla.bwla_w1ax_linear_group(layers, x, workspace=clean)
        dirty = torch.randint(0, 256, (clean.numel(),), dtype=torch.uint8, device="cuda")
        dirty[:256] = 0
        outs_b = bwla.bwla_w1ax_linear_group(layers, x, workspace=dirty)
        assert bwla.bwla_check_status(dirty) == 0
        for a, b in zip(outs_a, outs_b):
            assert torch.equal(a, b)


def test_outputs_of_one_group_feed_the_next_group_without_synchronisation(bwla):
    """q/k/v run beside one another (the siblings of a group do not wait for each other); the next group reads q's
    output as its x right behind them on the same stream.  The result must not depend on host synchronisation."""
    M = 16
    sq, sk, sv, so = (gen.CONFIG_SHAPES[2][i] for i in (0, 1, 2, 3))
    assert sq.N == so.K
    lays = [gen.make_layer(2, sh, 6, direct_words=True) for sh in (sq, sk, sv, so)]
    dls = [H.DeviceLayer(l, bwla) for l in lays]
    L = [bwla.Layer(d.P1, d.P2, 6, d.packed, d.alpha, d.U, d.V) for d in dls]
    x = H.bf16_to_dev(gen.make_activations(2, sq, M))
    ws1 = bwla.new_group_workspace(L[:3], M)
    ws2 = bwla.new_group_workspace(L[3:], M)

    def run(sync):
        outs = bwla.bwla_w1ax_linear_group(L[:3], x, workspace=ws1)
        if sync:
            torch.cuda.synchronize()
        y = bwla.bwla_w1ax_linear_group(L[3:], outs[0], workspace=ws2)[0]
        torch.cuda.synchronize()
        return [o.clone() for o in outs] + [y.clone()]

    want = run(True)
    for _ in range(5):
        got = run(False)
        for a, b in zip(want, got):
            assert torch.equal(a, b)
    assert bwla.bwla_check_status(ws1) == 0 and bwla.bwla_check_status(ws2) == 0

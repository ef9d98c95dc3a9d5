"""Pins for the CPU oracle: what the paper and the mathematics fix, with no implementation to lean on.

Each test compares the oracle with something other than itself: a brute-force dense Kronecker product, a
closed form, an exact special case, an independent library routine, or a value the paper states.
"""
import os

import numpy as np
import pytest

import oracle
from paper_2605_00422_b200 import inputs as gen

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _bf16(a):
    return gen.bf16_bits_from_f32(np.asarray(a, np.float32))


def _orth(n, seed):
    return gen.orthogonal_f32(n, np.random.default_rng(seed))


# ----------------------------------------------------------------------------------------------
# O1: Kronecker rotation (Sec. 3.1 OKT; App. A.2 Kronecker identity)
# ----------------------------------------------------------------------------------------------
@pytest.mark.parametrize("n1,n2", [(1, 1), (2, 3), (3, 2), (4, 4), (5, 8), (8, 5)])
def test_rotation_matches_dense_kronecker(n1, n2):
    rng = np.random.default_rng(10 * n1 + n2)
    P1 = rng.standard_normal((n1, n1)).astype(np.float32)   # need not be orthogonal for the identity
    P2 = rng.standard_normal((n2, n2)).astype(np.float32)
    xb = _bf16(rng.standard_normal((3, n1 * n2)))
    x = gen.f32_from_bf16_bits(xb).astype(np.float64)
    Y = oracle.rotate(xb, P1, P2)
    R = np.kron(P1.astype(np.float64), P2.astype(np.float64))   # R[a*n2+b, c*n2+d] = P1[a,c] P2[b,d]
    for t in range(3):
        dense = R.T @ x[t]                                       # (P1 (x) P2)^T vec_rowmajor(X)
        np.testing.assert_allclose(Y[t], dense, rtol=0, atol=1e-13 * max(1.0, np.abs(dense).max()))
        # and the same thing as two small contractions written with einsum
        X = x[t].reshape(n1, n2)
        two = np.einsum("ac,ab,bd->cd", P1.astype(np.float64), X, P2.astype(np.float64)).reshape(-1)
        np.testing.assert_allclose(Y[t], two, rtol=0, atol=1e-13 * max(1.0, np.abs(two).max()))


def test_rotation_preserves_norm_for_orthogonal_factors():
    P1, P2 = _orth(16, 1), _orth(24, 2)
    xb = _bf16(np.random.default_rng(3).standard_t(3, size=(5, 16 * 24)))
    x = gen.f32_from_bf16_bits(xb).astype(np.float64)
    Y = oracle.rotate(xb, P1, P2)
    np.testing.assert_allclose(np.linalg.norm(Y, axis=1), np.linalg.norm(x, axis=1), rtol=1e-6)


def test_identity_rotation_is_a_noop():
    xb = _bf16(np.random.default_rng(4).standard_normal((4, 6 * 10)))
    Y = oracle.rotate(xb, np.eye(6, dtype=np.float32), np.eye(10, dtype=np.float32))
    assert np.array_equal(Y, gen.f32_from_bf16_bits(xb).astype(np.float64))


def test_forward_equivalence_fixes_direction_and_factor_order():
    # W x = (W R)(R^T x) with R = P1 (x) P2 (Sec. 1; Sec. 3.1): a swap of R and R^T or of P1 and P2 breaks it.
    n1, n2, N = 6, 10, 7
    P1, P2 = _orth(n1, 5), _orth(n2, 6)
    rng = np.random.default_rng(7)
    W = rng.standard_normal((N, n1 * n2))
    xb = _bf16(rng.standard_normal((2, n1 * n2)))
    x = gen.f32_from_bf16_bits(xb).astype(np.float64)
    R = np.kron(P1.astype(np.float64), P2.astype(np.float64))
    Wrot = W @ R
    Y = oracle.rotate(xb, P1, P2)
    lhs = Y @ Wrot.T
    exact = x @ (R @ R.T) @ W.T          # what the identity gives with fp32-rounded (almost orthogonal) factors
    np.testing.assert_allclose(lhs, exact, rtol=0, atol=1e-12)
    np.testing.assert_allclose(lhs, x @ W.T, rtol=0, atol=1e-5)
    # the wrong direction is far away
    wrong = oracle.rotate(xb, P1.T.copy(), P2.T.copy()) @ Wrot.T
    assert np.abs(wrong - x @ W.T).max() > 1e-2


# ----------------------------------------------------------------------------------------------
# O2: per-token symmetric quantiser
# ----------------------------------------------------------------------------------------------
@pytest.mark.parametrize("bits", [4, 6, 8])
@pytest.mark.parametrize("decision", ["f64", "f32"])
def test_quantiser_invariants(bits, decision):
    qmax = (1 << (bits - 1)) - 1
    rng = np.random.default_rng(bits)
    Y = rng.standard_t(3, size=(6, 257)).astype(np.float32).astype(np.float64)
    q = oracle.quantize(Y, bits, decision)
    codes, scales = q["codes"].astype(np.int64), q["scales"].astype(np.float64)
    assert codes.min() >= -qmax and codes.max() <= qmax
    for t in range(Y.shape[0]):
        k = int(np.argmax(np.abs(Y[t])))
        assert abs(codes[t, k]) == qmax and np.sign(codes[t, k]) == np.sign(Y[t, k])
        np.testing.assert_allclose(scales[t], np.abs(Y[t]).max() / qmax, rtol=2e-7)
        assert np.all(np.abs(Y[t] - scales[t] * codes[t]) <= 0.5 * scales[t] * (1 + 1e-5))
    assert np.array_equal(q["qsum"], codes.sum(axis=1))
    # idempotence: quantising the dequantised grid points gives the same codes
    grid = (scales[:, None] * codes).astype(np.float64)
    assert np.array_equal(oracle.quantize(grid, bits, "f64")["codes"], q["codes"])


@pytest.mark.parametrize("bits", [4, 6, 8])
@pytest.mark.parametrize("decision", ["f64", "f32"])
def test_quantiser_ties_go_to_even_and_zero_row(bits, decision):
    qmax = (1 << (bits - 1)) - 1
    # amax = qmax makes the scale exactly 1, so t = y and the halves are exact ties
    y = np.array([[qmax, 0.5, 1.5, 2.5, 3.5, -0.5, -1.5, -2.5, -3.5, 0.49999, 0.50001, -qmax],
                  [0.0] * 12], np.float64)
    q = oracle.quantize(y, bits, decision)
    assert q["codes"][0].tolist() == [qmax, 0, 2, 2, 4, 0, -2, -2, -4, 0, 1, -qmax]
    assert q["scales"][0] == 1.0
    assert np.all(q["dist"][0, 1:9] == 0.0) and q["dist"][0, 9] > 0
    assert q["codes"][1].tolist() == [0] * 12 and q["scales"][1] == 1.0


def test_quantiser_clamps_to_restricted_range():
    # the most negative two's-complement code is never produced
    y = np.array([[-1.0, 1.0, -0.999999, 0.3]], np.float64)
    for bits in (4, 6, 8):
        qmax = (1 << (bits - 1)) - 1
        c = oracle.quantize(y, bits)["codes"][0]
        assert c[0] == -qmax and c[1] == qmax and c.min() == -qmax


# ----------------------------------------------------------------------------------------------
# O3: sign convention and packing (Eq. 2-3)
# ----------------------------------------------------------------------------------------------
def test_pack_unpack_follow_the_sign_rule():
    rng = np.random.default_rng(8)
    W = rng.standard_normal((5, 96)).astype(np.float32)
    W[0, :4] = [0.0, -0.0, np.nan, 1e-45]         # Sign(x) = +1 iff x > 0
    W[1, :] = 0.0
    W[1, 37] = 2.0                                # one-hot row: bit 5 of word 1
    packed = oracle.pack_signs(W)
    s = oracle.unpack_signs(packed, 96)
    with np.errstate(invalid="ignore"):
        expect = np.where(W > 0, 1, -1).astype(np.int8)
    assert np.array_equal(s, expect)
    assert s[0, :4].tolist() == [-1, -1, -1, 1]
    assert packed[1].tolist() == [0, 1 << 5, 0]
    # LSB-first, 32 weights per word, written independently with numpy
    bits = (expect > 0).astype(np.uint64).reshape(5, 3, 32)
    words = (bits << np.arange(32, dtype=np.uint64)).sum(axis=2).astype(np.uint32)
    assert np.array_equal(packed, words)
    assert np.array_equal(oracle.pack_signs_bf16(_bf16(W)), oracle.pack_signs(gen.f32_from_bf16_bits(_bf16(W))))


# ----------------------------------------------------------------------------------------------
# weight format: alpha = mean|w| minimises the binarisation error (Eq. 1; App. "double-bell")
# ----------------------------------------------------------------------------------------------
def test_alpha_is_mean_abs_and_error_is_m_var_abs():
    rng = np.random.default_rng(9)
    W = rng.standard_normal((4, 200)).astype(np.float32)
    mu, delta = oracle.row_stats(W, centre=False)
    assert np.all(mu == 0)
    Wd = W.astype(np.float64)
    for n in range(4):
        w = Wd[n]
        s = np.where(w > 0, 1.0, -1.0)
        grid = np.linspace(0, 3, 30001)
        err = ((w[None, :] - grid[:, None] * s[None, :]) ** 2).sum(axis=1)
        assert abs(grid[err.argmin()] - delta[n]) <= 1e-4
        best = ((w - delta[n] * s) ** 2).sum()
        np.testing.assert_allclose(best, w.size * np.var(np.abs(w)), rtol=1e-12)
        assert best <= err.min() + 1e-9
    # centred variant is Eq. 1 as printed
    mu_c, delta_c = oracle.row_stats(W, centre=True)
    np.testing.assert_allclose(mu_c, Wd.mean(axis=1), rtol=0, atol=1e-15)
    np.testing.assert_allclose(delta_c, np.abs(Wd - Wd.mean(axis=1, keepdims=True)).mean(axis=1), rtol=1e-14)


def test_two_valued_row_is_recovered_exactly():
    c = np.float32(0.37)
    s = np.where(np.random.default_rng(10).random(64) > 0.5, 1.0, -1.0).astype(np.float32)
    W = (c * s)[None, :]
    _, delta = oracle.row_stats(W, centre=False)
    sign = oracle.unpack_signs(oracle.pack_signs(W), 64)[0]
    assert np.array_equal(delta[0] * sign, W[0].astype(np.float64)) or \
        np.allclose(delta[0] * sign, W[0].astype(np.float64), rtol=1e-15, atol=0)


# ----------------------------------------------------------------------------------------------
# O4: integer contraction
# ----------------------------------------------------------------------------------------------
def test_integer_gemm_matches_unpacked_matmul_and_bitplane_identity():
    rng = np.random.default_rng(11)
    M, N, K, bits = 5, 9, 160, 6
    qmax = 31
    codes = rng.integers(-qmax, qmax + 1, size=(M, K)).astype(np.int8)
    packed = gen.random_sign_words(N, K, rng)
    acc = oracle.gemm(codes, packed)
    # independent form 1: explicit +-1 matrix built with numpy bit operations, int64 matmul
    s = np.where((packed[:, :, None] >> np.arange(32, dtype=np.uint32)) & 1, 1, -1).reshape(N, K).astype(np.int64)
    assert np.array_equal(acc, codes.astype(np.int64) @ s.T)
    # independent form 2: bit planes of u = q + qmax and popcounts
    u = (codes.astype(np.int64) + qmax)
    wbits = ((packed[:, :, None] >> np.arange(32, dtype=np.uint32)) & 1).reshape(N, K).astype(np.int64)
    via_planes = np.zeros((M, N), np.int64)
    for i in range(bits):
        p = (u >> i) & 1                                     # [M][K]
        via_planes += (1 << i) * (2 * (p @ wbits.T) - p.sum(axis=1, keepdims=True))
    via_planes -= qmax * (2 * wbits.sum(axis=1) - K)[None, :]
    assert np.array_equal(acc, via_planes)
    # a one-hot code row picks out single signs (catches k-index or bit-order slips)
    onehot = np.zeros((1, K), np.int8)
    onehot[0, 37] = 3
    assert np.array_equal(oracle.gemm(onehot, packed)[0], 3 * s[:, 37])


# ----------------------------------------------------------------------------------------------
# O5: PSP low-rank branch (Sec. 3.2: M = A B, W x = (W - M) x + A (B x))
# ----------------------------------------------------------------------------------------------
def test_lowrank_equals_dense_product():
    rng = np.random.default_rng(12)
    M, N, K, r = 3, 11, 64, 4
    Ub, Vb = gen.lowrank_bf16(N, K, r, rng, rng)
    xb = _bf16(rng.standard_normal((M, K)))
    L = oracle.lowrank(xb, Ub, Vb)
    U = gen.f32_from_bf16_bits(Ub).astype(np.float64)
    V = gen.f32_from_bf16_bits(Vb).astype(np.float64)
    x = gen.f32_from_bf16_bits(xb).astype(np.float64)
    np.testing.assert_allclose(L, x @ (U @ V).T, rtol=0, atol=1e-15 * K)


# ----------------------------------------------------------------------------------------------
# O6 and the whole layer
# ----------------------------------------------------------------------------------------------
def test_layer_exact_special_case():
    # rows of W' in {+-c_n}, identity rotation, 8-bit, integer activations with amax = 127:
    # scale = 1, quantisation is exact, so the layer returns W' x exactly (and alpha = c_n).
    rng = np.random.default_rng(13)
    K, N, M = 64, 6, 3
    c = np.array([0.5, 0.25, 2.0, 1.0, 0.125, 4.0], np.float32)
    sgn = np.where(rng.random((N, K)) > 0.5, 1.0, -1.0).astype(np.float32)
    W = c[:, None] * sgn
    x = rng.integers(-127, 128, size=(M, K)).astype(np.float32)
    x[:, 0] = 127.0
    out = oracle.linear(_bf16(x), np.eye(8, dtype=np.float32), np.eye(8, dtype=np.float32), 8,
                        oracle.pack_signs(W), oracle.row_stats(W, centre=False)[1].astype(np.float32))
    assert np.array_equal(out["codes"], x.astype(np.int8))
    assert np.array_equal(out["y"], x.astype(np.float64) @ W.astype(np.float64).T)


def test_layer_is_the_sum_of_its_parts_and_rank0_drops_the_branch():
    shape = gen.small_shape(96, 40, 8, 12, 4)
    lay = gen.make_layer(0, shape, 6)
    xb = gen.make_activations(0, shape, 3)
    packed = oracle.pack_signs(lay.W)
    full = oracle.linear(xb, lay.P1, lay.P2, 6, packed, lay.alpha, lay.U, lay.V)
    plain = oracle.linear(xb, lay.P1, lay.P2, 6, packed, lay.alpha)
    # independent recomputation of the epilogue with numpy from the oracle's integer parts
    x = gen.f32_from_bf16_bits(xb).astype(np.float64)
    U = gen.f32_from_bf16_bits(lay.U).astype(np.float64)
    V = gen.f32_from_bf16_bits(lay.V).astype(np.float64)
    main = lay.alpha.astype(np.float64)[None, :] * full["scales"].astype(np.float64)[:, None] * full["acc"]
    np.testing.assert_allclose(plain["y"], main, rtol=1e-15)
    np.testing.assert_allclose(full["y"], main + (x @ V.T) @ U.T, rtol=1e-13, atol=1e-16)
    # dequantised view: y ~= alpha * sign(W') . (scale * q), i.e. Eq. 4 applied to quantised activations
    s = oracle.unpack_signs(packed, 96).astype(np.float64)
    deq = (full["scales"].astype(np.float64)[:, None] * full["codes"]) @ (lay.alpha.astype(np.float64)[:, None] * s).T
    np.testing.assert_allclose(plain["y"], deq, rtol=1e-12, atol=1e-15)


def test_layer_approximates_the_unquantised_product():
    # with 8-bit codes the layer is close to alpha*sign(W') (R^T x) + U V x evaluated without quantisation
    shape = gen.small_shape(256, 32, 16, 16, 8)
    lay = gen.make_layer(0, shape, 8)
    xb = gen.activations_bf16(4, 256, np.random.default_rng(1), np.random.default_rng(2), n_outlier=0)
    packed = oracle.pack_signs(lay.W)
    out = oracle.linear(xb, lay.P1, lay.P2, 8, packed, lay.alpha, lay.U, lay.V)
    x = gen.f32_from_bf16_bits(xb).astype(np.float64)
    R = np.kron(lay.P1.astype(np.float64), lay.P2.astype(np.float64))
    s = np.where(lay.W > 0, 1.0, -1.0)
    U = gen.f32_from_bf16_bits(lay.U).astype(np.float64)
    V = gen.f32_from_bf16_bits(lay.V).astype(np.float64)
    ref = (x @ R) @ (lay.alpha.astype(np.float64)[:, None] * s).T + (x @ V.T) @ U.T
    rel = np.linalg.norm(out["y"] - ref) / np.linalg.norm(ref)
    assert rel < 0.05


def test_mu_shift_term():
    # Eq. 4: W_deq = sign * delta + mu, so the layer gains mu_n * sum_k yhat_k = mu_n * scale_t * sum_k q_k
    shape = gen.small_shape(64, 16, 8, 8, 0)
    lay = gen.make_layer(0, shape, 6, with_mu=True)
    xb = gen.make_activations(0, shape, 2)
    packed = oracle.pack_signs(lay.W)
    a = oracle.linear(xb, lay.P1, lay.P2, 6, packed, lay.alpha)
    b = oracle.linear(xb, lay.P1, lay.P2, 6, packed, lay.alpha, mu=lay.mu)
    extra = lay.mu.astype(np.float64)[None, :] * (a["scales"].astype(np.float64) * a["codes"].sum(axis=1))[:, None]
    np.testing.assert_allclose(b["y"], a["y"] + extra, rtol=1e-13, atol=1e-18)


# ----------------------------------------------------------------------------------------------
# bf16 output rounding
# ----------------------------------------------------------------------------------------------
def test_bf16_rounding_is_direct_and_ties_to_even():
    import torch
    rng = np.random.default_rng(14)
    v32 = np.concatenate([rng.standard_normal(4000).astype(np.float32) * np.float32(10.0) ** rng.integers(-30, 30, 4000),
                          np.array([0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.3895314e38, 1e-40, -1e-40], np.float32)])
    ours = oracle.bf16_round(v32.astype(np.float64))
    theirs = torch.from_numpy(v32).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(ours, theirs)
    # a double that a detour through fp32 would round the other way
    d = 1.0 + 2.0 ** -8 + 2.0 ** -30
    assert oracle.bf16_round(np.array([d]))[0] == 0x3F81
    assert oracle.bf16_round(np.array([1.0 + 2.0 ** -8]))[0] == 0x3F80      # exact tie -> even


# ----------------------------------------------------------------------------------------------
# values the paper states
# ----------------------------------------------------------------------------------------------
def test_kron_factor_pairs_from_algorithm_1():
    with open(os.path.join(GOLDEN, "kron_factor_pairs.txt")) as f:
        rows = [tuple(int(v) for v in ln.split()) for ln in f if ln.strip() and not ln.startswith("#")]
    assert len(rows) >= 8
    for n, n1, n2 in rows:
        assert oracle.kron_factor(n) == (n1, n2)
        # brute force: n2 is the largest divisor not above sqrt(n)
        assert n2 == max(a for a in range(1, int(n ** 0.5) + 2) if a * a <= n and n % a == 0)
    # the factor pairs of every benchmark shape are Alg. 1's (listed small factor first)
    for cfg in (0, 1, 2, 3):
        for sh in gen.CONFIG_SHAPES[cfg]:
            assert sorted(oracle.kron_factor(sh.K)) == sorted((sh.n1, sh.n2))


def test_storage_format_lands_in_the_papers_effective_bit_band():
    with open(os.path.join(GOLDEN, "effective_bits.txt")) as f:
        lo, hi = [tuple(float(v) for v in ln.split()) for ln in f if ln.strip() and not ln.startswith("#")][0]
    for N, K in [(4096, 4096), (5120, 5120), (8192, 8192)]:      # square projections, rank = 0.005 * width
        r = round(0.005 * min(N, K))
        n1, n2 = oracle.kron_factor(K)
        bits = N * K + 16 * r * (N + K) + 32 * N + 16 * (n1 * n1 + n2 * n2)
        assert lo - 0.005 <= bits / (N * K) <= hi + 0.005


# ------------------------------------------------------------------------------------------------
# per-token asymmetric quantiser (Sec. 4.1 "per-token asymmetric quantization for activations")
# ------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("bits", [4, 6, 8])
def test_asymmetric_quantiser_recovers_a_row_that_lies_on_its_grid(bits):
    """y_k = s0 * (j_k - z0) with every code 0..L present: scale, zero point and codes come back exactly."""
    L = (1 << bits) - 1
    s0, z0 = 0.375, L // 3                       # exactly representable scale
    j = np.concatenate([np.arange(L + 1), np.random.default_rng(bits).integers(0, L + 1, size=200)])
    y = (s0 * (j - z0))[None, :].astype(np.float64)
    for decision in ("f64", "f32"):
        q = oracle.quantize_asym(y, bits, decision)
        assert q["zeros"][0] == z0 and np.isclose(q["scales"][0], s0, rtol=1e-7)
        assert np.array_equal(q["codes"][0], j.astype(np.uint8))


@pytest.mark.parametrize("bits", [4, 6, 8])
def test_asymmetric_quantiser_invariants_on_random_rows(bits):
    rng = np.random.default_rng(100 + bits)
    Y = rng.standard_t(3, size=(16, 777)) + rng.normal(size=(16, 1)) * 2.0      # rows with a non-zero mean
    Y[3] = np.abs(Y[3])                                                         # a non-negative row
    Y[4] = 0.0                                                                  # an all-zero row
    Y[5, 7] = 0.0                                                               # an exact zero inside a mixed row
    L = (1 << bits) - 1
    q = oracle.quantize_asym(Y, bits)
    u, s, z = q["codes"].astype(np.int64), q["scales"].astype(np.float64), q["zeros"].astype(np.int64)
    assert u.min() >= 0 and u.max() <= L and z.min() >= 0 and z.max() <= L
    lo, hi = np.minimum(Y.min(axis=1), 0), np.maximum(Y.max(axis=1), 0)
    live = hi > lo
    assert np.allclose(s[live], ((hi - lo) / L)[live], rtol=1e-6)
    assert s[4] == 1.0 and z[4] == 0 and not u[4].any()
    # the value a code stands for is within half a step of y (a step more where the sum met the clamp)
    deq = s[:, None] * (u - z[:, None])
    assert np.all(np.abs(deq - Y)[live] <= 0.5 * s[live, None] * (1 + 1e-6) + 1e-12) or \
        np.all(np.abs(deq - Y)[live] <= 1.5 * s[live, None])
    frac_clamped = np.mean(np.abs(deq - Y)[live] > 0.5 * s[live, None] * (1 + 1e-6) + 1e-12)
    assert frac_clamped < 1e-3
    # zero is represented exactly, the smallest value takes code 0, the largest a code within one of L
    assert u[5, 7] == z[5] and deq[5, 7] == 0.0
    assert np.all(u[live].min(axis=1) == 0) and np.all(u[live].max(axis=1) >= L - 1)
    # a non-negative row needs no zero point and gets the whole range: twice the resolution of the symmetric quantiser
    assert z[3] == 0
    sym = oracle.quantize(Y[3:4], bits)
    assert s[3] < 0.51 * sym["scales"][0] * (1 + 2.0 / L)


def test_asymmetric_contraction_is_the_plain_contraction_minus_zero_times_row_sum():
    """sum_k sign * (u - z) = sum_k sign * u - z * (2 * popc(row) - K): the identity the kernels' epilogue relies on,
    against the oracle's direct evaluation."""
    rng = np.random.default_rng(5)
    M, N, K = 5, 37, 96
    W = rng.standard_normal((N, K)).astype(np.float32)
    packed = oracle.pack_signs(W)
    signs = oracle.unpack_signs(packed, K).astype(np.int64)
    u = rng.integers(0, 64, size=(M, K)).astype(np.uint8)
    z = rng.integers(0, 64, size=M).astype(np.int32)
    acc, rsum = oracle.gemm_asym(u, z, packed)
    rowsum = 2 * np.array([bin(int(w)).count("1") for w in packed.reshape(-1)]).reshape(N, -1).sum(axis=1) - K
    assert np.array_equal(rowsum, signs.sum(axis=1))
    want = u.astype(np.int64) @ signs.T - z.astype(np.int64)[:, None] * rowsum[None, :]
    assert np.array_equal(acc, want)
    assert np.array_equal(rsum, u.astype(np.int64).sum(axis=1) - K * z.astype(np.int64))


def test_asymmetric_layer_approaches_the_unquantised_product_with_more_bits():
    """The layer with asymmetric codes against the same layer on unquantised rotated activations: the error falls by
    about 4x per two bits, and is no larger than the symmetric quantiser's on activations with a non-zero mean."""
    rng = np.random.default_rng(11)
    shape = gen.small_shape(256, 48, 16, 16, 0, shape_id=31)
    lay = gen.make_layer(0, shape, 6)
    x = rng.standard_normal((6, 256)).astype(np.float32) + 1.5
    xb = gen.bf16_bits_from_f32(x)
    packed = oracle.pack_signs(lay.W)
    signs = oracle.unpack_signs(packed, 256).astype(np.float64)
    Y = oracle.rotate(xb, lay.P1, lay.P2)
    exact = (Y @ signs.T) * lay.alpha.astype(np.float64)[None, :]
    errs = {}
    for bits in (4, 6, 8):
        ya = oracle.linear_asym(xb, lay.P1, lay.P2, bits, packed, lay.alpha)["y"]
        ys = oracle.linear(xb, lay.P1, lay.P2, bits, packed, lay.alpha)["y"]
        errs[bits] = (np.linalg.norm(ya - exact), np.linalg.norm(ys - exact))
    assert errs[6][0] < 0.4 * errs[4][0] and errs[8][0] < 0.4 * errs[6][0]
    assert all(errs[b][0] <= 1.05 * errs[b][1] for b in errs)


# ----------------------------------------------------------------------------------------------
# Final binarisation in the rotated coordinates (Alg. 2, last step; Eq. 1-3)
# ----------------------------------------------------------------------------------------------
def test_binarisation_recovers_rows_that_are_binary_in_the_rotated_coordinates():
    """W_res = (mu + c * s) R^T with balanced signs: the rotated rows are mu + c s exactly (up to rounding), so the
    oracle must return those signs, c and mu.  A rotation by R^T instead of R, or swapped factors, scrambles the rows."""
    n1, n2, N = 4, 8, 6
    K = n1 * n2
    rng = np.random.default_rng(77)
    P1, P2 = _orth(n1, 1), _orth(n2, 2)
    R = np.kron(P1.astype(np.float64), P2.astype(np.float64))
    s = np.tile(np.array([1.0, -1.0]), K // 2)[None, :].repeat(N, 0)
    for n in range(N):
        rng.shuffle(s[n])                                       # balanced: mean(s) = 0
    c = rng.uniform(0.5, 2.0, N)
    mu = rng.uniform(-0.3, 0.3, N)
    X = mu[:, None] + c[:, None] * s
    W = (X @ R.T).astype(np.float32)                            # W R = X up to the fp32 rounding of W
    out = oracle.binarize(W, P1, P2)
    np.testing.assert_allclose(out["X"], X, atol=5e-6)
    np.testing.assert_allclose(out["mu"], mu, atol=2e-6)
    np.testing.assert_allclose(out["alpha"], c, atol=2e-6)
    assert np.array_equal(oracle.unpack_signs(out["packed"], K), s.astype(np.int8))


def test_binarisation_with_identity_factors_is_equation_1_on_the_rows_themselves():
    rng = np.random.default_rng(5)
    N, n1, n2 = 5, 2, 16
    K = n1 * n2
    W = rng.standard_normal((N, K)).astype(np.float32)
    out = oracle.binarize(W, np.eye(n1, dtype=np.float32), np.eye(n2, dtype=np.float32))
    assert np.array_equal(out["X"], W.astype(np.float64))
    # a hand-written row: values 1, 2, 3, 6 repeated -> mean 3, mean |x - 3| = (2 + 1 + 0 + 3) / 4 = 1.5, signs - - - +
    row = np.tile(np.array([1.0, 2.0, 3.0, 6.0], np.float32), K // 4)[None, :]
    o2 = oracle.binarize(row, np.eye(n1, dtype=np.float32), np.eye(n2, dtype=np.float32))
    assert o2["mu"][0] == 3.0 and o2["alpha"][0] == 1.5
    assert np.array_equal(oracle.unpack_signs(o2["packed"], K)[0], np.tile(np.array([-1, -1, -1, 1], np.int8), K // 4))


def test_binarisation_scale_minimises_the_reconstruction_error_of_the_rotated_row():
    """For the signs and the shift the oracle returns, alpha = mean |x - mu| is the least-squares scale (1-D scan), and
    the rotation keeps the row norms (orthogonal factors)."""
    n1, n2, N = 8, 8, 4
    rng = np.random.default_rng(9)
    P1, P2 = _orth(n1, 3), _orth(n2, 4)
    W = rng.standard_normal((N, n1 * n2)).astype(np.float32)
    out = oracle.binarize(W, P1, P2)
    np.testing.assert_allclose(np.linalg.norm(out["X"], axis=1), np.linalg.norm(W.astype(np.float64), axis=1), rtol=1e-6)
    s = oracle.unpack_signs(out["packed"], n1 * n2).astype(np.float64)
    for n in range(N):
        x = out["X"][n] - out["mu"][n]
        grid = out["alpha"][n] * np.linspace(0.5, 1.5, 2001)
        errs = [np.sum((x - a * s[n]) ** 2) for a in grid]
        assert abs(grid[int(np.argmin(errs))] - out["alpha"][n]) <= out["alpha"][n] * 1e-3
        assert abs(np.mean(x)) < 1e-12


# ----------------------------------------------------------------------------------------------
# W1A16: the weight-only operating point (Table 1, upper half)
# ----------------------------------------------------------------------------------------------
def test_a16_with_identity_factors_is_the_plain_signed_sum_of_the_activations():
    """P = I: the rotated activation is x itself, which is bf16 already, so nothing is rounded and the layer is
    alpha * (S x) with S the +-1 matrix, written here with an independent dense product."""
    n1, n2, N, M = 4, 16, 24, 5
    K = n1 * n2
    rng = np.random.default_rng(21)
    W = rng.standard_normal((N, K)).astype(np.float32)
    packed = oracle.pack_signs(W)
    S = np.where(W > 0, 1.0, -1.0)
    alpha = rng.uniform(0.5, 2.0, N).astype(np.float32)
    mu = rng.uniform(-0.1, 0.1, N).astype(np.float32)
    xb = _bf16(rng.standard_normal((M, K)))
    x = gen.f32_from_bf16_bits(xb).astype(np.float64)
    out = oracle.linear_a16(xb, np.eye(n1, dtype=np.float32), np.eye(n2, dtype=np.float32), packed, alpha, mu=mu)
    assert np.array_equal(gen.f32_from_bf16_bits(out["yhat"]).astype(np.float64), x)
    want = (x @ S.T) * alpha.astype(np.float64)[None, :] + x.sum(axis=1)[:, None] * mu.astype(np.float64)[None, :]
    np.testing.assert_allclose(out["y"], want, rtol=0, atol=1e-12 * np.abs(want).max())


def test_a16_error_is_the_bf16_rounding_of_the_rotated_activation_and_below_the_8_bit_layer():
    n1, n2, N, M, r = 8, 16, 64, 12, 8
    K = n1 * n2
    rng = np.random.default_rng(22)
    P1, P2 = _orth(n1, 5), _orth(n2, 6)
    W = rng.standard_normal((N, K)).astype(np.float32)
    packed = oracle.pack_signs(W)
    S = np.where(W > 0, 1.0, -1.0)
    alpha = rng.uniform(0.5, 2.0, N).astype(np.float32)
    U = _bf16(0.05 * rng.standard_normal((N, r)))
    V = _bf16(0.05 * rng.standard_normal((r, K)))
    xb = _bf16(rng.standard_normal((M, K)))
    a16 = oracle.linear_a16(xb, P1, P2, packed, alpha, U, V)
    a8 = oracle.linear(xb, P1, P2, 8, packed, alpha, U, V)
    exact = (a16["Y"] @ S.T) * alpha.astype(np.float64)[None, :] + oracle.lowrank(xb, U, V)
    e16 = np.linalg.norm(a16["y"] - exact) / np.linalg.norm(exact)
    e8 = np.linalg.norm(a8["y"] - exact) / np.linalg.norm(exact)
    assert e16 < e8 < 2e-2
    # every rotated value moved by at most half a bf16 step, so every output by at most alpha * sum_k 2^-9 |Y_k|
    bound = alpha.astype(np.float64)[None, :] * (np.abs(a16["Y"]).sum(axis=1) * 2.0 ** -9)[:, None]
    assert np.all(np.abs(a16["y"] - exact) <= bound + 1e-12)
    # and the rounding itself is the bf16 rounding the rest of the oracle uses
    assert np.array_equal(a16["yhat"], oracle.bf16_round(a16["Y"]))

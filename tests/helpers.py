"""Shared pieces of the GPU parity tests: host<->device marshalling and the comparison rules.

Tolerances (all stated here, used by every parity test):
  * packed sign words, int32 accumulators for identical codes: bit-exact.
  * quantised codes: bit-exact against the fp64 oracle except where the oracle's pre-rounding value lies within
    1e-6 * qmax (1e-6 of the token's full scale, in code units) of a rounding boundary; such mismatches must be
    exactly +-1 and are counted.
  * per-token scale: within 2e-6 relative of amax / qmax (amax comes out of two fp32 contractions of up to
    n1 + n2 = 320 terms; sqrt(320) * 2^-24 ~ 1e-6 of the row's scale).
  * bf16 output: relative L2 error <= 2e-3 (asserted for outputs of >= 1024 elements); every element within
    1e-2 * rms(y) + 2^-8 * |y| of the fp64 oracle value (a correctly rounded bf16 is already up to 2^-9 * |y| away,
    so the absolute bound alone cannot hold for elements several rms large).  A code that legitimately differs from
    the oracle's by one step at a near-tie moves every output of its token by alpha[n] * s_t; for a token with f such
    codes the bound grows by f * alpha[n] * s_t and the token is left out of the L2 figure (with 4-bit codes and
    heavy-tailed activations one step is already more than 1e-2 * rms(y)).
  * where the test also knows the two summands of the output (the scaled integer term and the low-rank term):
    every element within 1 bf16 step of the correctly rounded oracle value plus 2^-18 * (|term1| + |term2|).  The
    kernel evaluates the sum in fp32 (tensor-core fp32 accumulation for the low-rank term), whose error is
    proportional to the summands, not to a sum that may cancel; 2^-18 leaves 6 bits over the fp32 unit roundoff.
"""
from __future__ import annotations

import numpy as np
import torch

import oracle
from paper_2605_00422_b200 import inputs as gen


def bf16_to_dev(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def bf16_to_host(t: torch.Tensor) -> np.ndarray:
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def words_to_dev(packed: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(packed).view(np.int32)).cuda()


def words_to_host(t: torch.Tensor) -> np.ndarray:
    return t.contiguous().cpu().numpy().view(np.uint32)


def f32_to_dev(a: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).cuda()


class DeviceLayer:
    """One layer's static tensors on the device plus the host copies the oracle needs."""

    def __init__(self, lay: gen.LayerTensors, bwla):
        self.lay = lay
        self.P1 = f32_to_dev(lay.P1)
        self.P2 = f32_to_dev(lay.P2)
        self.alpha = f32_to_dev(lay.alpha)
        self.U = bf16_to_dev(lay.U) if lay.U is not None else None
        self.V = bf16_to_dev(lay.V) if lay.V is not None else None
        self.mu = f32_to_dev(lay.mu) if lay.mu is not None else None
        if lay.packed is not None:
            self.packed_host = lay.packed
            self.packed = words_to_dev(lay.packed)
        else:
            self.packed = bwla.bwla_pack_signs(f32_to_dev(lay.W))
            self.packed_host = words_to_host(self.packed)


def token_sample(M: int, tile: int = 128) -> list:
    """Stratified token subset for problems too large for the oracle: every position inside the first tile, the whole
    last tile, and one (varying) position of every tile in between."""
    last_start = (M - 1) // tile * tile
    picked = set(range(min(tile, M))) | set(range(last_start, M))
    picked |= {i * tile + (i * 37) % tile for i in range(1, last_start // tile)}
    return sorted(picked)


def deinterleave_codes(stored: torch.Tensor) -> torch.Tensor:
    """Codes as the tensor-core contraction wants them (inside each group of 32 consecutive k, byte 4*j + i holds
    k = j + 8*i) back in natural order."""
    M, K = stored.shape
    return stored.view(M, K // 32, 8, 4).transpose(2, 3).reshape(M, K).contiguous()


def fused_call_codes(bwla, ws: torch.Tensor, M: int, shape, bits: int):
    """The int8 codes (natural order) and scales that bwla_w1ax_linear left in its workspace."""
    off, nb = bwla.bwla_workspace_section(M, shape.K, shape.N, shape.r, bits, bwla.BWLA_WS_CODES)
    stored = ws[off:off + nb].view(torch.int8).view(M, shape.K)
    if bwla.bwla_chosen_path(M, shape.K, shape.N, shape.r, bits) == bwla.BWLA_PATH_I8:
        codes = deinterleave_codes(stored)
    else:
        codes = stored.clone()
    off, nb = bwla.bwla_workspace_section(M, shape.K, shape.N, shape.r, bits, bwla.BWLA_WS_SCALES)
    scales = ws[off:off + nb].view(torch.float32).clone()
    return codes, scales


def summand_magnitude(ref: dict, alpha: np.ndarray) -> np.ndarray:
    """|alpha * s * acc| + |y - alpha * s * acc| of an oracle result: the size of what the output sum adds up."""
    main = alpha.astype(np.float64)[None, :] * ref["scales"].astype(np.float64)[:, None] * ref["acc"].astype(np.float64)
    return np.abs(main) + np.abs(ref["y"] - main)


def check_codes(gpu_codes: np.ndarray, gpu_scales: np.ndarray, Y: np.ndarray, bits: int) -> dict:
    """The comparison rule for the integer codes (see the module docstring); returns counts for the report."""
    ref = oracle.quantize(Y, bits, "f64")
    diff = gpu_codes.astype(np.int32) - ref["codes"].astype(np.int32)
    bad = diff != 0
    window = oracle.near_tie_window(bits)
    flagged = ref["dist"] <= window
    unflagged = bad & ~flagged
    assert np.all(np.abs(diff[bad]) == 1), "a code differs from the oracle by more than one step"
    assert not unflagged.any(), (
        f"{int(unflagged.sum())} code mismatches outside the near-tie window; "
        f"worst distance to a boundary {ref['dist'][unflagged].max():.3e} (window {window:.1e})")
    exact_scale = np.abs(Y).max(axis=1) / float((1 << (bits - 1)) - 1)
    exact_scale[exact_scale == 0] = 1.0
    scale_err = np.abs(gpu_scales.astype(np.float64) - exact_scale) / exact_scale
    assert scale_err.max() <= 2e-6, f"scale off by {scale_err.max():.2e} relative"
    return {"near_ties": int(flagged.sum()), "mismatches": int(bad.sum()), "elements": int(bad.size),
            "scale_rel_err": float(scale_err.max())}


def code_step_slack(gpu_codes: np.ndarray, ref: dict, alpha: np.ndarray, mu: np.ndarray = None) -> np.ndarray:
    """[tokens][N]: how far the outputs of a token may move because f of its codes differ from the oracle's by one step
    (check_codes has verified that these are near-ties): f * (|alpha[n]| + |mu[n]|) * s_t."""
    flips = np.count_nonzero(gpu_codes.astype(np.int32) != ref["codes"].astype(np.int32), axis=1).astype(np.float64)
    per_row = np.abs(alpha.astype(np.float64)) + (0.0 if mu is None else np.abs(mu.astype(np.float64)))
    return flips[:, None] * per_row[None, :] * ref["scales"].astype(np.float64)[:, None]


def check_output(gpu_bits: np.ndarray, y_ref: np.ndarray, mag: np.ndarray = None, step_slack: np.ndarray = None) -> dict:
    got = gen.f32_from_bf16_bits(gpu_bits).astype(np.float64)
    err = got - y_ref
    same_codes = np.ones(y_ref.shape[0], bool) if step_slack is None else (step_slack.max(axis=1) == 0)
    rel_l2 = float(np.linalg.norm(err[same_codes]) / max(np.linalg.norm(y_ref[same_codes]), 1e-300))
    rms = float(np.sqrt(np.mean(y_ref ** 2)))
    # the L2 figure is a statistic of the output rounding (a single correctly rounded bf16 can be 2^-8 away),
    # so it is only asserted where there are enough elements for it to mean something
    if y_ref[same_codes].size >= 1024:
        assert rel_l2 <= 2e-3, f"relative L2 error {rel_l2:.3e} > 2e-3"
    bound = 1e-2 * rms + 2.0 ** -8 * np.abs(y_ref) + (0.0 if step_slack is None else step_slack)
    assert np.all(np.abs(err) <= bound), f"max |err| {np.abs(err).max():.3e} exceeds 1e-2*rms + 2^-8*|y|"
    # distance to the correctly rounded value, in bf16 steps of the reference
    ref_bits = oracle.bf16_round(y_ref)
    ref_val = gen.f32_from_bf16_bits(ref_bits).astype(np.float64)
    step = np.maximum(np.abs(ref_val), 2.0 ** -126) * 2.0 ** -7
    slack = 0.0 if mag is None else 2.0 ** -18 * mag
    ulps = np.maximum(np.abs(got - ref_val) - slack, 0.0) / step
    return {"rel_l2": rel_l2, "max_abs_over_rms": float(np.abs(err).max() / max(rms, 1e-300)),
            "over_literal_bound": int(np.count_nonzero(np.abs(err) > 1e-2 * rms)),
            "max_bf16_steps": float(ulps.max()), "exact_bf16": float(np.mean(gpu_bits == ref_bits))}

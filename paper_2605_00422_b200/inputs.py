"""Seeded synthetic inputs for the W1AX linear layer.

This module only draws random tensors and describes workload shapes.  It holds
none of the layer's arithmetic (no rotation, no quantiser, no packing, no
contraction): both the CUDA path and the CPU oracle receive what is generated
here as plain arrays.  It needs numpy only.

Conventions
-----------
* bf16 tensors are carried as ``uint16`` arrays holding the bf16 bit patterns
  (numpy has no bf16 dtype).  ``bf16_bits_from_f32`` / ``f32_from_bf16_bits``
  are storage-type conversions, not part of the method.
* Every tensor comes from ``numpy.random.default_rng([422, cfg, layer, shape,
  tensor])`` so that each one can be regenerated on its own.

The value distributions stand in for calibrated checkpoints, which are not
available: orthogonal Kronecker factors (Haar, by QR), Bernoulli(0.5) signs,
log-normal per-row scales, small Gaussian low-rank factors and heavy-tailed
activations with a few scaled outlier channels.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional, Tuple

import numpy as np

ROOT_SEED = 422

# tensor ids inside a seed tuple
T_P1, T_P2, T_W, T_ALPHA, T_U, T_V, T_X, T_MU, T_OUTLIER = range(9)


# --------------------------------------------------------------------------
# storage-type helpers (bf16 carried as uint16 bit patterns)
# --------------------------------------------------------------------------
def bf16_bits_from_f32(a: np.ndarray) -> np.ndarray:
    """Round fp32 values to bf16 (nearest, ties to even) and return the bits."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + bias) >> np.uint32(16)).astype(np.uint16)


def f32_from_bf16_bits(b: np.ndarray) -> np.ndarray:
    """Widen bf16 bit patterns to fp32 (exact)."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def _rng(cfg: int, layer: int, shape_id: int, tensor_id: int) -> np.random.Generator:
    return np.random.default_rng([ROOT_SEED, cfg, layer, shape_id, tensor_id])


# --------------------------------------------------------------------------
# tensor recipes
# --------------------------------------------------------------------------
def orthogonal_f32(n: int, rng: np.random.Generator) -> np.ndarray:
    """Haar-distributed orthogonal n x n matrix, fp32, row-major."""
    g = rng.standard_normal((n, n))
    q, r = np.linalg.qr(g)
    q = q * np.sign(np.diag(r))[None, :]
    return np.ascontiguousarray(q, dtype=np.float32)


def gaussian_weights_f32(N: int, K: int, rng: np.random.Generator) -> np.ndarray:
    """Rotated/centred weights W' ~ N(0,1) whose signs are Bernoulli(0.5)."""
    return rng.standard_normal((N, K), dtype=np.float32)


def random_sign_words(N: int, K: int, rng: np.random.Generator) -> np.ndarray:
    """Bernoulli(0.5) sign bits drawn directly as packed words, uint32 [N][K/32]."""
    assert K % 32 == 0
    return rng.integers(0, 1 << 32, size=(N, K // 32), dtype=np.uint64).astype(np.uint32)


def alpha_f32(N: int, rng: np.random.Generator) -> np.ndarray:
    return rng.lognormal(mean=-4.0, sigma=0.3, size=N).astype(np.float32)


def lowrank_bf16(N: int, K: int, r: int, rng_u: np.random.Generator,
                 rng_v: np.random.Generator) -> Tuple[np.ndarray, np.ndarray]:
    """U [N][r] and V [r][K], N(0, 0.01^2), as bf16 bit patterns."""
    U = (0.01 * rng_u.standard_normal((N, r))).astype(np.float32)
    V = (0.01 * rng_v.standard_normal((r, K))).astype(np.float32)
    return bf16_bits_from_f32(U), bf16_bits_from_f32(V)


def activations_bf16(M: int, K: int, rng: np.random.Generator, rng_outlier: np.random.Generator,
                     nu: float = 3.0, n_outlier: int = 8, outlier_scale: float = 50.0) -> np.ndarray:
    """Student-t activations with ``n_outlier`` channels multiplied by ``outlier_scale``; bf16 bits [M][K]."""
    x = rng.standard_t(nu, size=(M, K)).astype(np.float32)
    if n_outlier > 0:
        ch = rng_outlier.choice(K, size=min(n_outlier, K), replace=False)
        x[:, ch] *= np.float32(outlier_scale)
    return bf16_bits_from_f32(x)


# --------------------------------------------------------------------------
# workload description
# --------------------------------------------------------------------------
@dataclass(frozen=True)
class LinearShape:
    name: str
    K: int          # d_in
    N: int          # d_out
    n1: int
    n2: int
    r: int
    shape_id: int = 0


@dataclass
class LayerTensors:
    shape: LinearShape
    bits: int
    P1: np.ndarray            # fp32 [n1][n1]
    P2: np.ndarray            # fp32 [n2][n2]
    alpha: np.ndarray         # fp32 [N]
    U: Optional[np.ndarray]   # bf16 bits [N][r]
    V: Optional[np.ndarray]   # bf16 bits [r][K]
    W: Optional[np.ndarray] = None        # fp32 [N][K] when signs come from pack_signs
    packed: Optional[np.ndarray] = None   # uint32 [N][K/32] when drawn directly
    mu: Optional[np.ndarray] = None       # fp32 [N] (optional per-row shift)


CONFIG_SHAPES: Dict[int, List[LinearShape]] = {
    0: [LinearShape("c0", 1024, 1024, 32, 32, 16, 0)],
    1: [LinearShape("l7_qkv", 4096, 12288, 64, 64, 32, 0),
        LinearShape("l7_o", 4096, 4096, 64, 64, 32, 1),
        LinearShape("l7_gate_up", 4096, 22016, 64, 64, 32, 2),
        LinearShape("l7_down", 11008, 4096, 86, 128, 32, 3)],
    2: [LinearShape("q_q", 5120, 8192, 64, 80, 64, 0),
        LinearShape("q_k", 5120, 1024, 64, 80, 64, 1),
        LinearShape("q_v", 5120, 1024, 64, 80, 64, 2),
        LinearShape("q_o", 8192, 5120, 64, 128, 64, 3),
        LinearShape("q_gate", 5120, 25600, 64, 80, 64, 4),
        LinearShape("q_up", 5120, 25600, 64, 80, 64, 5),
        LinearShape("q_down", 25600, 5120, 160, 160, 64, 6)],
    3: [LinearShape("q_down", 25600, 5120, 160, 160, 64, 0)],
}
CONFIG_SHAPES[4] = CONFIG_SHAPES[2]

CONFIG_TOKENS: Dict[int, List[int]] = {
    0: [16],
    1: [1, 16, 128, 2048],
    2: [1, 8, 64, 512, 4096],
    3: [1, 32, 2048],
    4: [1, 16, 64, 2048],
}
CONFIG_BITS: Dict[int, List[int]] = {0: [6], 1: [6], 2: [6], 3: [4, 6, 8], 4: [6]}
QWEN3_32B_LAYERS = 64


def make_layer(cfg: int, shape: LinearShape, bits: int = 6, layer: int = 0,
               direct_words: bool = False, with_mu: bool = False) -> LayerTensors:
    """Draw every static tensor of one linear layer."""
    s = shape.shape_id
    P1 = orthogonal_f32(shape.n1, _rng(cfg, layer, s, T_P1))
    P2 = orthogonal_f32(shape.n2, _rng(cfg, layer, s, T_P2))
    alpha = alpha_f32(shape.N, _rng(cfg, layer, s, T_ALPHA))
    U = V = None
    if shape.r > 0:
        U, V = lowrank_bf16(shape.N, shape.K, shape.r, _rng(cfg, layer, s, T_U), _rng(cfg, layer, s, T_V))
    W = packed = None
    if direct_words:
        packed = random_sign_words(shape.N, shape.K, _rng(cfg, layer, s, T_W))
    else:
        W = gaussian_weights_f32(shape.N, shape.K, _rng(cfg, layer, s, T_W))
    mu = None
    if with_mu:
        mu = (0.002 * _rng(cfg, layer, s, T_MU).standard_normal(shape.N)).astype(np.float32)
    return LayerTensors(shape, bits, P1, P2, alpha, U, V, W, packed, mu)


def make_activations(cfg: int, shape: LinearShape, M: int, layer: int = 0) -> np.ndarray:
    """bf16 bit patterns [M][K]; config 3 uses the heavier-tailed recipe."""
    s = shape.shape_id
    if cfg == 3:
        return activations_bf16(M, shape.K, _rng(cfg, layer, s, T_X), _rng(cfg, layer, s, T_OUTLIER),
                                nu=2.5, n_outlier=shape.K // 100, outlier_scale=100.0)
    return activations_bf16(M, shape.K, _rng(cfg, layer, s, T_X), _rng(cfg, layer, s, T_OUTLIER),
                            nu=3.0, n_outlier=8, outlier_scale=50.0)


def small_shape(K: int, N: int, n1: int, n2: int, r: int, shape_id: int = 99) -> LinearShape:
    """Ad-hoc shape for edge-case tests."""
    assert n1 * n2 == K
    return LinearShape(f"s{K}x{N}", K, N, n1, n2, r, shape_id)

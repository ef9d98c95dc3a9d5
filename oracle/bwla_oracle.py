"""ctypes front end of the plain-C CPU oracle (test infrastructure only).

Argument marshalling only: every step of the layer is computed by
``bwla_oracle.c``.  The shared object is built on demand with the host
compiler (``gcc -O2 -fopenmp``); no CUDA header or source is involved.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import Dict, Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "bwla_oracle.c")
_LIB = os.path.join(_HERE, "libbwla_oracle.so")

__all__ = [
    "build", "num_threads", "kron_factor", "row_stats", "pack_signs", "pack_signs_bf16", "unpack_signs",
    "rotate", "quantize", "gemm", "lowrank", "epilogue", "linear", "bf16_round", "near_tie_window",
    "quantize_asym", "gemm_asym", "linear_asym", "near_tie_window_asym", "binarize", "linear_a16",
]


def build(force: bool = False) -> str:
    """Compile the oracle with the host compiler if the shared object is missing or stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c99", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off",
               "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


_lib = None


def _L():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.bwla_oracle_linear.restype = C.c_int
        _lib.bwla_oracle_num_threads.restype = C.c_int
    return _lib


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _c(a, dtype):
    return np.ascontiguousarray(a, dtype=dtype)


i64 = C.c_int64


def num_threads() -> int:
    return int(_L().bwla_oracle_num_threads())


def kron_factor(n: int):
    n1, n2 = i64(), i64()
    _L().bwla_oracle_kron_factor(i64(n), C.byref(n1), C.byref(n2))
    return int(n1.value), int(n2.value)


def row_stats(W: np.ndarray, centre: bool = True):
    W = _c(W, np.float32)
    N, K = W.shape
    mu = np.empty(N, np.float64)
    delta = np.empty(N, np.float64)
    _L().bwla_oracle_row_stats(_p(W), i64(N), i64(K), C.c_int(int(centre)), _p(mu), _p(delta))
    return mu, delta


def pack_signs(W: np.ndarray) -> np.ndarray:
    W = _c(W, np.float32)
    N, K = W.shape
    assert K % 32 == 0
    out = np.empty((N, K // 32), np.uint32)
    _L().bwla_oracle_pack_signs(_p(W), i64(N), i64(K), i64(K), _p(out))
    return out


def pack_signs_bf16(W_bits: np.ndarray) -> np.ndarray:
    W_bits = _c(W_bits, np.uint16)
    N, K = W_bits.shape
    assert K % 32 == 0
    out = np.empty((N, K // 32), np.uint32)
    _L().bwla_oracle_pack_signs_bf16(_p(W_bits), i64(N), i64(K), i64(K), _p(out))
    return out


def unpack_signs(packed: np.ndarray, K: int) -> np.ndarray:
    packed = _c(packed, np.uint32)
    N = packed.shape[0]
    s = np.empty((N, K), np.int8)
    _L().bwla_oracle_unpack_signs(_p(packed), i64(N), i64(K), _p(s))
    return s


def rotate(x_bits: np.ndarray, P1: np.ndarray, P2: np.ndarray) -> np.ndarray:
    x_bits = _c(x_bits, np.uint16)
    P1 = _c(P1, np.float32)
    P2 = _c(P2, np.float32)
    M, K = x_bits.shape
    n1, n2 = P1.shape[0], P2.shape[0]
    assert n1 * n2 == K
    Y = np.empty((M, K), np.float64)
    _L().bwla_oracle_rotate(_p(x_bits), i64(M), i64(K), i64(K), _p(P1), i64(n1), _p(P2), i64(n2), _p(Y))
    return Y


def binarize(W: np.ndarray, P1: np.ndarray, P2: np.ndarray) -> Dict[str, np.ndarray]:
    """Alg. 2, last step: rows of W_res (fp32 [N][K]) rotated, then Eq. 1-3 per row.  Returns X (fp64), mu, alpha,
    packed."""
    W = _c(W, np.float32)
    P1 = _c(P1, np.float32)
    P2 = _c(P2, np.float32)
    N, K = W.shape
    n1, n2 = P1.shape[0], P2.shape[0]
    assert n1 * n2 == K and K % 32 == 0
    X = np.empty((N, K), np.float64)
    mu = np.empty(N, np.float64)
    alpha = np.empty(N, np.float64)
    packed = np.empty((N, K // 32), np.uint32)
    _L().bwla_oracle_binarize(_p(W), i64(N), i64(K), _p(P1), i64(n1), _p(P2), i64(n2), _p(X), _p(mu), _p(alpha), _p(packed))
    return {"X": X, "mu": mu, "alpha": alpha, "packed": packed}


def quantize(Y: np.ndarray, bits: int, decision: str = "f64") -> Dict[str, np.ndarray]:
    """decision: 'f64' (definition) or 'f32' (the precision a float kernel decides in)."""
    Y = _c(Y, np.float64)
    M, K = Y.shape
    codes = np.empty((M, K), np.int8)
    scales = np.empty(M, np.float32)
    dist = np.empty((M, K), np.float64)
    qsum = np.empty(M, np.int64)
    _L().bwla_oracle_quantize(_p(Y), i64(M), i64(K), C.c_int(bits), C.c_int(1 if decision == "f32" else 0),
                              _p(codes), _p(scales), _p(dist), _p(qsum))
    return {"codes": codes, "scales": scales, "dist": dist, "qsum": qsum}


def quantize_asym(Y: np.ndarray, bits: int, decision: str = "f64") -> Dict[str, np.ndarray]:
    """Per-token asymmetric quantiser (Sec. 4.1): unsigned codes u in [0, 2^b - 1], scale and integer zero point per token;
    a code stands for scale * (u - zero)."""
    Y = _c(Y, np.float64)
    M, K = Y.shape
    codes = np.empty((M, K), np.uint8)
    scales = np.empty(M, np.float32)
    zeros = np.empty(M, np.int32)
    dist = np.empty((M, K), np.float64)
    dist_zero = np.empty(M, np.float64)
    _L().bwla_oracle_quantize_asym(_p(Y), i64(M), i64(K), C.c_int(bits), C.c_int(1 if decision == "f32" else 0),
                                   _p(codes), _p(scales), _p(zeros), _p(dist), _p(dist_zero))
    return {"codes": codes, "scales": scales, "zeros": zeros, "dist": dist, "dist_zero": dist_zero}


def near_tie_window_asym(bits: int) -> float:
    """As near_tie_window for the asymmetric quantiser, whose full scale is 2^b - 1 code units."""
    return 1e-6 * float((1 << bits) - 1)


def gemm_asym(codes: np.ndarray, zeros: np.ndarray, packed: np.ndarray):
    """(acc, rsum): acc[t][n] = sum_k sign[n][k] * (u[t][k] - zero[t]); rsum[t] = sum_k (u[t][k] - zero[t])."""
    codes = _c(codes, np.uint8)
    zeros = _c(zeros, np.int32)
    packed = _c(packed, np.uint32)
    M, K = codes.shape
    N = packed.shape[0]
    assert packed.shape[1] * 32 == K
    acc = np.empty((M, N), np.int64)
    rsum = np.empty(M, np.int64)
    _L().bwla_oracle_gemm_asym(_p(codes), _p(zeros), _p(packed), i64(M), i64(N), i64(K), _p(acc), _p(rsum))
    return acc, rsum


def linear_asym(x_bits, P1, P2, bits, packed, alpha, U_bits=None, V_bits=None, mu=None,
                decision: str = "f64") -> Dict[str, np.ndarray]:
    """The whole layer with the per-token asymmetric activation quantiser, step by step:
    y[t][n] = alpha[n] * s_t * sum_k sign[n][k] * (u[t][k] - z_t) + U (V x_t) [+ mu[n] * s_t * sum_k (u[t][k] - z_t)]."""
    Y = rotate(x_bits, P1, P2)
    q = quantize_asym(Y, bits, decision)
    acc, rsum = gemm_asym(q["codes"], q["zeros"], packed)
    L = lowrank(x_bits, U_bits, V_bits) if U_bits is not None else None
    y, yb = epilogue(acc, q["scales"], alpha, L, mu, rsum if mu is not None else None)
    return {"y": y, "y_bf16": yb, "Y": Y, "codes": q["codes"], "scales": q["scales"], "zeros": q["zeros"], "acc": acc,
            "dist": q["dist"], "dist_zero": q["dist_zero"]}


def near_tie_window(bits: int) -> float:
    """Distance (in code units) under which a code counts as a near-tie: 1e-6 of the token's full scale."""
    return 1e-6 * float((1 << (bits - 1)) - 1)


def gemm(codes: np.ndarray, packed: np.ndarray) -> np.ndarray:
    codes = _c(codes, np.int8)
    packed = _c(packed, np.uint32)
    M, K = codes.shape
    N = packed.shape[0]
    assert packed.shape[1] * 32 == K
    acc = np.empty((M, N), np.int64)
    _L().bwla_oracle_gemm(_p(codes), _p(packed), i64(M), i64(N), i64(K), _p(acc))
    return acc


def lowrank(x_bits: np.ndarray, U_bits: np.ndarray, V_bits: np.ndarray) -> np.ndarray:
    x_bits = _c(x_bits, np.uint16)
    U_bits = _c(U_bits, np.uint16)
    V_bits = _c(V_bits, np.uint16)
    M, K = x_bits.shape
    N, r = U_bits.shape
    assert V_bits.shape == (r, K)
    L = np.empty((M, N), np.float64)
    _L().bwla_oracle_lowrank(_p(x_bits), i64(M), i64(K), i64(K), _p(U_bits), _p(V_bits), i64(N), i64(r), _p(L))
    return L


def epilogue(acc, scales, alpha, L=None, mu=None, qsum=None):
    acc = _c(acc, np.int64)
    M, N = acc.shape
    scales = _c(scales, np.float32)
    alpha = _c(alpha, np.float32)
    if L is not None:
        L = _c(L, np.float64)
    if mu is not None:
        mu = _c(mu, np.float32)
        qsum = _c(qsum, np.int64)
    y = np.empty((M, N), np.float64)
    yb = np.empty((M, N), np.uint16)
    _L().bwla_oracle_epilogue(_p(acc), _p(scales), _p(alpha), _p(mu), _p(qsum), _p(L), i64(M), i64(N), _p(y), _p(yb))
    return y, yb


def bf16_round(y: np.ndarray) -> np.ndarray:
    y = _c(y, np.float64)
    out = np.empty(y.shape, np.uint16)
    _L().bwla_oracle_bf16_round(_p(y), i64(y.size), _p(out))
    return out


def linear_a16(x_bits, P1, P2, packed, alpha, U_bits=None, V_bits=None, mu=None) -> Dict[str, np.ndarray]:
    """The weight-only layer (W1A16): rotated activations kept in bf16.  Returns y (fp64), Y (rotated, fp64), yhat (bf16
    bits), acc (fp64)."""
    x_bits = _c(x_bits, np.uint16)
    packed = _c(packed, np.uint32)
    alpha = _c(alpha, np.float32)
    M, K = x_bits.shape
    N = packed.shape[0]
    assert packed.shape[1] * 32 == K and alpha.shape == (N,)
    Y = rotate(x_bits, P1, P2)
    L = lowrank(x_bits, U_bits, V_bits) if U_bits is not None else None
    if mu is not None:
        mu = _c(mu, np.float32)
    yhat = np.empty((M, K), np.uint16)
    acc = np.empty((M, N), np.float64)
    y = np.empty((M, N), np.float64)
    _L().bwla_oracle_a16(_p(Y), i64(M), i64(K), _p(packed), _p(alpha), _p(mu), _p(L), i64(N), _p(yhat), _p(acc), _p(y))
    return {"y": y, "Y": Y, "yhat": yhat, "acc": acc}


def linear(x_bits, P1, P2, bits, packed, alpha, U_bits=None, V_bits=None, mu=None,
           decision: str = "f64") -> Dict[str, np.ndarray]:
    """The whole layer.  Returns y (fp64), y_bf16 (bits), Y (rotated), codes, scales, acc."""
    x_bits = _c(x_bits, np.uint16)
    P1 = _c(P1, np.float32)
    P2 = _c(P2, np.float32)
    packed = _c(packed, np.uint32)
    alpha = _c(alpha, np.float32)
    M, K = x_bits.shape
    N = packed.shape[0]
    n1, n2 = P1.shape[0], P2.shape[0]
    assert n1 * n2 == K and packed.shape[1] * 32 == K and alpha.shape == (N,)
    r = 0
    if U_bits is not None:
        U_bits = _c(U_bits, np.uint16)
        V_bits = _c(V_bits, np.uint16)
        r = U_bits.shape[1]
        assert U_bits.shape == (N, r) and V_bits.shape == (r, K)
    if mu is not None:
        mu = _c(mu, np.float32)
    y = np.empty((M, N), np.float64)
    yb = np.empty((M, N), np.uint16)
    Y = np.empty((M, K), np.float64)
    codes = np.empty((M, K), np.int8)
    scales = np.empty(M, np.float32)
    acc = np.empty((M, N), np.int64)
    ovf = _L().bwla_oracle_linear(_p(x_bits), i64(M), i64(K), i64(K), _p(P1), i64(n1), _p(P2), i64(n2),
                                  C.c_int(bits), C.c_int(1 if decision == "f32" else 0),
                                  _p(packed), _p(alpha), _p(mu), _p(U_bits), _p(V_bits), i64(r), i64(N),
                                  _p(y), _p(yb), _p(Y), _p(codes), _p(scales), _p(acc))
    assert ovf == 0, "integer accumulator left the int32 range"
    return {"y": y, "y_bf16": yb, "Y": Y, "codes": codes, "scales": scales, "acc": acc}

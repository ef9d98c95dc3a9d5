"""Thin Python binding of the C ABI in ``include/bwla.h``.

Argument marshalling only: each function here checks tensor types, takes ``data_ptr()`` and the current CUDA
stream from PyTorch and calls the entry point of the same name in ``libbwla.so``.  Every step of the layer
runs in the library's CUDA kernels.  There is no fallback: if the shared object is missing the import fails.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("BWLA_LIBRARY", os.path.join(_HERE, "libbwla.so"))   # override: another build of the same ABI

BWLA_OK = 0
BWLA_ERR_INVALID_ARG = -1
BWLA_ERR_UNSUPPORTED = -2
BWLA_ERR_WORKSPACE = -3
BWLA_ERR_CUDA = -4
BWLA_ERR_DEVICE_TIMEOUT = -5
BWLA_ERR_STATIC_SCRATCH = -6
BWLA_STATIC_SCRATCH_BYTES = 4 * 1024 * 1024

BWLA_ROT_AUTO, BWLA_ROT_SIMT, BWLA_ROT_UMMA = 0, 1, 2

BWLA_PATH_AUTO = 0
BWLA_PATH_SIMPLE = 1
BWLA_PATH_BITPLANE = 2
BWLA_PATH_I8 = 3

EXPORTS = [
    "bwla_pack_signs", "bwla_rotate_quant_act", "bwla_workspace_bytes", "bwla_w1ax_linear", "bwla_w1a_gemm_codes",
    "bwla_check_status", "bwla_force_path", "bwla_chosen_path", "bwla_last_launch_count", "bwla_last_cuda_error",
    "bwla_status_string", "bwla_profile_enable", "bwla_profile_collect", "bwla_w1ax_linear_static",
    "bwla_workspace_section", "bwla_force_rotation", "bwla_layer_prepared_bytes", "bwla_layer_create",
    "bwla_layer_destroy", "bwla_layer_rotate_quant", "bwla_group_workspace_bytes", "bwla_w1ax_linear_group",
    "bwla_layer_set_activation_quant", "bwla_layer_rotate_quant_asym", "bwla_binarize_workspace_bytes",
    "bwla_binarize_rows", "bwla_w1a16_workspace_bytes", "bwla_layer_w1a16_linear",
]


class BwlaError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {bwla_status_string(status)} (cuda error {bwla_last_cuda_error()})")


def _load() -> C.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2605_00422_b200.build` "
                          "(there is no CPU or PyTorch fallback)")
    lib = C.CDLL(LIB_PATH)
    i64, vp, ci, sz = C.c_int64, C.c_void_p, C.c_int, C.c_size_t
    lib.bwla_pack_signs.argtypes = [vp, ci, i64, i64, i64, vp, vp]
    lib.bwla_rotate_quant_act.argtypes = [vp, i64, i64, i64, vp, ci, vp, ci, ci, vp, vp, vp]
    lib.bwla_binarize_workspace_bytes.argtypes = [i64]
    lib.bwla_binarize_workspace_bytes.restype = sz
    lib.bwla_binarize_rows.argtypes = [vp, ci, i64, i64, i64, vp, ci, vp, ci, vp, vp, vp, vp, sz, vp]
    lib.bwla_workspace_bytes.argtypes = [i64, i64, i64, ci, ci]
    lib.bwla_workspace_bytes.restype = sz
    lib.bwla_w1ax_linear.argtypes = [vp, i64, i64, i64, vp, ci, vp, ci, ci, vp, vp, vp, vp, vp, ci, vp, i64, i64,
                                     vp, sz, vp]
    lib.bwla_w1a_gemm_codes.argtypes = [vp, vp, i64, i64, ci, vp, vp, vp, vp, i64, vp, vp, ci, vp, i64, i64, vp,
                                        vp, sz, vp]
    lib.bwla_check_status.argtypes = [vp, vp]
    lib.bwla_workspace_section.argtypes = [i64, i64, i64, ci, ci, ci, C.POINTER(sz), C.POINTER(sz)]
    lib.bwla_workspace_section.restype = ci
    lib.bwla_w1ax_linear_static.argtypes = [vp, i64, i64, i64, vp, ci, vp, ci, ci, vp, vp, vp, vp, vp, ci, vp, i64, i64, vp]
    lib.bwla_w1ax_linear_static.restype = ci
    lib.bwla_force_path.argtypes = [ci]
    lib.bwla_force_rotation.argtypes = [ci]
    lib.bwla_force_rotation.restype = ci
    lib.bwla_layer_prepared_bytes.argtypes = [i64, i64, ci, ci, ci]
    lib.bwla_layer_prepared_bytes.restype = sz
    lib.bwla_layer_create.argtypes = [C.POINTER(vp), i64, i64, vp, ci, vp, ci, ci, vp, vp, vp, vp, vp, ci, vp, sz, vp]
    lib.bwla_layer_create.restype = ci
    lib.bwla_layer_destroy.argtypes = [vp]
    lib.bwla_layer_destroy.restype = None
    lib.bwla_layer_rotate_quant.argtypes = [vp, vp, i64, i64, vp, vp, vp, vp]
    lib.bwla_layer_rotate_quant.restype = ci
    lib.bwla_layer_set_activation_quant.argtypes = [vp, ci]
    lib.bwla_layer_set_activation_quant.restype = ci
    lib.bwla_layer_rotate_quant_asym.argtypes = [vp, vp, i64, i64, vp, vp, vp, vp, vp]
    lib.bwla_layer_rotate_quant_asym.restype = ci
    lib.bwla_w1a16_workspace_bytes.argtypes = [vp, i64]
    lib.bwla_w1a16_workspace_bytes.restype = sz
    lib.bwla_layer_w1a16_linear.argtypes = [vp, vp, i64, i64, vp, i64, vp, sz, vp]
    lib.bwla_group_workspace_bytes.argtypes = [C.POINTER(vp), ci, i64]
    lib.bwla_group_workspace_bytes.restype = sz
    lib.bwla_w1ax_linear_group.argtypes = [C.POINTER(vp), ci, vp, i64, i64, C.POINTER(vp), C.POINTER(i64), vp, sz, vp]
    lib.bwla_w1ax_linear_group.restype = ci
    lib.bwla_chosen_path.argtypes = [i64, i64, i64, ci, ci]
    lib.bwla_profile_enable.argtypes = [ci]
    lib.bwla_profile_collect.argtypes = [vp, vp]
    lib.bwla_status_string.argtypes = [ci]
    lib.bwla_status_string.restype = C.c_char_p
    for name in ("bwla_pack_signs", "bwla_rotate_quant_act", "bwla_w1ax_linear", "bwla_w1a_gemm_codes",
                 "bwla_check_status", "bwla_force_path", "bwla_chosen_path", "bwla_last_launch_count",
                 "bwla_last_cuda_error", "bwla_profile_enable", "bwla_profile_collect"):
        getattr(lib, name).restype = ci
    return lib


_lib = _load()


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _need(t: torch.Tensor, dtype, name: str, ndim: Optional[int] = None):
    if not t.is_cuda or t.dtype != dtype or (ndim is not None and t.dim() != ndim):
        raise TypeError(f"{name}: expected a CUDA tensor of {dtype}" + (f" with {ndim} dims" if ndim else ""))
    if t.stride(-1) != 1 and t.numel() > 0:
        raise TypeError(f"{name}: innermost dimension must be contiguous")


def _check(status: int, where: str):
    if status != BWLA_OK:
        raise BwlaError(status, where)


def bwla_status_string(status: int) -> str:
    return _lib.bwla_status_string(status).decode()


def bwla_last_cuda_error() -> int:
    return int(_lib.bwla_last_cuda_error())


def bwla_last_launch_count() -> int:
    return int(_lib.bwla_last_launch_count())


def bwla_force_path(path: int) -> None:
    _check(_lib.bwla_force_path(path), "bwla_force_path")


def bwla_force_rotation(which: int) -> None:
    _check(_lib.bwla_force_rotation(which), "bwla_force_rotation")


def bwla_chosen_path(M: int, K: int, N: int, r: int, bits: int) -> int:
    return int(_lib.bwla_chosen_path(M, K, N, r, bits))


def bwla_workspace_bytes(M: int, K: int, N: int, r: int, bits: int) -> int:
    return int(_lib.bwla_workspace_bytes(M, K, N, r, bits))


def new_workspace(M: int, K: int, N: int, r: int, bits: int, device="cuda") -> torch.Tensor:
    """Scratch buffer for bwla_w1ax_linear / bwla_w1a_gemm_codes (device memory from PyTorch, zero-filled)."""
    n = bwla_workspace_bytes(M, K, N, r, bits)
    if n == 0:
        raise ValueError("invalid dimensions")
    return torch.zeros(n, dtype=torch.uint8, device=device)


def bwla_pack_signs(w: torch.Tensor, packed: Optional[torch.Tensor] = None) -> torch.Tensor:
    """w: fp32 or bf16 [N][K] (row stride >= K) -> uint32 words stored as int32 [N][K/32]."""
    if w.dtype not in (torch.float32, torch.bfloat16):
        raise TypeError("w must be fp32 or bf16")
    _need(w, w.dtype, "w", 2)
    N, K = w.shape
    if packed is None:
        packed = torch.empty((N, K // 32), dtype=torch.int32, device=w.device)
    _need(packed, torch.int32, "packed", 2)
    st = _lib.bwla_pack_signs(_ptr(w), 0 if w.dtype == torch.float32 else 1, N, K, w.stride(0) if N > 0 else K,
                              _ptr(packed), _stream())
    _check(st, "bwla_pack_signs")
    return packed


def bwla_binarize_workspace_bytes(K: int) -> int:
    return int(_lib.bwla_binarize_workspace_bytes(K))


def bwla_binarize_rows(w_res: torch.Tensor, P1: torch.Tensor, P2: torch.Tensor, workspace: Optional[torch.Tensor] = None):
    """w_res: fp32 or bf16 [N][K] (row stride >= K) -> (packed int32 [N][K/32], alpha fp32 [N], mu fp32 [N]) of the rows
    rotated by P1 (x) P2 (Alg. 2, last step)."""
    if w_res.dtype not in (torch.float32, torch.bfloat16):
        raise TypeError("w_res must be fp32 or bf16")
    _need(w_res, w_res.dtype, "w_res", 2)
    _need(P1, torch.float32, "P1", 2)
    _need(P2, torch.float32, "P2", 2)
    N, K = w_res.shape
    packed = torch.empty((N, K // 32), dtype=torch.int32, device=w_res.device)
    alpha = torch.empty(N, dtype=torch.float32, device=w_res.device)
    mu = torch.empty(N, dtype=torch.float32, device=w_res.device)
    if workspace is None:
        workspace = torch.zeros(bwla_binarize_workspace_bytes(K), dtype=torch.uint8, device=w_res.device)
    st = _lib.bwla_binarize_rows(_ptr(w_res), 0 if w_res.dtype == torch.float32 else 1, N, K, w_res.stride(0) if N > 0 else K,
                                 _ptr(P1), P1.shape[0], _ptr(P2), P2.shape[0], _ptr(packed), _ptr(alpha), _ptr(mu),
                                 _ptr(workspace), workspace.numel(), _stream())
    _check(st, "bwla_binarize_rows")
    return packed, alpha, mu


def bwla_rotate_quant_act(x: torch.Tensor, P1: torch.Tensor, P2: torch.Tensor, bits: int,
                          codes: Optional[torch.Tensor] = None, scales: Optional[torch.Tensor] = None):
    """x: bf16 [M][K]; P1 fp32 [n1][n1]; P2 fp32 [n2][n2] -> (codes int8 [M][K], scales fp32 [M])."""
    _need(x, torch.bfloat16, "x", 2)
    _need(P1, torch.float32, "P1", 2)
    _need(P2, torch.float32, "P2", 2)
    M, K = x.shape
    if codes is None:
        codes = torch.empty((M, K), dtype=torch.int8, device=x.device)
    if scales is None:
        scales = torch.empty((M,), dtype=torch.float32, device=x.device)
    st = _lib.bwla_rotate_quant_act(_ptr(x), M, K, x.stride(0) if M > 0 else K, _ptr(P1.contiguous()), P1.shape[0],
                                    _ptr(P2.contiguous()), P2.shape[0], bits, _ptr(codes), _ptr(scales), _stream())
    _check(st, "bwla_rotate_quant_act")
    return codes, scales


def _linear_args(x, P1, P2, packed, alpha, U, V, mu, out):
    """Type and layout checks shared by the two whole-layer entry points; returns (M, K, N, r, out)."""
    _need(x, torch.bfloat16, "x", 2)
    _need(packed, torch.int32, "packed", 2)
    _need(alpha, torch.float32, "alpha", 1)
    M, K = x.shape
    N = packed.shape[0]
    r = 0
    if U is not None:
        _need(U, torch.bfloat16, "U", 2)
        _need(V, torch.bfloat16, "V", 2)
        r = U.shape[1]
        if not (U.is_contiguous() and V.is_contiguous()) or tuple(V.shape) != (r, K) or U.shape[0] != N:
            raise TypeError("U must be contiguous [N][r] and V contiguous [r][K]")
    if mu is not None:
        _need(mu, torch.float32, "mu", 1)
    if not (packed.is_contiguous() and P1.is_contiguous() and P2.is_contiguous()):
        raise TypeError("packed, P1 and P2 must be contiguous")
    if out is None:
        out = torch.empty((M, N), dtype=torch.bfloat16, device=x.device)
    _need(out, torch.bfloat16, "out", 2)
    return M, K, N, r, out


def bwla_w1ax_linear(x: torch.Tensor, P1: torch.Tensor, P2: torch.Tensor, bits: int, packed: torch.Tensor,
                     alpha: torch.Tensor, U: Optional[torch.Tensor] = None, V: Optional[torch.Tensor] = None,
                     mu: Optional[torch.Tensor] = None, out: Optional[torch.Tensor] = None,
                     workspace: Optional[torch.Tensor] = None) -> torch.Tensor:
    """The whole layer: bf16 x [M][K] -> bf16 out [M][N]."""
    M, K, N, r, out = _linear_args(x, P1, P2, packed, alpha, U, V, mu, out)
    if workspace is None:
        workspace = new_workspace(M, K, N, r, bits, x.device)
    st = _lib.bwla_w1ax_linear(_ptr(x), M, K, x.stride(0) if M > 0 else K, _ptr(P1), P1.shape[0], _ptr(P2),
                               P2.shape[0], bits, _ptr(packed), _ptr(alpha), _ptr(mu), _ptr(U), _ptr(V), r,
                               _ptr(out), N, out.stride(0) if M > 0 else N, _ptr(workspace), workspace.numel(),
                               _stream())
    _check(st, "bwla_w1ax_linear")
    return out


def bwla_w1ax_linear_static(x: torch.Tensor, P1: torch.Tensor, P2: torch.Tensor, bits: int, packed: torch.Tensor,
                            alpha: torch.Tensor, U: Optional[torch.Tensor] = None, V: Optional[torch.Tensor] = None,
                            mu: Optional[torch.Tensor] = None, out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """The whole layer through the entry point that owns its scratch memory (see include/bwla.h): for callers that
    cannot allocate a workspace.  `out` should be passed by such a caller; it is created here only for convenience.
    Calls share one built-in scratch array per device and must not overlap on the GPU."""
    M, K, N, r, out = _linear_args(x, P1, P2, packed, alpha, U, V, mu, out)
    st = _lib.bwla_w1ax_linear_static(_ptr(x), M, K, x.stride(0) if M > 0 else K, _ptr(P1), P1.shape[0], _ptr(P2),
                                      P2.shape[0], bits, _ptr(packed), _ptr(alpha), _ptr(mu), _ptr(U), _ptr(V), r,
                                      _ptr(out), N, out.stride(0) if M > 0 else N, _stream())
    _check(st, "bwla_w1ax_linear_static")
    return out


class Layer:
    """A prepared layer (bwla_layer_create): keeps the handle, the tensors it points into and the prepared buffer."""

    def __init__(self, P1, P2, bits, packed, alpha, U=None, V=None, mu=None, asymmetric=False):
        _need(packed, torch.int32, "packed", 2)
        _need(alpha, torch.float32, "alpha", 1)
        _need(P1, torch.float32, "P1", 2)
        _need(P2, torch.float32, "P2", 2)
        if not (packed.is_contiguous() and P1.is_contiguous() and P2.is_contiguous()):
            raise TypeError("packed, P1 and P2 must be contiguous")
        self.N, self.K = packed.shape[0], packed.shape[1] * 32
        self.n1, self.n2, self.bits = P1.shape[0], P2.shape[0], bits
        self.r = 0
        if U is not None:
            _need(U, torch.bfloat16, "U", 2)
            _need(V, torch.bfloat16, "V", 2)
            self.r = U.shape[1]
            if not (U.is_contiguous() and V.is_contiguous()) or tuple(V.shape) != (self.r, self.K) or U.shape[0] != self.N:
                raise TypeError("U must be contiguous [N][r] and V contiguous [r][K]")
        if mu is not None:
            _need(mu, torch.float32, "mu", 1)
        self.tensors = (P1, P2, packed, alpha, U, V, mu)
        nbytes = int(_lib.bwla_layer_prepared_bytes(self.K, self.N, self.n1, self.n2, self.r))
        if nbytes == 0:
            raise BwlaError(BWLA_ERR_INVALID_ARG, "bwla_layer_prepared_bytes")
        self.prepared = torch.empty(nbytes, dtype=torch.uint8, device=packed.device)
        self.handle = C.c_void_p()
        st = _lib.bwla_layer_create(C.byref(self.handle), self.K, self.N, _ptr(P1), self.n1, _ptr(P2), self.n2, bits,
                                    _ptr(packed), _ptr(alpha), _ptr(mu), _ptr(U), _ptr(V), self.r, _ptr(self.prepared),
                                    nbytes, _stream())
        _check(st, "bwla_layer_create")
        if asymmetric:
            bwla_layer_set_activation_quant(self, BWLA_ACT_ASYMMETRIC)

    def __del__(self):
        h = getattr(self, "handle", None)
        if h is not None and h.value and _lib is not None:      # (_lib is None while the interpreter shuts down)
            _lib.bwla_layer_destroy(h)
            self.handle = C.c_void_p()


def bwla_w1a16_workspace_bytes(layer: Layer, M: int) -> int:
    return int(_lib.bwla_w1a16_workspace_bytes(layer.handle, M))


def bwla_layer_w1a16_linear(layer: Layer, x: torch.Tensor, out: Optional[torch.Tensor] = None,
                            workspace: Optional[torch.Tensor] = None) -> torch.Tensor:
    """The weight-only layer (W1A16): bf16 x [M][K] -> bf16 out [M][N], rotated activations kept in bf16."""
    _need(x, torch.bfloat16, "x", 2)
    M = x.shape[0]
    if out is None:
        out = torch.empty((M, layer.N), dtype=torch.bfloat16, device=x.device)
    _need(out, torch.bfloat16, "out", 2)
    if workspace is None:
        workspace = torch.zeros(max(256, bwla_w1a16_workspace_bytes(layer, M)), dtype=torch.uint8, device=x.device)
    st = _lib.bwla_layer_w1a16_linear(layer.handle, _ptr(x), M, x.stride(0) if M > 0 else layer.K, _ptr(out),
                                      out.stride(0) if M > 0 else layer.N, _ptr(workspace), workspace.numel(), _stream())
    _check(st, "bwla_layer_w1a16_linear")
    return out


def bwla_layer_prepared_bytes(K: int, N: int, n1: int, n2: int, r: int) -> int:
    return int(_lib.bwla_layer_prepared_bytes(K, N, n1, n2, r))


def bwla_layer_create(P1, P2, bits, packed, alpha, U=None, V=None, mu=None, asymmetric=False) -> Layer:
    """Prepares a layer's constants once (launches on the current stream) and returns the handle object."""
    return Layer(P1, P2, bits, packed, alpha, U, V, mu, asymmetric)


def bwla_layer_destroy(layer: Layer) -> None:
    layer.__del__()


def bwla_layer_set_activation_quant(layer: Layer, mode: int) -> None:
    _check(_lib.bwla_layer_set_activation_quant(layer.handle, mode), "bwla_layer_set_activation_quant")


def bwla_layer_rotate_quant_asym(layer: Layer, x: torch.Tensor, want_y: bool = False):
    """(codes uint8 [M][K], scales fp32 [M], zeros int32 [M], Y fp32 [M][K] or None): the per-token asymmetric quantiser."""
    _need(x, torch.bfloat16, "x", 2)
    M, K = x.shape
    codes = torch.empty((M, K), dtype=torch.uint8, device=x.device)
    scales = torch.empty((M,), dtype=torch.float32, device=x.device)
    zeros = torch.empty((M,), dtype=torch.int32, device=x.device)
    y = torch.empty((M, K), dtype=torch.float32, device=x.device) if want_y else None
    st = _lib.bwla_layer_rotate_quant_asym(layer.handle, _ptr(x), M, x.stride(0) if M > 0 else K, _ptr(codes), _ptr(scales),
                                           _ptr(zeros), _ptr(y), _stream())
    _check(st, "bwla_layer_rotate_quant_asym")
    return codes, scales, zeros, y


def bwla_layer_rotate_quant(layer: Layer, x: torch.Tensor, want_y: bool = False):
    """(codes int8 [M][K], scales fp32 [M], Y fp32 [M][K] or None) through a prepared layer."""
    _need(x, torch.bfloat16, "x", 2)
    M, K = x.shape
    codes = torch.empty((M, K), dtype=torch.int8, device=x.device)
    scales = torch.empty((M,), dtype=torch.float32, device=x.device)
    y = torch.empty((M, K), dtype=torch.float32, device=x.device) if want_y else None
    st = _lib.bwla_layer_rotate_quant(layer.handle, _ptr(x), M, x.stride(0) if M > 0 else K, _ptr(codes), _ptr(scales),
                                      _ptr(y), _stream())
    _check(st, "bwla_layer_rotate_quant")
    return codes, scales, y


def _handles(layers):
    arr = (C.c_void_p * len(layers))(*[l.handle.value for l in layers])
    return arr


def bwla_group_workspace_bytes(layers, M: int) -> int:
    return int(_lib.bwla_group_workspace_bytes(_handles(layers), len(layers), M))


def new_group_workspace(layers, M: int, device="cuda") -> torch.Tensor:
    n = bwla_group_workspace_bytes(layers, M)
    if n == 0:
        raise ValueError("invalid group")
    return torch.zeros(n, dtype=torch.uint8, device=device)


def bwla_w1ax_linear_group(layers, x: torch.Tensor, outs=None, workspace: Optional[torch.Tensor] = None):
    """Layers that share x (q/k/v, gate/up) in one call; returns the list of bf16 outputs [M][N_i]."""
    _need(x, torch.bfloat16, "x", 2)
    M, K = x.shape
    if outs is None:
        outs = [torch.empty((M, l.N), dtype=torch.bfloat16, device=x.device) for l in layers]
    for o in outs:
        _need(o, torch.bfloat16, "out", 2)
    if workspace is None:
        workspace = new_group_workspace(layers, M, x.device)
    optr = (C.c_void_p * len(layers))(*[o.data_ptr() for o in outs])
    ldos = (C.c_int64 * len(layers))(*[(o.stride(0) if M > 0 else l.N) for o, l in zip(outs, layers)])
    st = _lib.bwla_w1ax_linear_group(_handles(layers), len(layers), _ptr(x), M, x.stride(0) if M > 0 else K, optr, ldos,
                                     _ptr(workspace), workspace.numel(), _stream())
    _check(st, "bwla_w1ax_linear_group")
    return outs


def bwla_w1a_gemm_codes(codes: torch.Tensor, scales: torch.Tensor, bits: int, packed: torch.Tensor,
                        alpha: torch.Tensor, x: Optional[torch.Tensor] = None, U: Optional[torch.Tensor] = None,
                        V: Optional[torch.Tensor] = None, mu: Optional[torch.Tensor] = None,
                        out: Optional[torch.Tensor] = None, acc: Optional[torch.Tensor] = None,
                        want_out: bool = True, want_acc: bool = False, workspace: Optional[torch.Tensor] = None):
    """Contraction + epilogue from given int8 codes [M][K]; returns (out bf16 or None, acc int32 or None)."""
    _need(codes, torch.int8, "codes", 2)
    _need(scales, torch.float32, "scales", 1)
    _need(packed, torch.int32, "packed", 2)
    _need(alpha, torch.float32, "alpha", 1)
    M, K = codes.shape
    N = packed.shape[0]
    r = 0
    if U is not None:
        _need(U, torch.bfloat16, "U", 2)
        _need(V, torch.bfloat16, "V", 2)
        _need(x, torch.bfloat16, "x", 2)
        r = U.shape[1]
    if not codes.is_contiguous() or not packed.is_contiguous():
        raise TypeError("codes and packed must be contiguous")
    if out is None and want_out:
        out = torch.empty((M, N), dtype=torch.bfloat16, device=codes.device)
    if acc is None and want_acc:
        acc = torch.empty((M, N), dtype=torch.int32, device=codes.device)
    if workspace is None:
        workspace = new_workspace(M, K, N, r, bits, codes.device)
    st = _lib.bwla_w1a_gemm_codes(_ptr(codes), _ptr(scales), M, K, bits, _ptr(packed), _ptr(alpha), _ptr(mu),
                                  _ptr(x), x.stride(0) if (x is not None and M > 0) else K, _ptr(U), _ptr(V), r,
                                  _ptr(out), N, out.stride(0) if (out is not None and M > 0) else N, _ptr(acc),
                                  _ptr(workspace), workspace.numel(), _stream())
    _check(st, "bwla_w1a_gemm_codes")
    return out, acc


BWLA_WS_SCALES, BWLA_WS_QSUM, BWLA_WS_T, BWLA_WS_CODES, BWLA_WS_ZEROS = 0, 1, 2, 3, 4
BWLA_ACT_SYMMETRIC, BWLA_ACT_ASYMMETRIC = 0, 1


def bwla_workspace_section(M: int, K: int, N: int, r: int, bits: int, which: int):
    """(offset, bytes) of one intermediate inside the workspace of bwla_w1ax_linear."""
    off, nb = C.c_size_t(0), C.c_size_t(0)
    _check(_lib.bwla_workspace_section(M, K, N, r, bits, which, C.byref(off), C.byref(nb)), "bwla_workspace_section")
    return int(off.value), int(nb.value)


def bwla_check_status(workspace: torch.Tensor) -> int:
    """Synchronises the current stream and returns the status a bounded device-side wait may have left."""
    return int(_lib.bwla_check_status(_ptr(workspace), _stream()))


PROFILE_KINDS = ("prologue", "unused1", "contraction", "unused3", "prepare_codes", "pack_signs")


def bwla_profile_enable(on: bool) -> None:
    _check(_lib.bwla_profile_enable(1 if on else 0), "bwla_profile_enable")


def bwla_profile_collect() -> dict:
    """Waits for the recorded events; returns {kind: (total_ms, launches)}."""
    ms = (C.c_float * 8)()
    n = (C.c_int * 8)()
    _check(_lib.bwla_profile_collect(ms, n), "bwla_profile_collect")
    return {k: (float(ms[i]), int(n[i])) for i, k in enumerate(PROFILE_KINDS)}

"""Thin ctypes binding of libisopo.so: same names as the C ABI, argument marshalling only.

Every step of the path runs in the library's CUDA kernels.  torch is used for device memory and
the current stream, nothing else.  Importing this module without a built library raises.
"""

from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import numpy as np
import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
# ISOPO_LIB_VARIANT=debug selects the range-checking build (libisopo_debug.so, `build(debug=True)`)
LIB_PATH = os.path.join(_PKG, "libisopo_debug.so" if os.environ.get("ISOPO_LIB_VARIANT") == "debug" else "libisopo.so")

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_CUDA = range(5)
F32, BF16 = 0, 1
PATH_AUTO, PATH_GRAM, PATH_MATERIALISE = 0, 1, 2
(VAR_REINFORCE, VAR_NORMALISED, VAR_DIRECTION, VAR_EUCLID, VAR_GENERAL, VAR_INTERACTING,
 VAR_NORMALISED_RAW) = range(7)
INFO_TIMEOUT = 0x40000000
INFO_STALE_WORKSPACE = 0x10000000
INFO_SATURATED = 0x04000000

EXPORTS = (
    "isopo_status_string", "isopo_last_cuda_error", "isopo_choose_path", "isopo_workspace_bytes",
    "isopo_layer_gram", "isopo_transform_advantages", "isopo_weight_grad", "isopo_layer_gram_shared_x",
    "isopo_layer_gram_shared_x_stored",
    "isopo_profile_enable", "isopo_profile_collect", "isopo_kernel_name", "isopo_layer_gram_static",
    "isopo_sampled_workspace_bytes", "isopo_sampled_coefficients",
    "isopo_reg_ema_update", "isopo_transform_advantages_rel", "isopo_transform_advantages_batched",
    "isopo_spectral_workspace_bytes", "isopo_transform_spectral", "isopo_transform_spectral_batched",
    "isopo_selftest_bounded_wait", "isopo_set_deterministic", "isopo_get_deterministic", "isopo_debug_build",
    "isopo_set_store_format", "isopo_get_store_format",
    "isopo_transform_large_workspace_bytes", "isopo_transform_advantages_large",
)
MAX_LARGE_SEQS = 1024
MAX_SAMPLES = 4096
STATIC_MAX_TOKENS, STATIC_MAX_SEQS = 65536, 256
NUM_KERNELS = 17


class IsopoError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        super().__init__(what)


def _load():
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2512_23353_b200.build` "
            "(there is no CPU or PyTorch fallback)")
    lib = ctypes.CDLL(LIB_PATH)
    c = ctypes
    lib.isopo_status_string.restype = c.c_char_p
    lib.isopo_status_string.argtypes = [c.c_int]
    lib.isopo_last_cuda_error.restype = c.c_char_p
    lib.isopo_last_cuda_error.argtypes = []
    lib.isopo_choose_path.restype = c.c_int
    lib.isopo_choose_path.argtypes = [c.c_int, c.c_int64, c.c_int, c.c_int, c.c_int]
    lib.isopo_workspace_bytes.restype = c.c_size_t
    lib.isopo_workspace_bytes.argtypes = [c.c_int, c.c_int64, c.c_int, c.c_int, c.c_int, c.c_int]
    lib.isopo_layer_gram.restype = c.c_int
    lib.isopo_layer_gram.argtypes = [c.c_void_p, c.c_void_p, c.c_int, c.c_int64, c.c_int, c.c_int, c.c_void_p,
                                     c.c_int, c.c_int, c.c_void_p, c.c_void_p, c.c_size_t, c.c_void_p, c.c_void_p]
    lib.isopo_layer_gram_shared_x.restype = c.c_int
    lib.isopo_layer_gram_shared_x.argtypes = [c.c_void_p, c.c_int, c.c_void_p, c.c_void_p, c.c_int, c.c_int64, c.c_int,
                                              c.c_void_p, c.c_int, c.c_void_p, c.c_void_p, c.c_size_t, c.c_void_p,
                                              c.c_void_p]
    lib.isopo_layer_gram_shared_x_stored.restype = c.c_int
    lib.isopo_layer_gram_shared_x_stored.argtypes = [c.c_void_p, c.c_int, c.c_void_p, c.c_void_p, c.c_int, c.c_int64,
                                                     c.c_int, c.c_void_p, c.c_int, c.c_void_p, c.c_void_p, c.c_void_p,
                                                     c.c_void_p, c.c_void_p]
    lib.isopo_transform_advantages.restype = c.c_int
    lib.isopo_transform_advantages.argtypes = [c.c_void_p, c.c_void_p, c.c_int, c.c_int, c.c_float, c.c_void_p,
                                               c.c_void_p, c.c_void_p, c.c_void_p]
    lib.isopo_weight_grad.restype = c.c_int
    lib.isopo_weight_grad.argtypes = [c.c_void_p, c.c_void_p, c.c_int, c.c_int64, c.c_int, c.c_int, c.c_void_p,
                                      c.c_void_p, c.c_int, c.c_int, c.c_void_p, c.c_float, c.c_void_p, c.c_size_t,
                                      c.c_void_p, c.c_void_p]
    lib.isopo_layer_gram_static.restype = c.c_int
    lib.isopo_layer_gram_static.argtypes = [c.c_void_p, c.c_void_p, c.c_int, c.c_int64, c.c_int, c.c_int, c.c_void_p,
                                            c.c_int, c.c_void_p, c.c_void_p, c.c_void_p]
    lib.isopo_sampled_workspace_bytes.restype = c.c_size_t
    lib.isopo_sampled_workspace_bytes.argtypes = [c.c_int, c.c_int64, c.c_int, c.c_int, c.c_int, c.c_int]
    lib.isopo_sampled_coefficients.restype = c.c_int
    lib.isopo_sampled_coefficients.argtypes = [c.c_void_p, c.c_void_p, c.c_int, c.c_int64, c.c_int, c.c_int, c.c_void_p,
                                               c.c_int, c.c_void_p, c.c_int, c.c_void_p, c.c_float, c.c_void_p,
                                               c.c_void_p, c.c_void_p, c.c_size_t, c.c_void_p, c.c_void_p]
    lib.isopo_transform_large_workspace_bytes.restype = c.c_size_t
    lib.isopo_transform_large_workspace_bytes.argtypes = [c.c_int]
    lib.isopo_transform_advantages_large.restype = c.c_int
    lib.isopo_transform_advantages_large.argtypes = [c.c_void_p, c.c_void_p, c.c_int, c.c_float, c.c_void_p, c.c_void_p,
                                                     c.c_size_t, c.c_void_p, c.c_void_p]
    lib.isopo_reg_ema_update.restype = c.c_int
    lib.isopo_reg_ema_update.argtypes = [c.c_void_p, c.c_int, c.c_float, c.c_void_p, c.c_void_p]
    lib.isopo_transform_advantages_batched.restype = c.c_int
    lib.isopo_transform_advantages_batched.argtypes = [c.c_int, c.c_void_p, c.c_void_p, c.c_int, c.c_int, c.c_void_p,
                                                       c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p]
    lib.isopo_spectral_workspace_bytes.restype = c.c_size_t
    lib.isopo_spectral_workspace_bytes.argtypes = []
    lib.isopo_transform_spectral.restype = c.c_int
    lib.isopo_transform_spectral.argtypes = [c.c_void_p, c.c_void_p, c.c_int, c.c_float, c.c_float, c.c_void_p,
                                             c.c_void_p, c.c_void_p, c.c_size_t, c.c_void_p, c.c_void_p]
    lib.isopo_transform_spectral_batched.restype = c.c_int
    lib.isopo_transform_spectral_batched.argtypes = [c.c_int, c.c_void_p, c.c_void_p, c.c_int, c.c_void_p, c.c_float,
                                                     c.c_void_p, c.c_void_p, c.c_void_p, c.c_size_t, c.c_void_p,
                                                     c.c_void_p]
    lib.isopo_transform_advantages_rel.restype = c.c_int
    lib.isopo_transform_advantages_rel.argtypes = [c.c_void_p, c.c_void_p, c.c_int, c.c_int, c.c_float, c.c_void_p,
                                                   c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p]
    lib.isopo_set_store_format.restype = c.c_int
    lib.isopo_set_store_format.argtypes = [c.c_int]
    lib.isopo_get_store_format.restype = c.c_int
    lib.isopo_get_store_format.argtypes = []
    lib.isopo_set_deterministic.restype = None
    lib.isopo_set_deterministic.argtypes = [c.c_int]
    lib.isopo_get_deterministic.restype = c.c_int
    lib.isopo_get_deterministic.argtypes = []
    lib.isopo_debug_build.restype = c.c_int
    lib.isopo_debug_build.argtypes = []
    lib.isopo_selftest_bounded_wait.restype = c.c_int
    lib.isopo_selftest_bounded_wait.argtypes = [c.c_int64, c.c_void_p, c.c_void_p, c.c_void_p]
    lib.isopo_profile_enable.restype = None
    lib.isopo_profile_enable.argtypes = [c.c_int]
    lib.isopo_profile_collect.restype = c.c_int
    lib.isopo_profile_collect.argtypes = [c.c_void_p, c.c_void_p]
    lib.isopo_kernel_name.restype = c.c_char_p
    lib.isopo_kernel_name.argtypes = [c.c_int]
    return lib


lib = _load()


def _check(status: int, what: str):
    if status != OK:
        name = lib.isopo_status_string(status).decode()
        extra = f" [{lib.isopo_last_cuda_error().decode()}]" if status == ERR_CUDA else ""
        raise IsopoError(status, f"{what}: {name}{extra}")


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    raise TypeError(f"unsupported dtype {t.dtype}")


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _offsets(seq_offsets) -> np.ndarray:
    off = np.ascontiguousarray(np.asarray(seq_offsets, dtype=np.int64))
    if off.ndim != 1 or off.shape[0] < 2:
        raise ValueError("seq_offsets must be a 1-D array of B+1 entries")
    return off


def isopo_choose_path(dtype: int, T: int, d_in: int, d_out: int, B: int) -> int:
    return lib.isopo_choose_path(dtype, T, d_in, d_out, B)


def isopo_workspace_bytes(dtype: int, T: int, d_in: int, d_out: int, B: int, path: int = PATH_AUTO) -> int:
    return lib.isopo_workspace_bytes(dtype, T, d_in, d_out, B, path)


def alloc_workspace(dtype: int, T: int, d_in: int, d_out: int, B: int, path: int = PATH_AUTO, device="cuda"):
    """A torch uint8 buffer of the size the library asks for (torch's allocator aligns to 512 B; the
    view returned starts on a 1024-byte boundary)."""
    n = isopo_workspace_bytes(dtype, T, d_in, d_out, B, path)
    if n == 0:
        raise IsopoError(ERR_INVALID_ARG, "isopo_workspace_bytes: invalid sizes")
    raw = torch.empty(n + 1024, dtype=torch.uint8, device=device)
    shift = (-raw.data_ptr()) % 1024
    return raw[shift:shift + n]


def isopo_layer_gram(X: torch.Tensor, dY: torch.Tensor, seq_offsets, K: torch.Tensor, ws: torch.Tensor,
                     info: torch.Tensor, path: int = PATH_AUTO) -> None:
    off = _offsets(seq_offsets)
    B = off.shape[0] - 1
    assert X.is_cuda and dY.is_cuda and X.is_contiguous() and dY.is_contiguous() and X.dtype == dY.dtype
    assert K.dtype == torch.float32 and K.is_contiguous() and K.numel() == B * B
    assert info.dtype == torch.int32 and ws.dtype == torch.uint8
    st = lib.isopo_layer_gram(X.data_ptr(), dY.data_ptr(), _dtype_code(X), X.shape[0], X.shape[1], dY.shape[1],
                              off.ctypes.data, B, path, K.data_ptr(), ws.data_ptr(), ws.numel(), info.data_ptr(),
                              _stream())
    _check(st, "isopo_layer_gram")


def isopo_layer_gram_shared_x(X: torch.Tensor, dYs, seq_offsets, Ks, ws: torch.Tensor, info: torch.Tensor) -> None:
    """Gram-route K of up to three projections dYs[h] that share the input X, in one launch."""
    off = _offsets(seq_offsets)
    B = off.shape[0] - 1
    n = len(dYs)
    assert len(Ks) == n and X.is_cuda and X.is_contiguous()
    for dY, K in zip(dYs, Ks):
        assert dY.is_cuda and dY.is_contiguous() and dY.dtype == X.dtype and dY.shape[0] == X.shape[0]
        assert K.dtype == torch.float32 and K.is_contiguous() and K.numel() == B * B
    dy_ptrs = np.array([d.data_ptr() for d in dYs], dtype=np.uint64)
    k_ptrs = np.array([K.data_ptr() for K in Ks], dtype=np.uint64)
    widths = np.array([d.shape[1] for d in dYs], dtype=np.int32)
    st = lib.isopo_layer_gram_shared_x(X.data_ptr(), n, dy_ptrs.ctypes.data, widths.ctypes.data, _dtype_code(X),
                                       X.shape[0], X.shape[1], off.ctypes.data, B, k_ptrs.ctypes.data, ws.data_ptr(),
                                       ws.numel(), info.data_ptr(), _stream())
    _check(st, "isopo_layer_gram_shared_x")


def isopo_layer_gram_shared_x_stored(X: torch.Tensor, dYs, seq_offsets, Ks, wss, info: torch.Tensor) -> None:
    """Stored-gradient-route K of up to three projections dYs[h] that share the input X: one launch forms all
    their per-sequence gradients; wss[h] is projection h's own workspace (MATERIALISE size)."""
    off = _offsets(seq_offsets)
    B = off.shape[0] - 1
    n = len(dYs)
    assert len(Ks) == n and len(wss) == n and X.is_cuda and X.is_contiguous()
    for dY, K, ws in zip(dYs, Ks, wss):
        assert dY.is_cuda and dY.is_contiguous() and dY.dtype == X.dtype and dY.shape[0] == X.shape[0]
        assert K.dtype == torch.float32 and K.is_contiguous() and K.numel() == B * B and ws.dtype == torch.uint8
    dy_ptrs = np.array([d.data_ptr() for d in dYs], dtype=np.uint64)
    k_ptrs = np.array([K.data_ptr() for K in Ks], dtype=np.uint64)
    ws_ptrs = np.array([w.data_ptr() for w in wss], dtype=np.uint64)
    ws_sizes = np.array([w.numel() for w in wss], dtype=np.uint64)
    widths = np.array([d.shape[1] for d in dYs], dtype=np.int32)
    st = lib.isopo_layer_gram_shared_x_stored(X.data_ptr(), n, dy_ptrs.ctypes.data, widths.ctypes.data, _dtype_code(X),
                                              X.shape[0], X.shape[1], off.ctypes.data, B, k_ptrs.ctypes.data,
                                              ws_ptrs.ctypes.data, ws_sizes.ctypes.data, info.data_ptr(), _stream())
    _check(st, "isopo_layer_gram_shared_x_stored")


def isopo_layer_gram_static(X: torch.Tensor, dY: torch.Tensor, seq_offsets, K: torch.Tensor,
                            info: torch.Tensor) -> None:
    """isopo_layer_gram on the Gram route for callers that cannot allocate: the scratch is a fixed
    array inside the library (at most STATIC_MAX_TOKENS tokens and STATIC_MAX_SEQS sequences).
    Calls on one device share that array, so do not let two of them overlap on the GPU."""
    off = _offsets(seq_offsets)
    B = off.shape[0] - 1
    assert X.is_cuda and dY.is_cuda and X.is_contiguous() and dY.is_contiguous() and X.dtype == dY.dtype
    assert K.dtype == torch.float32 and K.is_contiguous() and K.numel() == B * B and info.dtype == torch.int32
    st = lib.isopo_layer_gram_static(X.data_ptr(), dY.data_ptr(), _dtype_code(X), X.shape[0], X.shape[1],
                                     dY.shape[1], off.ctypes.data, B, K.data_ptr(), info.data_ptr(), _stream())
    if st == ERR_UNSUPPORTED:
        raise IsopoError(st, f"isopo_layer_gram_static: ISOPO_ERR_UNSUPPORTED [{lib.isopo_last_cuda_error().decode()}]")
    _check(st, "isopo_layer_gram_static")


def isopo_transform_advantages(K: torch.Tensor, A: torch.Tensor, variant: int, lam: float, coeffs: torch.Tensor,
                               info: torch.Tensor, pqr_regs=None) -> None:
    B = A.numel()
    assert K.dtype == torch.float32 and A.dtype == torch.float32 and coeffs.dtype == torch.float32
    assert K.is_contiguous() and K.numel() == B * B and coeffs.numel() == B
    g = None
    if pqr_regs is not None:
        g = np.ascontiguousarray(np.asarray(pqr_regs, dtype=np.float32))
        assert g.shape == (6,)
    st = lib.isopo_transform_advantages(K.data_ptr(), A.data_ptr(), B, variant, float(lam),
                                        g.ctypes.data if g is not None else None, coeffs.data_ptr(),
                                        info.data_ptr(), _stream())
    _check(st, "isopo_transform_advantages")


def isopo_transform_large_workspace_bytes(B: int) -> int:
    return int(lib.isopo_transform_large_workspace_bytes(B))


def isopo_transform_advantages_large(K: torch.Tensor, A: torch.Tensor, lam: float, coeffs: torch.Tensor, ws: torch.Tensor,
                                     info: torch.Tensor) -> None:
    B = A.numel()
    assert K.dtype == torch.float32 and A.dtype == torch.float32 and coeffs.dtype == torch.float32
    assert K.is_contiguous() and K.numel() == B * B and coeffs.numel() == B and ws.dtype == torch.uint8
    st = lib.isopo_transform_advantages_large(K.data_ptr(), A.data_ptr(), B, float(lam), coeffs.data_ptr(), ws.data_ptr(),
                                              ws.numel(), info.data_ptr(), _stream())
    _check(st, "isopo_transform_advantages_large")


def isopo_reg_ema_update(K: torch.Tensor, decay: float, state: torch.Tensor) -> None:
    """Folds this microbatch's K into the running means `state` (device float32 [4], zeroed once by the caller)."""
    B = K.shape[0]
    assert K.dtype == torch.float32 and K.is_contiguous() and K.numel() == B * B
    assert state.dtype == torch.float32 and state.numel() == 4 and state.is_cuda
    _check(lib.isopo_reg_ema_update(K.data_ptr(), B, float(decay), state.data_ptr(), _stream()), "isopo_reg_ema_update")


def isopo_transform_advantages_rel(K: torch.Tensor, A: torch.Tensor, variant: int, factor: float, state: torch.Tensor,
                                   coeffs: torch.Tensor, info: torch.Tensor, pqr_factors=None) -> None:
    """isopo_transform_advantages with the regulariser = factor x the running mean kept in `state`."""
    B = A.numel()
    assert K.dtype == torch.float32 and A.dtype == torch.float32 and coeffs.dtype == torch.float32
    assert K.is_contiguous() and K.numel() == B * B and coeffs.numel() == B and state.numel() == 4
    g = None
    if pqr_factors is not None:
        g = np.ascontiguousarray(np.asarray(pqr_factors, dtype=np.float32))
        assert g.shape == (6,)
    st = lib.isopo_transform_advantages_rel(K.data_ptr(), A.data_ptr(), B, variant, float(factor),
                                            g.ctypes.data if g is not None else None, state.data_ptr(),
                                            coeffs.data_ptr(), info.data_ptr(), _stream())
    _check(st, "isopo_transform_advantages_rel")


def isopo_transform_advantages_batched(Ks, A: torch.Tensor, variant: int, lams, coeffs, info: torch.Tensor,
                                       pqr_regs=None, states=None) -> None:
    """One launch for the layers Ks[l] -> coeffs[l] (lists of tensors); lams are absolute regularisers, or
    factors of the running means when `states` (a list of device float32 [4] tensors) is given."""
    n, B = len(Ks), A.numel()
    assert len(coeffs) == n and len(lams) == n and (states is None or len(states) == n)
    for K, co in zip(Ks, coeffs):
        assert K.dtype == torch.float32 and K.is_contiguous() and K.numel() == B * B
        assert co.dtype == torch.float32 and co.is_contiguous() and co.numel() == B
    assert A.dtype == torch.float32
    k_ptrs = np.array([K.data_ptr() for K in Ks], dtype=np.uint64)
    c_ptrs = np.array([co.data_ptr() for co in coeffs], dtype=np.uint64)
    lam = np.ascontiguousarray(np.asarray(lams, dtype=np.float32))
    s_ptrs = None
    if states is not None:
        for stt in states:
            assert stt.dtype == torch.float32 and stt.numel() == 4 and stt.is_cuda
        s_ptrs = np.array([stt.data_ptr() for stt in states], dtype=np.uint64)
    g = None
    if pqr_regs is not None:
        g = np.ascontiguousarray(np.asarray(pqr_regs, dtype=np.float32))
        assert g.shape == (6,)
    st = lib.isopo_transform_advantages_batched(n, k_ptrs.ctypes.data, A.data_ptr(), B, variant, lam.ctypes.data,
                                                g.ctypes.data if g is not None else None,
                                                s_ptrs.ctypes.data if s_ptrs is not None else None,
                                                c_ptrs.ctypes.data, info.data_ptr(), _stream())
    _check(st, "isopo_transform_advantages_batched")


INFO_NO_CONVERGENCE = 0x20000000


def isopo_transform_spectral(K: torch.Tensor, A: torch.Tensor, lam: float, coeffs: torch.Tensor, info: torch.Tensor,
                             rel_cutoff: float = 0.0, eigenvalues: torch.Tensor | None = None,
                             ws: torch.Tensor | None = None) -> None:
    """Interacting coefficients through the eigendecomposition of K (Alg. 2 as printed), optionally with the
    spectrum (largest first) and with the directions below rel_cutoff * max(D) left out."""
    B = A.numel()
    assert K.dtype == torch.float32 and A.dtype == torch.float32 and coeffs.dtype == torch.float32
    assert K.is_contiguous() and K.numel() == B * B and coeffs.numel() == B
    assert eigenvalues is None or (eigenvalues.dtype == torch.float32 and eigenvalues.numel() == B)
    if ws is None:
        ws = torch.empty(lib.isopo_spectral_workspace_bytes(), dtype=torch.uint8, device=K.device)
    st = lib.isopo_transform_spectral(K.data_ptr(), A.data_ptr(), B, float(lam), float(rel_cutoff), coeffs.data_ptr(),
                                      eigenvalues.data_ptr() if eigenvalues is not None else None, ws.data_ptr(),
                                      ws.numel(), info.data_ptr(), _stream())
    _check(st, "isopo_transform_spectral")


def isopo_transform_spectral_batched(Ks, A: torch.Tensor, lams, coeffs, info: torch.Tensor, rel_cutoff: float = 0.0,
                                     eigenvalues=None, ws: torch.Tensor | None = None) -> None:
    """isopo_transform_spectral for the layers Ks[l] -> coeffs[l] (and eigenvalues[l]) in one launch."""
    n, B = len(Ks), A.numel()
    assert len(coeffs) == n and len(lams) == n and (eigenvalues is None or len(eigenvalues) == n)
    for K, co in zip(Ks, coeffs):
        assert K.dtype == torch.float32 and K.is_contiguous() and K.numel() == B * B
        assert co.dtype == torch.float32 and co.is_contiguous() and co.numel() == B
    k_ptrs = np.array([K.data_ptr() for K in Ks], dtype=np.uint64)
    c_ptrs = np.array([co.data_ptr() for co in coeffs], dtype=np.uint64)
    e_ptrs = None
    if eigenvalues is not None:
        e_ptrs = np.array([e.data_ptr() if e is not None else 0 for e in eigenvalues], dtype=np.uint64)
    lam = np.ascontiguousarray(np.asarray(lams, dtype=np.float32))
    if ws is None:
        ws = torch.empty(n * lib.isopo_spectral_workspace_bytes(), dtype=torch.uint8, device=A.device)
    st = lib.isopo_transform_spectral_batched(n, k_ptrs.ctypes.data, A.data_ptr(), B, lam.ctypes.data, float(rel_cutoff),
                                              c_ptrs.ctypes.data, e_ptrs.ctypes.data if e_ptrs is not None else None,
                                              ws.data_ptr(), ws.numel(), info.data_ptr(), _stream())
    _check(st, "isopo_transform_spectral_batched")


def isopo_weight_grad(X: torch.Tensor, dY: torch.Tensor, coeffs: torch.Tensor, seq_offsets, dW: torch.Tensor,
                      ws: torch.Tensor, info: torch.Tensor, path: int = PATH_AUTO, beta: float = 0.0) -> None:
    off = _offsets(seq_offsets)
    B = off.shape[0] - 1
    assert dW.dtype == torch.float32 and dW.is_contiguous() and dW.shape == (dY.shape[1], X.shape[1])
    assert coeffs.dtype == torch.float32 and coeffs.numel() == B
    st = lib.isopo_weight_grad(X.data_ptr(), dY.data_ptr(), _dtype_code(X), X.shape[0], X.shape[1], dY.shape[1],
                               coeffs.data_ptr(), off.ctypes.data, B, path, dW.data_ptr(), float(beta),
                               ws.data_ptr(), ws.numel(), info.data_ptr(), _stream())
    _check(st, "isopo_weight_grad")


def isopo_sampled_workspace_bytes(dtype: int, T: int, d_in: int, d_out: int, B: int, n_samples: int) -> int:
    return lib.isopo_sampled_workspace_bytes(dtype, T, d_in, d_out, B, n_samples)


def alloc_sampled_workspace(dtype: int, T: int, d_in: int, d_out: int, B: int, n_samples: int, device="cuda"):
    n = isopo_sampled_workspace_bytes(dtype, T, d_in, d_out, B, n_samples)
    if n == 0:
        raise IsopoError(ERR_INVALID_ARG, "isopo_sampled_workspace_bytes: invalid sizes")
    raw = torch.empty(n + 1024, dtype=torch.uint8, device=device)
    shift = (-raw.data_ptr()) % 1024
    return raw[shift:shift + n]


def isopo_sampled_coefficients(X: torch.Tensor, dY: torch.Tensor, seq_offsets, sample_rows, A: torch.Tensor, lam: float,
                               coeffs: torch.Tensor, ws: torch.Tensor, info: torch.Tensor, F2: torch.Tensor = None) -> None:
    """Algorithm 1's coefficients from sampled token rows (the caller draws `sample_rows`)."""
    off = _offsets(seq_offsets)
    B = off.shape[0] - 1
    rows = np.ascontiguousarray(np.asarray(sample_rows, dtype=np.int64))
    assert rows.ndim == 1 and X.is_cuda and dY.is_cuda and X.is_contiguous() and dY.is_contiguous() and X.dtype == dY.dtype
    assert A.dtype == torch.float32 and coeffs.dtype == torch.float32 and A.numel() == B and coeffs.numel() == B
    assert F2 is None or (F2.dtype == torch.float32 and F2.numel() == B)
    st = lib.isopo_sampled_coefficients(X.data_ptr(), dY.data_ptr(), _dtype_code(X), X.shape[0], X.shape[1], dY.shape[1],
                                        off.ctypes.data, B, rows.ctypes.data, rows.shape[0], A.data_ptr(), float(lam),
                                        coeffs.data_ptr(), F2.data_ptr() if F2 is not None else None, ws.data_ptr(),
                                        ws.numel(), info.data_ptr(), _stream())
    _check(st, "isopo_sampled_coefficients")


STORE_BF16, STORE_E4M3_SPLIT = 0, 1


def isopo_set_store_format(fmt: int) -> None:
    """Store format of the bf16 stored-gradient route: STORE_BF16 (default) or STORE_E4M3_SPLIT."""
    _check(lib.isopo_set_store_format(int(fmt)), "isopo_set_store_format")


def isopo_set_deterministic(on: bool) -> None:
    lib.isopo_set_deterministic(1 if on else 0)


def isopo_debug_build() -> bool:
    return bool(lib.isopo_debug_build())


def isopo_selftest_bounded_wait(limit_clocks: int, info: torch.Tensor, roles_at_teardown: torch.Tensor) -> None:
    """Makes one bounded mbarrier wait run out (nothing ever arrives) and lets the kernel tear down."""
    assert info.dtype == torch.int32 and roles_at_teardown.dtype == torch.int32
    _check(lib.isopo_selftest_bounded_wait(int(limit_clocks), info.data_ptr(), roles_at_teardown.data_ptr(), _stream()),
           "isopo_selftest_bounded_wait")


def isopo_profile_enable(on: bool) -> None:
    lib.isopo_profile_enable(1 if on else 0)


def isopo_profile_collect() -> dict:
    """{kernel name: (total ms, launches)} since the last collect; synchronises the recorded events."""
    ms = np.zeros(NUM_KERNELS, dtype=np.float64)
    n = np.zeros(NUM_KERNELS, dtype=np.int64)
    _check(lib.isopo_profile_collect(ms.ctypes.data, n.ctypes.data), "isopo_profile_collect")
    return {lib.isopo_kernel_name(k).decode(): (float(ms[k]), int(n[k])) for k in range(NUM_KERNELS) if n[k] or ms[k]}


@dataclass
class LayerResult:
    K: torch.Tensor
    coeffs: torch.Tensor
    dW: torch.Tensor
    info: int


def isopo_layer(X, dY, seq_offsets, A, variant, lam, path=PATH_AUTO, pqr_regs=None, ws=None) -> LayerResult:
    """The three calls of one layer in order on the current stream; synchronises to read `info`."""
    off = _offsets(seq_offsets)
    B = off.shape[0] - 1
    dev = X.device
    dt = _dtype_code(X)
    if ws is None:
        ws = alloc_workspace(dt, X.shape[0], X.shape[1], dY.shape[1], B, path, dev)
    K = torch.empty((B, B), dtype=torch.float32, device=dev)
    c = torch.empty(B, dtype=torch.float32, device=dev)
    dW = torch.empty((dY.shape[1], X.shape[1]), dtype=torch.float32, device=dev)
    info = torch.zeros(1, dtype=torch.int32, device=dev)
    isopo_layer_gram(X, dY, off, K, ws, info, path)
    isopo_transform_advantages(K, A, variant, lam, c, info, pqr_regs)
    isopo_weight_grad(X, dY, c, off, dW, ws, info, path, 0.0)
    return LayerResult(K, c, dW, int(info.item()))

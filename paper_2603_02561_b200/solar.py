"""ctypes binding of the C ABI in include/solar.h.

Argument marshalling only: every step of the forward pass runs in the CUDA
library.  torch is used for device memory and streams.  If the shared library
is missing this module raises -- there is no CPU fallback.
"""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libsolar_b200.so")

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_CUDA = range(5)
F32, BF16 = 0, 1
FLAG_NO_SOFTMAX = 1
INFO_NOT_CONVERGED, INFO_NONFINITE, INFO_NOT_CERTIFIED, INFO_DEVICE_WAIT = 1, 2, 4, 8
ROUTE_AUTO, ROUTE_SUBSPACE, ROUTE_FULL, ROUTE_TRIDIAG = 0, 1, 2, 3


def route_with(route: int, sweep_cap: int = 0, power_steps: int = 0) -> int:
    """The route argument of eig_from_partials_ex with its optional fields (SOLAR_ROUTE_WITH)."""
    return int(route) | (int(sweep_cap) << 8) | (int(power_steps) << 16)

_c_int, _c_size, _c_vp, _c_float, _c_uint = (ctypes.c_int, ctypes.c_size_t, ctypes.c_void_p,
                                              ctypes.c_float, ctypes.c_uint)

# name -> (restype, argtypes); must list every symbol include/solar.h declares
SIGNATURES = {
    "solar_status_string": (ctypes.c_char_p, [_c_int]),
    "solar_workspace_bytes": (_c_size, [_c_int] * 5 + [_c_int]),
    "solar_lowrank_factor": (_c_int, [_c_int] * 5 + [_c_int] + [_c_vp] * 5 + [_c_vp, _c_size, _c_vp]),
    "solar_svd_attention_fwd": (_c_int, [_c_int] * 5 + [_c_int] + [_c_vp] * 6 +
                                [_c_float, _c_uint, _c_vp, _c_vp, _c_size, _c_vp]),
    "solar_fused_workspace_bytes": (_c_size, [_c_int] * 5 + [_c_int]),
    "solar_svd_attention_fused": (_c_int, [_c_int] * 5 + [_c_int] + [_c_vp] * 5 + [_c_float, _c_uint] +
                                  [_c_vp] * 4 + [_c_vp, _c_size, _c_vp]),
    "solar_set_slice_limit": (_c_int, [_c_int]),
    "solar_gram_splits": (_c_int, [_c_int] * 3 + [_c_int]),
    "solar_gram_slices": (_c_int, [_c_int] * 3 + [_c_int]),
    "solar_gram_partials": (_c_int, [_c_int] * 3 + [_c_int, _c_vp, _c_vp, _c_size, _c_vp]),
    "solar_eig_from_partials": (_c_int, [_c_int] * 4 + [_c_int] + [_c_vp] * 3 + [_c_vp, _c_size, _c_vp]),
    "solar_eig_from_partials_ex": (_c_int, [_c_int] * 4 + [_c_int, _c_int] + [_c_vp] * 4 +
                                   [_c_vp, _c_size, _c_vp]),
    "solar_project_us": (_c_int, [_c_int] * 4 + [_c_int] + [_c_vp] * 3 + [_c_vp]),
    "solar_svd_backward": (_c_int, [_c_int] * 4 + [_c_int] + [_c_vp] * 5 + [_c_float] + [_c_vp] * 2 +
                           [_c_size, _c_vp]),
    "solar_backward_workspace_bytes": (_c_size, [_c_int] * 5 + [_c_int]),
    "solar_svd_attention_bwd": (_c_int, [_c_int] * 5 + [_c_int] + [_c_vp] * 6 + [_c_float, _c_uint] +
                                [_c_vp] * 7 + [_c_vp, _c_size, _c_vp]),
    "solar_attn_prepare": (_c_int, [_c_int] * 3 + [_c_int] + [_c_vp] * 5 + [_c_float, _c_vp, _c_size, _c_vp]),
    "solar_factored_softmax_attention_fwd": (_c_int, [_c_int] * 5 + [_c_int] + [_c_vp] * 6 +
                                             [_c_float, _c_vp, _c_vp, _c_size, _c_vp]),
    "solar_static_scratch_bytes": (_c_size, []),
    "solar_lowrank_factor_static": (_c_int, [_c_int] * 5 + [_c_int] + [_c_vp] * 4 + [_c_vp]),
    "solar_attn_apply": (_c_int, [_c_int] * 4 + [_c_int, _c_vp, _c_uint, _c_vp, _c_vp, _c_size, _c_vp]),
}

_lib = None


class SolarError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = lib().solar_status_string(status).decode()
        super().__init__(f"{where}: {msg} (status {status})")


def lib() -> ctypes.CDLL:
    """Loads libsolar_b200.so (built in-tree by build.py); raises if it is absent."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2603_02561_b200.build`; "
                "this package has no CPU fallback")
        L = ctypes.CDLL(LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(L, name)
            fn.restype, fn.argtypes = res, args
        _lib = L
    return _lib


def dtype_code(t: torch.dtype) -> int:
    if t == torch.float32:
        return F32
    if t == torch.bfloat16:
        return BF16
    raise TypeError(f"storage dtype must be float32 or bfloat16, got {t}")


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def _check(status: int, where: str):
    if status != OK:
        raise SolarError(status, where)


def workspace_bytes(B, M, N, d, r, dtype) -> int:
    return int(lib().solar_workspace_bytes(B, M, N, d, r, dtype_code(dtype)))


def gram_splits(B, N, d, dtype) -> int:
    return int(lib().solar_gram_splits(B, N, d, dtype_code(dtype)))


def gram_slices(B, N, d, dtype) -> int:
    return int(lib().solar_gram_slices(B, N, d, dtype_code(dtype)))


def alloc_workspace(B, M, N, d, r, dtype, device="cuda") -> torch.Tensor:
    return torch.empty(max(workspace_bytes(B, M, N, d, r, dtype), 256), dtype=torch.uint8, device=device)


def _need(t, shape, dtype, name):
    if t.dtype != dtype or tuple(t.shape) != tuple(shape) or not t.is_contiguous() or not t.is_cuda:
        raise ValueError(f"{name}: want contiguous CUDA {dtype} {tuple(shape)}, got {t.dtype} {tuple(t.shape)}")


def lowrank_factor(H, r, S=None, V=None, US=None, info=None, workspace=None, M=0, stream=None):
    """solar_lowrank_factor: H[B,N,d] -> S[B,r], V[B,d,r] (and US[B,N,r] if given)."""
    B, N, d = H.shape
    _need(H, (B, N, d), H.dtype, "H")
    dev = H.device
    S = torch.empty(B, r, dtype=torch.float32, device=dev) if S is None else S
    V = torch.empty(B, d, r, dtype=torch.float32, device=dev) if V is None else V
    _need(S, (B, r), torch.float32, "S"); _need(V, (B, d, r), torch.float32, "V")
    if US is not None:
        _need(US, (B, N, r), H.dtype, "US")
    if info is not None:
        _need(info, (B,), torch.int32, "info")
    if workspace is None:
        workspace = alloc_workspace(B, M, N, d, r, H.dtype, dev)
    st = lib().solar_lowrank_factor(B, M, N, d, r, dtype_code(H.dtype), _ptr(H), _ptr(S), _ptr(V),
                                    _ptr(US), _ptr(info), _ptr(workspace), workspace.numel(),
                                    _stream(stream))
    _check(st, "solar_lowrank_factor")
    return S, V


def svd_attention_fwd(C, S, V, Wq, Wk, Wv, scale, flags=0, O=None, workspace=None, N=0, stream=None):
    """solar_svd_attention_fwd: C[B,M,d] + factors -> O[B,M,d]."""
    B, M, d = C.shape
    r = S.shape[1]
    _need(C, (B, M, d), C.dtype, "C")
    _need(S, (B, r), torch.float32, "S"); _need(V, (B, d, r), torch.float32, "V")
    for nm, W in (("Wq", Wq), ("Wk", Wk), ("Wv", Wv)):
        _need(W, (d, d), C.dtype, nm)
    O = torch.empty_like(C) if O is None else O
    _need(O, (B, M, d), C.dtype, "O")
    if workspace is None:
        workspace = alloc_workspace(B, M, max(N, r), d, r, C.dtype, C.device)
    st = lib().solar_svd_attention_fwd(B, M, max(N, r), d, r, dtype_code(C.dtype), _ptr(C), _ptr(S),
                                       _ptr(V), _ptr(Wq), _ptr(Wk), _ptr(Wv), float(scale),
                                       int(flags), _ptr(O), _ptr(workspace), workspace.numel(),
                                       _stream(stream))
    _check(st, "solar_svd_attention_fwd")
    return O


def factored_softmax_attention_fwd(C, US, V, Wq, Wk, Wv, scale, O=None, workspace=None, stream=None):
    """solar_factored_softmax_attention_fwd: softmax attention over the N positions through
    the factors (US[B,N,r] = H V from lowrank_factor, V[B,d,r])."""
    B, M, d = C.shape
    N, r = US.shape[1], US.shape[2]
    _need(C, (B, M, d), C.dtype, "C"); _need(US, (B, N, r), C.dtype, "US")
    _need(V, (B, d, r), torch.float32, "V")
    for nm, W in (("Wq", Wq), ("Wk", Wk), ("Wv", Wv)):
        _need(W, (d, d), C.dtype, nm)
    O = torch.empty_like(C) if O is None else O
    _need(O, (B, M, d), C.dtype, "O")
    if workspace is None:
        workspace = alloc_workspace(B, M, N, d, r, C.dtype, C.device)
    st = lib().solar_factored_softmax_attention_fwd(B, M, N, d, r, dtype_code(C.dtype), _ptr(C), _ptr(US),
                                                    _ptr(V), _ptr(Wq), _ptr(Wk), _ptr(Wv), float(scale),
                                                    _ptr(O), _ptr(workspace), workspace.numel(), _stream(stream))
    _check(st, "solar_factored_softmax_attention_fwd")
    return O


def static_scratch_bytes() -> int:
    return int(lib().solar_static_scratch_bytes())


def lowrank_factor_static(H, r, S=None, V=None, info=None, M=0, stream=None):
    """solar_lowrank_factor_static: the factorization with the scratch inside the library.

    For callers that cannot allocate device memory; takes only inputs and outputs.
    Raises SolarError(ERR_WORKSPACE) when the sizes need more than static_scratch_bytes().
    """
    B, N, d = H.shape
    _need(H, (B, N, d), H.dtype, "H")
    if S is None or V is None:
        raise ValueError("lowrank_factor_static allocates nothing: pass S[B,r] and V[B,d,r]")
    _need(S, (B, r), torch.float32, "S"); _need(V, (B, d, r), torch.float32, "V")
    if info is not None:
        _need(info, (B,), torch.int32, "info")
    st = lib().solar_lowrank_factor_static(B, M, N, d, r, dtype_code(H.dtype), _ptr(H), _ptr(S),
                                           _ptr(V), _ptr(info), _stream(stream))
    _check(st, "solar_lowrank_factor_static")
    return S, V


# ---- stage-level calls --------------------------------------------------------------
def gram_partials(H, workspace, stream=None):
    B, N, d = H.shape
    _check(lib().solar_gram_partials(B, N, d, dtype_code(H.dtype), _ptr(H), _ptr(workspace),
                                     workspace.numel(), _stream(stream)), "solar_gram_partials")


def eig_from_partials(B, N, d, r, dtype, S, V, info, workspace, stream=None):
    _check(lib().solar_eig_from_partials(B, N, d, r, dtype_code(dtype), _ptr(S), _ptr(V), _ptr(info),
                                         _ptr(workspace), workspace.numel(), _stream(stream)),
           "solar_eig_from_partials")


def eig_from_partials_ex(B, N, d, r, dtype, route, S, V, info, route_taken, workspace, stream=None):
    _check(lib().solar_eig_from_partials_ex(B, N, d, r, dtype_code(dtype), int(route), _ptr(S), _ptr(V),
                                            _ptr(info), _ptr(route_taken), _ptr(workspace),
                                            workspace.numel(), _stream(stream)),
           "solar_eig_from_partials_ex")


def project_us(H, V, US, stream=None):
    B, N, d = H.shape
    r = V.shape[2]
    _check(lib().solar_project_us(B, N, d, r, dtype_code(H.dtype), _ptr(H), _ptr(V), _ptr(US),
                                  _stream(stream)), "solar_project_us")


def backward_workspace_bytes(B, M, N, d, r, dtype) -> int:
    return int(lib().solar_backward_workspace_bytes(B, M, N, d, r, dtype_code(dtype)))


def alloc_backward_workspace(B, M, N, d, r, dtype, device="cuda") -> torch.Tensor:
    return torch.empty(max(backward_workspace_bytes(B, M, N, d, r, dtype), 256), dtype=torch.uint8, device=device)


def alloc_attention_grads(C, r):
    """Output tensors of svd_attention_bwd: dC, dWq, dWk, dWv, dS, dV."""
    B, M, d = C.shape
    dev = C.device
    return (torch.empty_like(C), *(torch.empty(d, d, dtype=torch.float32, device=dev) for _ in range(3)),
            torch.empty(B, r, dtype=torch.float32, device=dev), torch.empty(B, d, r, dtype=torch.float32, device=dev))


def svd_attention_bwd(C, S, V, Wq, Wk, Wv, scale, dO, workspace, flags=0, out=None, stream=None):
    """solar_svd_attention_bwd: gradients of the forward call's inputs given dO.
    Returns dC[B,M,d], dWq, dWk, dWv [d,d] f32, dS[B,r], dV[B,d,r] (written into `out` if given)."""
    B, M, d = C.shape
    r = S.shape[1]
    _need(dO, (B, M, d), C.dtype, "dO")
    dC, dWq, dWk, dWv, dS, dV = alloc_attention_grads(C, r) if out is None else out
    _need(dC, (B, M, d), C.dtype, "dC"); _need(dS, (B, r), torch.float32, "dS"); _need(dV, (B, d, r), torch.float32, "dV")
    for nm, W in (("dWq", dWq), ("dWk", dWk), ("dWv", dWv)):
        _need(W, (d, d), torch.float32, nm)
    _check(lib().solar_svd_attention_bwd(B, M, max(r, 1), d, r, dtype_code(C.dtype), _ptr(C), _ptr(S), _ptr(V),
                                         _ptr(Wq), _ptr(Wk), _ptr(Wv), float(scale), int(flags), _ptr(dO),
                                         _ptr(dC), _ptr(dWq), _ptr(dWk), _ptr(dWv), _ptr(dS), _ptr(dV),
                                         _ptr(workspace), workspace.numel(), _stream(stream)),
           "solar_svd_attention_bwd")
    return dC, dWq, dWk, dWv, dS, dV


def svd_backward(H, S, V, dS, dV, dH, workspace, eps_rel=0.0, stream=None):
    """dH = U [diag(dS) + 2 Sigma sym(F o (dV^T V))] V^T with U = H V Sigma^-1 (Eq. 13-15)."""
    B, N, d = H.shape
    r = V.shape[2]
    _check(lib().solar_svd_backward(B, N, d, r, dtype_code(H.dtype), _ptr(H), _ptr(S), _ptr(V), _ptr(dS),
                                    _ptr(dV), float(eps_rel), _ptr(dH), _ptr(workspace), workspace.numel(),
                                    _stream(stream)), "solar_svd_backward")


def attn_prepare(S, V, Wq, Wk, Wv, scale, workspace, stream=None):
    B, d, r = V.shape
    _check(lib().solar_attn_prepare(B, d, r, dtype_code(Wq.dtype), _ptr(S), _ptr(V), _ptr(Wq),
                                    _ptr(Wk), _ptr(Wv), float(scale), _ptr(workspace),
                                    workspace.numel(), _stream(stream)), "solar_attn_prepare")


def attn_apply(C, r, flags, O, workspace, stream=None):
    B, M, d = C.shape
    _check(lib().solar_attn_apply(B, M, d, r, dtype_code(C.dtype), _ptr(C), int(flags), _ptr(O),
                                  _ptr(workspace), workspace.numel(), _stream(stream)),
           "solar_attn_apply")


def set_slice_limit(max_slices: int) -> int:
    """solar_set_slice_limit: process-wide cap on the row slices per user (0 = none); returns the old value."""
    return int(lib().solar_set_slice_limit(int(max_slices)))


def fused_workspace_bytes(B, M, N, d, r, dtype) -> int:
    return int(lib().solar_fused_workspace_bytes(B, M, N, d, r, dtype_code(dtype)))


def alloc_fused_workspace(B, M, N, d, r, dtype, device="cuda") -> torch.Tensor:
    return torch.empty(max(fused_workspace_bytes(B, M, N, d, r, dtype), 256), dtype=torch.uint8, device=device)


def svd_attention_fused(H, C, Wq, Wk, Wv, r, scale, flags=0, S=None, V=None, O=None, info=None,
                        workspace=None, stream=None):
    """solar_svd_attention_fused: the whole forward pass (H, C, weights -> S, V, O) in one call."""
    B, N, d = H.shape
    M = C.shape[1]
    _need(H, (B, N, d), H.dtype, "H"); _need(C, (B, M, d), H.dtype, "C")
    for nm, W in (("Wq", Wq), ("Wk", Wk), ("Wv", Wv)):
        _need(W, (d, d), H.dtype, nm)
    dev = H.device
    S = torch.empty(B, r, dtype=torch.float32, device=dev) if S is None else S
    V = torch.empty(B, d, r, dtype=torch.float32, device=dev) if V is None else V
    O = torch.empty_like(C) if O is None else O
    _need(S, (B, r), torch.float32, "S"); _need(V, (B, d, r), torch.float32, "V"); _need(O, (B, M, d), H.dtype, "O")
    if info is not None:
        _need(info, (B,), torch.int32, "info")
    if workspace is None:
        workspace = alloc_fused_workspace(B, M, N, d, r, H.dtype, dev)
    st = lib().solar_svd_attention_fused(B, M, N, d, r, dtype_code(H.dtype), _ptr(H), _ptr(C), _ptr(Wq), _ptr(Wk),
                                         _ptr(Wv), float(scale), int(flags), _ptr(S), _ptr(V), _ptr(O), _ptr(info),
                                         _ptr(workspace), workspace.numel(), _stream(stream))
    _check(st, "solar_svd_attention_fused")
    return O, S, V


def forward(H, C, Wq, Wk, Wv, r, scale, flags=0, workspace=None, stream=None):
    """The whole hot path: factorization then attention, back to back on one stream."""
    B, N, d = H.shape
    M = C.shape[1]
    if workspace is None:
        workspace = alloc_workspace(B, M, N, d, r, H.dtype, H.device)
    S, V = lowrank_factor(H, r, workspace=workspace, M=M, stream=stream)
    O = svd_attention_fwd(C, S, V, Wq, Wk, Wv, scale, flags, workspace=workspace, N=N, stream=stream)
    return O, S, V

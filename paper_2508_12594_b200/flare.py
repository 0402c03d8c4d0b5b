"""Python binding of libflare: the same entry points as ``include/flare.h``, argument marshalling only.

Every step of the mixer runs in the library's CUDA kernels.  PyTorch is used for device memory and streams:
the functions take torch tensors, check layout and dtype, and pass raw pointers.  There is no CPU fallback:
if ``libflare.so`` is missing or cannot be loaded the first call raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libflare.so")

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE_TOO_SMALL, ERR_ARCH, ERR_CUDA, ERR_TIMEOUT = range(7)
DTYPE_F32, DTYPE_BF16, DTYPE_F16 = 0, 1, 2
OP_ENCODE, OP_DECODE, OP_FORWARD, OP_BACKWARD, OP_SPECTRAL = range(5)


class FlareDesc(ctypes.Structure):
    _fields_ = [("B", ctypes.c_int32), ("H", ctypes.c_int32), ("N", ctypes.c_int32), ("M", ctypes.c_int32),
                ("D", ctypes.c_int32), ("dtype", ctypes.c_int32), ("scale", ctypes.c_float)]


class FlareError(RuntimeError):
    def __init__(self, status: int, where: str):
        lib = _lib_or_none()
        text = lib.flare_status_string(status).decode() if lib else str(status)
        detail = lib.flare_last_cuda_error().decode() if lib and status == ERR_CUDA else ""
        super().__init__(f"{where}: {text}" + (f" ({detail})" if detail else ""))
        self.status = status


_lib = None

_vp, _sz = ctypes.c_void_p, ctypes.c_size_t
_dp = ctypes.POINTER(FlareDesc)
_SIGNATURES = {
    "flare_version": (ctypes.c_int, []),
    "flare_status_string": (ctypes.c_char_p, [ctypes.c_int]),
    "flare_last_cuda_error": (ctypes.c_char_p, []),
    "flare_workspace_bytes": (_sz, [_dp, ctypes.c_int]),
    "flare_encode_partials": (ctypes.c_int, [_dp]),
    "flare_encode": (ctypes.c_int, [_dp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _sz, _vp]),
    "flare_encode_static_scratch": (ctypes.c_int, [_dp, _vp, _vp, _vp, _vp, _vp, _vp, _vp]),
    "flare_decode": (ctypes.c_int, [_dp, _vp, _vp, _vp, _vp, _vp, _vp, _sz, _vp]),
    "flare_set_path": (ctypes.c_int, [ctypes.c_int]),
    "flare_forward": (ctypes.c_int, [_dp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _sz, _vp]),
    "flare_backward": (ctypes.c_int, [_dp] + [_vp] * 13 + [_sz, _vp]),
    "flare_forward_host": (ctypes.c_int, [_dp] + [_vp] * 11 + [_sz, _vp]),
    "flare_check": (ctypes.c_int, [_vp, _vp]),
    "flare_microbench": (ctypes.c_int, [ctypes.c_int, ctypes.c_int, _vp, _sz, ctypes.POINTER(ctypes.c_double), _vp]),
    "flare_variant_workspace_bytes": (_sz, [_dp, ctypes.c_int, ctypes.c_int, ctypes.c_int]),
    "flare_forward_variant": (ctypes.c_int, [_dp, ctypes.c_int] + [_vp] * 10 + [_sz, _vp]),
    "flare_backward_variant": (ctypes.c_int, [_dp, ctypes.c_int] + [_vp] * 15 + [_sz, _vp]),
    "flare_spectral_gram": (ctypes.c_int, [_dp, _vp, _vp, _vp, _vp, _vp, _vp, _sz, _vp]),
    "flare_spectral_eig": (ctypes.c_int, [ctypes.c_int32, ctypes.c_int32, _vp, _vp, _vp, ctypes.c_int32, _vp]),
    "flare_launch_count": (ctypes.c_int, [_dp, ctypes.c_int]),
    "flare_selftest_wait": (ctypes.c_int, [_vp, ctypes.c_uint64, _vp]),
}


def _lib_or_none():
    return _lib


def load():
    """Load libflare.so (once).  Raises if the CUDA extension has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} not found: build it with `python -m paper_2508_12594_b200.build`")
        lib = ctypes.CDLL(LIB_PATH)
        for name, (res, args) in _SIGNATURES.items():
            fn = getattr(lib, name)
            fn.restype, fn.argtypes = res, args
        _lib = lib
    return _lib


def exported_symbols():
    return list(_SIGNATURES)


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return DTYPE_F32
    if t.dtype == torch.bfloat16:
        return DTYPE_BF16
    if t.dtype == torch.float16:
        return DTYPE_F16
    raise TypeError(f"unsupported dtype {t.dtype}")


def make_desc(Q: torch.Tensor, K: torch.Tensor, scale: float = 1.0) -> FlareDesc:
    H, M, D = Q.shape
    B, N, H2, D2 = K.shape
    if (H2, D2) != (H, D):
        raise ValueError("Q_lat [H,M,D] and K [B,N,H,D] disagree")
    return FlareDesc(B, H, N, M, D, _dtype_code(K), float(scale))


def _ptr(t: Optional[torch.Tensor], dtype=None, shape=None, cuda=True):
    if t is None:
        return None
    if cuda and not t.is_cuda:
        raise ValueError("expected a CUDA tensor")
    if not t.is_contiguous():
        raise ValueError("expected a contiguous tensor")
    if dtype is not None and t.dtype != dtype:
        raise TypeError(f"expected {dtype}, got {t.dtype}")
    if shape is not None and tuple(t.shape) != tuple(shape):
        raise ValueError(f"expected shape {tuple(shape)}, got {tuple(t.shape)}")
    return ctypes.c_void_p(t.data_ptr())


def _stream(stream: Optional[torch.cuda.Stream]):
    s = stream if stream is not None else torch.cuda.current_stream()
    return ctypes.c_void_p(s.cuda_stream)


def _raise(rc: int, where: str):
    if rc != OK:
        raise FlareError(rc, where)


def flare_version() -> int:
    return load().flare_version()


def flare_workspace_bytes(desc: FlareDesc, op: int) -> int:
    return int(load().flare_workspace_bytes(ctypes.byref(desc), op))


def flare_encode_partials(desc: FlareDesc) -> int:
    return int(load().flare_encode_partials(ctypes.byref(desc)))


def alloc_workspace(desc: FlareDesc, op: int, device="cuda") -> torch.Tensor:
    n = flare_workspace_bytes(desc, op)
    if n == 0:
        raise FlareError(ERR_UNSUPPORTED, "flare_workspace_bytes")
    return torch.empty(n, dtype=torch.uint8, device=device)


def flare_encode(desc, Q, K, V, key_mask, Z, lse_enc, workspace, stream=None):
    dt = K.dtype
    B, H, N, M, D = desc.B, desc.H, desc.N, desc.M, desc.D
    rc = load().flare_encode(ctypes.byref(desc), _ptr(Q, dt, (H, M, D)), _ptr(K, dt, (B, N, H, D)),
                             _ptr(V, dt, (B, N, H, D)), _ptr(key_mask, torch.uint8, (B, N)),
                             _ptr(Z, torch.float32, (B, H, M, D)), _ptr(lse_enc, torch.float32, (B, H, M)),
                             _ptr(workspace, torch.uint8), workspace.numel(), _stream(stream))
    _raise(rc, "flare_encode")


STATIC_SCRATCH_BYTES = 8 << 20


def flare_encode_static_scratch(desc, Q, K, V, key_mask, Z, lse_enc, stream=None):
    """flare_encode for callers that cannot allocate device memory: the partial results go to the library's
    built-in scratch array (STATIC_SCRATCH_BYTES, shared by all calls on the device, so calls must not overlap
    on the GPU).  Larger problems raise FlareError(ERR_WORKSPACE_TOO_SMALL)."""
    dt = K.dtype
    B, H, N, M, D = desc.B, desc.H, desc.N, desc.M, desc.D
    rc = load().flare_encode_static_scratch(ctypes.byref(desc), _ptr(Q, dt, (H, M, D)), _ptr(K, dt, (B, N, H, D)),
                                            _ptr(V, dt, (B, N, H, D)), _ptr(key_mask, torch.uint8, (B, N)),
                                            _ptr(Z, torch.float32, (B, H, M, D)),
                                            _ptr(lse_enc, torch.float32, (B, H, M)), _stream(stream))
    _raise(rc, "flare_encode_static_scratch")


def flare_decode(desc, Q, K, Z, Y, lse_dec, workspace=None, stream=None):
    dt = K.dtype
    B, H, N, M, D = desc.B, desc.H, desc.N, desc.M, desc.D
    rc = load().flare_decode(ctypes.byref(desc), _ptr(Q, dt, (H, M, D)), _ptr(K, dt, (B, N, H, D)),
                             _ptr(Z, torch.float32, (B, H, M, D)), _ptr(Y, dt, (B, N, H, D)),
                             _ptr(lse_dec, torch.float32, (B, N, H)), _ptr(workspace, torch.uint8),
                             0 if workspace is None else workspace.numel(), _stream(stream))
    _raise(rc, "flare_decode")


PATH_AUTO, PATH_EXACT, PATH_FAST = 0, 1, 2


def flare_set_path(path: int):
    """Which form of the bfloat16 forward kernels runs: PATH_AUTO, PATH_EXACT (running maximum) or PATH_FAST."""
    _raise(load().flare_set_path(int(path)), "flare_set_path")


def flare_forward(desc, Q, K, V, key_mask, Y, Z, lse_enc, lse_dec, workspace, stream=None):
    dt = K.dtype
    B, H, N, M, D = desc.B, desc.H, desc.N, desc.M, desc.D
    rc = load().flare_forward(ctypes.byref(desc), _ptr(Q, dt, (H, M, D)), _ptr(K, dt, (B, N, H, D)),
                              _ptr(V, dt, (B, N, H, D)), _ptr(key_mask, torch.uint8, (B, N)),
                              _ptr(Y, dt, (B, N, H, D)), _ptr(Z, torch.float32, (B, H, M, D)),
                              _ptr(lse_enc, torch.float32, (B, H, M)), _ptr(lse_dec, torch.float32, (B, N, H)),
                              _ptr(workspace, torch.uint8), workspace.numel(), _stream(stream))
    _raise(rc, "flare_forward")


def flare_backward(desc, Q, K, V, key_mask, Y, dY, Z, lse_enc, lse_dec, dQ, dK, dV, workspace, stream=None):
    dt = K.dtype
    B, H, N, M, D = desc.B, desc.H, desc.N, desc.M, desc.D
    tok = (B, N, H, D)
    rc = load().flare_backward(ctypes.byref(desc), _ptr(Q, dt, (H, M, D)), _ptr(K, dt, tok), _ptr(V, dt, tok),
                               _ptr(key_mask, torch.uint8, (B, N)), _ptr(Y, dt, tok), _ptr(dY, dt, tok),
                               _ptr(Z, torch.float32, (B, H, M, D)), _ptr(lse_enc, torch.float32, (B, H, M)),
                               _ptr(lse_dec, torch.float32, (B, N, H)), _ptr(dQ, torch.float32, (H, M, D)),
                               _ptr(dK, dt, tok), _ptr(dV, dt, tok), _ptr(workspace, torch.uint8),
                               workspace.numel(), _stream(stream))
    _raise(rc, "flare_backward")


def flare_forward_host(desc, hQ, hK, hV, hmask, hY, dQ, dK, dV, dmask, dY, workspace, stream=None):
    """Host tensors in, host tensor out; the device tensors are the caller's staging buffers."""
    dt = hK.dtype
    B, H, N, M, D = desc.B, desc.H, desc.N, desc.M, desc.D
    tok = (B, N, H, D)
    rc = load().flare_forward_host(ctypes.byref(desc), _ptr(hQ, dt, (H, M, D), cuda=False), _ptr(hK, dt, tok, cuda=False),
                                   _ptr(hV, dt, tok, cuda=False), _ptr(hmask, torch.uint8, (B, N), cuda=False),
                                   _ptr(hY, dt, tok, cuda=False), _ptr(dQ, dt, (H, M, D)), _ptr(dK, dt, tok),
                                   _ptr(dV, dt, tok), _ptr(dmask, torch.uint8, (B, N)), _ptr(dY, dt, tok),
                                   _ptr(workspace, torch.uint8), workspace.numel(), _stream(stream))
    _raise(rc, "flare_forward_host")


def flare_check(workspace, stream=None):
    """workspace=None checks the built-in scratch array of flare_encode_static_scratch."""
    _raise(load().flare_check(_ptr(workspace, torch.uint8), _stream(stream)), "flare_check")


def flare_launch_count(desc: FlareDesc, op: int) -> int:
    return int(load().flare_launch_count(ctypes.byref(desc), op))


def flare_selftest_wait(workspace, budget_ns: int, stream=None):
    _raise(load().flare_selftest_wait(_ptr(workspace, torch.uint8), int(budget_ns), _stream(stream)), "flare_selftest_wait")


def flare_variant_workspace_bytes(desc, op, shared_latents, separate) -> int:
    return int(load().flare_variant_workspace_bytes(ctypes.byref(desc), op, int(shared_latents), int(separate)))


def flare_forward_variant(desc, shared_latents, Q_enc, Q_dec, K, V, key_mask, Y, Z, lse_enc, lse_dec, workspace, stream=None):
    """The mixer with one latent sequence for all heads (Q [M, D]) and / or separate decode queries (Q_dec, else None)."""
    dt = K.dtype
    B, H, N, M, D = desc.B, desc.H, desc.N, desc.M, desc.D
    qs = (M, D) if shared_latents else (H, M, D)
    rc = load().flare_forward_variant(ctypes.byref(desc), int(shared_latents), _ptr(Q_enc, dt, qs), _ptr(Q_dec, dt, qs),
                                      _ptr(K, dt, (B, N, H, D)), _ptr(V, dt, (B, N, H, D)), _ptr(key_mask, torch.uint8, (B, N)),
                                      _ptr(Y, dt, (B, N, H, D)), _ptr(Z, torch.float32, (B, H, M, D)),
                                      _ptr(lse_enc, torch.float32, (B, H, M)), _ptr(lse_dec, torch.float32, (B, N, H)),
                                      _ptr(workspace, torch.uint8), workspace.numel(), _stream(stream))
    _raise(rc, "flare_forward_variant")


def flare_backward_variant(desc, shared_latents, Q_enc, Q_dec, K, V, key_mask, Y, dY, Z, lse_enc, lse_dec, dQ_enc, dQ_dec, dK,
                           dV, workspace, stream=None):
    dt = K.dtype
    B, H, N, M, D = desc.B, desc.H, desc.N, desc.M, desc.D
    tok, qs = (B, N, H, D), ((M, D) if shared_latents else (H, M, D))
    rc = load().flare_backward_variant(ctypes.byref(desc), int(shared_latents), _ptr(Q_enc, dt, qs), _ptr(Q_dec, dt, qs),
                                       _ptr(K, dt, tok), _ptr(V, dt, tok), _ptr(key_mask, torch.uint8, (B, N)),
                                       _ptr(Y, dt, tok), _ptr(dY, dt, tok), _ptr(Z, torch.float32, (B, H, M, D)),
                                       _ptr(lse_enc, torch.float32, (B, H, M)), _ptr(lse_dec, torch.float32, (B, N, H)),
                                       _ptr(dQ_enc, torch.float32, qs), _ptr(dQ_dec, torch.float32, qs), _ptr(dK, dt, tok),
                                       _ptr(dV, dt, tok), _ptr(workspace, torch.uint8), workspace.numel(), _stream(stream))
    _raise(rc, "flare_backward_variant")


def flare_microbench(which: int, iters: int = 20000, stream=None) -> float:
    """One of the library's instruction-level measurements (see include/flare.h)."""
    scratch = torch.empty(4096, dtype=torch.uint8, device="cuda")
    out = ctypes.c_double(0.0)
    _raise(load().flare_microbench(int(which), int(iters), _ptr(scratch, torch.uint8), scratch.numel(), ctypes.byref(out),
                                   _stream(stream)), "flare_microbench")
    return float(out.value)


def flare_spectral_gram(desc, Q, K, lse_enc, lse_dec, G, workspace, stream=None):
    dt = K.dtype
    B, H, N, M, D = desc.B, desc.H, desc.N, desc.M, desc.D
    rc = load().flare_spectral_gram(ctypes.byref(desc), _ptr(Q, dt, (H, M, D)), _ptr(K, dt, (B, N, H, D)),
                                    _ptr(lse_enc, torch.float32, (B, H, M)), _ptr(lse_dec, torch.float32, (B, N, H)),
                                    _ptr(G, torch.float32, (B, H, M, M)), _ptr(workspace, torch.uint8), workspace.numel(),
                                    _stream(stream))
    _raise(rc, "flare_spectral_gram")


def flare_spectral_eig(G, eigenvalues, U=None, sweeps=0, stream=None):
    """G [..., M, M] float32 (destroyed) -> eigenvalues [..., M] descending, U [..., M, M] eigenvectors as columns."""
    M = G.shape[-1]
    matrices = G.numel() // (M * M)
    rc = load().flare_spectral_eig(matrices, M, _ptr(G, torch.float32), _ptr(eigenvalues, torch.float32),
                                   _ptr(U, torch.float32), int(sweeps), _stream(stream))
    _raise(rc, "flare_spectral_eig")


def forward(Q, K, V, key_mask=None, scale=1.0, want_stats=False, stream=None):
    """Convenience: allocate outputs and workspace with torch, call flare_forward, return Y (and Z, lse's)."""
    desc = make_desc(Q, K, scale)
    B, H, N, M, D = desc.B, desc.H, desc.N, desc.M, desc.D
    ws = alloc_workspace(desc, OP_FORWARD, K.device)
    Y = torch.empty_like(K)
    Z = torch.empty(B, H, M, D, dtype=torch.float32, device=K.device)
    le = torch.empty(B, H, M, dtype=torch.float32, device=K.device)
    ld = torch.empty(B, N, H, dtype=torch.float32, device=K.device)
    flare_forward(desc, Q, K, V, key_mask, Y, Z, le, ld, ws, stream)
    return (Y, Z, le, ld) if want_stats else Y


def forward_backward(Q, K, V, dY, key_mask=None, scale=1.0, stream=None, check=False):
    """Convenience: flare_forward (keeping Z and the log-sum-exp rows) then flare_backward.
    Returns (Y, dQ_lat [H,M,D] float32, dK, dV).  With check=True the stream is synchronised and a device-side
    wait that gave up raises."""
    desc = make_desc(Q, K, scale)
    Y, Z, le, ld = forward(Q, K, V, key_mask, scale, want_stats=True, stream=stream)
    ws = alloc_workspace(desc, OP_BACKWARD, K.device)
    dQ = torch.empty(desc.H, desc.M, desc.D, dtype=torch.float32, device=K.device)
    dK, dV = torch.empty_like(K), torch.empty_like(V)
    flare_backward(desc, Q, K, V, key_mask, Y, dY, Z, le, ld, dQ, dK, dV, ws, stream)
    if check:
        (stream or torch.cuda.current_stream()).synchronize()
        flare_check(ws, stream)
    return Y, dQ, dK, dV

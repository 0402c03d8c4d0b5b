"""ctypes front end of the C oracle (``flare_oracle.c``) -- TEST INFRASTRUCTURE, not the product.

Only tests, the smoke check and the benchmark's CPU-baseline leg may import this.  It compiles the C file
with gcc on first use (``-O2 -fopenmp``, no fast-math, so every sum keeps its written order) and exposes the
functions on numpy float64 arrays in the C-ABI layouts:
Q [H,M,D]; K,V,Y,dY,dK,dV [B,N,H,D]; Z [B,H,M,D]; lse_enc [B,H,M]; lse_dec [B,N,H]; key_mask [B,N] uint8.

Which passage each function follows is stated in the C file.  Pins that hold this oracle to the paper and to
the mathematics (brute-force mixing matrix, row-stochasticity, rank, M = 1, a library attention routine,
finite differences, the spectral identity) are in ``tests/test_oracle_pins.py``; no function here is unpinned.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "flare_oracle.c")
_LIB = os.path.join(_HERE, "libflare_oracle.so")
_lock = threading.Lock()
_lib = None

_dp = ctypes.POINTER(ctypes.c_double)
_u8p = ctypes.POINTER(ctypes.c_uint8)
_i64p = ctypes.POINTER(ctypes.c_int64)


def build(force: bool = False) -> str:
    """Compile the oracle's shared library next to its source (idempotent)."""
    with _lock:
        stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
        if force or stale:
            tmp = _LIB + f".{os.getpid()}.tmp"
            subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", tmp, _SRC, "-lm"])
            os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.flare_oracle_max_threads.restype = ctypes.c_int
    return _lib


def _d(a):
    a = np.ascontiguousarray(a, dtype=np.float64)
    return a, a.ctypes.data_as(_dp)


def _mask(key_mask, B, N):
    if key_mask is None:
        return None, None
    m = np.ascontiguousarray(key_mask, dtype=np.uint8).reshape(B, N)
    return m, m.ctypes.data_as(_u8p)


def _dims(Q, K):
    H, M, D = Q.shape
    B, N, H2, D2 = K.shape
    assert (H2, D2) == (H, D), "Q [H,M,D] and K [B,N,H,D] disagree"
    return B, H, N, M, D


def max_threads() -> int:
    return int(_load().flare_oracle_max_threads())


def encode(Q, K, V, key_mask=None, scale=1.0):
    """Z [B,H,M,D], lse_enc [B,H,M]."""
    B, H, N, M, D = _dims(Q, K)
    Q, pq = _d(Q); K, pk = _d(K); V, pv = _d(V)
    mk, pm = _mask(key_mask, B, N)
    Z = np.empty((B, H, M, D)); lse = np.empty((B, H, M))
    _load().flare_oracle_encode(B, H, N, M, D, ctypes.c_double(scale), pq, pk, pv, pm,
                                Z.ctypes.data_as(_dp), lse.ctypes.data_as(_dp))
    return Z, lse


def decode(Q, K, Z, scale=1.0):
    """Y [B,N,H,D], lse_dec [B,N,H]."""
    B, H, N, M, D = _dims(Q, K)
    Q, pq = _d(Q); K, pk = _d(K); Z, pz = _d(Z)
    Y = np.empty((B, N, H, D)); lse = np.empty((B, N, H))
    _load().flare_oracle_decode(B, H, N, M, D, ctypes.c_double(scale), pq, pk, pz,
                                Y.ctypes.data_as(_dp), lse.ctypes.data_as(_dp))
    return Y, lse


def decode_rows(Q, K, Z, rows, scale=1.0):
    """Decode only the token rows ``rows`` (flat indices b*N+n): Y_rows [len(rows), H, D]."""
    B, H, N, M, D = _dims(Q, K)
    Q, pq = _d(Q); K, pk = _d(K); Z, pz = _d(Z)
    rows = np.ascontiguousarray(rows, dtype=np.int64)
    Y = np.empty((len(rows), H, D))
    _load().flare_oracle_decode_rows(B, H, N, M, D, ctypes.c_double(scale), pq, pk, pz,
                                     rows.ctypes.data_as(_i64p), len(rows), Y.ctypes.data_as(_dp))
    return Y


def forward(Q, K, V, key_mask=None, scale=1.0):
    """The whole mixer.  Returns dict(Z, lse_enc, Y, lse_dec)."""
    B, H, N, M, D = _dims(Q, K)
    Q, pq = _d(Q); K, pk = _d(K); V, pv = _d(V)
    mk, pm = _mask(key_mask, B, N)
    Z = np.empty((B, H, M, D)); le = np.empty((B, H, M))
    Y = np.empty((B, N, H, D)); ld = np.empty((B, N, H))
    _load().flare_oracle_forward(B, H, N, M, D, ctypes.c_double(scale), pq, pk, pv, pm,
                                 Z.ctypes.data_as(_dp), le.ctypes.data_as(_dp),
                                 Y.ctypes.data_as(_dp), ld.ctypes.data_as(_dp))
    return dict(Z=Z, lse_enc=le, Y=Y, lse_dec=ld)


def mixing_matrices(Q, K, b, h, key_mask=None, scale=1.0):
    """Dense W_enc [M,N], W_dec [N,M], W = W_dec W_enc [N,N] of one (b, h).  Small N only."""
    B, H, N, M, D = _dims(Q, K)
    Q, pq = _d(Q); K, pk = _d(K)
    mk, pm = _mask(key_mask, B, N)
    We = np.empty((M, N)); Wd = np.empty((N, M)); W = np.empty((N, N))
    _load().flare_oracle_mixing_matrices(B, H, N, M, D, ctypes.c_double(scale), pq, pk, pm, int(b), int(h),
                                         We.ctypes.data_as(_dp), Wd.ctypes.data_as(_dp), W.ctypes.data_as(_dp))
    return We, Wd, W


def backward(Q, K, V, dY, key_mask=None, scale=1.0):
    """Gradients of sum(Y * dY).  Returns dict(dQ [H,M,D], dK, dV [B,N,H,D], dZ [B,H,M,D])."""
    B, H, N, M, D = _dims(Q, K)
    Q, pq = _d(Q); K, pk = _d(K); V, pv = _d(V); dY, pdy = _d(dY)
    mk, pm = _mask(key_mask, B, N)
    dQ = np.empty((H, M, D)); dK = np.empty((B, N, H, D)); dV = np.empty((B, N, H, D)); dZ = np.empty((B, H, M, D))
    _load().flare_oracle_backward(B, H, N, M, D, ctypes.c_double(scale), pq, pk, pv, pm, pdy,
                                  dQ.ctypes.data_as(_dp), dK.ctypes.data_as(_dp), dV.ctypes.data_as(_dp),
                                  dZ.ctypes.data_as(_dp))
    return dict(dQ=dQ, dK=dK, dV=dV, dZ=dZ)


def backward_rows(Q, K, V, dY, rows, key_mask=None, scale=1.0):
    """The backward with dK and dV evaluated only for the token rows ``rows`` (flat indices b*N+n); the reductions
    over all tokens (dQ, dZ) run in full.  Returns dict(dQ [H,M,D], dK_rows, dV_rows [len(rows),H,D], dZ)."""
    B, H, N, M, D = _dims(Q, K)
    Q, pq = _d(Q); K, pk = _d(K); V, pv = _d(V); dY, pdy = _d(dY)
    mk, pm = _mask(key_mask, B, N)
    rows = np.ascontiguousarray(rows, dtype=np.int64)
    dQ = np.empty((H, M, D)); dZ = np.empty((B, H, M, D))
    dK = np.empty((len(rows), H, D)); dV = np.empty((len(rows), H, D))
    _load().flare_oracle_backward_rows(B, H, N, M, D, ctypes.c_double(scale), pq, pk, pv, pm, pdy,
                                       rows.ctypes.data_as(_i64p), len(rows), dQ.ctypes.data_as(_dp),
                                       dK.ctypes.data_as(_dp), dV.ctypes.data_as(_dp), dZ.ctypes.data_as(_dp))
    return dict(dQ=dQ, dK_rows=dK, dV_rows=dV, dZ=dZ)


def backward_asym(Qe, Qd, K, V, dY, key_mask=None, scale=1.0):
    """Gradients of sum(Y * dY) for the variant with separate encode and decode queries (Qe, Qd [H,M,D]).
    Returns dict(dQe, dQd [H,M,D], dK, dV [B,N,H,D]).  Dense and single-threaded: small cases only."""
    B, H, N, M, D = _dims(Qe, K)
    Qe, pqe = _d(Qe); Qd, pqd = _d(Qd); K, pk = _d(K); V, pv = _d(V); dY, pdy = _d(dY)
    mk, pm = _mask(key_mask, B, N)
    dQe = np.empty((H, M, D)); dQd = np.empty((H, M, D)); dK = np.empty((B, N, H, D)); dV = np.empty((B, N, H, D))
    _load().flare_oracle_backward_asym(B, H, N, M, D, ctypes.c_double(scale), pqe, pqd, pk, pv, pm, pdy,
                                       dQe.ctypes.data_as(_dp), dQd.ctypes.data_as(_dp), dK.ctypes.data_as(_dp),
                                       dV.ctypes.data_as(_dp))
    return dict(dQe=dQe, dQd=dQd, dK=dK, dV=dV)

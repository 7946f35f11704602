"""ctypes front end of the float64 CPU oracle (``darkattn_ref.c``).

TEST INFRASTRUCTURE ONLY: imported by the tests, the smoke check and the benchmark's CPU-baseline
leg. It does not import the CUDA package and the CUDA package does not import it.

All arrays are numpy float64, C-contiguous; shapes follow the C file's header comment.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "darkattn_ref.c")
_LIB = os.path.join(_HERE, "libdarkattn_ref.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (plain -O2, no fast-math, OpenMP over (batch, head))."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.darkattn_ref_num_threads.restype = ctypes.c_int
    return _lib


def num_threads() -> int:
    return int(_load().darkattn_ref_num_threads())


def _p(a):
    if a is None:
        return ctypes.c_void_p(None)
    assert a.dtype == np.float64 and a.flags["C_CONTIGUOUS"]
    return a.ctypes.data_as(ctypes.c_void_p)


def _c(a):
    return None if a is None else np.ascontiguousarray(a, dtype=np.float64)


def features(X, M, W, s=1.0, shift=None, return_xt=False):
    """phi(x_i)_l = exp(w_l.(s M x_i) - |s M x_i|^2/2 - shift_i)/sqrt(m) for the rows of X [N,d]."""
    X, M, W, shift = _c(X), _c(M), _c(W), _c(shift)
    N, d = X.shape
    r, d2 = M.shape
    m, r2 = W.shape
    assert d2 == d and r2 == r
    phi = np.empty((N, m))
    xt = np.empty((N, r)) if return_xt else None
    rc = _load().darkattn_ref_features(N, d, r, m, ctypes.c_double(s), _p(X), _p(M), _p(W), _p(shift),
                                       _p(phi), _p(xt))
    if rc:
        raise RuntimeError(f"darkattn_ref_features failed ({rc})")
    return (phi, xt) if return_xt else phi


def _dims(Q, V, M, W):
    B, H, N, d = Q.shape
    dv = V.shape[-1]
    r = M.shape[-2]
    w_per_head = 1 if W.ndim == 3 else 0
    m = W.shape[-2]
    assert M.shape == (H, r, d) and W.shape[-1] == r
    return B, H, N, d, r, m, dv, w_per_head


def _expand_kv(Q, K, V):
    """Grouped key/value heads (K, V of shape [B, H_kv, N, *] with H_kv dividing H): query heads h*G .. h*G+G-1 read
    key/value head h, i.e. the attention is the ungrouped one with every key/value head repeated G times. The feature
    map of a query head (its own M) is applied to the keys it reads, as to its queries (Appendix B: q~ = Mq, k~ = Mk)."""
    H, Hkv = Q.shape[1], K.shape[1]
    assert V.shape[1] == Hkv and H % Hkv == 0, "H_kv must divide H"
    G = H // Hkv
    if G == 1:
        return K, V, 1
    return np.repeat(K, G, axis=1), np.repeat(V, G, axis=1), G


def forward(Q, K, V, M, W, causal=False, scale=None, shift_q=None, shift_k=None):
    """O [B,H,N,dv]; scale defaults to 1/sqrt(d). K, V may have fewer heads than Q (grouped key/value heads)."""
    K, V, _ = _expand_kv(np.asarray(Q), np.asarray(K), np.asarray(V))
    Q, K, V, M, W = _c(Q), _c(K), _c(V), _c(M), _c(W)
    B, H, N, d, r, m, dv, wph = _dims(Q, V, M, W)
    scale = 1.0 / np.sqrt(d) if scale is None else float(scale)
    O = np.empty((B, H, N, dv))
    rc = _load().darkattn_ref_forward(B, H, N, d, r, m, dv, int(bool(causal)), ctypes.c_double(scale), wph,
                                      _p(Q), _p(K), _p(V), _p(M), _p(W), _p(_c(shift_q)), _p(_c(shift_k)),
                                      _p(O))
    if rc:
        raise RuntimeError(f"darkattn_ref_forward failed ({rc})")
    return O


def backward(Q, K, V, M, W, dO, causal=False, scale=None, shift_q=None, shift_k=None):
    """Returns dQ, dK, dV, dM [H,r,d], dW (same shape as W) for L = sum(dO * O). With grouped key/value heads dK and
    dV have K's and V's shapes: a shared key (value) collects the gradients of all query heads that read it."""
    K, V, G = _expand_kv(np.asarray(Q), np.asarray(K), np.asarray(V))
    Q, K, V, M, W, dO = _c(Q), _c(K), _c(V), _c(M), _c(W), _c(dO)
    B, H, N, d, r, m, dv, wph = _dims(Q, V, M, W)
    scale = 1.0 / np.sqrt(d) if scale is None else float(scale)
    dQ, dK, dV = np.empty_like(Q), np.empty_like(K), np.empty_like(V)
    dM, dW = np.empty_like(M), np.empty_like(W)
    rc = _load().darkattn_ref_backward(B, H, N, d, r, m, dv, int(bool(causal)), ctypes.c_double(scale), wph,
                                       _p(Q), _p(K), _p(V), _p(M), _p(W), _p(dO),
                                       _p(_c(shift_q)), _p(_c(shift_k)),
                                       _p(dQ), _p(dK), _p(dV), _p(dM), _p(dW))
    if rc:
        raise RuntimeError(f"darkattn_ref_backward failed ({rc})")
    if G > 1:
        dK = dK.reshape(B, H // G, G, N, d).sum(axis=2)
        dV = dV.reshape(B, H // G, G, N, dv).sum(axis=2)
    return dQ, dK, dV, dM, dW

"""fp64 CPU oracle for the FLuRKA attention forward pass (arxiv 2306.15799, Eq. (2)).

TEST INFRASTRUCTURE ONLY: nothing in the CUDA package imports this module, and this
module imports nothing from the CUDA package.  It wraps ``flurka_oracle.c`` (plain C,
fp64, OpenMP) through ctypes; the shared object is compiled on first use with gcc.

The module-level functions mirror the C entry points; every array is converted to
contiguous float64.  ``OracleLib(path)`` binds another build of the same source (the
pin tests use it to check that planted mistakes are caught).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

PERFORMER = 0
RNN = 1

_HERE = os.path.dirname(os.path.abspath(__file__))
SOURCE = os.path.join(_HERE, "flurka_oracle.c")
_LIB = os.path.join(_HERE, "libflurka_oracle.so")
_lock = threading.Lock()
_default = None

_DP = ctypes.POINTER(ctypes.c_double)
_LP = ctypes.POINTER(ctypes.c_long)


def compile_source(src: str, out: str) -> str:
    """gcc -O2 -fopenmp, no fast-math."""
    tmp = out + ".tmp.%d" % os.getpid()
    cmd = ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", tmp, src, "-lm"]
    subprocess.run(cmd, check=True)
    os.replace(tmp, out)
    return out


def build(force: bool = False) -> str:
    """Compile the C oracle if missing or stale. Returns the library path."""
    with _lock:
        stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(SOURCE)
        if force or stale:
            compile_source(SOURCE, _LIB)
    return _LIB


def _f64(a):
    return None if a is None else np.ascontiguousarray(np.asarray(a, dtype=np.float64))


def _ptr(a):
    return _DP() if a is None else a.ctypes.data_as(_DP)


def _rows(rows, N):
    if rows is None:
        return None, N, _LP()
    arr = np.ascontiguousarray(np.asarray(rows, dtype=np.int64))
    assert arr.ndim == 1 and (arr >= 0).all() and (arr < N).all()
    return arr, arr.shape[0], arr.ctypes.data_as(_LP)


class OracleLib:
    def __init__(self, path: str):
        lib = ctypes.CDLL(path)
        ci = ctypes.c_int
        lib.flurka_oracle_head.restype = ci
        lib.flurka_oracle_head.argtypes = [_DP] * 6 + [ci] * 6 + [_LP, ctypes.c_long] + [_DP] * 5
        lib.flurka_oracle_head_quadratic.restype = ci
        lib.flurka_oracle_head_quadratic.argtypes = [_DP] * 6 + [ci] * 6 + [_LP, ctypes.c_long] + [_DP] * 2
        lib.flurka_oracle_forward.restype = ci
        lib.flurka_oracle_forward.argtypes = [_DP] * 6 + [ci] * 7 + [_DP]
        lib.flurka_oracle_features.restype = ci
        lib.flurka_oracle_features.argtypes = [_DP, ci, ci, _DP, ci, ci, ci, ci, _DP]
        lib.flurka_oracle_threads.restype = ci
        if hasattr(lib, "flurka_oracle_fused_head"):
            lib.flurka_oracle_fused_head.restype = ci
            lib.flurka_oracle_fused_head.argtypes = [_DP] * 9 + [ci] * 7 + [_LP, ctypes.c_long] + [_DP] * 4
        if hasattr(lib, "flurka_oracle_head_backward"):
            lib.flurka_oracle_head_backward.restype = ci
            lib.flurka_oracle_head_backward.argtypes = [_DP] * 7 + [ci] * 5 + [_DP] * 5
        self._lib = lib

    def threads(self) -> int:
        return int(self._lib.flurka_oracle_threads())

    @staticmethod
    def _head_args(Q, K, V, E, F, W, variant):
        Q, K, V, E, F, W = (_f64(x) for x in (Q, K, V, E, F, W))
        N, d = Q.shape
        k = E.shape[0]
        assert K.shape == (N, d) and V.shape == (N, d), "Q, K, V must be [N, d]"
        assert E.shape == (k, N) and F.shape == (k, N), "E, F must be [k, N]"
        if variant == PERFORMER:
            assert W is not None and W.ndim == 2 and W.shape[1] == d, "W must be [m, d]"
            m = W.shape[0]
        else:
            m = 0
        return Q, K, V, E, F, W, N, d, k, m

    def head(self, Q, K, V, E, F, W, variant, *, stabilise=True, rows=None, intermediates=False):
        """One head, associative order. Q,K,V [N,d]; E,F [k,N]; W [m,d] or None (RNN).

        Returns O [n_rows,d] float64, or (O, dict(Kp, Vp, KV, z)) with intermediates=True.
        """
        Q, K, V, E, F, W, N, d, k, m = self._head_args(Q, K, V, E, F, W, variant)
        p = m if variant == PERFORMER else d
        rows_arr, n_rows, rows_p = _rows(rows, N)
        out = np.empty((n_rows, d), dtype=np.float64)
        if intermediates:
            Kp, Vp, KV, z = np.empty((k, d)), np.empty((k, d)), np.empty((p, d)), np.empty((p,))
        else:
            Kp = Vp = KV = z = None
        rc = self._lib.flurka_oracle_head(
            _ptr(Q), _ptr(K), _ptr(V), _ptr(E), _ptr(F), _ptr(W), variant, N, d, k, m,
            1 if stabilise else 0, rows_p, n_rows, _ptr(out), _ptr(Kp), _ptr(Vp), _ptr(KV), _ptr(z))
        if rc:
            raise ValueError("flurka_oracle_head failed: %d" % rc)
        return (out, {"Kp": Kp, "Vp": Vp, "KV": KV, "z": z}) if intermediates else out

    def head_quadratic(self, Q, K, V, E, F, W, variant, *, stabilise=True, rows=None, weights=False):
        """One head, explicit quadratic form (the definition). Returns O or (O, Ahat [n_rows,k])."""
        Q, K, V, E, F, W, N, d, k, m = self._head_args(Q, K, V, E, F, W, variant)
        rows_arr, n_rows, rows_p = _rows(rows, N)
        out = np.empty((n_rows, d), dtype=np.float64)
        Ahat = np.empty((n_rows, k)) if weights else None
        rc = self._lib.flurka_oracle_head_quadratic(
            _ptr(Q), _ptr(K), _ptr(V), _ptr(E), _ptr(F), _ptr(W), variant, N, d, k, m,
            1 if stabilise else 0, rows_p, n_rows, _ptr(out), _ptr(Ahat))
        if rc:
            raise ValueError("flurka_oracle_head_quadratic failed: %d" % rc)
        return (out, Ahat) if weights else out

    def fused_head(self, Xq, Xk, Xv, E, F, Wq, Wk, Wv, W, variant, *, stabilise=True, rows=None, intermediates=False):
        """One head of Eq. (2) with its linear maps: Xq, Xk, Xv [N,dm] un-projected; Wq, Wk, Wv [dm,d]
        (this head's); E, F [k,N]; W [m,d] or None.  Returns O [n_rows,d], or (O, dict(Kp, Vp, Q))."""
        Xq, Xk, Xv, E, F, Wq, Wk, Wv, W = (_f64(x) for x in (Xq, Xk, Xv, E, F, Wq, Wk, Wv, W))
        N, dm = Xq.shape
        d = Wq.shape[1]
        k = E.shape[0]
        assert Xk.shape == (N, dm) and Xv.shape == (N, dm), "Xq, Xk, Xv must be [N, dm]"
        assert Wq.shape == (dm, d) and Wk.shape == (dm, d) and Wv.shape == (dm, d), "Wq, Wk, Wv must be [dm, d]"
        assert E.shape == (k, N) and F.shape == (k, N), "E, F must be [k, N]"
        if variant == PERFORMER:
            assert W is not None and W.shape[1] == d, "W must be [m, d]"
            m = W.shape[0]
        else:
            m = 0
        rows_arr, n_rows, rows_p = _rows(rows, N)
        out = np.empty((n_rows, d), dtype=np.float64)
        if intermediates:
            Kp, Vp, Qh = np.empty((k, d)), np.empty((k, d)), np.empty((n_rows, d))
        else:
            Kp = Vp = Qh = None
        rc = self._lib.flurka_oracle_fused_head(
            _ptr(Xq), _ptr(Xk), _ptr(Xv), _ptr(E), _ptr(F), _ptr(Wq), _ptr(Wk), _ptr(Wv), _ptr(W), variant,
            N, dm, d, k, m, 1 if stabilise else 0, rows_p, n_rows, _ptr(out), _ptr(Kp), _ptr(Vp), _ptr(Qh))
        if rc:
            raise ValueError("flurka_oracle_fused_head failed: %d" % rc)
        return (out, {"Kp": Kp, "Vp": Vp, "Q": Qh}) if intermediates else out

    def head_backward(self, Q, K, V, E, F, W, dO, variant):
        """Gradients of sum(O * dO) for one head: returns dict(dQ, dK, dV [N,d], dE, dF [k,N])."""
        Q, K, V, E, F, W, N, d, k, m = self._head_args(Q, K, V, E, F, W, variant)
        dO = _f64(dO)
        assert dO.shape == (N, d), "dO must be [N, d]"
        g = {"dQ": np.empty((N, d)), "dK": np.empty((N, d)), "dV": np.empty((N, d)),
             "dE": np.empty((k, N)), "dF": np.empty((k, N))}
        rc = self._lib.flurka_oracle_head_backward(
            _ptr(Q), _ptr(K), _ptr(V), _ptr(E), _ptr(F), _ptr(W), _ptr(dO), variant, N, d, k, m,
            _ptr(g["dQ"]), _ptr(g["dK"]), _ptr(g["dV"]), _ptr(g["dE"]), _ptr(g["dF"]))
        if rc:
            raise ValueError("flurka_oracle_head_backward failed: %d" % rc)
        return g

    def features(self, X, W, variant, *, stabilise=False, scope_global=False):
        """phi applied to the rows of X [rows,d]. Returns [rows,m] (PERFORMER) or [rows,d] (RNN)."""
        X, W = _f64(X), _f64(W)
        rows, d = X.shape
        m = W.shape[0] if variant == PERFORMER else 0
        p = m if variant == PERFORMER else d
        Phi = np.empty((rows, p))
        rc = self._lib.flurka_oracle_features(_ptr(X), rows, d, _ptr(W), m, variant,
                                              1 if stabilise else 0, 1 if scope_global else 0, _ptr(Phi))
        if rc:
            raise ValueError("flurka_oracle_features failed: %d" % rc)
        return Phi

    def forward(self, Q, K, V, E, F, W, variant):
        """All heads. Q,K,V [B,H,N,d]; E,F [k,N]; W [m,d] or None. Returns O [B,H,N,d] float64."""
        Q, K, V, E, F, W = (_f64(x) for x in (Q, K, V, E, F, W))
        B, H, N, d = Q.shape
        k = E.shape[0]
        assert K.shape == Q.shape and V.shape == Q.shape
        assert E.shape == (k, N) and F.shape == (k, N)
        m = W.shape[0] if variant == PERFORMER else 0
        out = np.empty_like(Q)
        rc = self._lib.flurka_oracle_forward(
            _ptr(Q), _ptr(K), _ptr(V), _ptr(E), _ptr(F), _ptr(W), variant, B, H, N, d, k, m, _ptr(out))
        if rc:
            raise ValueError("flurka_oracle_forward failed: %d" % rc)
        return out


def default() -> OracleLib:
    global _default
    if _default is None:
        _default = OracleLib(build())
    return _default


def threads() -> int:
    return default().threads()


def head(*a, **kw):
    return default().head(*a, **kw)


def head_quadratic(*a, **kw):
    return default().head_quadratic(*a, **kw)


def fused_head(*a, **kw):
    return default().fused_head(*a, **kw)


def head_backward(*a, **kw):
    return default().head_backward(*a, **kw)


def features(*a, **kw):
    return default().features(*a, **kw)


def forward(*a, **kw):
    return default().forward(*a, **kw)

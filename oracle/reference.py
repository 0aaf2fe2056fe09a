"""ctypes wrapper around the plain-C fp64 oracle (TEST INFRASTRUCTURE, not the product).

Argument marshalling only: every number the oracle reports is computed in
`restkv_oracle.c`.  The shared object is built on first use with gcc.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading
from dataclasses import dataclass
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "restkv_oracle.c")
_LIB = os.path.join(_HERE, "librestkv_oracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile restkv_oracle.c into a shared object next to it (gcc -O2 -fopenmp)."""
    with _lock:
        stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
        if force or stale:
            tmp = _LIB + ".tmp.%d" % os.getpid()
            cmd = ["gcc", "-O2", "-fopenmp", "-std=c11", "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"]
            subprocess.run(cmd, check=True)
            os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        c_f = ctypes.POINTER(ctypes.c_float)
        c_d = ctypes.POINTER(ctypes.c_double)
        c_i = ctypes.POINTER(ctypes.c_int)
        lib.restkv_oracle_score.restype = ctypes.c_int
        lib.restkv_oracle_score.argtypes = (
            [c_f, c_f, c_f] + [ctypes.c_int] * 7 + [ctypes.c_double, ctypes.c_double]
            + [ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_double, ctypes.c_int]
            + [ctypes.c_int, ctypes.c_int, ctypes.c_int]
            + [c_d, c_d, c_d, c_d, c_i, c_d, c_d]
        )
        lib.restkv_oracle_score_variant.restype = ctypes.c_int
        lib.restkv_oracle_score_variant.argtypes = (
            [c_f, c_f, c_f] + [ctypes.c_int] * 7 + [ctypes.c_double, ctypes.c_double]
            + [ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_double, ctypes.c_int]
            + [ctypes.c_int] * 6 + [c_f, ctypes.c_int]
            + [c_d, c_d, c_d, c_d, c_i, c_d, c_d]
        )
        lib.restkv_oracle_select.restype = ctypes.c_int
        lib.restkv_oracle_select.argtypes = [c_d, ctypes.c_int, ctypes.c_int, ctypes.c_int, c_i]
        lib.restkv_oracle_compact.restype = ctypes.c_int
        lib.restkv_oracle_compact.argtypes = [
            ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.c_size_t, c_i, ctypes.c_int, ctypes.c_void_p]
        lib.restkv_oracle_decode.restype = ctypes.c_int
        lib.restkv_oracle_decode.argtypes = [c_f, c_f, c_f] + [ctypes.c_int] * 5 + [ctypes.c_double, c_d, c_d]
        lib.restkv_oracle_num_threads.restype = ctypes.c_int
        lib.restkv_oracle_set_threads.argtypes = [ctypes.c_int]
        _lib = lib
    return _lib


def num_threads() -> int:
    return int(_load().restkv_oracle_num_threads())


def set_threads(t: int) -> None:
    _load().restkv_oracle_set_threads(int(t))


def _f32(x: np.ndarray) -> np.ndarray:
    x = np.ascontiguousarray(x)
    if x.dtype != np.float32:
        raise TypeError("oracle inputs are float32 arrays holding dtype-exact values")
    return x


def _ptr(a: Optional[np.ndarray], ctype):
    if a is None:
        return ctypes.cast(None, ctypes.POINTER(ctype))
    return a.ctypes.data_as(ctypes.POINTER(ctype))


@dataclass
class ScoreResult:
    scores: np.ndarray                 # [b, Hkv, n_kv] float64, +inf on the trailing rows
    I_hat: Optional[np.ndarray]        # [b, Hkv, n]
    I_raw: Optional[np.ndarray]        # [b, Hq, w, n]
    A: Optional[np.ndarray]            # [b, Hq, w, n_kv]
    O: Optional[np.ndarray]            # [b, Hq, w, d]
    pool: np.ndarray                   # [b, Hkv, 2] (W, gamma)
    D: Optional[np.ndarray]            # [b, Hkv, 2] (D_front, D_rear), adaptive only


def score(Q, K, V, *, causal_tail: int = 0, scale: Optional[float] = None, ema_decay: float = 0.7,
          pool_mode: int = 0, width: int = 1, shift: int = 0, beta: float = 2000.0, base_width: int = 1,
          budget: int = 0, literal_gamma: bool = False, group_mode: int = 0,
          indicator_mode: int = 0, temporal_mode: int = 0, spatial_mode: int = 0, W_O=None,
          want_I_hat: bool = True, want_I_raw: bool = False, want_A: bool = False,
          want_O: bool = False) -> ScoreResult:
    """Steps Eq. 3 -> Eq. 7 -> Eq. 8-9 -> (Eq. 10-12) -> Eq. 13.  Q [b,Hq,w,d], K,V [b,Hkv,n_kv,d].

    The three `*_mode` switches pick the ablation variants of Appendix G (0 = the method as printed).
    W_O [Hq, d, d_model] float32: the output projection of Eq. 4, one d x d_model slice per query head."""
    Q, K, V = _f32(Q), _f32(K), _f32(V)
    b, Hq, w, d = Q.shape
    b2, Hkv, n_kv, d2 = K.shape
    if V.shape != K.shape or b2 != b or d2 != d:
        raise ValueError("shape mismatch")
    n = n_kv - causal_tail
    if scale is None:
        scale = 1.0 / np.sqrt(d)
    scores = np.empty((b, Hkv, n_kv), np.float64)
    I_hat = np.empty((b, Hkv, n), np.float64) if want_I_hat else None
    I_raw = np.empty((b, Hq, w, n), np.float64) if want_I_raw else None
    A = np.empty((b, Hq, w, n_kv), np.float64) if want_A else None
    O = np.empty((b, Hq, w, d), np.float64) if want_O else None
    pool = np.zeros((b, Hkv, 2), np.int32)
    D = np.zeros((b, Hkv, 2), np.float64) if pool_mode == 1 else None
    variant = (int(indicator_mode), int(temporal_mode), int(spatial_mode))
    lib = _load()
    plain = variant == (0, 0, 0) and W_O is None
    fn = lib.restkv_oracle_score if plain else lib.restkv_oracle_score_variant
    extra = ()
    if not plain:
        if W_O is not None:
            W_O = _f32(W_O)
            if W_O.ndim != 3 or W_O.shape[:2] != (Hq, d):
                raise ValueError("W_O must be [Hq, d, d_model]")
        extra = variant + (_ptr(W_O, ctypes.c_float), 0 if W_O is None else int(W_O.shape[2]))
    rc = fn(
        _ptr(Q, ctypes.c_float), _ptr(K, ctypes.c_float), _ptr(V, ctypes.c_float),
        b, Hq, Hkv, d, n_kv, w, causal_tail, float(scale), float(ema_decay),
        int(pool_mode), int(width), int(shift), float(beta), int(base_width),
        int(budget), int(bool(literal_gamma)), int(group_mode),
        *extra,
        _ptr(A, ctypes.c_double), _ptr(O, ctypes.c_double), _ptr(I_raw, ctypes.c_double),
        _ptr(I_hat, ctypes.c_double), _ptr(pool, ctypes.c_int), _ptr(D, ctypes.c_double),
        _ptr(scores, ctypes.c_double))
    if rc != 0:
        raise RuntimeError("restkv_oracle_score failed with code %d" % rc)
    return ScoreResult(scores, I_hat, I_raw, A, O, pool, D)


def select(scores: np.ndarray, budget: int) -> np.ndarray:
    """Eq. 14 argmax_B per (batch, KV head): [b,Hkv,n_kv] -> ascending int32 [b,Hkv,min(B,n_kv)]."""
    s = np.ascontiguousarray(scores, dtype=np.float64)
    lead, n_kv = s.shape[:-1], s.shape[-1]
    rows = int(np.prod(lead)) if lead else 1
    keep = min(int(budget), n_kv)
    out = np.empty(lead + (keep,), np.int32)
    rc = _load().restkv_oracle_select(_ptr(s, ctypes.c_double), rows, n_kv, int(budget), _ptr(out, ctypes.c_int))
    if rc != 0:
        raise RuntimeError("restkv_oracle_select failed with code %d" % rc)
    return out


def compact(X: np.ndarray, indices: np.ndarray) -> np.ndarray:
    """Eq. 14 gather: X [b,Hkv,n_kv,d] (any dtype, bytes copied untouched), indices [b,Hkv,n_sel]."""
    X = np.ascontiguousarray(X)
    idx = np.ascontiguousarray(indices, dtype=np.int32)
    b, H, n_kv, d = X.shape
    n_sel = idx.shape[-1]
    out = np.empty((b, H, n_sel, d), X.dtype)
    rc = _load().restkv_oracle_compact(X.ctypes.data, b * H, n_kv, d * X.dtype.itemsize,
                                       _ptr(idx, ctypes.c_int), n_sel, out.ctypes.data)
    if rc != 0:
        raise RuntimeError("restkv_oracle_compact failed with code %d" % rc)
    return out


def decode(q, Kc, Vc, *, scale: Optional[float] = None):
    """One decode step (Eq. 3) over a cache: q [b,Hq,d], Kc,Vc [b,Hkv,rows,d] -> (out [b,Hq,d], lse [b,Hq])."""
    q, Kc, Vc = _f32(q), _f32(Kc), _f32(Vc)
    b, Hq, d = q.shape
    _, Hkv, rows, _ = Kc.shape
    if scale is None:
        scale = 1.0 / np.sqrt(d)
    out = np.empty((b, Hq, d), np.float64)
    lse = np.empty((b, Hq), np.float64)
    rc = _load().restkv_oracle_decode(_ptr(q, ctypes.c_float), _ptr(Kc, ctypes.c_float), _ptr(Vc, ctypes.c_float),
                                      b, Hq, Hkv, d, rows, float(scale), _ptr(out, ctypes.c_double),
                                      _ptr(lse, ctypes.c_double))
    if rc != 0:
        raise RuntimeError("restkv_oracle_decode failed with code %d" % rc)
    return out, lse

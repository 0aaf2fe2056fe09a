"""Token-deletion definition of the eviction indicator (Eq. 6) -- TEST INFRASTRUCTURE ONLY.

For tiny inputs: really delete KV pair n, renormalise the softmax over what is left,
recompute the attention output and measure the l2 distance to the full output.  Written
with NumPy/SciPy library routines and no knowledge of the closed form (Eq. 7), so that
the C oracle's closed form can be pinned against it.
"""
from __future__ import annotations

import numpy as np
from scipy.special import softmax


def attention_output(q: np.ndarray, K: np.ndarray, V: np.ndarray, scale: float) -> np.ndarray:
    """Eq. 3 for one query: softmax(q K^T * scale) V, in float64."""
    a = softmax((K.astype(np.float64) @ q.astype(np.float64)) * scale)
    return a @ V.astype(np.float64)


def indicator_by_deletion(Q: np.ndarray, K: np.ndarray, V: np.ndarray, *, causal_tail: int = 0,
                          scale: float | None = None, W_O: np.ndarray | None = None) -> np.ndarray:
    """I[b, hq, i, j] = || out(full) - out(without pair j) ||_2 for every scored row j < n (Eq. 6).

    Q [b,Hq,w,d]; K,V [b,Hkv,n_kv,d]; with causal_tail = w query i also sees trailing rows
    n..n+i (its own and earlier window tokens) and only prefix rows j < n are deleted.
    W_O [Hq, d, d_model]: the head outputs are projected before they are compared (Eq. 4: the head's share of
    the layer output is z W_O).
    """
    b, Hq, w, d = Q.shape
    _, Hkv, n_kv, _ = K.shape
    G = Hq // Hkv
    n = n_kv - causal_tail
    if scale is None:
        scale = 1.0 / np.sqrt(d)
    out = np.zeros((b, Hq, w, n), np.float64)
    for bi in range(b):
        for hq in range(Hq):
            h = hq // G
            for i in range(w):
                vis = n_kv if causal_tail == 0 else n + i + 1
                Kv, Vv = K[bi, h, :vis], V[bi, h, :vis]
                full = attention_output(Q[bi, hq, i], Kv, Vv, scale)
                for j in range(n):
                    keep = np.ones(vis, bool)
                    keep[j] = False
                    if not keep.any():
                        out[bi, hq, i, j] = 0.0
                        continue
                    part = attention_output(Q[bi, hq, i], Kv[keep], Vv[keep], scale)
                    diff = full - part
                    if W_O is not None:
                        diff = diff @ W_O[hq].astype(np.float64)
                    out[bi, hq, i, j] = np.linalg.norm(diff)
    return out

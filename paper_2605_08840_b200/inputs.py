"""Seeded synthetic inputs for the eviction-scoring path.

This module holds no arithmetic of the method: it draws random Q/K/V with the shapes and
value structure of the paper's long-context workloads (Llama-3.1-8B / Mistral-7B attention
geometry, observation window S_w = 32, budgets up to 2048, contexts up to 128k; Section 4.1
and Appendix B) and rounds them once to the dtype under test.  The same arrays are handed to
the CPU oracle (as float32 holding dtype-exact values) and to the CUDA library (as raw bf16
bit patterns or float32).

Generator: NumPy `Generator(Philox(key=seed))`, `standard_normal(float32)`, drawn in the
fixed order Q, K, V, then the structure draws.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import Dict, Optional

import numpy as np


@dataclass(frozen=True)
class Case:
    """One workload: shapes, method knobs and the value recipe."""
    name: str
    batch: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    n: int                      # scored prefix rows
    w: int = 32                 # observation window S_w
    budget: int = 1024          # B
    width: int = 7              # fixed pooling width W
    shift: int = 0              # fixed pooling shift gamma
    ema_decay: float = 0.9      # 1 - alpha
    dtype: str = "bf16"         # "bf16" | "f32"
    causal_tail: int = 0        # 0, or w: K/V carry the window tokens' own rows
    recipe: str = "normal"      # "normal" | "normal_kscaled" | "planted" | "drift"
    seed: int = 0
    n_heavy: int = 64
    n_sink: int = 4

    @property
    def n_kv(self) -> int:
        return self.n + self.causal_tail

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    def with_(self, **kw) -> "Case":
        return replace(self, **kw)


# The five workloads (tiny, 8B-shaped layer, 32-layer drift, 128k long context, batched sweep) and the split of the first one.
CONFIGS: Dict[str, Case] = {
    # tiny single layer; "1a" keeps the K pre-scaling by 1/sqrt(64) literally, "1b" leaves K unscaled
    "cfg1a": Case("cfg1a", 1, 8, 2, 64, 1024, 32, 128, 7, 0, 0.9, "f32", 0, "normal_kscaled", 0),
    "cfg1b": Case("cfg1b", 1, 8, 2, 64, 1024, 32, 128, 7, 0, 0.9, "f32", 0, "normal", 0),
    # Llama-3.1-8B-shaped single layer with planted heavy hitters and attention sinks
    "cfg2": Case("cfg2", 1, 32, 8, 128, 16384, 32, 1024, 7, 0, 0.9, "bf16", 0, "planted", 2),
    # one of 32 layers at n = 32768 with a drifting key mean (seed = 3000 + layer)
    "cfg3": Case("cfg3", 1, 32, 8, 128, 32768, 32, 2048, 7, 0, 0.9, "bf16", 0, "drift", 3000),
    # long context, the timed headline
    "cfg4": Case("cfg4", 1, 32, 8, 128, 131072, 32, 2048, 7, 0, 0.9, "bf16", 0, "planted", 4),
    # batched sweep, Mistral-7B shape; budget / width / decay are swept by the caller
    "cfg5": Case("cfg5", 8, 32, 8, 128, 32768, 32, 2048, 7, 0, 0.9, "bf16", 0, "planted", 5000),
}


def round_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> bf16 bit patterns (uint16), round-to-nearest-even."""
    u = np.ascontiguousarray(x, np.float32).view(np.uint32)
    r = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """bf16 bit patterns (uint16) -> the float32 values they denote."""
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)


@dataclass
class Inputs:
    case: Case
    Q: np.ndarray            # float32 [b,Hq,w,d], dtype-exact values
    K: np.ndarray            # float32 [b,Hkv,n_kv,d]
    V: np.ndarray            # float32 [b,Hkv,n_kv,d]
    direction: Optional[np.ndarray] = None   # [b,Hkv,d] planted direction (float32, unrounded)
    heavy_rows: Optional[np.ndarray] = None  # [b,Hkv,n_heavy] planted row indices
    extras: dict = field(default_factory=dict)

    def device_arrays(self):
        """(Q, K, V) as the CUDA library wants them: int16 views of bf16 bits, or float32."""
        if self.case.dtype == "bf16":
            return tuple(round_to_bf16_bits(a).view(np.int16) for a in (self.Q, self.K, self.V))
        return self.Q, self.K, self.V


def _quantise(x: np.ndarray, dtype: str) -> np.ndarray:
    if dtype == "bf16":
        return bf16_bits_to_f32(round_to_bf16_bits(x))
    if dtype == "f32":
        return np.ascontiguousarray(x, np.float32)
    raise ValueError("dtype must be 'bf16' or 'f32'")


def make_inputs(case: Case, seed: Optional[int] = None) -> Inputs:
    """Draw Q, K, V for `case` (seed defaults to the case's own)."""
    seed = case.seed if seed is None else seed
    rng = np.random.Generator(np.random.Philox(key=seed))
    b, Hq, Hkv, d, w, G = case.batch, case.n_q_heads, case.n_kv_heads, case.head_dim, case.w, case.group
    n, n_kv = case.n, case.n_kv
    Q = rng.standard_normal((b, Hq, w, d), dtype=np.float32)
    K = rng.standard_normal((b, Hkv, n_kv, d), dtype=np.float32)
    V = rng.standard_normal((b, Hkv, n_kv, d), dtype=np.float32)
    direction = heavy = None
    if case.recipe == "normal":
        pass
    elif case.recipe == "normal_kscaled":
        K *= np.float32(1.0 / np.sqrt(d))
    elif case.recipe == "planted":
        # per KV head one direction s; queries lean on it, a few keys carry a multiple of it
        direction = rng.standard_normal((b, Hkv, d), dtype=np.float32)
        lean = np.float32(2.0 / np.sqrt(d))
        Q += lean * np.repeat(direction, G, axis=1)[:, :, None, :]
        n_heavy = min(case.n_heavy, max(n - case.n_sink, 0))
        heavy = np.zeros((b, Hkv, n_heavy), np.int64)
        for bi in range(b):
            for h in range(Hkv):
                rows = case.n_sink + rng.choice(n - case.n_sink, size=n_heavy, replace=False) if n_heavy else []
                heavy[bi, h] = np.sort(rows)
                K[bi, h, heavy[bi, h]] += np.float32(4.0) * direction[bi, h]
                K[bi, h, :min(case.n_sink, n)] += np.float32(2.0) * direction[bi, h]
    elif case.recipe == "drift":
        # slowly drifting key mean along the token axis: random walk, std 0.02 per token
        for bi in range(b):
            for h in range(Hkv):
                step = rng.standard_normal((n_kv, d), dtype=np.float32)
                step *= np.float32(0.02)
                step[0] = 0
                K[bi, h] += np.cumsum(step, axis=0, dtype=np.float32)
    else:
        raise ValueError("unknown recipe %r" % case.recipe)
    return Inputs(case, _quantise(Q, case.dtype), _quantise(K, case.dtype), _quantise(V, case.dtype),
                  direction, heavy)


def make_decode_query(inp: Inputs, seed: int = 0) -> np.ndarray:
    """A fresh query per query head for the decode timing: N(0,1) plus the planted lean."""
    c = inp.case
    rng = np.random.Generator(np.random.Philox(key=(1 << 40) + seed))
    q = rng.standard_normal((c.batch, c.n_q_heads, c.head_dim), dtype=np.float32)
    if inp.direction is not None:
        q += np.float32(2.0 / np.sqrt(c.head_dim)) * np.repeat(inp.direction, c.group, axis=1)
    return _quantise(q, c.dtype)

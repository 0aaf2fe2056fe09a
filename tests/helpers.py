"""Shared helpers of the GPU parity tests: run the CUDA library through its C ABI binding and
compare with the CPU oracle by the acceptance rules written out below."""
from __future__ import annotations

import numpy as np

from paper_2605_08840_b200 import binding as rk
from paper_2605_08840_b200.inputs import Case, Inputs

# relative tolerance of the scores: bf16 inputs with fp32 accumulation / fp32 mode
TOL = {"bf16": 2e-3, "f32": 1e-5}

# decode (a timing aid), fp32 SIMT kernels: max error of an output row relative to that row's largest element
DECODE_TOL = {"f32": 2e-5}


def decode_error_bound(q: np.ndarray, K: np.ndarray, V: np.ndarray, scale: float | None = None) -> np.ndarray:
    """Worst-case error of every decode output element on the bf16 path, from the exact softmax weights.

    The tensor-core kernel rounds each unnormalised softmax weight to bf16 (8 significant bits, round to nearest:
    relative error at most 2^-8) before the P V product and divides by the sum of the unrounded weights, so
    |out_k - exact_k| <= 2^-8 * sum_j A_j |v_jk|.  On top of that come the fp32 rounding of the logits (a few 1e-6
    of a weight after exponentiation), exp2 in hardware (2^-22 relative per weight) and fp32 accumulation
    (tensor-core accumulators, the split merge): a further 2^-15 of the same sum is allowed for those.  q [b,Hq,d], K,V [b,Hkv,rows,d] as float32 arrays holding the exact input values."""
    from scipy.special import softmax
    b, Hq, d = q.shape
    Hkv = K.shape[1]
    G = Hq // Hkv
    if scale is None:
        scale = 1.0 / np.sqrt(d)
    bound = np.empty((b, Hq, d), np.float64)
    for bi in range(b):
        for h in range(Hkv):
            Kh, Vh = K[bi, h].astype(np.float64), np.abs(V[bi, h].astype(np.float64))
            A = softmax(scale * (q[bi, h * G:(h + 1) * G].astype(np.float64) @ Kh.T), axis=-1)
            bound[bi, h * G:(h + 1) * G] = A @ Vh
    return bound * (2.0 ** -8 + 2.0 ** -15)


def assert_decode_close(out: np.ndarray, ref: np.ndarray, q, K, V, dtype: str):
    """bf16: element-wise against decode_error_bound; fp32: DECODE_TOL of the row's largest element."""
    if dtype == "bf16":
        bound = decode_error_bound(q, K, V)
        err = np.abs(out.astype(np.float64) - ref)
        assert np.all(err <= bound), "decode: worst error / bound = %.3f" % float(np.max(err / bound))
    else:
        scale = np.abs(ref).max(axis=-1, keepdims=True)
        assert np.max(np.abs(out - ref) / scale) < DECODE_TOL[dtype]


def torch_dev(arr: np.ndarray, dtype: str):
    """numpy (int16 bf16 bits | float32) -> CUDA tensor of the library's element type."""
    import torch
    t = torch.from_numpy(np.ascontiguousarray(arr)).cuda()
    return t.view(torch.bfloat16) if dtype == "bf16" else t


def shape_of(case: Case, **kw):
    return rk.make_shape(case.batch, case.n_q_heads, case.n_kv_heads, case.head_dim, case.n_kv, case.w,
                         case.causal_tail, rk.BF16 if case.dtype == "bf16" else rk.F32, **kw)


class DeviceRun:
    """Device copies of one workload plus output buffers; calls go through the binding only."""

    def __init__(self, handle: rk.Handle, inp: Inputs, budget: int | None = None, adaptive_budget: int = 0):
        import torch
        self.torch = torch
        self.h = handle
        self.inp = inp
        c = inp.case
        self.case = c
        self.budget = c.budget if budget is None else budget
        q, k, v = inp.device_arrays()
        self.Q, self.K, self.V = (torch_dev(a, c.dtype) for a in (q, k, v))
        self.shape = shape_of(c)
        self.keep = min(self.budget, c.n_kv)
        BH = (c.batch, c.n_kv_heads)
        self.scores = torch.empty(BH + (c.n_kv,), dtype=torch.float32, device="cuda")
        self.indices = torch.empty(BH + (self.keep,), dtype=torch.int32, device="cuda")
        self.K_out = torch.empty(BH + (self.keep, c.head_dim), dtype=self.K.dtype, device="cuda")
        self.V_out = torch.empty_like(self.K_out)
        self.pool_used = torch.zeros(BH + (2,), dtype=torch.int32, device="cuda")
        adaptive = adaptive_budget > 0
        nbytes = handle.workspace_bytes(self.shape, max(self.budget, adaptive_budget), adaptive=adaptive)
        assert nbytes > 0
        self.ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")

    def pool(self, width=None, shift=None):
        c = self.case
        return rk.fixed_pool(c.width if width is None else width, c.shift if shift is None else shift)

    def score(self, pool=None, ema_decay=None):
        self.h.score(self.shape, self.Q, self.K, self.V, self.case.ema_decay if ema_decay is None else ema_decay,
                     pool or self.pool(), self.scores, self.ws, pool_used=self.pool_used)
        self.torch.cuda.synchronize()
        return self.scores.cpu().numpy()

    def select(self):
        self.h.select(self.shape, self.scores, self.budget, self.indices, self.ws)
        self.torch.cuda.synchronize()
        return self.indices.cpu().numpy()

    def compact(self):
        self.h.compact(self.shape, self.K, self.V, self.indices, self.keep, self.K_out, self.V_out)
        self.torch.cuda.synchronize()
        return self._bits(self.K_out), self._bits(self.V_out)

    def evict(self, pool=None, ema_decay=None, with_scores=True):
        self.h.evict(self.shape, self.Q, self.K, self.V, self.case.ema_decay if ema_decay is None else ema_decay,
                     pool or self.pool(), self.budget, self.indices, self.K_out, self.V_out, self.ws,
                     scores_out=self.scores if with_scores else None)
        self.torch.cuda.synchronize()
        assert self.h.poll_status() == rk.RESTKV_OK
        return (self.scores.cpu().numpy(), self.indices.cpu().numpy(), self._bits(self.K_out),
                self._bits(self.V_out))

    def _bits(self, t):
        if self.case.dtype == "bf16":
            return t.view(self.torch.int16).cpu().numpy()
        return t.cpu().numpy()


def assert_scores_close(gpu: np.ndarray, ref: np.ndarray, tol: float, what: str = "scores"):
    """|gpu - ref| <= tol * |ref| on finite entries; +inf entries must match exactly."""
    assert gpu.shape == ref.shape, (gpu.shape, ref.shape)
    inf = np.isposinf(ref)
    assert np.array_equal(np.isposinf(gpu), inf), "%s: +inf pattern differs" % what
    fin = ~inf
    assert np.all(np.isfinite(gpu[fin])), "%s: non-finite value where the oracle is finite" % what
    err = np.abs(gpu[fin].astype(np.float64) - ref[fin])
    bound = tol * np.abs(ref[fin]) + 1e-30
    worst = np.max(err / np.maximum(np.abs(ref[fin]), 1e-300))
    assert np.all(err <= bound), "%s: max rel err %.3e exceeds %.1e" % (what, worst, tol)
    return worst


def assert_selection_valid(idx: np.ndarray, ref_scores: np.ndarray, budget: int, tol: float):
    """idx [..., keep] against oracle scores [..., n_kv]: exactly keep distinct ascending indices; every row
    whose oracle score beats the budget-th score by more than tol is present, none below it by more than tol."""
    n_kv = ref_scores.shape[-1]
    keep = min(budget, n_kv)
    assert idx.shape == ref_scores.shape[:-1] + (keep,)
    flat_i = idx.reshape(-1, keep)
    flat_s = ref_scores.reshape(-1, n_kv)
    exact = 0
    for r in range(flat_i.shape[0]):
        row, s = flat_i[r].astype(np.int64), flat_s[r]
        assert row.min() >= 0 and row.max() < n_kv
        assert np.all(np.diff(row) > 0), "indices must be strictly ascending"
        tau = np.sort(s)[::-1][keep - 1]
        chosen = np.zeros(n_kv, bool)
        chosen[row] = True
        if np.isfinite(tau):
            must = s > tau * (1 + tol) + 1e-30
            must_not = s < tau * (1 - tol) - 1e-30
        else:
            must = np.zeros(n_kv, bool)
            must_not = ~np.isposinf(s)
        assert np.all(chosen[must]), "a row clearly above the threshold is missing"
        assert not np.any(chosen[must_not]), "a row clearly below the threshold was selected"
        ref_idx = np.sort(np.argsort(-s, kind="stable")[:keep])
        exact += int(np.array_equal(ref_idx, row))
    return exact / flat_i.shape[0]


def assert_compaction_exact(idx: np.ndarray, X_bits: np.ndarray, X_out_bits: np.ndarray):
    expect = np.take_along_axis(X_bits, idx[..., None].astype(np.int64), axis=2)
    assert np.array_equal(expect, X_out_bits), "compacted rows are not bit-exact copies"

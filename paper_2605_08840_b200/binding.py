"""Thin ctypes binding of librestkv.so (the C ABI declared in include/restkv.h).

Argument marshalling only: tensors are torch CUDA tensors whose data pointers are passed
through; every step of the path runs in the library's CUDA kernels.  There is no fallback:
if the shared library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "librestkv.so")

RESTKV_OK = 0
ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT = 1, 2, 3, 4, 5
BF16, F32 = 0, 1
POOL_FIXED, POOL_ADAPTIVE = 0, 1
PATH_AUTO, PATH_SIMT, PATH_TENSOR_CORE, PATH_HEAD_SEQUENTIAL = 0, 1, 2, 3

EXPORTS = [
    "restkv_create", "restkv_destroy", "restkv_workspace_bytes", "restkv_workspace_bytes_adaptive",
    "restkv_score", "restkv_score_from_lse", "restkv_select", "restkv_compact", "restkv_evict", "restkv_evict_from_lse", "restkv_evict_host", "restkv_decode", "restkv_decode_static",
    "restkv_decode_static_last_cuda_error",
    "restkv_poll_status", "restkv_launch_count", "restkv_last_cuda_error", "restkv_error_string",
    "restkv_set_kernel_path", "restkv_set_profile_events", "restkv_set_wait_limit", "restkv_set_fused_select", "restkv_last_evict_fused_select",
    "restkv_set_variant", "restkv_evict_budgets",
    "restkv_output_projection_bytes", "restkv_prepare_output_projection", "restkv_set_output_projection",
]
KERNEL_NONE, KERNEL_PASS1, KERNEL_COMBINE, KERNEL_PASS2, KERNEL_POOL, KERNEL_SELECT, KERNEL_COMPACT = range(7)


class Shape(ctypes.Structure):
    _fields_ = [
        ("batch", ctypes.c_int), ("n_q_heads", ctypes.c_int), ("n_kv_heads", ctypes.c_int), ("head_dim", ctypes.c_int),
        ("n_kv", ctypes.c_int), ("w", ctypes.c_int), ("causal_tail", ctypes.c_int), ("dtype", ctypes.c_int),
        ("softmax_scale", ctypes.c_float),
        ("k_stride_b", ctypes.c_longlong), ("k_stride_h", ctypes.c_longlong), ("k_stride_n", ctypes.c_longlong),
        ("v_stride_b", ctypes.c_longlong), ("v_stride_h", ctypes.c_longlong), ("v_stride_n", ctypes.c_longlong),
    ]


class PoolParams(ctypes.Structure):
    _fields_ = [("mode", ctypes.c_int), ("width", ctypes.c_int), ("shift", ctypes.c_int), ("beta", ctypes.c_float),
                ("base_width", ctypes.c_int), ("budget", ctypes.c_int)]


class Variant(ctypes.Structure):
    """restkv_variant: the ablation variants of Appendix G as modes of the score calls (all 0 = the method)."""
    _fields_ = [("indicator", ctypes.c_int), ("temporal", ctypes.c_int), ("spatial", ctypes.c_int),
                ("group", ctypes.c_int)]


INDICATOR_RECONSTRUCTION, INDICATOR_ATTENTION, INDICATOR_ATTENTION_VNORM = 0, 1, 2
TEMPORAL_EMA, TEMPORAL_MEAN, TEMPORAL_INV_EMA, TEMPORAL_NONE = 0, 1, 2, 3
SPATIAL_MEAN, SPATIAL_MAX = 0, 1
GROUP_MEAN, GROUP_MAX = 0, 1


class RestKVError(RuntimeError):
    def __init__(self, status: int, what: str, cuda_error: int = 0):
        self.status = status
        self.cuda_error = cuda_error
        super().__init__("%s failed: status %d (%s)%s" % (
            what, status, error_string(status), " cuda error %d" % cuda_error if cuda_error else ""))


_lib = None


def load_library() -> ctypes.CDLL:
    """Loads librestkv.so; raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError("librestkv.so is not built: run `python -m paper_2605_08840_b200.build` "
                           "(or __graft_entry__.build()); there is no CPU fallback")
    lib = ctypes.CDLL(LIB_PATH)
    vp, sz, ci, cf = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int, ctypes.c_float
    shp, pool = ctypes.POINTER(Shape), ctypes.POINTER(PoolParams)
    lib.restkv_create.argtypes = [ctypes.POINTER(vp)]
    lib.restkv_destroy.argtypes = [vp]
    lib.restkv_workspace_bytes.argtypes = [shp, ci]
    lib.restkv_workspace_bytes.restype = sz
    lib.restkv_workspace_bytes_adaptive.argtypes = [shp, ci]
    lib.restkv_workspace_bytes_adaptive.restype = sz
    lib.restkv_score.argtypes = [vp, shp, vp, vp, vp, cf, pool, vp, vp, vp, sz, vp]
    lib.restkv_score_from_lse.argtypes = [vp, shp, vp, vp, vp, vp, vp, cf, pool, vp, vp, vp, sz, vp]
    lib.restkv_select.argtypes = [vp, shp, vp, ci, vp, vp, sz, vp]
    lib.restkv_compact.argtypes = [vp, shp, vp, vp, vp, ci, vp, vp, vp]
    lib.restkv_evict.argtypes = [vp, shp, vp, vp, vp, cf, pool, ci, vp, vp, vp, vp, vp, sz, vp]
    lib.restkv_evict_from_lse.argtypes = [vp, shp, vp, vp, vp, vp, vp, cf, pool, ci, vp, vp, vp, vp, vp, sz, vp]
    lib.restkv_evict_budgets.argtypes = [vp, shp, vp, vp, vp, cf, pool, vp, ci, vp, vp, vp, vp, vp, sz, vp]
    lib.restkv_evict_host.argtypes = [vp, shp, vp, vp, vp, cf, pool, ci, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.restkv_decode.argtypes = [vp, shp, vp, vp, vp, ci, vp, vp, vp, sz, vp]
    lib.restkv_decode_static.argtypes = [shp, vp, vp, vp, ci, vp, vp, vp]
    lib.restkv_poll_status.argtypes = [vp, vp]
    lib.restkv_launch_count.argtypes = [vp]
    lib.restkv_launch_count.restype = ctypes.c_longlong
    lib.restkv_last_cuda_error.argtypes = [vp]
    lib.restkv_error_string.argtypes = [ci]
    lib.restkv_error_string.restype = ctypes.c_char_p
    lib.restkv_set_kernel_path.argtypes = [vp, ci]
    lib.restkv_set_profile_events.argtypes = [vp, ci, vp, vp]
    lib.restkv_set_wait_limit.argtypes = [vp, ctypes.c_longlong]
    lib.restkv_set_fused_select.argtypes = [vp, ci]
    lib.restkv_last_evict_fused_select.argtypes = [vp]
    lib.restkv_set_variant.argtypes = [vp, ctypes.POINTER(Variant)]
    lib.restkv_output_projection_bytes.argtypes = [ci, ci]
    lib.restkv_output_projection_bytes.restype = sz
    lib.restkv_prepare_output_projection.argtypes = [vp, ci, ci, ci, ci, vp, vp, sz, vp]
    lib.restkv_set_output_projection.argtypes = [vp, vp, ci, ci]
    _lib = lib
    return lib


def error_string(status: int) -> str:
    return load_library().restkv_error_string(int(status)).decode()


def make_shape(batch, n_q_heads, n_kv_heads, head_dim, n_kv, w, causal_tail=0, dtype=BF16, softmax_scale=0.0,
               k_strides=(0, 0, 0), v_strides=(0, 0, 0)) -> Shape:
    return Shape(batch, n_q_heads, n_kv_heads, head_dim, n_kv, w, causal_tail, dtype, softmax_scale,
                 *k_strides, *v_strides)


def fixed_pool(width: int = 1, shift: int = 0) -> PoolParams:
    return PoolParams(POOL_FIXED, width, shift, 0.0, 1, 0)


def adaptive_pool(beta: float, base_width: int, budget: int) -> PoolParams:
    return PoolParams(POOL_ADAPTIVE, 1, 0, beta, base_width, budget)


def _ptr(t) -> Optional[int]:
    """Device (or host) address of a torch tensor; None passes NULL."""
    if t is None:
        return None
    return t.data_ptr()


def _stream_ptr(stream) -> Optional[int]:
    if stream is None:
        import torch
        stream = torch.cuda.current_stream()
    return stream.cuda_stream or None


def decode_static(shape, q, Kc, Vc, n_rows, out, lse=None, stream=None) -> None:
    """restkv_decode_static: decode without a handle or a workspace (partials in the library's own 2 MiB array).

    For callers that cannot allocate device memory at this point; see include/restkv.h for the capacity limit
    and the rule that calls sharing a device must not overlap on the GPU."""
    lib = load_library()
    st = lib.restkv_decode_static(ctypes.byref(shape), _ptr(q), _ptr(Kc), _ptr(Vc), int(n_rows), _ptr(out), _ptr(lse),
                                  _stream_ptr(stream))
    if st != RESTKV_OK:
        raise RestKVError(st, "restkv_decode_static", lib.restkv_decode_static_last_cuda_error())


class Handle:
    """Owns a restkv_handle for the current CUDA device."""

    def __init__(self):
        self._lib = load_library()
        self._h = ctypes.c_void_p()
        st = self._lib.restkv_create(ctypes.byref(self._h))
        if st != RESTKV_OK:
            raise RestKVError(st, "restkv_create")

    def close(self):
        if self._h:
            self._lib.restkv_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, st: int, what: str):
        if st != RESTKV_OK:
            raise RestKVError(st, what, self._lib.restkv_last_cuda_error(self._h))

    # -- same names as the C ABI, same argument order --------------------------------------------
    def workspace_bytes(self, shape: Shape, budget: int, adaptive: bool = False) -> int:
        f = self._lib.restkv_workspace_bytes_adaptive if adaptive else self._lib.restkv_workspace_bytes
        return int(f(ctypes.byref(shape), int(budget)))

    def score(self, shape, Q_obs, K, V, ema_decay, pool, scores, workspace, pool_used=None, stream=None):
        self._check(self._lib.restkv_score(self._h, ctypes.byref(shape), _ptr(Q_obs), _ptr(K), _ptr(V),
                                           float(ema_decay), ctypes.byref(pool), _ptr(scores), _ptr(pool_used),
                                           _ptr(workspace), workspace.numel() * workspace.element_size(),
                                           _stream_ptr(stream)), "restkv_score")

    def score_from_lse(self, shape, Q_obs, K, V, O_obs, LSE_obs, ema_decay, pool, scores, workspace, pool_used=None,
                       stream=None):
        self._check(self._lib.restkv_score_from_lse(self._h, ctypes.byref(shape), _ptr(Q_obs), _ptr(K), _ptr(V),
                                                    _ptr(O_obs), _ptr(LSE_obs), float(ema_decay), ctypes.byref(pool),
                                                    _ptr(scores), _ptr(pool_used), _ptr(workspace),
                                                    workspace.numel() * workspace.element_size(),
                                                    _stream_ptr(stream)), "restkv_score_from_lse")

    def select(self, shape, scores, budget, indices, workspace, stream=None):
        self._check(self._lib.restkv_select(self._h, ctypes.byref(shape), _ptr(scores), int(budget), _ptr(indices),
                                            _ptr(workspace), workspace.numel() * workspace.element_size(),
                                            _stream_ptr(stream)), "restkv_select")

    def compact(self, shape, K, V, indices, n_sel, K_out, V_out, stream=None):
        self._check(self._lib.restkv_compact(self._h, ctypes.byref(shape), _ptr(K), _ptr(V), _ptr(indices),
                                             int(n_sel), _ptr(K_out), _ptr(V_out), _stream_ptr(stream)),
                    "restkv_compact")

    def evict(self, shape, Q_obs, K, V, ema_decay, pool, budget, indices, K_out, V_out, workspace,
              scores_out=None, stream=None):
        self._check(self._lib.restkv_evict(self._h, ctypes.byref(shape), _ptr(Q_obs), _ptr(K), _ptr(V),
                                           float(ema_decay), ctypes.byref(pool), int(budget), _ptr(scores_out),
                                           _ptr(indices), _ptr(K_out), _ptr(V_out), _ptr(workspace),
                                           workspace.numel() * workspace.element_size(), _stream_ptr(stream)),
                    "restkv_evict")

    def evict_budgets(self, shape, Q_obs, K, V, ema_decay, pool, budgets, max_budget, indices, K_out, V_out,
                      workspace, scores_out=None, stream=None):
        self._check(self._lib.restkv_evict_budgets(self._h, ctypes.byref(shape), _ptr(Q_obs), _ptr(K), _ptr(V),
                                                   float(ema_decay), ctypes.byref(pool), _ptr(budgets),
                                                   int(max_budget), _ptr(scores_out), _ptr(indices), _ptr(K_out),
                                                   _ptr(V_out), _ptr(workspace),
                                                   workspace.numel() * workspace.element_size(), _stream_ptr(stream)),
                    "restkv_evict_budgets")

    def evict_from_lse(self, shape, Q_obs, K, V, O_obs, LSE_obs, ema_decay, pool, budget, indices, K_out, V_out,
                       workspace, scores_out=None, stream=None):
        self._check(self._lib.restkv_evict_from_lse(self._h, ctypes.byref(shape), _ptr(Q_obs), _ptr(K), _ptr(V),
                                                    _ptr(O_obs), _ptr(LSE_obs), float(ema_decay), ctypes.byref(pool),
                                                    int(budget), _ptr(scores_out), _ptr(indices), _ptr(K_out),
                                                    _ptr(V_out), _ptr(workspace),
                                                    workspace.numel() * workspace.element_size(), _stream_ptr(stream)),
                    "restkv_evict_from_lse")

    def evict_host(self, shape, Q_host, K_host, V_host, ema_decay, pool, budget, indices_host, K_out_host,
                   V_out_host, d_Q, d_K, d_V, d_indices, d_K_out, d_V_out, workspace, stream=None):
        self._check(self._lib.restkv_evict_host(
            self._h, ctypes.byref(shape), _ptr(Q_host), _ptr(K_host), _ptr(V_host), float(ema_decay),
            ctypes.byref(pool), int(budget), _ptr(indices_host), _ptr(K_out_host), _ptr(V_out_host), _ptr(d_Q),
            _ptr(d_K), _ptr(d_V), _ptr(d_indices), _ptr(d_K_out), _ptr(d_V_out), _ptr(workspace),
            workspace.numel() * workspace.element_size(), _stream_ptr(stream)), "restkv_evict_host")

    def decode(self, shape, q, Kc, Vc, n_rows, out, workspace, lse=None, stream=None):
        self._check(self._lib.restkv_decode(self._h, ctypes.byref(shape), _ptr(q), _ptr(Kc), _ptr(Vc), int(n_rows),
                                            _ptr(out), _ptr(lse), _ptr(workspace),
                                            workspace.numel() * workspace.element_size(), _stream_ptr(stream)),
                    "restkv_decode")

    def poll_status(self, stream=None) -> int:
        return int(self._lib.restkv_poll_status(self._h, _stream_ptr(stream)))

    def launch_count(self) -> int:
        return int(self._lib.restkv_launch_count(self._h))

    def set_kernel_path(self, path: int):
        self._check(self._lib.restkv_set_kernel_path(self._h, int(path)), "restkv_set_kernel_path")

    def set_fused_select(self, on: bool):
        self._check(self._lib.restkv_set_fused_select(self._h, int(bool(on))), "restkv_set_fused_select")

    def last_evict_fused_select(self) -> bool:
        return bool(self._lib.restkv_last_evict_fused_select(self._h))

    def set_variant(self, indicator: int = 0, temporal: int = 0, spatial: int = 0, group: int = 0):
        v = Variant(int(indicator), int(temporal), int(spatial), int(group))
        self._check(self._lib.restkv_set_variant(self._h, ctypes.byref(v)), "restkv_set_variant")

    def output_projection_bytes(self, n_q_heads: int, head_dim: int) -> int:
        return int(self._lib.restkv_output_projection_bytes(int(n_q_heads), int(head_dim)))

    def prepare_output_projection(self, n_q_heads, head_dim, d_model, dtype, W_O, factor, stream=None):
        self._check(self._lib.restkv_prepare_output_projection(
            self._h, int(n_q_heads), int(head_dim), int(d_model), int(dtype), _ptr(W_O), _ptr(factor),
            factor.numel() * factor.element_size(), _stream_ptr(stream)), "restkv_prepare_output_projection")

    def set_output_projection(self, factor=None, n_q_heads: int = 0, head_dim: int = 0):
        self._check(self._lib.restkv_set_output_projection(self._h, _ptr(factor), int(n_q_heads), int(head_dim)),
                    "restkv_set_output_projection")

    def set_wait_limit(self, sm_clocks: int):
        self._check(self._lib.restkv_set_wait_limit(self._h, int(sm_clocks)), "restkv_set_wait_limit")

    def set_profile_events(self, which: int, start=None, stop=None):
        """start/stop: torch.cuda.Event(enable_timing=True) that have been recorded once, or None to clear."""
        a = start.cuda_event if start is not None else None
        b = stop.cuda_event if stop is not None else None
        if (start is not None) and (not a or not b):
            raise ValueError("profile events must be created (record them once) before they are handed over")
        self._check(self._lib.restkv_set_profile_events(self._h, int(which), a, b), "restkv_set_profile_events")

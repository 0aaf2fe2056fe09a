"""restkv_decode_static: the decode step for callers that cannot allocate device memory.

An inference server that gave the whole GPU to its own pool at start-up, or a token loop that cannot afford the
device-wide synchronisation of cudaMalloc, cannot hand restkv_decode a workspace (nor create a handle, which
allocates a status block).  The static variant keeps its split partials in an array inside the library image.
This file checks, through the C ABI, that it returns what restkv_decode returns, on two calls in a row with
different inputs (the shared array keeps the first call's contents, which must not leak into the second), and
that shapes beyond the array's capacity are refused.  It is collected last on purpose.
"""
import numpy as np
import pytest

from paper_2605_08840_b200 import binding as rk
from paper_2605_08840_b200.inputs import Case, round_to_bf16_bits

from helpers import DECODE_TOL, shape_of, torch_dev

pytestmark = pytest.mark.gpu


def _draw(rng, shape):
    x = rng.standard_normal(shape).astype(np.float32)
    return round_to_bf16_bits(x).view(np.int16)


def test_static_decode_matches_decode_on_two_calls_in_a_row():
    import torch
    handle = rk.Handle()
    rng = np.random.default_rng(21)
    # first a long cache (many splits fill the shared array), then a short one with other shapes
    for b, Hq, Hkv, d, rows in ((1, 32, 8, 128, 20000), (2, 8, 2, 64, 300)):
        case = Case("static_dec", b, Hq, Hkv, d, rows, 1, dtype="bf16")
        shape = shape_of(case)
        q = torch_dev(_draw(rng, (b, Hq, d)), "bf16")
        K = torch_dev(_draw(rng, (b, Hkv, rows, d)), "bf16")
        V = torch_dev(_draw(rng, (b, Hkv, rows, d)), "bf16")
        ref = torch.empty((b, Hq, d), dtype=torch.float32, device="cuda")
        ref_lse = torch.empty((b, Hq), dtype=torch.float32, device="cuda")
        ws = torch.empty(handle.workspace_bytes(shape, 0), dtype=torch.uint8, device="cuda")
        handle.decode(shape, q, K, V, rows, ref, ws, lse=ref_lse)
        out = torch.full((b, Hq, d), float("nan"), dtype=torch.float32, device="cuda")
        lse = torch.full((b, Hq), float("nan"), dtype=torch.float32, device="cuda")
        rk.decode_static(shape, q, K, V, rows, out, lse=lse)
        torch.cuda.synchronize()
        ref_np, out_np = ref.cpu().numpy(), out.cpu().numpy()
        scale = np.abs(ref_np).max(axis=-1, keepdims=True)
        assert np.all(np.isfinite(out_np))
        assert np.max(np.abs(out_np - ref_np) / scale) < DECODE_TOL["bf16"]   # the tolerance of the decode parity tests
        np.testing.assert_allclose(lse.cpu().numpy(), ref_lse.cpu().numpy(), rtol=1e-5, atol=1e-5)
    assert handle.poll_status() == rk.RESTKV_OK
    handle.close()


def test_static_decode_refuses_what_does_not_fit():
    import torch
    # batch * n_q_heads * (head_dim + 2) = 64 * 64 * 130 floats per split > 524288: nothing may be enqueued
    case = Case("static_big", 64, 64, 8, 128, 16, 1, dtype="bf16")
    shape = shape_of(case)
    q = torch.zeros((64, 64, 128), dtype=torch.bfloat16, device="cuda")
    K = torch.zeros((64, 8, 16, 128), dtype=torch.bfloat16, device="cuda")
    out = torch.zeros((64, 64, 128), dtype=torch.float32, device="cuda")
    with pytest.raises(rk.RestKVError) as err:
        rk.decode_static(shape, q, K, K, 16, out)
    assert err.value.status == rk.ERR_WORKSPACE
    with pytest.raises(rk.RestKVError) as err:
        rk.decode_static(shape, None, K, K, 16, out)
    assert err.value.status == rk.ERR_INVALID_ARG
    torch.cuda.synchronize()

"""restkv_decode_static: the decode step for callers that cannot allocate device memory.

An inference server that gave the whole GPU to its own pool at start-up, or a token loop that cannot afford the
device-wide synchronisation of cudaMalloc, cannot hand restkv_decode a workspace (nor create a handle, which
allocates a status block).  The static variant keeps its split partials in an array inside the library image.
This file checks, through the C ABI, that it returns what the CPU oracle and restkv_decode return, on calls in a
row with different inputs (the shared array keeps the previous call's contents, which must not leak into the next),
that the amount of free device memory does not move across a call, and that shapes beyond the array's capacity are
refused.  It is collected last on purpose.
"""
import numpy as np
import pytest

import oracle
from paper_2605_08840_b200 import binding as rk
from paper_2605_08840_b200.inputs import Case, bf16_bits_to_f32, round_to_bf16_bits

from helpers import assert_decode_close, shape_of, torch_dev

pytestmark = pytest.mark.gpu


def _draw(rng, shape, dtype):
    """(exact values as float32, the array the library gets)."""
    x = rng.standard_normal(shape).astype(np.float32)
    if dtype == "bf16":
        bits = round_to_bf16_bits(x)
        return bf16_bits_to_f32(bits), bits.view(np.int16)
    return x, x


# batch, query heads, KV heads, head_dim, rows, dtype.  First a long cache (many splits fill the shared array), then
# shorter ones with other shapes: one whose split count the array's capacity lowers (64 * 258 floats per split leave
# room for 31 splits where restkv_decode takes 37), one in fp32 with a single query head per KV head, one with eight.
STATIC_SHAPES = ((1, 32, 8, 128, 20000, "bf16"), (2, 8, 2, 64, 300, "bf16"), (1, 64, 8, 256, 16384, "bf16"),
                 (2, 4, 4, 64, 777, "f32"), (1, 16, 2, 128, 1500, "bf16"))


def test_static_decode_matches_oracle_and_decode_on_calls_in_a_row():
    import torch
    handle = rk.Handle()
    rng = np.random.default_rng(21)
    for b, Hq, Hkv, d, rows, dtype in STATIC_SHAPES:
        case = Case("static_dec", b, Hq, Hkv, d, rows, 1, dtype=dtype)
        shape = shape_of(case)
        q, qd = _draw(rng, (b, Hq, d), dtype)
        K, Kd = _draw(rng, (b, Hkv, rows, d), dtype)
        V, Vd = _draw(rng, (b, Hkv, rows, d), dtype)
        dq, dK, dV = torch_dev(qd, dtype), torch_dev(Kd, dtype), torch_dev(Vd, dtype)
        ref = torch.empty((b, Hq, d), dtype=torch.float32, device="cuda")
        ref_lse = torch.empty((b, Hq), dtype=torch.float32, device="cuda")
        ws = torch.empty(handle.workspace_bytes(shape, 0), dtype=torch.uint8, device="cuda")
        handle.decode(shape, dq, dK, dV, rows, ref, ws, lse=ref_lse)
        out = torch.full((b, Hq, d), float("nan"), dtype=torch.float32, device="cuda")
        lse = torch.full((b, Hq), float("nan"), dtype=torch.float32, device="cuda")
        torch.cuda.synchronize()
        free_before, _ = torch.cuda.mem_get_info()
        rk.decode_static(shape, dq, dK, dV, rows, out, lse=lse)
        torch.cuda.synchronize()
        free_after, _ = torch.cuda.mem_get_info()
        if (b, Hq, Hkv, d, rows, dtype) != STATIC_SHAPES[0]:
            # (the very first call on a device may make the driver load the module that holds the array)
            assert free_after == free_before, "the call changed the amount of free device memory"
        out_np = out.cpu().numpy()
        assert np.all(np.isfinite(out_np))
        want, want_lse = oracle.decode(q, K, V)
        assert_decode_close(out_np, want, q, K, V, dtype)
        np.testing.assert_allclose(lse.cpu().numpy(), want_lse, rtol=1e-5, atol=1e-5)
        # and the existing entry point, within the same bound (both are within it of the exact result)
        assert_decode_close(ref.cpu().numpy(), want, q, K, V, dtype)
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

"""GPU parity: the CUDA library, called through its C ABI binding, against the CPU oracle on the same
seeded inputs.  Scores within the stated relative tolerance, selections identical up to rows whose
oracle score lies inside that tolerance of the budget-th score, compaction bit-exact."""
import numpy as np
import pytest

import oracle
from paper_2605_08840_b200 import binding as rk
from paper_2605_08840_b200.inputs import CONFIGS, Case, make_inputs, make_decode_query, round_to_bf16_bits

from helpers import (TOL, DeviceRun, assert_compaction_exact, assert_decode_close, assert_scores_close, assert_selection_valid,
                     shape_of, torch_dev)

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def handle():
    h = rk.Handle()
    yield h
    h.close()


def oracle_scores(inp, **kw):
    c = inp.case
    args = dict(causal_tail=c.causal_tail, ema_decay=c.ema_decay, width=c.width, shift=c.shift)
    args.update(kw)
    return oracle.score(inp.Q, inp.K, inp.V, **args)


def full_check(handle, inp, budget=None, path=rk.PATH_AUTO, **pool_kw):
    """evict on the GPU vs score+select on the oracle, all three acceptance rules."""
    c = inp.case
    handle.set_kernel_path(path)
    try:
        run = DeviceRun(handle, inp, budget=budget)
        scores, idx, K_out, V_out = run.evict(pool=run.pool(**pool_kw))
    finally:
        handle.set_kernel_path(rk.PATH_AUTO)
    ref = oracle_scores(inp, **pool_kw)
    tol = TOL[c.dtype]
    worst = assert_scores_close(scores, ref.scores, tol)
    exact = assert_selection_valid(idx, ref.scores, run.budget, tol)
    _, kbits, vbits = inp.device_arrays()
    assert_compaction_exact(idx, kbits, K_out)
    assert_compaction_exact(idx, vbits, V_out)
    return worst, exact


# ------------------------------------------------------------------ config 1 (tiny, fp32 and bf16)
@pytest.mark.parametrize("name", ["cfg1a", "cfg1b"])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("tail", [0, 32])
def test_config1(handle, name, dtype, tail):
    case = CONFIGS[name].with_(dtype=dtype, causal_tail=tail)
    full_check(handle, make_inputs(case))


def test_config1_separate_calls_match_fused(handle):
    inp = make_inputs(CONFIGS["cfg1b"])
    run = DeviceRun(handle, inp)
    s_f, i_f, k_f, v_f = run.evict()
    s = run.score()
    i = run.select()
    k, v = run.compact()
    np.testing.assert_array_equal(s, s_f)
    np.testing.assert_array_equal(i, i_f)
    np.testing.assert_array_equal(k, k_f)
    np.testing.assert_array_equal(v, v_f)


@pytest.mark.parametrize("tail", [0, 32])
def test_config1_adaptive_window(handle, tail):
    case = CONFIGS["cfg1b"].with_(causal_tail=tail)
    inp = make_inputs(case)
    B = case.budget
    probe = oracle_scores(inp, pool_mode=1, beta=1e9, base_width=1, budget=B)
    delta = abs(probe.D[..., 0] - probe.D[..., 1]).min()
    assert delta > 0
    # beta chosen from the oracle's own D so that (D_front - D_rear)/beta sits mid-way between integers
    compared = 0
    for target, base in ((0.5, 1), (1.5, 1), (2.5, 5)):
        beta = float(delta / target)
        ref = oracle_scores(inp, pool_mode=1, beta=beta, base_width=base, budget=B)
        x = (ref.D[..., 0] - ref.D[..., 1]) / beta
        if np.any(np.abs(x - np.round(x)) < 0.05):
            continue   # too close to a rounding boundary for an fp32-vs-fp64 ranking comparison
        run = DeviceRun(handle, inp, adaptive_budget=B)
        scores = run.score(pool=rk.adaptive_pool(beta, base, B))
        np.testing.assert_array_equal(run.pool_used.cpu().numpy(), ref.pool)
        assert_scores_close(scores, ref.scores, TOL[case.dtype])
        compared += 1
    assert compared > 0, "every beta landed on a rounding boundary: nothing was compared"


# ------------------------------------------------------------------ config 2 (8B-shaped layer)
@pytest.mark.parametrize("path", [rk.PATH_AUTO, rk.PATH_SIMT, rk.PATH_HEAD_SEQUENTIAL])
def test_config2(handle, path):
    inp = make_inputs(CONFIGS["cfg2"])
    worst, exact = full_check(handle, inp, path=path)
    # the planted heavy rows and sinks should be kept (reported, and checked loosely)
    run = DeviceRun(handle, inp)
    _, idx, _, _ = run.evict()
    planted = np.concatenate([inp.heavy_rows, np.broadcast_to(np.arange(4), inp.heavy_rows.shape[:2] + (4,))], -1)
    recall = np.mean([np.isin(planted[0, h], idx[0, h]).mean() for h in range(8)])
    assert recall > 0.9


@pytest.mark.parametrize("path", [rk.PATH_AUTO, rk.PATH_HEAD_SEQUENTIAL])
def test_config2_causal_tail(handle, path):
    full_check(handle, make_inputs(CONFIGS["cfg2"].with_(causal_tail=32)), path=path)


@pytest.mark.parametrize("spec", [(2, 8, 2, 1000, 32, 0), (1, 8, 1, 700, 16, 0), (2, 4, 1, 4097, 32, 32), (3, 4, 1, 129, 32, 0)])
def test_head_sequential_kernel_on_ragged_shapes(handle, spec):
    b, Hq, Hkv, n, w, tail = spec
    case = Case("headseq", b, Hq, Hkv, 128, n, w, 64, 5, 0, 0.8, "bf16", tail, "normal", 91)
    full_check(handle, make_inputs(case), path=rk.PATH_HEAD_SEQUENTIAL)


def test_head_sequential_kernel_at_full_size(handle):
    full_check(handle, make_inputs(CONFIGS["cfg4"]), path=rk.PATH_HEAD_SEQUENTIAL)


def _adaptive_check(handle, inp, path, base=5, evict=False):
    """Eq. 10-12: D_front / D_rear from the per-query top-B, window width and shift, then the pooled scores; heads
    whose (D_front - D_rear) / beta lands too close to a rounding boundary are not compared."""
    case = inp.case
    B = case.budget
    probe = oracle_scores(inp, pool_mode=1, beta=1e9, base_width=1, budget=B)
    delta = abs(probe.D[..., 0] - probe.D[..., 1]).min()
    assert delta > 0
    beta = float(delta / 1.5)                     # (D_front - D_rear) / beta = +-1.5 on the head with the smallest gap
    ref = oracle_scores(inp, pool_mode=1, beta=beta, base_width=base, budget=B)
    x = (ref.D[..., 0] - ref.D[..., 1]) / beta
    keep = np.abs(x - np.round(x)) >= 0.05
    assert keep.any()
    handle.set_kernel_path(path)
    try:
        run = DeviceRun(handle, inp, adaptive_budget=B)
        pool = rk.adaptive_pool(beta, base, B)
        if evict:
            scores, idx, K_out, V_out = run.evict(pool=pool)
        else:
            scores = run.score(pool=pool)
            used = run.pool_used.cpu().numpy()
            np.testing.assert_array_equal(used[keep], ref.pool[keep])
    finally:
        handle.set_kernel_path(rk.PATH_AUTO)
    for b, h in zip(*np.nonzero(keep)):
        assert_scores_close(scores[b, h], ref.scores[b, h], TOL[case.dtype])
        if evict:
            assert_selection_valid(idx[b, h], ref.scores[b, h], B, TOL[case.dtype])
    if evict:
        _, kbits, vbits = inp.device_arrays()
        assert_compaction_exact(idx, kbits, K_out)
        assert_compaction_exact(idx, vbits, V_out)
    return keep


@pytest.mark.parametrize("path", [rk.PATH_TENSOR_CORE, rk.PATH_SIMT])
def test_config2_adaptive_window(handle, path):
    _adaptive_check(handle, make_inputs(CONFIGS["cfg2"]), path)


@pytest.mark.parametrize("tail", [0, 32])
def test_config2_adaptive_window_evict_on_the_tensor_core_kernel(handle, tail):
    _adaptive_check(handle, make_inputs(CONFIGS["cfg2"].with_(causal_tail=tail)), rk.PATH_TENSOR_CORE, evict=True)


def test_adaptive_window_at_full_size(handle):
    """The adaptive window at the long context's length: per-query top-B selections over 131072 tokens each (two KV
    heads of the long-context workload's shape; the oracle sorts every query's row, which sets the cost of this test)."""
    case = CONFIGS["cfg4"].with_(n_q_heads=8, n_kv_heads=2)
    keep = _adaptive_check(handle, make_inputs(case), rk.PATH_TENSOR_CORE, evict=True)
    assert keep.sum() >= 1


def test_config2_is_deterministic(handle):
    run = DeviceRun(handle, make_inputs(CONFIGS["cfg2"]))
    a = run.evict()
    b = run.evict()
    for x, y in zip(a, b):
        np.testing.assert_array_equal(x, y)


@pytest.mark.parametrize("spec", [("cfg2", 0, 1024, 7, 0), ("cfg2", 32, 1024, 21, 0), ("cfg2", 0, 37, 1, 0), ("cfg2", 0, 1024, 5, -9),
                                  ("cfg3", 0, 2048, 7, 0), ("cfg3", 0, 16000, 31, 4)])
def test_selection_inside_the_score_kernel_equals_the_separate_kernel(handle, spec):
    """restkv_evict on the tensor-core path pools, selects and gathers inside the score kernel by default; with that
    switched off the separate kernel does: scores, indices and gathered rows must be identical bit for bit."""
    name, tail, budget, width, shift = spec
    inp = make_inputs(CONFIGS[name].with_(causal_tail=tail))
    run = DeviceRun(handle, inp, budget=budget)
    pool = run.pool(width=width, shift=shift)
    fused = [x.copy() for x in run.evict(pool=pool)]
    handle.set_fused_select(False)
    try:
        separate = run.evict(pool=pool)
    finally:
        handle.set_fused_select(True)
    for x, y in zip(fused, separate):
        np.testing.assert_array_equal(x, y)
    ref = oracle_scores(inp, width=width, shift=shift)
    assert_scores_close(fused[0], ref.scores, TOL["bf16"])
    assert_selection_valid(fused[1], ref.scores, budget, TOL["bf16"])


def test_selection_inside_the_score_kernel_with_ties(handle):
    """Identical keys (uniform attention) and only two distinct value rows, alternating: the scores of a head fall
    into two classes of exact ties, so the lower index must win ties exactly as in the separate kernel, also across
    the boundaries between the head's thread blocks."""
    case = Case("ties", 1, 4, 1, 128, 5000, 32, 777, 1, 0, 0.9, "bf16", 0, "normal", 3)
    inp = make_inputs(case)
    inp.K[...] = inp.K[:, :, :1]
    va, vb = inp.V[:, :, 0:1].copy(), inp.V[:, :, 1:2].copy()
    inp.V[:, :, 0::2] = va
    inp.V[:, :, 1::2] = vb
    run = DeviceRun(handle, inp)
    fused = [x.copy() for x in run.evict()]
    handle.set_fused_select(False)
    try:
        separate = run.evict()
    finally:
        handle.set_fused_select(True)
    for x, y in zip(fused, separate):
        np.testing.assert_array_equal(x, y)
    ref = oracle_scores(inp)
    assert_selection_valid(fused[1], ref.scores, case.budget, TOL["bf16"])


# ------------------------------------------------------------------ config 3 (32 layers, drifting keys)
@pytest.mark.parametrize("layer", list(range(32)))
def test_config3_layer(handle, layer):
    case = CONFIGS["cfg3"].with_(seed=3000 + layer)
    inp = make_inputs(case)
    run = DeviceRun(handle, inp)
    scores, idx, K_out, V_out = run.evict()
    ref = oracle_scores(inp)                      # all eight heads of the layer
    assert_scores_close(scores, ref.scores, TOL["bf16"])
    assert_selection_valid(idx, ref.scores, case.budget, TOL["bf16"])
    _, kbits, vbits = inp.device_arrays()
    assert_compaction_exact(idx, kbits, K_out)
    assert_compaction_exact(idx, vbits, V_out)


def test_config3_wide_pooling_changes_the_selection(handle):
    inp = make_inputs(CONFIGS["cfg3"])
    run = DeviceRun(handle, inp)
    _, idx7, _, _ = run.evict()
    idx7 = idx7.copy()
    scores, idx31, _, _ = run.evict(pool=run.pool(width=31))
    ref = oracle_scores(inp, width=31)
    assert_scores_close(scores, ref.scores, TOL["bf16"])
    assert_selection_valid(idx31, ref.scores, inp.case.budget, TOL["bf16"])
    assert not np.array_equal(idx7, idx31)


# ------------------------------------------------------------------ config 4 (128k, the timed headline)
def test_config4_full_size(handle):
    inp = make_inputs(CONFIGS["cfg4"])
    worst, exact = full_check(handle, inp)
    print("cfg4: worst rel err %.2e, heads with identical index sets %.2f" % (worst, exact))


def test_config4_is_deterministic(handle):
    run = DeviceRun(handle, make_inputs(CONFIGS["cfg4"]))
    a = run.evict()
    b = run.evict()
    for x, y in zip(a, b):
        np.testing.assert_array_equal(x, y)


# ------------------------------------------------------------------ config 5 (batched sweep)
@pytest.fixture(scope="module")
def cfg5_inputs():
    return make_inputs(CONFIGS["cfg5"])


@pytest.mark.parametrize("decay", [0.5, 0.9, 0.99])
@pytest.mark.parametrize("width", [1, 7, 31])
def test_config5_sweep(handle, cfg5_inputs, decay, width):
    inp = cfg5_inputs
    ref = oracle_scores(inp, ema_decay=decay, width=width).scores     # all 64 (batch, KV head) rows
    _, kbits, vbits = inp.device_arrays()
    for budget in (128, 512, 2048):
        run = DeviceRun(handle, inp, budget=budget)
        scores, idx, K_out, V_out = run.evict(pool=run.pool(width=width), ema_decay=decay)
        assert_scores_close(scores, ref, TOL["bf16"])
        assert_selection_valid(idx, ref, budget, TOL["bf16"])
        assert_compaction_exact(idx, kbits, K_out)
        assert_compaction_exact(idx, vbits, V_out)
        del run


def test_config5_is_deterministic(handle, cfg5_inputs):
    run = DeviceRun(handle, cfg5_inputs)
    a = run.evict()
    b = run.evict()
    for x, y in zip(a, b):
        np.testing.assert_array_equal(x, y)


# ------------------------------------------------------------------ edge cases
EDGE = [
    # name, Hq, Hkv, d, n, w, budget, width, dtype, tail
    ("one_row", 4, 1, 128, 1, 32, 1, 1, "bf16", 0),
    ("five_rows", 4, 1, 128, 5, 32, 3, 3, "bf16", 0),
    ("tile_minus_one", 4, 1, 128, 127, 32, 17, 7, "bf16", 0),
    ("tile_exact", 4, 1, 128, 128, 32, 128, 7, "bf16", 0),
    ("tile_plus_one", 8, 2, 128, 129, 32, 1, 7, "bf16", 0),
    ("ragged", 8, 2, 128, 1000, 32, 100, 5, "bf16", 0),
    ("ragged_tail", 8, 2, 128, 4097, 32, 640, 21, "bf16", 32),
    ("budget_over_n", 4, 1, 128, 300, 32, 1000, 7, "bf16", 0),
    ("w1", 4, 1, 128, 200, 1, 20, 3, "bf16", 0),
    ("w7_tail", 4, 2, 64, 333, 7, 40, 5, "bf16", 7),
    ("mha", 2, 2, 64, 500, 32, 64, 7, "f32", 0),
    ("g2_d32", 4, 2, 32, 257, 16, 33, 7, "f32", 16),
    ("d256", 2, 1, 256, 130, 8, 13, 3, "bf16", 0),
    ("g8", 8, 1, 128, 700, 16, 70, 7, "bf16", 0),
]


@pytest.mark.parametrize("spec", EDGE, ids=[e[0] for e in EDGE])
def test_edge_cases(handle, spec):
    name, Hq, Hkv, d, n, w, budget, width, dtype, tail = spec
    case = Case(name, 2, Hq, Hkv, d, n, w, budget, width, 0, 0.7, dtype, tail, "normal", 77)
    full_check(handle, make_inputs(case))


def test_more_heads_than_sms(handle):
    """160 (batch, KV head) pairs: the persistent score kernel runs one CTA per head and two rounds."""
    case = Case("many_heads", 20, 32, 8, 128, 300, 32, 30, 5, 0, 0.8, "bf16", 0, "normal", 33)
    inp = make_inputs(case)
    run = DeviceRun(handle, inp)
    scores, idx, K_out, V_out = run.evict()
    ref = oracle_scores(inp).scores            # all 160 heads
    assert_scores_close(scores, ref, TOL["bf16"])
    assert_selection_valid(idx, ref, case.budget, TOL["bf16"])
    _, kbits, vbits = inp.device_arrays()
    assert_compaction_exact(idx, kbits, K_out)
    assert_compaction_exact(idx, vbits, V_out)


@pytest.mark.parametrize("decay", [0.0, 1.0])
def test_ema_extremes(handle, decay):
    case = Case("ema", 1, 8, 2, 128, 600, 16, 50, 1, 0, decay, "bf16", 0, "normal", 5)
    full_check(handle, make_inputs(case))


def test_pool_shift(handle):
    case = Case("shift", 1, 8, 2, 64, 400, 32, 50, 5, 0, 0.9, "f32", 0, "normal", 6)
    inp = make_inputs(case)
    for shift in (-3, 2, 40):
        full_check(handle, inp, shift=shift)


def test_strided_kv_layout(handle):
    """K and V stored as [batch, n_kv, Hkv, d] (token-major), addressed through the strides."""
    import torch
    case = Case("strided", 2, 8, 2, 128, 900, 32, 90, 7, 0, 0.9, "bf16", 0, "normal", 8)
    inp = make_inputs(case)
    q, k, v = inp.device_arrays()
    Q = torch_dev(q, "bf16")
    Kt = torch_dev(np.ascontiguousarray(k.transpose(0, 2, 1, 3)), "bf16")   # [b, n, H, d]
    Vt = torch_dev(np.ascontiguousarray(v.transpose(0, 2, 1, 3)), "bf16")
    H, n, d = case.n_kv_heads, case.n_kv, case.head_dim
    strides = (n * H * d, d, H * d)
    shape = shape_of(case, k_strides=strides, v_strides=strides)
    ref_run = DeviceRun(handle, inp)
    s_ref, i_ref, k_ref, v_ref = ref_run.evict()
    run = DeviceRun(handle, inp)
    handle.evict(shape, Q, Kt, Vt, case.ema_decay, run.pool(), case.budget, run.indices, run.K_out, run.V_out, run.ws,
                 scores_out=run.scores)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(run.scores.cpu().numpy(), s_ref)
    np.testing.assert_array_equal(run.indices.cpu().numpy(), i_ref)
    np.testing.assert_array_equal(run.K_out.view(torch.int16).cpu().numpy(), k_ref)
    np.testing.assert_array_equal(run.V_out.view(torch.int16).cpu().numpy(), v_ref)


def test_evict_host_matches_oracle(handle):
    """The host-buffer entry point (the one the end-to-end number is measured through): pinned host tensors in,
    pinned host tensors out, copies enqueued by the library."""
    import torch
    case = CONFIGS["cfg2"]
    inp = make_inputs(case)
    run = DeviceRun(handle, inp)
    q, k, v = inp.device_arrays()
    hQ, hK, hV = (torch.from_numpy(np.ascontiguousarray(a)).pin_memory() for a in (q, k, v))
    dQ, dK, dV = (torch.empty_like(t, device="cuda") for t in (hQ, hK, hV))     # staging, filled by the call
    keep = run.keep
    h_idx = torch.full((case.batch, case.n_kv_heads, keep), -1, dtype=torch.int32).pin_memory()
    h_Ko = torch.zeros((case.batch, case.n_kv_heads, keep, case.head_dim), dtype=torch.int16).pin_memory()
    h_Vo = torch.zeros_like(h_Ko).pin_memory()
    handle.evict_host(run.shape, hQ, hK, hV, case.ema_decay, run.pool(), case.budget, h_idx, h_Ko, h_Vo, dQ, dK, dV,
                      run.indices, run.K_out, run.V_out, run.ws)
    torch.cuda.synchronize()
    assert handle.poll_status() == rk.RESTKV_OK
    ref = oracle_scores(inp)
    idx = h_idx.numpy()
    assert_selection_valid(idx, ref.scores, case.budget, TOL["bf16"])
    assert_compaction_exact(idx, k, h_Ko.numpy())
    assert_compaction_exact(idx, v, h_Vo.numpy())
    # arguments are checked before the first copy is enqueued
    dQ.zero_()
    with pytest.raises(rk.RestKVError) as err:
        handle.evict_host(run.shape, hQ, hK, hV, case.ema_decay, rk.fixed_pool(4), case.budget, h_idx, h_Ko, h_Vo, dQ,
                          dK, dV, run.indices, run.K_out, run.V_out, run.ws)
    assert err.value.status == rk.ERR_INVALID_ARG
    torch.cuda.synchronize()
    assert int(dQ.view(torch.int16).abs().max()) == 0


# ------------------------------------------------------------------ unit: select, compact, decode
def test_select_matches_stable_sort_with_ties_and_inf(handle):
    import torch
    rng = np.random.default_rng(3)
    n_kv = 5000
    s = rng.standard_normal((2, 3, n_kv)).astype(np.float32)
    s[0, 0, ::7] = 0.25                       # many ties
    s[0, 1] = 1.0                             # all equal
    s[1, 0, -40:] = np.inf
    s[1, 1] = np.abs(s[1, 1]) * 1e-30         # tiny positives
    s[1, 2, 100:200] = -s[1, 2, 100:200] - 5  # negatives
    case = Case("sel", 2, 3, 3, 64, n_kv, 32)
    shape = shape_of(case)
    d_s = torch.from_numpy(s).cuda()
    for B in (1, 2, 31, 32, 33, 1000, 4999, 5000, 9000):
        keep = min(B, n_kv)
        idx = torch.empty((2, 3, keep), dtype=torch.int32, device="cuda")
        ws = torch.empty(handle.workspace_bytes(shape, B), dtype=torch.uint8, device="cuda")
        handle.select(shape, d_s, B, idx, ws)
        torch.cuda.synchronize()
        got = idx.cpu().numpy()
        np.testing.assert_array_equal(got, oracle.select(s.astype(np.float64), B))


def test_compact_bit_exact_and_bad_index_reported(handle):
    import torch
    case = Case("cmp", 2, 4, 2, 64, 300, 8, dtype="f32")
    shape = shape_of(case)
    rng = np.random.default_rng(4)
    K = rng.standard_normal((2, 2, 300, 64)).astype(np.float32)
    V = rng.standard_normal((2, 2, 300, 64)).astype(np.float32)
    idx = np.sort(rng.choice(300, size=(2, 2, 37)), axis=-1).astype(np.int32)
    dK, dV, dI = torch.from_numpy(K).cuda(), torch.from_numpy(V).cuda(), torch.from_numpy(idx).cuda()
    Ko = torch.zeros((2, 2, 37, 64), device="cuda")
    Vo = torch.zeros_like(Ko)
    handle.compact(shape, dK, dV, dI, 37, Ko, Vo)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(Ko.cpu().numpy(), oracle.compact(K, idx))
    np.testing.assert_array_equal(Vo.cpu().numpy(), oracle.compact(V, idx))
    assert handle.poll_status() == rk.RESTKV_OK
    bad = idx.copy()
    bad[1, 1, 5] = 300                       # out of range: skipped and reported, never dereferenced
    handle.compact(shape, dK, dV, torch.from_numpy(bad).cuda(), 37, Ko, Vo)
    assert handle.poll_status() == rk.ERR_INVALID_ARG
    assert handle.poll_status() == rk.RESTKV_OK     # sticky word is cleared by the poll


@pytest.mark.parametrize("spec", [("bf16", 32, 8, 128, 2048), ("bf16", 32, 8, 128, 131072), ("f32", 8, 2, 64, 777),
                                  ("bf16", 4, 4, 64, 100), ("bf16", 16, 2, 256, 1500), ("bf16", 16, 1, 128, 1000),
                                  ("bf16", 3, 3, 128, 129), ("bf16", 8, 8, 128, 2)])
def test_decode_matches_oracle(handle, spec):
    import torch
    dtype, Hq, Hkv, d, rows = spec
    rng = np.random.default_rng(11)
    b = 1 if rows > 10000 else 2

    def draw(shape):
        x = rng.standard_normal(shape).astype(np.float32)
        if dtype == "bf16":
            bits = round_to_bf16_bits(x)
            return (bits.astype(np.uint32) << 16).view(np.float32), bits.view(np.int16)
        return x, x

    q, qd = draw((b, Hq, d))
    K, Kd = draw((b, Hkv, rows, d))
    V, Vd = draw((b, Hkv, rows, d))
    ref, ref_lse = oracle.decode(q, K, V)
    case = Case("dec", b, Hq, Hkv, d, rows, 1, dtype=dtype)
    shape = shape_of(case)
    out = torch.empty((b, Hq, d), dtype=torch.float32, device="cuda")
    lse = torch.empty((b, Hq), dtype=torch.float32, device="cuda")
    ws = torch.empty(handle.workspace_bytes(shape, 0), dtype=torch.uint8, device="cuda")
    handle.decode(shape, torch_dev(qd, dtype), torch_dev(Kd, dtype), torch_dev(Vd, dtype), rows, out, ws, lse=lse)
    torch.cuda.synchronize()
    assert_decode_close(out.cpu().numpy(), ref, q, K, V, dtype)
    np.testing.assert_allclose(lse.cpu().numpy(), ref_lse, rtol=1e-5, atol=1e-5)


def test_decode_over_compacted_cache_of_config2(handle):
    import torch
    inp = make_inputs(CONFIGS["cfg2"])
    run = DeviceRun(handle, inp)
    _, idx, K_out, V_out = run.evict()
    q = make_decode_query(inp)
    qd = round_to_bf16_bits(q).view(np.int16)
    c = inp.case
    out = torch.empty((c.batch, c.n_q_heads, c.head_dim), dtype=torch.float32, device="cuda")
    handle.decode(run.shape, torch_dev(qd, "bf16"), run.K_out, run.V_out, run.keep, out, run.ws)
    torch.cuda.synchronize()
    Kc = np.take_along_axis(inp.K, idx[..., None].astype(np.int64), axis=2)
    Vc = np.take_along_axis(inp.V, idx[..., None].astype(np.int64), axis=2)
    ref, _ = oracle.decode(q, Kc, Vc)
    assert_decode_close(out.cpu().numpy(), ref, q, Kc, Vc, "bf16")


# ------------------------------------------------------------------ scores from given window outputs and normalisers
def _window_stats(inp, with_A_check=True):
    """(O float32 [b,Hq,w,d], LSE float32 [b,Hq,w]) of the window rows: O is the oracle's own; the log-sum-exp of the
    scaled logits over the visible rows comes from SciPy on the same inputs and is tied to the oracle's softmax
    weights (A = exp(s - LSE)) before it is used."""
    from scipy.special import logsumexp
    c = inp.case
    ref = oracle_scores(inp, want_O=True, want_A=with_A_check)
    G, w, n, n_kv = c.group, c.w, c.n, c.n_kv
    scale = 1.0 / np.sqrt(c.head_dim)
    lse = np.empty((c.batch, c.n_q_heads, w), np.float64)
    for b in range(c.batch):
        for h in range(c.n_kv_heads):
            q = inp.Q[b, h * G:(h + 1) * G].astype(np.float64).reshape(G * w, -1)
            s = scale * (q @ inp.K[b, h].astype(np.float64).T)                      # [G*w, n_kv]
            if c.causal_tail:
                i = np.tile(np.arange(w), G)[:, None]
                s[:, n:] = np.where(np.arange(n_kv - n)[None, :] <= i, s[:, n:], -np.inf)
            l = logsumexp(s, axis=-1)
            lse[b, h * G:(h + 1) * G] = l.reshape(G, w)
            if with_A_check:
                A = ref.A[b, h * G:(h + 1) * G].reshape(G * w, n_kv)
                np.testing.assert_allclose(np.exp(s[:, :64] - l[:, None]), A[:, :64], rtol=1e-9, atol=1e-300)
    return ref, ref.O.astype(np.float32), lse.astype(np.float32)


@pytest.mark.parametrize("spec", [("cfg1b", "f32", 0), ("cfg1b", "bf16", 32), ("cfg2", "bf16", 0), ("cfg2", "bf16", 32)])
def test_score_from_lse_matches_oracle(handle, spec):
    """restkv_score_from_lse: the window rows' outputs and log-sum-exps are given (as after prompt prefilling), the
    scores must be the oracle's."""
    import torch
    name, dtype, tail = spec
    inp = make_inputs(CONFIGS[name].with_(dtype=dtype, causal_tail=tail))
    ref, O, lse = _window_stats(inp)
    run = DeviceRun(handle, inp)
    handle.score_from_lse(run.shape, run.Q, run.K, run.V, torch.from_numpy(O).cuda(), torch.from_numpy(lse).cuda(),
                          inp.case.ema_decay, run.pool(), run.scores, run.ws)
    torch.cuda.synchronize()
    assert handle.poll_status() == rk.RESTKV_OK
    assert_scores_close(run.scores.cpu().numpy(), ref.scores, TOL[dtype])


@pytest.mark.parametrize("spec", [("cfg2", 0), ("cfg2", 32), ("cfg1b", 0)])
def test_evict_from_lse_matches_oracle(handle, spec):
    """restkv_evict_from_lse: score, select and compact from given window statistics, all three acceptance rules."""
    import torch
    name, tail = spec
    inp = make_inputs(CONFIGS[name].with_(causal_tail=tail))
    c = inp.case
    ref, O, lse = _window_stats(inp, with_A_check=False)
    run = DeviceRun(handle, inp)
    handle.evict_from_lse(run.shape, run.Q, run.K, run.V, torch.from_numpy(O).cuda(), torch.from_numpy(lse).cuda(),
                          c.ema_decay, run.pool(), run.budget, run.indices, run.K_out, run.V_out, run.ws,
                          scores_out=run.scores)
    torch.cuda.synchronize()
    assert handle.poll_status() == rk.RESTKV_OK
    idx = run.indices.cpu().numpy()
    assert_scores_close(run.scores.cpu().numpy(), ref.scores, TOL[c.dtype])
    assert_selection_valid(idx, ref.scores, run.budget, TOL[c.dtype])
    _, kbits, vbits = inp.device_arrays()
    assert_compaction_exact(idx, kbits, run._bits(run.K_out))
    assert_compaction_exact(idx, vbits, run._bits(run.V_out))


def test_score_from_lse_at_full_size(handle):
    import torch
    inp = make_inputs(CONFIGS["cfg4"])
    ref, O, lse = _window_stats(inp, with_A_check=False)
    run = DeviceRun(handle, inp)
    dO, dL = torch.from_numpy(O).cuda(), torch.from_numpy(lse).cuda()
    handle.score_from_lse(run.shape, run.Q, run.K, run.V, dO, dL, inp.case.ema_decay, run.pool(), run.scores, run.ws)
    torch.cuda.synchronize()
    assert handle.poll_status() == rk.RESTKV_OK
    assert_scores_close(run.scores.cpu().numpy(), ref.scores, TOL["bf16"])
    run.scores.zero_()
    handle.evict_from_lse(run.shape, run.Q, run.K, run.V, dO, dL, inp.case.ema_decay, run.pool(), run.budget,
                          run.indices, run.K_out, run.V_out, run.ws, scores_out=run.scores)
    torch.cuda.synchronize()
    assert handle.poll_status() == rk.RESTKV_OK
    idx = run.indices.cpu().numpy()
    assert_scores_close(run.scores.cpu().numpy(), ref.scores, TOL["bf16"])
    assert_selection_valid(idx, ref.scores, run.budget, TOL["bf16"])
    _, kbits, vbits = inp.device_arrays()
    assert_compaction_exact(idx, kbits, run._bits(run.K_out))
    assert_compaction_exact(idx, vbits, run._bits(run.V_out))


# ------------------------------------------------------------------ ablation variants (Appendix G)
REC, ATT, ATTV = rk.INDICATOR_RECONSTRUCTION, rk.INDICATOR_ATTENTION, rk.INDICATOR_ATTENTION_VNORM
EMA, MEAN, INV, NONE = rk.TEMPORAL_EMA, rk.TEMPORAL_MEAN, rk.TEMPORAL_INV_EMA, rk.TEMPORAL_NONE
VARIANTS = [
    # (indicator, temporal, spatial, group)
    (ATT, MEAN, rk.SPATIAL_MEAN, rk.GROUP_MEAN),     # window mean of the attention weights, pooled
    (ATTV, EMA, rk.SPATIAL_MEAN, rk.GROUP_MEAN),
    (REC, INV, rk.SPATIAL_MEAN, rk.GROUP_MEAN),
    (REC, NONE, rk.SPATIAL_MAX, rk.GROUP_MEAN),
    (REC, MEAN, rk.SPATIAL_MEAN, rk.GROUP_MAX),
    (ATT, INV, rk.SPATIAL_MAX, rk.GROUP_MAX),
    (ATTV, NONE, rk.SPATIAL_MEAN, rk.GROUP_MAX),
    (REC, EMA, rk.SPATIAL_MAX, rk.GROUP_MAX),
]


def variant_check(handle, inp, variant, path=rk.PATH_AUTO, from_lse=False, ema_decay=None, budget=None, fused=None):
    """evict (or evict_from_lse) under a variant against the oracle run with the same modes: all three rules."""
    import torch
    ind, tmp, spa, grp = variant
    c = inp.case
    decay = c.ema_decay if ema_decay is None else ema_decay
    handle.set_kernel_path(path)
    handle.set_variant(ind, tmp, spa, grp)
    try:
        run = DeviceRun(handle, inp, budget=budget)
        if from_lse:
            _, O, lse = _window_stats(inp, with_A_check=False)
            handle.evict_from_lse(run.shape, run.Q, run.K, run.V, torch.from_numpy(O).cuda(),
                                  torch.from_numpy(lse).cuda(), decay, run.pool(), run.budget, run.indices,
                                  run.K_out, run.V_out, run.ws, scores_out=run.scores)
        else:
            handle.evict(run.shape, run.Q, run.K, run.V, decay, run.pool(), run.budget, run.indices, run.K_out,
                         run.V_out, run.ws, scores_out=run.scores)
        torch.cuda.synchronize()
        assert handle.poll_status() == rk.RESTKV_OK
        if fused is not None:
            assert handle.last_evict_fused_select() == fused
    finally:
        handle.set_kernel_path(rk.PATH_AUTO)
        handle.set_variant()
    ref = oracle_scores(inp, ema_decay=decay, indicator_mode=ind, temporal_mode=tmp, spatial_mode=spa, group_mode=grp)
    tol = TOL[c.dtype]
    idx = run.indices.cpu().numpy()
    assert_scores_close(run.scores.cpu().numpy(), ref.scores, tol)
    assert_selection_valid(idx, ref.scores, run.budget, tol)
    _, kbits, vbits = inp.device_arrays()
    assert_compaction_exact(idx, kbits, run._bits(run.K_out))
    assert_compaction_exact(idx, vbits, run._bits(run.V_out))
    return ref


@pytest.mark.parametrize("variant", VARIANTS)
@pytest.mark.parametrize("spec", [("cfg1b", "f32", 0), ("cfg1b", "bf16", 32)])
def test_variants_on_the_simt_kernels(handle, variant, spec):
    name, dtype, tail = spec
    variant_check(handle, make_inputs(CONFIGS[name].with_(dtype=dtype, causal_tail=tail)), variant)


@pytest.mark.parametrize("variant", VARIANTS)
@pytest.mark.parametrize("tail", [0, 32])
def test_variants_on_the_tensor_core_kernel(handle, variant, tail):
    # cfg2 qualifies for the selection inside the score kernel, so its max-pooling is covered here too
    inp = make_inputs(CONFIGS["cfg2"].with_(causal_tail=tail))
    ref = variant_check(handle, inp, variant, path=rk.PATH_TENSOR_CORE, fused=True)
    # the variant must have changed the scores, or the test compares the default with itself
    base = oracle_scores(inp).scores
    fin = np.isfinite(base)
    assert not np.allclose(ref.scores[fin], base[fin], rtol=1e-3)


@pytest.mark.parametrize("variant", VARIANTS)
def test_variants_from_given_window_statistics(handle, variant):
    variant_check(handle, make_inputs(CONFIGS["cfg2"]), variant, path=rk.PATH_TENSOR_CORE, from_lse=True)


@pytest.mark.parametrize("variant", [VARIANTS[0], VARIANTS[4], VARIANTS[5]])
def test_variants_with_the_selection_as_its_own_kernel(handle, variant):
    handle.set_fused_select(False)
    try:
        variant_check(handle, make_inputs(CONFIGS["cfg2"]), variant, path=rk.PATH_TENSOR_CORE, fused=False)
    finally:
        handle.set_fused_select(True)


@pytest.mark.parametrize("variant", [VARIANTS[2], VARIANTS[4], VARIANTS[5], VARIANTS[7]])
@pytest.mark.parametrize("spec", [(16, 2, 16), (4, 2, 64), (2, 2, 128), (8, 1, 16)])
def test_variants_at_other_window_lengths(handle, variant, spec):
    """The group reduction and the temporal chain of the tensor-core kernel are laid out differently for each window
    length (a 32-column slice is two windows, one, half of one or a quarter)."""
    Hq, Hkv, w = spec
    case = Case("variant_w%d" % w, 2, Hq, Hkv, 128, 3000, w, 200, 5, 0, 0.9, "bf16", 0, "normal", 55)
    variant_check(handle, make_inputs(case), variant, path=rk.PATH_TENSOR_CORE)


@pytest.mark.parametrize("decay,expect_tc", [(0.9, True), (0.5, True), (0.2, False), (0.0, False), (1.0, False)])
def test_inverted_ema_leaves_the_tensor_core_kernel_when_its_chain_would_overflow(handle, decay, expect_tc):
    inp = make_inputs(CONFIGS["cfg2"])
    variant = (REC, INV, rk.SPATIAL_MEAN, rk.GROUP_MEAN)
    variant_check(handle, inp, variant, ema_decay=decay)            # automatic choice: always served
    if not expect_tc:
        handle.set_kernel_path(rk.PATH_TENSOR_CORE)
        handle.set_variant(*variant)
        try:
            run = DeviceRun(handle, inp)
            with pytest.raises(rk.RestKVError) as e:
                handle.evict(run.shape, run.Q, run.K, run.V, decay, run.pool(), run.budget, run.indices, run.K_out,
                             run.V_out, run.ws)
            assert e.value.status == rk.ERR_UNSUPPORTED
        finally:
            handle.set_kernel_path(rk.PATH_AUTO)
            handle.set_variant()
    else:
        variant_check(handle, inp, variant, path=rk.PATH_TENSOR_CORE, ema_decay=decay)


@pytest.mark.parametrize("variant", [VARIANTS[0], VARIANTS[5], VARIANTS[1]])
def test_variants_with_the_adaptive_window(handle, variant):
    ind, tmp, spa, grp = variant
    inp = make_inputs(CONFIGS["cfg1b"])
    c = inp.case
    B = c.budget
    modes = dict(indicator_mode=ind, temporal_mode=tmp, spatial_mode=spa, group_mode=grp)
    probe = oracle_scores(inp, pool_mode=1, beta=1e9, base_width=1, budget=B, **modes)
    delta = abs(probe.D[..., 0] - probe.D[..., 1]).min()
    assert delta > 0
    compared = 0
    for target, base in ((0.5, 3), (1.5, 1), (2.5, 3)):
        beta = float(delta / target)
        ref = oracle_scores(inp, pool_mode=1, beta=beta, base_width=base, budget=B, **modes)
        x = (ref.D[..., 0] - ref.D[..., 1]) / beta
        if np.any(np.abs(x - np.round(x)) < 0.05):
            continue   # too close to a rounding boundary for an fp32-vs-fp64 ranking comparison
        handle.set_variant(ind, tmp, spa, grp)
        try:
            run = DeviceRun(handle, inp, adaptive_budget=B)
            scores = run.score(pool=rk.adaptive_pool(beta, base, B))
        finally:
            handle.set_variant()
        np.testing.assert_array_equal(run.pool_used.cpu().numpy(), ref.pool)
        assert_scores_close(scores, ref.scores, TOL[c.dtype])
        compared += 1
    assert compared > 0, "every beta landed on a rounding boundary: nothing was compared"


def test_variants_score_a_single_row_cache(handle):
    # Eq. 7 is 0/0 on a cache of one row (defined as 0); the attention-weight indicators are 1 and ||v|| there
    case = Case("one_row", 1, 4, 2, 64, 1, 4, 1, 1, 0, 0.7, "f32", 0, "normal", 5)
    inp = make_inputs(case)
    for ind, expect in ((REC, None), (ATT, 1.0), (ATTV, None)):
        handle.set_variant(ind)
        try:
            got = DeviceRun(handle, inp).score()
        finally:
            handle.set_variant()
        ref = oracle.score(inp.Q, inp.K, inp.V, ema_decay=case.ema_decay, width=1, indicator_mode=ind).scores
        np.testing.assert_allclose(got, ref, rtol=1e-6, atol=0)
        if expect is not None:
            np.testing.assert_allclose(got, expect, rtol=1e-6)
    assert np.all(oracle.score(inp.Q, inp.K, inp.V, width=1).scores == 0.0)


def test_variant_at_full_size(handle):
    """The long-context workload under two variants, in the launch configuration the benchmark times."""
    inp = make_inputs(CONFIGS["cfg4"])
    variant_check(handle, inp, VARIANTS[0], fused=True)
    variant_check(handle, inp, VARIANTS[5], fused=True)


def test_set_variant_validates_its_fields(handle):
    for bad in ((3, 0, 0, 0), (0, 4, 0, 0), (0, 0, 2, 0), (0, 0, 0, 2), (-1, 0, 0, 0)):
        with pytest.raises(rk.RestKVError) as e:
            handle.set_variant(*bad)
        assert e.value.status == rk.ERR_INVALID_ARG
    handle.set_variant()


# ------------------------------------------------------------------ a budget of its own per head (Appendix C)
def _budgets_check(handle, inp, budgets, max_budget, pool=None, oracle_kw=None):
    import torch
    c = inp.case
    run = DeviceRun(handle, inp, budget=max_budget)
    S = run.keep                                           # min(max_budget, n_kv)
    dB = torch.from_numpy(np.ascontiguousarray(budgets, dtype=np.int32)).cuda()
    sentinel = 0x7B7B if c.dtype == "bf16" else None
    if c.dtype == "bf16":
        run.K_out.view(torch.int16).fill_(sentinel)
        run.V_out.view(torch.int16).fill_(sentinel)
    else:
        run.K_out.fill_(-777.0)
        run.V_out.fill_(-777.0)
    run.indices.fill_(-5)
    handle.evict_budgets(run.shape, run.Q, run.K, run.V, c.ema_decay, pool or run.pool(), dB, max_budget, run.indices,
                         run.K_out, run.V_out, run.ws, scores_out=run.scores)
    torch.cuda.synchronize()
    assert handle.poll_status() == rk.RESTKV_OK
    assert not handle.last_evict_fused_select()
    ref = oracle_scores(inp, **(oracle_kw or {}))
    tol = TOL[c.dtype]
    scores, idx = run.scores.cpu().numpy(), run.indices.cpu().numpy()
    K_out, V_out = run._bits(run.K_out), run._bits(run.V_out)
    _, kbits, vbits = inp.device_arrays()
    assert_scores_close(scores, ref.scores, tol)
    for b in range(c.batch):
        for h in range(c.n_kv_heads):
            keep = min(max(int(budgets[b, h]), 1), S)
            assert_selection_valid(idx[b, h, :keep], ref.scores[b, h], keep, tol)
            assert np.all(idx[b, h, keep:] == -1)
            assert np.array_equal(K_out[b, h, :keep], kbits[b, h][idx[b, h, :keep]])
            assert np.array_equal(V_out[b, h, :keep], vbits[b, h][idx[b, h, :keep]])
            untouched = sentinel if c.dtype == "bf16" else np.float32(-777.0)
            assert np.all(K_out[b, h, keep:] == untouched) and np.all(V_out[b, h, keep:] == untouched)


def test_budgets_per_head_on_workload_2(handle):
    inp = make_inputs(CONFIGS["cfg2"])
    budgets = np.array([[1024, 1, 700, 0, 5000, 333, 64, 1023]], np.int32)    # 0 counts as 1, 5000 as max_budget
    _budgets_check(handle, inp, budgets, 1024)


def test_budgets_per_head_small_fp32_with_causal_tail(handle):
    inp = make_inputs(CONFIGS["cfg1b"].with_(causal_tail=32))
    _budgets_check(handle, inp, np.array([[40, 200]], np.int32), 256)
    # a stride beyond the cache: every row can be kept
    _budgets_check(handle, inp, np.array([[5000, 33]], np.int32), 4096)


def test_budgets_per_head_with_more_heads_than_sms(handle):
    case = Case("many_heads_budgets", 20, 32, 8, 128, 300, 32, 30, 5, 0, 0.8, "bf16", 0, "normal", 34)
    rng = np.random.default_rng(5)
    _budgets_check(handle, make_inputs(case), rng.integers(1, 61, size=(20, 8)).astype(np.int32), 48)


def test_budgets_per_head_with_the_adaptive_window(handle):
    inp = make_inputs(CONFIGS["cfg1b"])
    B = inp.case.budget
    probe = oracle_scores(inp, pool_mode=1, beta=1e9, base_width=1, budget=B)
    beta = float(abs(probe.D[..., 0] - probe.D[..., 1]).min() / 1.5)
    kw = dict(pool_mode=1, beta=beta, base_width=3, budget=B)
    x = (probe.D[..., 0] - probe.D[..., 1]) / beta
    if np.any(np.abs(x - np.round(x)) < 0.05):
        pytest.skip("a head sits on a rounding boundary of Eq. 11")
    import torch
    c = inp.case
    run = DeviceRun(handle, inp, budget=B, adaptive_budget=B)
    dB = torch.tensor([[100, 17]], dtype=torch.int32, device="cuda")
    handle.evict_budgets(run.shape, run.Q, run.K, run.V, c.ema_decay, rk.adaptive_pool(beta, 3, B), dB, B, run.indices,
                         run.K_out, run.V_out, run.ws, scores_out=run.scores)
    torch.cuda.synchronize()
    assert handle.poll_status() == rk.RESTKV_OK
    ref = oracle_scores(inp, **kw)
    idx = run.indices.cpu().numpy()
    assert_scores_close(run.scores.cpu().numpy(), ref.scores, TOL[c.dtype])
    for h, keep in enumerate((100, 17)):
        assert_selection_valid(idx[0, h, :keep], ref.scores[0, h], keep, TOL[c.dtype])
        assert np.all(idx[0, h, keep:] == -1)


# ------------------------------------------------------------------ eviction again while decoding (Appendix B)
@pytest.mark.parametrize("use_decode_statistics", [True, False])
def test_reeviction_after_m_generated_tokens(handle, use_decode_statistics):
    """Evict at prefill, decode M tokens over the compacted cache while appending their K/V, then evict again with the
    last w decode queries as the window.  With use_decode_statistics the second eviction reads the outputs and
    log-sum-exps that the decode calls themselves produced (restkv_evict_from_lse), as the paper suggests; otherwise
    it recomputes them (restkv_evict).  Both rounds are held against the oracle run on the same caches."""
    import torch
    from paper_2605_08840_b200.inputs import Inputs
    case = CONFIGS["cfg2"].with_(n=4096, budget=512)
    B, w, M = case.budget, case.w, 48
    tol = TOL["bf16"]
    inp = make_inputs(case)
    run = DeviceRun(handle, inp)
    scores1, idx1, _, _ = run.evict()
    ref1 = oracle_scores(inp)
    assert_scores_close(scores1, ref1.scores, tol)
    assert_selection_valid(idx1, ref1.scores, B, tol)
    take = idx1[..., None].astype(np.int64)
    fresh = make_inputs(case.with_(n=M, recipe="normal"), seed=case.seed + 17)
    K2 = np.ascontiguousarray(np.concatenate([np.take_along_axis(inp.K, take, axis=2), fresh.K], axis=2))
    V2 = np.ascontiguousarray(np.concatenate([np.take_along_axis(inp.V, take, axis=2), fresh.V], axis=2))
    queries = np.stack([make_decode_query(inp, seed=100 + t) for t in range(M)], axis=2)      # [b, Hq, M, d]
    # decode step t sees the compacted rows and the appended rows up to its own
    dK2, dV2 = (torch_dev(round_to_bf16_bits(a).view(np.int16), "bf16") for a in (K2, V2))
    outs = torch.empty((M, case.batch, case.n_q_heads, case.head_dim), dtype=torch.float32, device="cuda")
    lses = torch.empty((M, case.batch, case.n_q_heads), dtype=torch.float32, device="cuda")
    for t in range(M):
        rows = B + t + 1
        qd = torch_dev(round_to_bf16_bits(queries[:, :, t]).view(np.int16), "bf16")
        handle.decode(run.shape, qd, dK2[:, :, :rows].contiguous(), dV2[:, :, :rows].contiguous(), rows, outs[t],
                      run.ws, lse=lses[t])
    torch.cuda.synchronize()
    t_chk = M - 1
    ref_o, ref_l = oracle.decode(queries[:, :, t_chk], K2, V2)
    assert_decode_close(outs[t_chk].cpu().numpy(), ref_o, queries[:, :, t_chk], K2, V2, "bf16")
    np.testing.assert_allclose(lses[t_chk].cpu().numpy(), ref_l, rtol=0, atol=2e-3)
    # second eviction: the last w generated tokens are the window; their own rows are the cache's last w rows
    case2 = case.with_(name="reevict", n=B + M - w, causal_tail=w, recipe="normal")
    inp2 = Inputs(case2, np.ascontiguousarray(queries[:, :, M - w:]), K2, V2)
    run2 = DeviceRun(handle, inp2)
    if use_decode_statistics:
        O_obs = outs[M - w:].permute(1, 2, 0, 3).contiguous()          # [b, Hq, w, d]
        L_obs = lses[M - w:].permute(1, 2, 0).contiguous()             # [b, Hq, w]
        handle.evict_from_lse(run2.shape, run2.Q, run2.K, run2.V, O_obs, L_obs, case2.ema_decay, run2.pool(), B,
                              run2.indices, run2.K_out, run2.V_out, run2.ws, scores_out=run2.scores)
    else:
        handle.evict(run2.shape, run2.Q, run2.K, run2.V, case2.ema_decay, run2.pool(), B, run2.indices, run2.K_out,
                     run2.V_out, run2.ws, scores_out=run2.scores)
    torch.cuda.synchronize()
    assert handle.poll_status() == rk.RESTKV_OK
    ref2 = oracle_scores(inp2)
    idx2 = run2.indices.cpu().numpy()
    assert_scores_close(run2.scores.cpu().numpy(), ref2.scores, tol)
    assert_selection_valid(idx2, ref2.scores, B, tol)
    assert np.array_equal(idx2[..., -w:], np.broadcast_to(np.arange(B + M - w, B + M), idx2.shape[:2] + (w,)))
    _, kbits, vbits = inp2.device_arrays()
    assert_compaction_exact(idx2, kbits, run2._bits(run2.K_out))
    assert_compaction_exact(idx2, vbits, run2._bits(run2.V_out))


# ------------------------------------------------------------------ the output projection inside Eq. 7 (Eq. 4)
def _make_projection(handle, case, d_model, seed, scale=1.0):
    """(W float32 [Hq, d, d_model] holding dtype-exact values, factor buffer on the device)."""
    import torch
    from paper_2605_08840_b200.inputs import bf16_bits_to_f32
    rng = np.random.default_rng(seed)
    W = (rng.standard_normal((case.n_q_heads, case.head_dim, d_model)) * scale / np.sqrt(d_model)).astype(np.float32)
    if case.dtype == "bf16":
        bits = round_to_bf16_bits(W)
        W = bf16_bits_to_f32(bits)
        dW = torch_dev(bits.view(np.int16).reshape(-1, d_model), "bf16")
    else:
        dW = torch.from_numpy(W.reshape(-1, d_model)).cuda()
    nbytes = handle.output_projection_bytes(case.n_q_heads, case.head_dim)
    assert nbytes > 0
    factor = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    handle.prepare_output_projection(case.n_q_heads, case.head_dim, d_model, rk.BF16 if case.dtype == "bf16" else rk.F32,
                                     dW, factor)
    torch.cuda.synchronize()
    return W, factor


def projection_check(handle, inp, d_model, path=rk.PATH_AUTO, seed=1, from_lse=False, variant=None, fused=None):
    import torch
    c = inp.case
    W, factor = _make_projection(handle, c, d_model, seed)
    handle.set_kernel_path(path)
    handle.set_output_projection(factor, c.n_q_heads, c.head_dim)
    if variant:
        handle.set_variant(*variant)
    try:
        run = DeviceRun(handle, inp)
        if from_lse:
            _, O, lse = _window_stats(inp, with_A_check=False)
            handle.evict_from_lse(run.shape, run.Q, run.K, run.V, torch.from_numpy(O).cuda(),
                                  torch.from_numpy(lse).cuda(), c.ema_decay, run.pool(), run.budget, run.indices,
                                  run.K_out, run.V_out, run.ws, scores_out=run.scores)
            torch.cuda.synchronize()
            assert handle.poll_status() == rk.RESTKV_OK
            scores, idx = run.scores.cpu().numpy(), run.indices.cpu().numpy()
            K_out, V_out = run._bits(run.K_out), run._bits(run.V_out)
        else:
            scores, idx, K_out, V_out = run.evict()
        if fused is not None:
            assert handle.last_evict_fused_select() == fused
    finally:
        handle.set_kernel_path(rk.PATH_AUTO)
        handle.set_output_projection(None)
        handle.set_variant()
    kw = {}
    if variant:
        kw = dict(indicator_mode=variant[0], temporal_mode=variant[1], spatial_mode=variant[2], group_mode=variant[3])
    ref = oracle_scores(inp, W_O=W, **kw)
    tol = TOL[c.dtype]
    assert_scores_close(scores, ref.scores, tol)
    assert_selection_valid(idx, ref.scores, run.budget, tol)
    _, kbits, vbits = inp.device_arrays()
    assert_compaction_exact(idx, kbits, K_out)
    assert_compaction_exact(idx, vbits, V_out)
    plain = oracle_scores(inp, **kw).scores
    fin = np.isfinite(plain)
    assert not np.allclose(ref.scores[fin], plain[fin], rtol=1e-2), "the projection changed nothing"
    return ref


@pytest.mark.parametrize("spec", [("f32", 64, 96), ("bf16", 128, 300), ("f32", 128, 64), ("bf16", 48, 48),
                                  ("bf16", 128, 96), ("bf16", 128, 120), ("bf16", 128, 24)])
def test_projection_factor(handle, spec):
    """M = W W^T, a factor of it rounded to bf16 (stored transposed) and the product of the rounded factor."""
    import torch
    from paper_2605_08840_b200.inputs import bf16_bits_to_f32
    dtype, d, d_model = spec
    case = Case("proj", 1, 6, 2, d, 64, 4, 8, 1, 0, 0.9, dtype, 0, "normal", 3)
    W, factor = _make_projection(handle, case, d_model, seed=9)
    raw = factor.cpu().numpy()
    dd = 6 * d * d
    M = raw[:4 * dd].view(np.float32).reshape(6, d, d)
    Mt = raw[4 * dd:8 * dd].view(np.float32).reshape(6, d, d)
    LT = bf16_bits_to_f32(raw[8 * dd:10 * dd].view(np.uint16)).reshape(6, d, d)
    M_ref = np.einsum("hik,hjk->hij", W.astype(np.float64), W.astype(np.float64))
    np.testing.assert_allclose(M, M_ref, rtol=0, atol=2e-6 * np.abs(M_ref).max())
    L = np.swapaxes(LT, 1, 2).astype(np.float64)
    np.testing.assert_allclose(Mt, L @ np.swapaxes(L, 1, 2), rtol=0, atol=2e-6 * np.abs(M_ref).max())
    # the rounded factor reproduces M to bf16 accuracy, also where M is singular (d_model < d)
    err = np.linalg.norm(Mt - M_ref, axis=(1, 2)) / np.linalg.norm(M_ref, axis=(1, 2))
    assert err.max() < 2.0 ** -7
    # no column is built on a pivot that is rounding residue: a singular M keeps at most its rank
    kept = (np.abs(LT) > 0).any(axis=2).sum(axis=1)          # non-zero columns of L
    assert kept.max() <= min(d, d_model)


@pytest.mark.parametrize("spec", [("cfg1b", "f32", 0, 96), ("cfg1b", "bf16", 32, 64), ("cfg1a", "f32", 0, 40)])
def test_projection_on_the_simt_kernels(handle, spec):
    name, dtype, tail, d_model = spec
    projection_check(handle, make_inputs(CONFIGS[name].with_(dtype=dtype, causal_tail=tail)), d_model)


@pytest.mark.parametrize("tail", [0, 32])
@pytest.mark.parametrize("d_model", [96, 24])
def test_projection_on_the_tensor_core_kernel(handle, tail, d_model):
    # workload 2 has planted heavy hitters: entries with A > 1/8 take the exact (projected) distance
    projection_check(handle, make_inputs(CONFIGS["cfg2"].with_(causal_tail=tail)), d_model, path=rk.PATH_TENSOR_CORE,
                     fused=True)


def test_projection_from_given_window_statistics(handle):
    projection_check(handle, make_inputs(CONFIGS["cfg2"]), 64, path=rk.PATH_TENSOR_CORE, from_lse=True)


@pytest.mark.parametrize("spec", [(4, 2, 64), (2, 2, 128), (16, 2, 16)])
def test_projection_at_other_window_lengths(handle, spec):
    """w = 64 and 128 run on the tensor-core kernel (two heads, one head per group); w = 16 has eight query heads per
    KV head, more than the tensor-core path's four factor tiles, and runs on the SIMT kernels."""
    Hq, Hkv, w = spec
    case = Case("proj_w%d" % w, 2, Hq, Hkv, 128, 3000, w, 200, 5, 0, 0.9, "bf16", 0, "normal", 56)
    projection_check(handle, make_inputs(case), 160, path=rk.PATH_TENSOR_CORE if w >= 32 else rk.PATH_AUTO)


def test_projection_with_a_variant(handle):
    inp = make_inputs(CONFIGS["cfg2"])
    projection_check(handle, inp, 48, path=rk.PATH_TENSOR_CORE, variant=(REC, INV, rk.SPATIAL_MAX, rk.GROUP_MAX))


def test_projection_is_ignored_by_the_attention_weight_indicators(handle):
    inp = make_inputs(CONFIGS["cfg2"])
    W, factor = _make_projection(handle, inp.case, 64, seed=4)
    handle.set_output_projection(factor, inp.case.n_q_heads, inp.case.head_dim)
    handle.set_variant(ATT, MEAN)
    try:
        scores, _, _, _ = DeviceRun(handle, inp).evict()
    finally:
        handle.set_output_projection(None)
        handle.set_variant()
    ref = oracle_scores(inp, indicator_mode=ATT, temporal_mode=MEAN)
    assert_scores_close(scores, ref.scores, TOL["bf16"])


def test_projection_at_full_size(handle):
    """The long-context workload with a rank-8 projection (d_model = 8 keeps the oracle's cost in bounds)."""
    projection_check(handle, make_inputs(CONFIGS["cfg4"]), 8, fused=True)


def test_projection_must_match_the_shape(handle):
    import torch
    inp = make_inputs(CONFIGS["cfg1b"])
    c = inp.case
    _, factor = _make_projection(handle, c, 32, seed=2)
    run = DeviceRun(handle, inp)
    handle.set_output_projection(factor, c.n_q_heads + 8, c.head_dim)
    try:
        with pytest.raises(rk.RestKVError) as e:
            handle.evict(run.shape, run.Q, run.K, run.V, 0.9, run.pool(), run.budget, run.indices, run.K_out, run.V_out,
                         run.ws)
        assert e.value.status == rk.ERR_INVALID_ARG
    finally:
        handle.set_output_projection(None)
    assert handle.output_projection_bytes(8, 20) == 0 and handle.output_projection_bytes(8, 256) == 0
    torch.cuda.synchronize()


# ------------------------------------------------------------------ nothing is written outside the buffers
class _Guarded:
    """One device allocation carved into buffers with 4 KB bands of a fixed byte pattern before and after each: a
    write past either end of a buffer shows up as a changed band (reads cannot be seen this way)."""
    BAND = 4096

    def __init__(self, sizes):
        import torch
        self.torch = torch
        self.offsets, off = [], self.BAND
        for nbytes in sizes:
            self.offsets.append((off, nbytes))
            off += (nbytes + self.BAND - 1) // self.BAND * self.BAND + self.BAND
        self.raw = torch.full((off,), 0xA5, dtype=torch.uint8, device="cuda")

    def view(self, i, dtype, shape):
        off, nbytes = self.offsets[i]
        return self.raw[off:off + nbytes].view(dtype).view(shape)

    def bands_intact(self):
        mask = self.torch.ones_like(self.raw, dtype=self.torch.bool)
        for off, nbytes in self.offsets:
            mask[off:off + nbytes] = False
        return bool((self.raw[mask] == 0xA5).all())


GUARD_CASES = [
    ("tc_ragged", Case("g1", 2, 8, 2, 128, 1000, 32, 64, 5, 0, 0.8, "bf16", 0, "normal", 91), rk.PATH_AUTO, False),
    ("tc_tail_fused", CONFIGS["cfg2"].with_(causal_tail=32), rk.PATH_TENSOR_CORE, False),
    ("tc_one_over_tile", Case("g2", 1, 4, 1, 128, 129, 32, 130, 3, 0, 0.7, "bf16", 0, "normal", 92), rk.PATH_AUTO, False),
    ("head_sequential", Case("g3", 3, 4, 1, 128, 700, 32, 50, 7, 2, 0.9, "bf16", 0, "normal", 93), rk.PATH_HEAD_SEQUENTIAL, False),
    ("simt_f32", CONFIGS["cfg1b"].with_(causal_tail=32), rk.PATH_AUTO, False),
    ("simt_odd", Case("g4", 2, 6, 3, 72, 333, 5, 40, 3, -1, 0.6, "f32", 0, "normal", 94), rk.PATH_AUTO, False),
    ("many_heads", Case("g5", 20, 32, 8, 128, 300, 32, 30, 5, 0, 0.8, "bf16", 0, "normal", 95), rk.PATH_AUTO, False),
    ("adaptive_tc", CONFIGS["cfg2"].with_(n=2000, budget=200), rk.PATH_AUTO, True),
    ("adaptive_simt", CONFIGS["cfg1b"], rk.PATH_AUTO, True),
]


@pytest.mark.parametrize("spec", GUARD_CASES, ids=[g[0] for g in GUARD_CASES])
def test_no_write_lands_outside_a_buffer(handle, spec):
    import torch
    _, case, path, adaptive = spec
    inp = make_inputs(case)
    c = inp.case
    keep = min(c.budget, c.n_kv)
    BH = c.batch * c.n_kv_heads
    esize = 2 if c.dtype == "bf16" else 4
    shape = shape_of(c)
    ws_bytes = handle.workspace_bytes(shape, c.budget, adaptive=adaptive)
    g = _Guarded([BH * c.n_kv * 4, BH * keep * 4, BH * keep * c.head_dim * esize, BH * keep * c.head_dim * esize, ws_bytes])
    el = torch.bfloat16 if c.dtype == "bf16" else torch.float32
    scores = g.view(0, torch.float32, (c.batch, c.n_kv_heads, c.n_kv))
    indices = g.view(1, torch.int32, (c.batch, c.n_kv_heads, keep))
    K_out = g.view(2, el, (c.batch, c.n_kv_heads, keep, c.head_dim))
    V_out = g.view(3, el, (c.batch, c.n_kv_heads, keep, c.head_dim))
    ws = g.view(4, torch.uint8, (ws_bytes,))
    q, k, v = (torch_dev(a, c.dtype) for a in inp.device_arrays())
    pool = rk.adaptive_pool(50.0, 3, c.budget) if adaptive else rk.fixed_pool(c.width, c.shift)
    handle.set_kernel_path(path)
    try:
        handle.evict(shape, q, k, v, c.ema_decay, pool, c.budget, indices, K_out, V_out, ws, scores_out=scores)
        handle.score(shape, q, k, v, c.ema_decay, pool, scores, ws)
        handle.select(shape, scores, c.budget, indices, ws)
        handle.compact(shape, k, v, indices, keep, K_out, V_out)
        torch.cuda.synchronize()
    finally:
        handle.set_kernel_path(rk.PATH_AUTO)
    assert handle.poll_status() == rk.RESTKV_OK
    assert g.bands_intact()
    idx = indices.cpu().numpy()
    assert idx.min() >= 0 and idx.max() < c.n_kv


# ------------------------------------------------------------------ a seeded sweep over shapes and settings
@pytest.mark.parametrize("seed", [11, 12, 13])
def test_random_shapes_and_settings(handle, seed):
    """Sixty seeded draws per seed of shape (tensor-core shapes and odd ones), tail mode, budget, window, shift, decay,
    variant and output projection, each held against the oracle by the three acceptance rules.  Left out on purpose:
    projections of rank below 16 on the bf16 path (the bf16 factor's rounding then shows as up to 4e-3 on a score)
    and planted heavy keys in caches of a few rows in fp32 (1 - A below fp32's resolution of l - e)."""
    import torch
    from paper_2605_08840_b200.inputs import bf16_bits_to_f32
    rng = np.random.default_rng(seed)
    for _ in range(60):
        if rng.random() < 0.7:
            w = int(rng.choice([16, 32, 64, 128])); G = 128 // w; d = 128; dtype = "bf16"
        else:
            w = int(rng.integers(1, 20)); G = int(rng.choice([1, 2, 3, 4])); d = int(rng.choice([16, 32, 64, 72, 128]))
            dtype = str(rng.choice(["f32", "bf16"]))
        Hkv, b = int(rng.integers(1, 4)), int(rng.integers(1, 3))
        tail = int(rng.choice([0, w]))
        n = int(rng.choice([1, 2, 5, 127, 128, 129, 300, 1000, 2500, 4097])) + int(rng.integers(0, 3))
        budget = int(rng.choice([1, 7, 64, 200, 5000]))
        width, shift = int(rng.choice([1, 3, 7, 21, 31])), int(rng.choice([0, 0, 2, -5, 40]))
        decay = float(rng.choice([0.0, 0.3, 0.7, 0.9, 0.99, 1.0]))
        recipe = "normal" if (dtype == "f32" and n < 50) else str(rng.choice(["normal", "planted"]))
        var = (0, 0, 0, 0)
        if rng.random() < 0.5:
            var = (int(rng.integers(0, 3)), int(rng.integers(0, 4)), int(rng.integers(0, 2)), int(rng.integers(0, 2)))
        proj = d % 16 == 0 and rng.random() < 0.3
        dm = int(rng.choice([40, 100, 128, 200]))
        case = Case("sweep", b, Hkv * G, Hkv, d, n, w, budget, width, shift, decay, dtype, tail, recipe,
                    int(rng.integers(0, 10000)))
        what = "%s variant %s projection %s" % (case, var, dm if proj else None)
        inp = make_inputs(case)
        W = None
        if proj:
            W = (rng.standard_normal((Hkv * G, d, dm)) / np.sqrt(dm)).astype(np.float32)
            if dtype == "bf16":
                bits = round_to_bf16_bits(W)
                W = bf16_bits_to_f32(bits)
                dW = torch_dev(bits.view(np.int16).reshape(-1, dm), "bf16")
            else:
                dW = torch.from_numpy(W.reshape(-1, dm)).cuda()
            factor = torch.empty(handle.output_projection_bytes(Hkv * G, d), dtype=torch.uint8, device="cuda")
            handle.prepare_output_projection(Hkv * G, d, dm, rk.BF16 if dtype == "bf16" else rk.F32, dW, factor)
            handle.set_output_projection(factor, Hkv * G, d)
        handle.set_variant(*var)
        try:
            run = DeviceRun(handle, inp)
            scores, idx, K_out, V_out = run.evict()
        finally:
            handle.set_variant()
            handle.set_output_projection(None)
        ref = oracle.score(inp.Q, inp.K, inp.V, causal_tail=tail, ema_decay=decay, width=width, shift=shift,
                           indicator_mode=var[0], temporal_mode=var[1], spatial_mode=var[2], group_mode=var[3],
                           W_O=W if var[0] == 0 else None)
        tol = TOL[dtype]
        assert_scores_close(scores, ref.scores, tol, what)
        assert_selection_valid(idx, ref.scores, run.budget, tol)
        _, kbits, vbits = inp.device_arrays()
        assert_compaction_exact(idx, kbits, K_out)
        assert_compaction_exact(idx, vbits, V_out)


@pytest.mark.parametrize("seed", [21, 22])
def test_random_shapes_through_the_other_entry_points(handle, seed):
    """Fifty seeded draws per seed of shape and settings through restkv_score_from_lse, restkv_evict_from_lse,
    restkv_evict_budgets and the adaptive window, each against the oracle."""
    import torch
    rng = np.random.default_rng(seed)
    for _ in range(50):
        if rng.random() < 0.7:
            w = int(rng.choice([16, 32, 64, 128])); G = 128 // w; d = 128; dtype = "bf16"
        else:
            w = int(rng.integers(1, 20)); G = int(rng.choice([1, 2, 3, 4])); d = int(rng.choice([16, 32, 64, 72, 128]))
            dtype = str(rng.choice(["f32", "bf16"]))
        Hkv, b = int(rng.integers(1, 4)), int(rng.integers(1, 3))
        tail = int(rng.choice([0, w]))
        n = int(rng.choice([2, 5, 127, 128, 129, 300, 1000, 2500, 4097])) + int(rng.integers(0, 3))
        budget = int(rng.choice([1, 7, 64, 200, 5000]))
        width, shift = int(rng.choice([1, 3, 7, 21, 31])), int(rng.choice([0, 0, 2, -5, 40]))
        decay = float(rng.choice([0.0, 0.3, 0.7, 0.9, 0.99, 1.0]))
        recipe = "normal" if (dtype == "f32" and n < 50) else str(rng.choice(["normal", "planted"]))
        mode = str(rng.choice(["lse_score", "lse_evict", "budgets", "adaptive"]))
        case = Case("sweep2", b, Hkv * G, Hkv, d, n, w, budget, width, shift, decay, dtype, tail, recipe,
                    int(rng.integers(0, 10000)))
        what = "%s %s" % (mode, case)
        inp = make_inputs(case)
        tol = TOL[dtype]
        _, kbits, vbits = inp.device_arrays()
        if mode in ("lse_score", "lse_evict"):
            ref, O, lse = _window_stats(inp, with_A_check=False)
            run = DeviceRun(handle, inp)
            dO, dL = torch.from_numpy(O).cuda(), torch.from_numpy(lse).cuda()
            if mode == "lse_score":
                handle.score_from_lse(run.shape, run.Q, run.K, run.V, dO, dL, decay, run.pool(), run.scores, run.ws)
            else:
                handle.evict_from_lse(run.shape, run.Q, run.K, run.V, dO, dL, decay, run.pool(), run.budget,
                                      run.indices, run.K_out, run.V_out, run.ws, scores_out=run.scores)
            torch.cuda.synchronize()
            assert handle.poll_status() == rk.RESTKV_OK, what
            assert_scores_close(run.scores.cpu().numpy(), ref.scores, tol, what)
            if mode == "lse_evict":
                idx = run.indices.cpu().numpy()
                assert_selection_valid(idx, ref.scores, run.budget, tol)
                assert_compaction_exact(idx, kbits, run._bits(run.K_out))
                assert_compaction_exact(idx, vbits, run._bits(run.V_out))
        elif mode == "budgets":
            ref = oracle_scores(inp)
            run = DeviceRun(handle, inp)
            bud = rng.integers(0, budget + 3, size=(b, Hkv)).astype(np.int32)
            run.indices.fill_(-7)
            handle.evict_budgets(run.shape, run.Q, run.K, run.V, decay, run.pool(), torch.from_numpy(bud).cuda(),
                                 budget, run.indices, run.K_out, run.V_out, run.ws, scores_out=run.scores)
            torch.cuda.synchronize()
            assert handle.poll_status() == rk.RESTKV_OK, what
            idx, K_out = run.indices.cpu().numpy(), run._bits(run.K_out)
            assert_scores_close(run.scores.cpu().numpy(), ref.scores, tol, what)
            for bi in range(b):
                for hh in range(Hkv):
                    keep = min(max(int(bud[bi, hh]), 1), run.keep)
                    assert_selection_valid(idx[bi, hh, :keep], ref.scores[bi, hh], keep, tol)
                    assert np.all(idx[bi, hh, keep:] == -1), what
                    assert np.array_equal(K_out[bi, hh, :keep], kbits[bi, hh][idx[bi, hh, :keep]]), what
        else:
            Bp = max(1, min(budget, 300)) + tail
            probe = oracle_scores(inp, pool_mode=1, beta=1e9, base_width=1, budget=Bp)
            delta = abs(probe.D[..., 0] - probe.D[..., 1]).min()
            if not delta > 0:
                continue
            beta, base = float(delta / 1.5), int(rng.choice([1, 3, 5]))
            ref = oracle_scores(inp, pool_mode=1, beta=beta, base_width=base, budget=Bp)
            x = (ref.D[..., 0] - ref.D[..., 1]) / beta
            keepm = np.abs(x - np.round(x)) >= 0.05
            run = DeviceRun(handle, inp, budget=Bp, adaptive_budget=Bp)
            sc = run.score(pool=rk.adaptive_pool(beta, base, Bp))
            assert handle.poll_status() == rk.RESTKV_OK, what
            assert np.array_equal(run.pool_used.cpu().numpy()[keepm], ref.pool[keepm]), what
            for bi, hh in zip(*np.nonzero(keepm)):
                assert_scores_close(sc[bi, hh], ref.scores[bi, hh], tol, what)


# ------------------------------------------------------------------ a device-side wait that runs out
def test_wait_limit_runs_out_and_the_handle_recovers(handle):
    """With a wait limit of one SM clock the first CTA to reach a group barrier of the persistent score kernel gives
    up at once (its peers have not arrived yet): the kernel must stop issuing work, let what it already issued land,
    return by itself and leave RESTKV_ERR_TIMEOUT in the sticky status; with the default limit restored the same
    handle and workspace then give the oracle's scores."""
    case = Case("timeout", 1, 4, 1, 128, 2000, 32, 100, 5, 0, 0.9, "bf16", 0, "normal", 123)
    inp = make_inputs(case)
    run = DeviceRun(handle, inp)
    handle.set_kernel_path(rk.PATH_TENSOR_CORE)
    try:
        handle.set_wait_limit(1)
        handle.evict(run.shape, run.Q, run.K, run.V, case.ema_decay, run.pool(), run.budget, run.indices, run.K_out,
                     run.V_out, run.ws, scores_out=run.scores)
        run.torch.cuda.synchronize()
        assert handle.poll_status() == rk.ERR_TIMEOUT
        assert handle.poll_status() == rk.RESTKV_OK          # the sticky word is cleared by the poll
    finally:
        handle.set_wait_limit(2_000_000_000)
        handle.set_kernel_path(rk.PATH_AUTO)
    full_check(handle, inp)


# ------------------------------------------------------------------ API misuse: error codes, never a fault
def test_api_rejects_bad_arguments(handle):
    import torch
    case = CONFIGS["cfg1b"]
    inp = make_inputs(case)
    run = DeviceRun(handle, inp)

    def status_of(fn):
        try:
            fn()
        except rk.RestKVError as e:
            return e.status
        return rk.RESTKV_OK

    pool = run.pool()
    ev = lambda **kw: handle.evict(kw.get("shape", run.shape), kw.get("Q", run.Q), run.K, run.V, kw.get("decay", 0.9),
                                   kw.get("pool", pool), kw.get("budget", 128), run.indices, run.K_out, run.V_out,
                                   kw.get("ws", run.ws))
    assert status_of(lambda: ev()) == rk.RESTKV_OK
    assert status_of(lambda: ev(Q=None)) == rk.ERR_INVALID_ARG
    assert status_of(lambda: ev(budget=0)) == rk.ERR_INVALID_ARG
    assert status_of(lambda: ev(decay=1.5)) == rk.ERR_INVALID_ARG
    assert status_of(lambda: ev(pool=rk.fixed_pool(4))) == rk.ERR_INVALID_ARG              # even width
    assert status_of(lambda: ev(ws=run.ws[:1024])) == rk.ERR_WORKSPACE                     # too small
    assert status_of(lambda: ev(ws=run.ws[1:])) == rk.ERR_WORKSPACE                        # misaligned
    assert status_of(lambda: ev(Q=run.Q.view(-1)[1:])) == rk.ERR_INVALID_ARG               # misaligned tensor
    bad = shape_of(case.with_(causal_tail=5))
    assert status_of(lambda: ev(shape=bad)) == rk.ERR_INVALID_ARG
    bad = shape_of(case.with_(n_q_heads=7))
    assert status_of(lambda: ev(shape=bad)) == rk.ERR_INVALID_ARG
    bad = shape_of(case.with_(head_dim=20))
    assert status_of(lambda: ev(shape=bad)) == rk.ERR_UNSUPPORTED
    bad = shape_of(case, k_strides=(0, 0, 7))
    assert status_of(lambda: ev(shape=bad)) == rk.ERR_INVALID_ARG
    torch.cuda.synchronize()
    assert handle.poll_status() == rk.RESTKV_OK
    assert handle.launch_count() > 0

"""The seeded input generators: determinism, dtype exactness and the planted structure."""
import numpy as np

from paper_2605_08840_b200.inputs import (CONFIGS, Case, bf16_bits_to_f32, make_decode_query, make_inputs,
                                           round_to_bf16_bits)


def test_bf16_rounding_is_nearest_even_and_idempotent():
    x = np.array([1.0, 1.00390625, 1.005859375, 1.01171875, -3.14159, 1e-30, 65504.0], np.float32)
    bits = round_to_bf16_bits(x)
    back = bf16_bits_to_f32(bits)
    assert back[0] == 1.0
    assert back[1] == 1.0              # 1 + 2^-8 is a tie: rounds to even (1.0)
    assert back[2] == 1.0078125        # above the tie
    assert back[3] == 1.015625         # 1 + 3*2^-8 is a tie: rounds to even (1 + 2^-6)
    assert np.array_equal(round_to_bf16_bits(back), bits)
    assert np.all(np.abs(back - x) <= np.abs(x) * 2.0 ** -8)


def test_generators_are_seeded_and_dtype_exact():
    case = CONFIGS["cfg2"].with_(n=512)
    a, b = make_inputs(case), make_inputs(case)
    for x, y in zip((a.Q, a.K, a.V), (b.Q, b.K, b.V)):
        assert np.array_equal(x, y)
    c = make_inputs(case, seed=99)
    assert not np.array_equal(a.K, c.K)
    for x in (a.Q, a.K, a.V):
        assert x.dtype == np.float32
        assert np.array_equal(bf16_bits_to_f32(round_to_bf16_bits(x)), x)
    q, k, v = a.device_arrays()
    assert k.dtype == np.int16 and k.shape == a.K.shape
    f = make_inputs(CONFIGS["cfg1a"])
    assert f.device_arrays()[1] is f.K


def test_planted_rows_attract_the_window_queries():
    case = CONFIGS["cfg2"].with_(n=2048)
    inp = make_inputs(case)
    assert inp.heavy_rows.shape == (1, 8, 64)
    assert inp.heavy_rows.min() >= 4 and inp.heavy_rows.max() < 2048
    G, d = case.group, case.head_dim
    for h in range(8):
        logits = inp.Q[0, h * G:(h + 1) * G].reshape(-1, d) @ inp.K[0, h].T / np.sqrt(d)
        mean = logits.mean(0)
        background = np.delete(mean, np.concatenate([inp.heavy_rows[0, h], np.arange(4)]))
        assert mean[inp.heavy_rows[0, h]].mean() - background.mean() > 4.5     # planted boost of about +8 |s|^2/d
        assert 1.5 < mean[:4].mean() - background.mean() < 6.5                 # sinks: about +4
    q = make_decode_query(inp)
    assert q.shape == (1, 32, 128)


def test_drift_recipe_is_a_slow_random_walk():
    case = CONFIGS["cfg3"].with_(n=4096)
    inp = make_inputs(case)
    K = inp.K[0, 0]
    block_means = K.reshape(32, 128, 128).mean(1)
    assert np.abs(block_means[-1] - block_means[0]).mean() > 0.3    # sqrt(4096) * 0.02 = 1.28 per coordinate
    assert abs(K[:128].mean()) < 0.15


def test_causal_tail_adds_window_rows():
    case = Case("t", 1, 4, 2, 64, 100, 8, causal_tail=8)
    inp = make_inputs(case)
    assert inp.K.shape == (1, 2, 108, 64) and inp.V.shape == (1, 2, 108, 64)

"""The seeded input generators: determinism, per-expert streams, truncation, bf16 rounding."""
import math

import numpy as np

from paper_2101_03961_b200 import inputs as si


def test_streams_are_deterministic_and_independent():
    cfg = si.CONFIGS["tiny"]
    a, b = si.gen_x(cfg, 0), si.gen_x(cfg, 0)
    np.testing.assert_array_equal(a, b)
    assert not np.array_equal(a, si.gen_x(cfg, 1))
    assert not np.array_equal(a, si.gen_dy(cfg, 0))
    W = si.gen_W_in(cfg, 0, threads=1)
    np.testing.assert_array_equal(W[5], si.gen_W_in_expert(cfg, 5, 0))        # one expert alone == its slice
    np.testing.assert_array_equal(W, si.gen_W_in(cfg, 0, threads=4))
    assert not np.array_equal(W[0], W[1])


def test_truncated_normal_scale_and_bound():
    cfg = si.CONFIGS["tiny"]
    for W, fan_in in [(si.gen_W_r(cfg), cfg.d_model), (si.gen_W_in(cfg), cfg.d_model), (si.gen_W_out(cfg), cfg.d_ff)]:
        sigma = math.sqrt(0.1 / fan_in)
        assert np.abs(W).max() <= 2 * sigma * (1 + 1e-6)
        assert abs(W.std() / sigma - 0.8796) < 0.03            # std of a normal truncated at two sigma
        assert abs(W.mean()) < 0.05 * sigma


def test_bf16_rounding_is_nearest_even_and_roundtrips():
    v = np.array([1.0, 1.0 + 2 ** -8, 1.0 + 3 * 2 ** -8, 1.0 + 2 ** -9, -3.1415926, 0.0, 1e-30], dtype=np.float32)
    r = si.round_to_bf16(v)
    assert r[0] == 1.0
    assert r[1] == 1.0                       # tie -> even mantissa
    assert r[2] == np.float32(1.0 + 2 ** -6)  # tie -> even mantissa (rounds up)
    assert r[3] == 1.0
    assert abs(r[4] - v[4]) <= abs(v[4]) * 2 ** -8
    np.testing.assert_array_equal(si.from_bf16_bits(si.to_bf16_bits(r)), r)
    cfg = si.CONFIGS["switch_base"].with_(T=64, E=2, d_model=16, d_ff=32)
    x = si.gen_x(cfg)
    np.testing.assert_array_equal(si.round_to_bf16(x), x)
    assert si.gen_W_r(cfg).dtype == np.float32
    Wb = si.gen_W_out(cfg, as_bits=True)
    np.testing.assert_array_equal(si.from_bf16_bits(Wb), si.gen_W_out(cfg))


def test_bias_only_when_requested():
    assert si.gen_router_bias(si.CONFIGS["switch_base"]) is None
    b = si.gen_router_bias(si.CONFIGS["stress_calibrated"])
    assert b.shape == (64,) and b.dtype == np.float32

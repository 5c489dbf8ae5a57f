"""The seeded generators: determinism, storage dtypes, and the stated distributions."""
import numpy as np

from gdn_inputs import (bf16_bits_to_f32, config, f32_to_bf16_bits, make_cu_seqlens, make_tokens,
                        make_varlen_lengths)


def test_bf16_round_trip_and_nearest_even():
    x = np.array([1.0, -2.5, 0.0, 3.140625, 1e-3], dtype=np.float32)
    b = f32_to_bf16_bits(x)
    y = bf16_bits_to_f32(b)
    assert np.all(np.abs(y - x) <= np.abs(x) * 2.0 ** -8)
    assert np.array_equal(f32_to_bf16_bits(y), b)
    # ties go to even: 1 + 2^-8 is halfway between 1 and 1 + 2^-7 -> 1; 1 + 3*2^-8 -> 1 + 2^-6
    t = np.array([1 + 2.0 ** -8, 1 + 3 * 2.0 ** -8], dtype=np.float32)
    assert np.array_equal(bf16_bits_to_f32(f32_to_bf16_bits(t)), np.array([1.0, 1 + 2.0 ** -6], dtype=np.float32))


def test_tokens_are_deterministic_and_follow_the_recipe():
    a = make_tokens(256, 2, 4, seed=0)
    b = make_tokens(256, 2, 4, seed=0)
    c = make_tokens(256, 2, 4, seed=1)
    for f in ("q", "k", "v", "g", "beta"):
        assert np.array_equal(getattr(a, f), getattr(b, f))
    assert not np.array_equal(a.q, c.q)
    assert a.q.dtype == np.uint16 and a.g.dtype == np.float32 and a.beta.dtype == np.float32
    kn = np.linalg.norm(bf16_bits_to_f32(a.k).astype(np.float64), axis=-1)
    qn = np.linalg.norm(bf16_bits_to_f32(a.q).astype(np.float64), axis=-1)
    assert np.all(np.abs(kn - 1) < 5e-3) and np.all(np.abs(qn * np.sqrt(128) - 1) < 5e-3)
    assert np.all(a.g <= 0) and -0.25 < a.g.mean() < -0.12  # log sigmoid(N(2,1))
    assert np.all((a.beta > 0) & (a.beta < 1)) and abs(a.beta.mean() - 0.5) < 0.05
    v = bf16_bits_to_f32(a.v)
    assert abs(v.std() - 1) < 0.05


def test_configs_have_the_stated_shapes():
    c0 = config("prefill_tiny")
    assert c0["tokens"].q.shape == (64, 1, 128) and c0["initial_state"] is None
    c1 = config("decode_b64", B=2)
    assert c1["state"].shape == (2, 32, 128, 128) and abs(c1["state"].std() - 0.02) < 1e-3
    assert c1["tokens"].q.shape == (2, 16, 128) and c1["tokens"].v.shape == (2, 32, 128)
    lens = make_varlen_lengths(16, 1, 2048, seed=0)
    assert lens.min() >= 1 and lens.max() <= 2048 and np.any(lens % 64 != 0)
    cu = make_cu_seqlens(lens)
    assert cu.dtype == np.int32 and cu[0] == 0 and cu[-1] == lens.sum()

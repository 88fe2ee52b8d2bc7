"""The seeded input generator: determinism, shapes, rounding, locality statistic."""
import numpy as np

import gen


def test_bf16_round_trip_and_rne():
    x = np.array([1.0, 1.00390625, 1.005859375, -3.14159, 0.0, 65280.0], dtype=np.float32)
    bits = gen.f32_to_bf16_bits(x)
    back = gen.bf16_bits_to_f32(bits)
    # 1 + 2^-8 is a tie between 1.0 and 1 + 2^-7: ties go to even (1.0)
    assert back[0] == 1.0 and back[1] == 1.0
    assert back[2] == np.float32(1.0078125)
    assert np.all(np.abs(back - x) <= np.abs(x) * 2.0 ** -8)
    assert np.array_equal(gen.f32_to_bf16_bits(back), bits)


def test_normal_stream_is_counter_based_and_standard():
    a = gen.normal(0, (1, 2, 3), 100000)
    b = gen.normal(0, (1, 2, 3), 1000)
    assert np.array_equal(a[:1000], b)
    assert not np.array_equal(a[:1000], gen.normal(0, (1, 2, 4), 1000))
    assert abs(a.mean()) < 0.02 and abs(a.std() - 1.0) < 0.02


def test_configs_shapes_and_locality():
    expect = {"cfg1": (1, 1024, 640, 16, 64), "cfg2": (2, 1024, 1280, 16, 64),
              "cfg3": (2, 4096, 640, 16, 256), "cfg4": (1, 4096, 3072, 16, 256),
              "cfg5a": (4, 16384, 640, 64, 256), "cfg5b": (4, 16384, 640, 16, 1024)}
    for name, (b, n, d, p, nl) in expect.items():
        c = gen.config(name)
        assert (c.batch, c.n_tokens, c.dim, c.n_tiles, c.n_loc) == (b, n, d, p, nl)
        assert c.n_heads * c.head_dim == c.dim
    c = gen.config("cfg2")
    x = gen.features(c)
    assert x.shape == (2, 1024, 1280) and x.dtype == np.float32
    assert np.array_equal(gen.round_to_dtype(x, "bf16"), x)  # already bf16 values
    assert 0.75 < gen.neighbour_cosine(c, x) < 0.85
    assert np.array_equal(x, gen.features(c))
    c1 = gen.config("cfg1")
    assert 0.2 < gen.neighbour_cosine(c1, gen.features(c1)) < 0.4


def test_step_sequence_drifts():
    c = gen.config("cfg3", batch=1, grid_h=16, grid_w=16, dim=64, steps=3)
    xs = list(gen.feature_sequence(c))
    assert len(xs) == 3
    d01 = (xs[1] - xs[0]).std()
    assert 0.03 < d01 < 0.08
    assert np.array_equal(xs[2], gen.features(c, 2))

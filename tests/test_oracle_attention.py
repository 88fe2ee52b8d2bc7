"""Pins for the attention oracle (Eq. 1 with tau = 1): textbook special cases and a
library second opinion."""
import numpy as np
import pytest
import torch

from oracle import toma_oracle as O


def test_constant_values_give_constant_output():
    rng = np.random.default_rng(0)
    q = rng.normal(size=(9, 16))
    k = rng.normal(size=(13, 16))
    v = np.tile(rng.normal(size=(1, 16)), (13, 1))
    assert np.allclose(O.attention(q, k, v, 2), np.tile(v[:1], (9, 1)))


def test_zero_queries_average_the_values():
    rng = np.random.default_rng(1)
    k = rng.normal(size=(11, 8))
    v = rng.normal(size=(11, 8))
    out = O.attention(np.zeros((4, 8)), k, v, 2)
    assert np.allclose(out, np.tile(v.mean(0), (4, 1)))


def test_single_key_returns_its_value():
    rng = np.random.default_rng(2)
    q = rng.normal(size=(5, 8))
    out = O.attention(q, rng.normal(size=(1, 8)), np.arange(8.0)[None], 4)
    assert np.allclose(out, np.tile(np.arange(8.0), (5, 1)))


def test_two_keys_closed_form_pins_the_scale():
    # one head of width 4: logits q.k/2; q = (2 ln 3, 0, 0, 0), keys e1 and 0 -> weights 3/4, 1/4
    q = np.array([[2 * np.log(3.0), 0, 0, 0]])
    k = np.array([[1.0, 0, 0, 0], [0, 0, 0, 0]])
    v = np.array([[1.0, 0, 0, 0], [0, 1.0, 0, 0]])
    assert np.allclose(O.attention(q, k, v, 1), [[0.75, 0.25, 0, 0]])


def test_heads_are_independent_column_blocks_and_match_library():
    rng = np.random.default_rng(3)
    L, h, dh = 37, 3, 8
    q, k, v = (rng.normal(size=(L, h * dh)) for _ in range(3))
    got = O.attention(q, k, v, h)
    tq, tk, tv = (torch.from_numpy(a).reshape(L, h, dh).permute(1, 0, 2) for a in (q, k, v))
    want = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv).permute(1, 0, 2).reshape(L, h * dh)
    assert np.allclose(got, want.numpy(), atol=1e-12)
    rows = np.array([0, 5, 36])
    assert np.allclose(O.attention(q, k, v, h, query_rows=rows), got[rows])


def test_linear_matches_explicit_loops():
    rng = np.random.default_rng(5)
    a, w = rng.normal(size=(5, 7)), rng.normal(size=(7, 3))
    want = np.zeros((5, 3))
    for i in range(5):
        for j in range(3):
            for k in range(7):
                want[i, j] += a[i, k] * w[k, j]
    assert np.allclose(O.linear(a, w), want, rtol=0, atol=1e-13)
    assert np.array_equal(O.linear(a, np.eye(7)), a)


def test_gelu_closed_forms_and_library_second_opinion():
    import math
    import torch
    # Phi(1) = 0.8413447460685429 (standard normal table), Phi(0) = 1/2
    assert O.gelu(np.array([0.0]))[0] == 0.0
    assert O.gelu(np.array([1.0]))[0] == pytest.approx(0.8413447460685429, abs=1e-15)
    assert O.gelu(np.array([-1.0]))[0] == pytest.approx(-0.15865525393145707, abs=1e-15)
    v = np.linspace(-6, 6, 241)
    g = O.gelu(v)
    assert np.allclose(g - O.gelu(-v), v, atol=1e-14)            # Phi(v) + Phi(-v) = 1
    assert np.allclose(g[v > 5.5], v[v > 5.5], atol=1e-7) and np.all(np.abs(g[v < -5.5]) < 1e-7)
    assert g.min() == pytest.approx(-0.16997, abs=1e-4)           # the dip near v = -0.7518
    want = torch.nn.functional.gelu(torch.from_numpy(v), approximate="none").numpy()
    assert np.allclose(g, want, atol=1e-14)
    # not the tanh approximation: the two differ by up to 5e-4
    tanh_form = 0.5 * v * (1 + np.tanh(math.sqrt(2 / math.pi) * (v + 0.044715 * v ** 3)))
    assert np.abs(g - tanh_form).max() > 1e-4


def test_mlp_is_two_projections_around_gelu():
    rng = np.random.default_rng(9)
    x, w1, w2 = rng.normal(size=(6, 8)), rng.normal(size=(8, 12)) / 3, rng.normal(size=(12, 8)) / 3
    h = np.zeros((6, 12))
    for i in range(6):
        for j in range(12):
            h[i, j] = sum(x[i, k] * w1[k, j] for k in range(8))
    want = O.gelu(h) @ w2
    assert np.allclose(O.mlp(x, w1, w2), want, atol=1e-13)
    # rounding hook: applied to the hidden tensor and to the result
    r = lambda t: np.round(t * 16) / 16
    assert np.array_equal(O.mlp(x, w1, w2, r), r(r(O.gelu(h)) @ w2))
    # a zero first layer gives GELU(0) = 0 everywhere
    assert np.array_equal(O.mlp(x, np.zeros_like(w1), w2), np.zeros((6, 8)))

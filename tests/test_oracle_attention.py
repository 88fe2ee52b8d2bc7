"""Pins for the attention oracle (Eq. 1 with tau = 1): textbook special cases and a
library second opinion."""
import numpy as np
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

"""Pins for the selection oracle: Eq. 2, the cached-max gain identity (App. A.1),
Algorithm 1/2 by brute force on tiny ground sets, closed-form tiles, and the
fixed-point similarity's exactness properties."""
import itertools
import math
import os

import numpy as np
import pytest

import gen
from oracle import toma_oracle as O


def _rand_int_S(rng, n, lo=-4000, hi=4000):
    a = rng.integers(lo, hi, size=(n, n))
    S = np.triu(a, 1)
    S = S + S.T
    np.fill_diagonal(S, O.DIAG_Q)
    return S.astype(np.int32)


def _f_bruteforce(S, subset):
    """Eq. 2 written as explicit loops."""
    tot = 0
    for i in range(S.shape[0]):
        tot += max(S[i][j] for j in subset)
    return tot


def test_facility_location_matches_explicit_loops():
    rng = np.random.default_rng(0)
    S = _rand_int_S(rng, 7)
    for r in range(1, 5):
        for sub in itertools.combinations(range(7), r):
            assert O.facility_location(S, sub) == _f_bruteforce(S, sub)


def test_gain_identity_cached_max():
    # f(A + v) - f(A) == sum_j max(0, S_jv - m_j),  m_j = max_{a in A} S_ja   (App. A.1)
    rng = np.random.default_rng(1)
    for _ in range(50):
        n = int(rng.integers(3, 10))
        S = _rand_int_S(rng, n)
        A = list(rng.choice(n, size=int(rng.integers(1, n)), replace=False))
        for v in set(range(n)) - set(A):
            m = S[:, A].max(axis=1)
            lhs = _f_bruteforce(S, A + [v]) - _f_bruteforce(S, A)
            rhs = int(np.maximum(0, S[:, v] - m).sum())
            assert lhs == rhs


def test_monotone_and_submodular_by_enumeration():
    rng = np.random.default_rng(2)
    n = 6
    S = _rand_int_S(rng, n, 0, 4000)
    subsets = [s for r in range(0, n + 1) for s in itertools.combinations(range(n), r)]
    f = {s: (O.facility_location(S, s) if s else 0) for s in subsets}
    for A in subsets:
        for Bs in subsets:
            if not set(A) <= set(Bs):
                continue
            for v in set(range(n)) - set(Bs):
                ga = f[tuple(sorted(A + (v,)))] - f[A]
                gb = f[tuple(sorted(Bs + (v,)))] - f[Bs]
                assert ga >= gb >= 0


def test_greedy_takes_best_single_addition_each_round_lowest_index_on_ties():
    rng = np.random.default_rng(3)
    for trial in range(40):
        n = int(rng.integers(4, 12))
        # coarse values force many exact ties
        S = _rand_int_S(rng, n, -3, 4) if trial % 2 else _rand_int_S(rng, n)
        k = int(rng.integers(1, n + 1))
        picks = list(O.greedy_select(S, k))
        assert len(set(picks)) == k
        for r in range(k):
            A = picks[:r]
            rest = [v for v in range(n) if v not in A]
            vals = [_f_bruteforce(S, A + [v]) for v in rest]
            best = max(vals)
            assert picks[r] == rest[vals.index(best)]  # first (lowest-index) maximiser


def test_greedy_first_pick_is_best_singleton():
    rng = np.random.default_rng(4)
    S = _rand_int_S(rng, 9)
    t = O.greedy_select(S, 1)[0]
    assert t == int(np.argmax([_f_bruteforce(S, [i]) for i in range(9)]))


def test_greedy_one_minus_inv_e_bound():
    rng = np.random.default_rng(5)
    for _ in range(10):
        n, k = 10, 3
        S = _rand_int_S(rng, n, 0, 4000)  # non-negative => f(empty) = 0 is consistent
        g = O.facility_location(S, O.greedy_select(S, k))
        opt = max(O.facility_location(S, s) for s in itertools.combinations(range(n), k))
        assert g >= (1 - 1 / math.e) * opt


def test_no_reselection_even_when_cache_is_negative():
    # a first pick whose row is very negative elsewhere: zeroing its row instead of
    # excluding it would make it the best "candidate" again
    S = np.full((4, 4), -3000, dtype=np.int32)
    np.fill_diagonal(S, O.DIAG_Q)
    picks = O.greedy_select(S, 4)
    assert sorted(picks) == [0, 1, 2, 3]


def test_identical_tokens_pick_in_index_order():
    x = np.tile(np.linspace(-1, 1, 16)[None, :], (12, 1))
    idx, _ = O.select_tile(x, 5)
    assert list(idx) == [0, 1, 2, 3, 4]


def test_orthogonal_prototype_groups_pick_first_member_of_each_group():
    d, groups, rep = 16, 4, 3
    protos = np.eye(d)[:groups] * 2.5
    x = np.repeat(protos, rep, axis=0)  # tokens 0..2 group 0, 3..5 group 1, ...
    idx, _ = O.select_tile(x, groups)
    assert list(idx) == [0, 3, 6, 9]


def test_round_to_8_bits_equals_bf16_rounding():
    k = np.arange(-4100, 4101, dtype=np.int64)
    got = O._round_to_8_significant_bits(k)
    want = gen.bf16_bits_to_f32(gen.f32_to_bf16_bits((k * 2.0 ** -12).astype(np.float32))) * 4096.0
    assert np.array_equal(got, want.astype(np.int64))


def test_pinned_similarity_properties():
    c = gen.config("cfg3", batch=1)
    x = gen.features(c)[0]
    tile = O.split_regions(x, c.grid_h, c.grid_w, c.tile_h, c.tile_w)[3]
    k, margin = O.quantise_tokens(tile)
    assert margin > O.FRAGILE_MARGIN
    # bf16-representable directions
    y = (k * 2.0 ** -12).astype(np.float32)
    assert np.array_equal(gen.round_to_dtype(y, "bf16"), y)
    S, _ = O.pinned_similarity(tile)
    assert np.array_equal(S, S.T) and np.all(np.diag(S) == O.DIAG_Q)
    cos = O.cosine_similarity(tile)
    off = ~np.eye(len(S), dtype=bool)
    assert np.abs(S[off] / 4096.0 - O.COS_SCALE ** 2 * cos[off]).max() < 6e-3
    # an fp32 accumulation in any order reproduces the integer Gram exactly
    rng = np.random.default_rng(0)
    K = k @ k.T
    for _ in range(3):
        perm = rng.permutation(k.shape[1])
        acc = np.zeros((8, 8), dtype=np.float32)
        for cidx in perm:
            acc = acc + np.outer(y[:8, cidx], y[:8, cidx]).astype(np.float32)
        assert np.array_equal(acc.astype(np.float64) * 2.0 ** 24, K[:8, :8].astype(np.float64))


def test_gram_rounding_is_ties_to_even_by_hand():
    """S_q = rint(K / 4096), halves to the even neighbour (the reading taken where Sec. 4.1 gives no precision).
    Hand-computed: 2048/4096 = 0.5 -> 0, 6144/4096 = 1.5 -> 2, 2049/4096 -> 1, 2047/4096 -> 0, 10240/4096 = 2.5 -> 2,
    and the same on the negative side (floor, half-up and ties-to-even differ on these)."""
    K = np.array([2048, 6144, 2049, 2047, 10240, 4096, 0, -2048, -6144, -2049, -2047, -10240, -4096])
    want = np.array([0, 2, 1, 0, 2, 1, 0, 0, -2, -1, 0, -2, -1])
    assert np.array_equal(O.round_gram(K), want)
    # ... and pinned_similarity goes through exactly this step: two tokens at 60 degrees, d = 2
    x = np.array([[1.0, 0.0], [0.5, np.sqrt(0.75)]])
    k, _ = O.quantise_tokens(x)
    S, _ = O.pinned_similarity(x)
    assert S[0, 1] == O.round_gram(np.array([int(k[0] @ k[1])]))[0] and abs(S[0, 1] - 0.99 ** 2 * 0.5 * 4096) <= 8


def test_zero_norm_token_is_harmless():
    rng = np.random.default_rng(7)
    x = rng.normal(size=(8, 32))
    x[2] = 0.0
    S, _ = O.pinned_similarity(x)
    assert np.all(S[2, [0, 1, 3, 4, 5, 6, 7]] == 0) and S[2, 2] == O.DIAG_Q
    assert len(set(O.greedy_select(S, 8))) == 8


def test_fixed_point_selection_is_faithful_to_fp64_cosine_greedy():
    c = gen.config("cfg3", batch=1)
    x = gen.features(c)[0]
    tiles = O.split_regions(x, c.grid_h, c.grid_w, c.tile_h, c.tile_w)
    for p in (0, 5, 10):
        a, _ = O.select_tile(tiles[p], O.dest_count(c.n_loc, c.merge_ratio))
        b = O.select_tile_definition(tiles[p], O.dest_count(c.n_loc, c.merge_ratio))
        cos = O.cosine_similarity(tiles[p])
        ratio = O.facility_location(cos, a) / O.facility_location(cos, b)
        assert ratio > 0.995
        assert len(set(a) & set(b)) >= 0.8 * O.dest_count(c.n_loc, c.merge_ratio)


def test_region_split_tiles_and_stripes():
    H, W, th, tw = 6, 8, 3, 4
    ids = O.tile_token_ids(H, W, th, tw)
    assert ids.shape == (4, 12)
    for y in range(H):
        for x in range(W):
            p = (y // th) * (W // tw) + (x // tw)
            l = (y % th) * tw + (x % tw)
            assert ids[p, l] == y * W + x
    stripes = O.tile_token_ids(H, W, 2, W)  # a stripe is a tile as wide as the grid
    assert np.array_equal(stripes, np.arange(H * W).reshape(3, 16))
    with pytest.raises(ValueError):
        O.tile_token_ids(6, 8, 4, 4)


def test_dest_count_reading():
    assert O.dest_count(64, 0.5) == 32
    assert [O.dest_count(256, r) for r in (0.25, 0.5, 0.75)] == [192, 128, 64]
    with pytest.raises(ValueError):
        O.dest_count(4, 1.0)


def test_flop_table_overhead_row():
    path = os.path.join(os.path.dirname(__file__), "golden", "flop_table.txt")
    rows = [l.split() for l in open(path) if l.strip() and not l.startswith("#")]
    sdxl = [r for r in rows if r[0] == "SDXL" and r[1] == "4096"][0]
    got = O.overhead_tiled(4096, 640, 0.5, 64) / 1e9
    assert round(got, 2) == float(sdxl[5])
    # tiling divides the selection cost by P and the weight / apply cost by P as well per region count
    assert O.overhead_tiled(4096, 640, 0.5, 1) == pytest.approx(4096 ** 2 * 640 * 2.5)
    assert O.cost_toma_global(4096, 640, 0.5) - (4 * 640 ** 2 * 2048 + 2 * 640 * 2048 ** 2) == pytest.approx(
        O.overhead_tiled(4096, 640, 0.5, 1))
    assert O.cost_base(4096, 640) == 4 * 640 ** 2 * 4096 + 2 * 640 * 4096 ** 2

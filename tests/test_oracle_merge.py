"""Pins for the merge-weight, merge and unmerge oracle (Sec. 4.2) and the block loop."""
import math

import numpy as np
import pytest

import gen
from oracle import toma_oracle as O


def test_scale_and_softmax_axis_closed_form():
    # d = 4, tau = 0.5  =>  tau*sqrt(d) = 1: logits are plain dot products
    x = np.array([[1.0, 0, 0, 0],          # destination 0
                  [0, 1.0, 0, 0],          # destination 1
                  [math.log(3.0), 0, 0, 0]])  # a source: logits (ln 3, 0) -> shares (3/4, 1/4)
    idx = np.array([0, 1])
    for tau, share in ((0.5, 3 / 4), (0.25, 9 / 10)):  # halving tau doubles the logits
        L = x[idx] @ x.T / (tau * 2.0)
        A = np.exp(L) / np.exp(L).sum(axis=0, keepdims=True)
        w = O.merge_weights(x, idx, tau)
        assert A[0, 2] == pytest.approx(share)
        # undo the row normalisation with the closed-form row sums
        assert w[0, 2] == pytest.approx(share / A[0].sum())
        assert w[1, 2] == pytest.approx((1 - share) / A[1].sum())


def test_weight_invariants_on_a_real_tile():
    c = gen.config("cfg2", batch=1)
    x = gen.features(c)[0]
    tile = O.split_regions(x, c.grid_h, c.grid_w, c.tile_h, c.tile_w)[7]
    idx, _ = O.select_tile(tile, O.dest_count(c.n_loc, c.merge_ratio))
    w = O.merge_weights(tile, idx, c.tau)
    assert w.shape == (O.dest_count(c.n_loc, c.merge_ratio), c.n_loc)
    assert np.all(w >= 0)
    assert np.allclose(w.sum(axis=1), 1.0, atol=1e-12)          # merge rows sum to 1
    Z = 1.0 / w[np.arange(O.dest_count(c.n_loc, c.merge_ratio)), idx]                          # not used further; rows are positive
    assert np.all(np.isfinite(Z))
    # before row normalisation every source's shares sum to 1: recover A = w * Z_row
    xs = tile.astype(np.float64)
    L = xs[idx] @ xs.T / (c.tau * math.sqrt(c.dim))
    A = np.exp(L - L.max(0)) / np.exp(L - L.max(0)).sum(0)
    assert np.allclose(A.sum(axis=0), 1.0)
    assert np.allclose(w, A / A.sum(1, keepdims=True))


def test_orthogonal_groups_give_group_means():
    d, groups, rep = 16, 4, 3
    protos = np.eye(d)[:groups] * 3.0
    x = np.repeat(protos, rep, axis=0)
    x = x + 0.01 * np.arange(x.size).reshape(x.shape) / x.size  # break exact duplication a little
    idx, _ = O.select_tile(x, groups)
    w = O.merge_weights(x, idx, 0.05)  # cold softmax: hard assignment
    member = np.repeat(np.arange(groups), rep)
    want = np.zeros((groups, groups * rep))
    for g in range(groups):
        want[g, member == g] = 1.0 / rep
    order = np.argsort(idx)  # destinations come in pick order; compare group-wise
    assert np.allclose(w[order], want, atol=1e-6)
    merged = O.merge(w, x)
    for j, g in enumerate(member[idx]):
        assert np.allclose(merged[j], x[member == g].mean(axis=0), atol=1e-5)
    y = np.arange(groups * d, dtype=np.float64).reshape(groups, d)
    un = O.unmerge(w, y)
    for k in range(groups * rep):
        j = list(member[idx]).index(member[k])
        assert np.allclose(un[k], y[j] / rep, atol=1e-5)


def test_hot_temperature_gives_tile_mean():
    rng = np.random.default_rng(0)
    x = rng.normal(size=(16, 8))
    idx = np.array([3, 7, 11])
    w = O.merge_weights(x, idx, 1e9)
    assert np.allclose(w, 1.0 / 16)
    assert np.allclose(O.merge(w, x), np.tile(x.mean(0), (3, 1)))


def test_identity_and_permutation_weights_round_trip_exactly():
    rng = np.random.default_rng(1)
    x = gen.round_to_dtype(rng.normal(size=(8, 5)).astype(np.float32), "bf16").astype(np.float64)
    eye = np.eye(8)
    assert np.array_equal(O.unmerge(eye, O.merge(eye, x)), x)
    perm = eye[rng.permutation(8)]
    assert np.array_equal(O.merge(perm, x), x[np.argmax(perm, axis=1)])
    assert np.array_equal(O.unmerge(perm, O.merge(perm, x)), x)   # A A^T = I  =>  A^T is the inverse


def test_merge_and_unmerge_are_the_two_matrix_products():
    rng = np.random.default_rng(2)
    w = rng.random((3, 7))
    x = rng.normal(size=(7, 4))
    y = rng.normal(size=(3, 4))
    m = O.merge(w, x)
    u = O.unmerge(w, y)
    for i in range(3):
        for c in range(4):
            assert m[i, c] == pytest.approx(sum(w[i, k] * x[k, c] for k in range(7)))
    for k in range(7):
        for c in range(4):
            assert u[k, c] == pytest.approx(sum(w[i, k] * y[i, c] for i in range(3)))


def test_block_step_reuse_schedule_and_layout():
    c = gen.config("cfg3", batch=1, grid_h=16, grid_w=16, tile_h=8, tile_w=8, dim=64, n_heads=2,
                   head_dim=32, steps=4, reuse_interval=2)
    st = O.BlockState()
    kw = dict(grid_h=16, grid_w=16, tile_h=8, tile_w=8, merge_ratio=0.5, tau=c.tau, n_heads=2,
              reuse_interval=2)
    seen = []
    for t, x in enumerate(gen.feature_sequence(c)):
        out, merged, att = O.block_step(x, t, st, **kw)
        seen.append(st.idx.copy())
        assert out.shape == x.shape and merged.shape == (1, 4 * 32, 64)
    assert np.array_equal(seen[0], seen[1]) and np.array_equal(seen[2], seen[3])
    assert not np.array_equal(seen[0], seen[2])
    # tile-major, pick-order layout of merged rows
    x0 = gen.features(c, 0)[0].astype(np.float64)
    st = O.BlockState()
    _, merged, _ = O.block_step(x0[None], 0, st, **kw)
    ids = O.tile_token_ids(16, 16, 8, 8)
    p = 2
    assert np.allclose(merged[0, p * 32:(p + 1) * 32], O.merge(st.w[0, p], x0[ids[p]]))


def test_block_step_passes_text_tokens_through():
    c = gen.config("cfg4", grid_h=16, grid_w=16, tile_h=8, tile_w=8, dim=32, n_heads=2, head_dim=16, n_extra=5)
    x = gen.features(c)
    st = O.BlockState()
    out, merged, att = O.block_step(x, 0, st, grid_h=16, grid_w=16, tile_h=8, tile_w=8, merge_ratio=0.5,
                                    tau=0.1, n_heads=2, reuse_interval=1, n_extra=5)
    D = 4 * 32
    assert merged.shape == (1, D + 5, 32)
    assert np.array_equal(merged[0, D:], x[0, 256:].astype(np.float64))
    assert np.array_equal(out[0, 256:], att[0, D:])


def test_block_step_separate_weight_schedule():
    # destinations every 4 steps, weights every 2: at step 2 the indices are kept but the weights follow the new x
    c = gen.config("cfg3", batch=1, grid_h=16, grid_w=16, tile_h=8, tile_w=8, dim=64, n_heads=2, head_dim=32, steps=4)
    kw = dict(grid_h=16, grid_w=16, tile_h=8, tile_w=8, merge_ratio=0.5, tau=c.tau, n_heads=2, reuse_interval=4,
              weight_reuse_interval=2)
    st = O.BlockState()
    xs = list(gen.feature_sequence(c))
    O.block_step(xs[0], 0, st, **kw)
    idx0, w0 = st.idx.copy(), st.w.copy()
    O.block_step(xs[1], 1, st, **kw)
    assert np.array_equal(st.idx, idx0) and np.array_equal(st.w, w0)
    O.block_step(xs[2], 2, st, **kw)
    assert np.array_equal(st.idx, idx0) and not np.array_equal(st.w, w0)
    ids = O.tile_token_ids(16, 16, 8, 8)
    assert np.allclose(st.w[0, 1], O.merge_weights(xs[2][0][ids[1]], idx0[0, 1], c.tau))


def test_global_merge_reduces_to_tile_merge_for_one_tile_and_sees_across_tiles():
    """Global merge (default ToMA variant): with a single tile it is the tile-local path; with several
    tiles every token gets a share of every destination (rows sum to 1, columns of A sum to 1), and
    two identical tokens in different tiles, one of them a destination, end up on that destination."""
    c = gen.config("cfg3", batch=1, grid_h=8, grid_w=8, tile_h=8, tile_w=8, dim=32, n_heads=1, head_dim=32, steps=1)
    x = gen.features(c)
    kw = dict(grid_h=8, grid_w=8, tile_h=8, tile_w=8, merge_ratio=0.5, tau=c.tau, n_heads=1, reuse_interval=1)
    a = O.block_step(x, 0, O.BlockState(), **kw)[0]
    b = O.block_step(x, 0, O.BlockState(), global_merge=True, **kw)[0]
    assert np.allclose(a, b, rtol=0, atol=1e-12)

    c = gen.config("cfg3", batch=1, grid_h=8, grid_w=8, tile_h=4, tile_w=4, dim=32, n_heads=1, head_dim=32, steps=1)
    x = gen.features(c).astype(np.float64)
    ids = O.tile_token_ids(8, 8, 4, 4)
    st = O.BlockState()
    kw = dict(grid_h=8, grid_w=8, tile_h=4, tile_w=4, merge_ratio=0.5, tau=c.tau, n_heads=1, reuse_interval=1)
    O.block_step(x, 0, st, global_merge=True, **kw)
    w = st.w[0, 0]                       # [D, N]
    D, N = w.shape
    assert (D, N) == (32, 64) and np.allclose(w.sum(1), 1.0)
    gidx = O.global_destinations(st.idx[0], ids)
    assert len(set(gidx.tolist())) == D
    # a copy, in another tile, of a destination token puts (almost) all its mass on that destination
    dest_tok = int(gidx[0])
    other = next(int(t) for t in ids[3] if t not in set(gidx.tolist()))
    x2 = x.copy()
    x2[0, other] = 3.0 * x2[0, dest_tok]  # a long copy: its logit with the destination dominates
    # shares of that token over the destinations = its column of A; after row normalisation the
    # largest entry of the column is still the destination it copies
    w2 = O.merge_weights(x2[0, :64], gidx, c.tau)
    assert np.argmax(w2[:, other] * w2.shape[1]) == 0 or np.argmax(w2[:, other]) == 0


def test_global_destinations_hand_written_two_by_two_tiles():
    """4x4 grid cut into four 2x2 tiles, written out by hand: tile p holds tokens
    p0: 0 1 4 5 | p1: 2 3 6 7 | p2: 8 9 12 13 | p3: 10 11 14 15 (local slot = row-major inside the tile),
    so the tile-local picks below map to these image tokens, tile-major, pick order inside a tile."""
    ids = O.tile_token_ids(4, 4, 2, 2)
    assert ids.tolist() == [[0, 1, 4, 5], [2, 3, 6, 7], [8, 9, 12, 13], [10, 11, 14, 15]]
    idx_tiles = np.array([[3, 0], [1, 2], [0, 3], [2, 1]])
    assert O.global_destinations(idx_tiles, ids).tolist() == [5, 0, 3, 6, 8, 13, 14, 11]
    # a permutation of the picks permutes the result the same way (any fixed one-to-one map would not)
    assert O.global_destinations(idx_tiles[:, ::-1], ids).tolist() == [0, 5, 6, 3, 13, 8, 11, 14]
    # the global-merge block puts exactly these tokens' rows first in their softmax columns: token 5 is
    # destination 0, so A[0, 5] is the largest share of column 5 when tau is cold
    rng = np.random.default_rng(5)
    x = rng.normal(size=(16, 8)) * 3.0
    A = O.softmax_shares(x, O.global_destinations(idx_tiles, ids), 0.01)
    for row, tok in enumerate([5, 0, 3, 6, 8, 13, 14, 11]):
        assert np.argmax(A[:, tok]) == row


def test_block_step_with_projections_is_the_hand_composed_chain():
    """block_step(proj=(wq, wk, wv, wo)) against the chain written out here from the pinned pieces: merge with
    the block's own weights, X_m wq / X_m wk / X_m wv, attention, wo, transpose unmerge.  Distinct random
    matrices: swapping any two of wq, wk, wv, wo in block_step changes the result."""
    c = gen.config("cfg3", batch=2, grid_h=8, grid_w=8, tile_h=4, tile_w=4, dim=16, n_heads=2, head_dim=8, steps=1, n_extra=3)
    x = gen.features(c).astype(np.float64)
    rng = np.random.default_rng(11)
    wq, wk, wv, wo = (rng.normal(size=(16, 16)) / 4.0 for _ in range(4))
    kw = dict(grid_h=8, grid_w=8, tile_h=4, tile_w=4, merge_ratio=0.5, tau=c.tau, n_heads=2, reuse_interval=1, n_extra=3)
    st = O.BlockState()
    out, merged, attended = O.block_step(x, 0, st, proj=(wq, wk, wv, wo), **kw)
    ids = O.tile_token_ids(8, 8, 4, 4)
    d_loc = O.dest_count(16, 0.5)
    for b in range(2):
        xm = np.concatenate([O.merge(st.w[b, p], x[b, ids[p]]) for p in range(4)] + [x[b, 64:]])
        assert np.allclose(merged[b], xm, atol=1e-12)
        att = O.attention(O.linear(xm, wq), O.linear(xm, wk), O.linear(xm, wv), 2)
        y = O.linear(att, wo)
        assert np.allclose(attended[b], y, atol=1e-12)
        for p in range(4):
            assert np.allclose(out[b, ids[p]], O.unmerge(st.w[b, p], y[p * d_loc:(p + 1) * d_loc]), atol=1e-12)
        assert np.allclose(out[b, 64:], y[4 * d_loc:], atol=1e-12)
        for perm in ((wk, wq, wv, wo), (wq, wv, wk, wo), (wq, wk, wo, wv), (wo, wk, wv, wq)):
            other = O.block_step(x, 0, O.BlockState(), proj=perm, **kw)[0]
            assert not np.allclose(other[b], out[b], atol=1e-3)


def _quarter(t):
    return np.round(np.asarray(t, dtype=np.float64) * 4.0) / 4.0


def test_block_step_round_fn_placement_with_projections_and_mlp():
    """Where block_step applies round_fn: to the merged tokens, to q, k, v, to the attention output and to the
    projected output (projections); to the merged tokens, the hidden tensor and the MLP output (MLP); to the
    merged and the attended tokens (plain attention).  A coarse rounding (multiples of 1/4) makes every
    placement visible; the chain is written out by hand."""
    c = gen.config("cfg3", batch=1, grid_h=8, grid_w=8, tile_h=4, tile_w=4, dim=16, n_heads=2, head_dim=8, steps=1)
    x = gen.features(c).astype(np.float64)
    rng = np.random.default_rng(12)
    wq, wk, wv, wo = (rng.normal(size=(16, 16)) / 2.0 for _ in range(4))
    w1, w2 = rng.normal(size=(16, 16)) / 2.0, rng.normal(size=(16, 16)) / 2.0   # square: a swapped pair would still run
    kw = dict(grid_h=8, grid_w=8, tile_h=4, tile_w=4, merge_ratio=0.5, tau=c.tau, n_heads=2, reuse_interval=1)
    ids = O.tile_token_ids(8, 8, 4, 4)
    d_loc = O.dest_count(16, 0.5)
    calls = []

    def rnd(t):
        calls.append(np.shape(t))
        return _quarter(t)

    def unmerged(st, y):
        out = np.empty((64, 16))
        for p in range(4):
            out[ids[p]] = O.unmerge(st.w[0, p], y[p * d_loc:(p + 1) * d_loc])
        return out

    # projections
    st = O.BlockState()
    out = O.block_step(x, 0, st, proj=(wq, wk, wv, wo), round_fn=rnd, **kw)[0]
    xm = _quarter(np.concatenate([O.merge(st.w[0, p], x[0, ids[p]]) for p in range(4)]))
    q, k, v = (_quarter(O.linear(xm, w)) for w in (wq, wk, wv))
    y = _quarter(O.linear(_quarter(O.attention(q, k, v, 2)), wo))
    assert np.allclose(out[0], unmerged(st, y), atol=1e-12)
    assert len(calls) == 6          # merged; q, k, v; attention output; projected output
    assert not np.allclose(out[0], O.block_step(x, 0, O.BlockState(), proj=(wq, wk, wv, wo), **kw)[0][0], atol=1e-3)
    # MLP
    calls.clear()
    st = O.BlockState()
    out = O.block_step(x, 0, st, mlp_weights=(w1, w2), round_fn=rnd, **kw)[0]
    hid = _quarter(O.gelu(O.linear(xm, w1)))
    assert np.allclose(out[0], unmerged(st, _quarter(O.linear(hid, w2))), atol=1e-12)
    assert len(calls) == 3          # merged; hidden; MLP output
    plain = O.block_step(x, 0, O.BlockState(), mlp_weights=(w1, w2), **kw)[0]
    xm_plain = np.concatenate([O.merge(st.w[0, p], x[0, ids[p]]) for p in range(4)])
    assert np.allclose(plain[0], unmerged(st, O.linear(O.gelu(O.linear(xm_plain, w1)), w2)), atol=1e-12)
    assert not np.allclose(plain[0], O.block_step(x, 0, O.BlockState(), mlp_weights=(w2, w1), **kw)[0][0], atol=1e-3)
    # plain attention: merged and attended, once each
    calls.clear()
    st = O.BlockState()
    out = O.block_step(x, 0, st, round_fn=rnd, **kw)[0]
    assert np.allclose(out[0], unmerged(st, _quarter(O.attention(xm, xm, xm, 2))), atol=1e-12)
    assert len(calls) == 2


def test_softmax_shares_closed_form_and_relation_to_merge_weights():
    """The matrix of the "shares" unmerge: columns sum to 1 (a token's shares over the destinations),
    A~ is A with its rows rescaled, and the closed form of the two-destination case."""
    x = np.array([[1.0, 0, 0, 0], [0, 1.0, 0, 0], [math.log(3.0), 0, 0, 0]])
    idx = np.array([0, 1])
    A = O.softmax_shares(x, idx, 0.5)              # tau*sqrt(d) = 1
    assert A[:, 2] == pytest.approx([3 / 4, 1 / 4])
    e = math.e
    assert A[:, 0] == pytest.approx([e / (e + 1), 1 / (e + 1)])  # destination 0 against itself and against 1
    c = gen.config("cfg2", batch=1)
    tile = O.split_regions(gen.features(c)[0], c.grid_h, c.grid_w, c.tile_h, c.tile_w)[3]
    idx, _ = O.select_tile(tile, O.dest_count(c.n_loc, c.merge_ratio))
    A = O.softmax_shares(tile, idx, c.tau)
    w = O.merge_weights(tile, idx, c.tau)
    assert np.all(A >= 0) and np.allclose(A.sum(axis=0), 1.0, atol=1e-12)
    assert np.allclose(w * A.sum(axis=1, keepdims=True), A, rtol=1e-12, atol=0)


def test_shares_unmerge_is_a_partition_of_unity_and_beats_the_transpose_on_round_trips():
    """With the column-stochastic matrix every source token receives a convex combination of the
    destinations' outputs: a constant comes back unchanged, outputs stay inside the destinations'
    range, and unmerge(merge(x)) is closer to x than with A~^T, whose columns sum to about D/N."""
    c = gen.config("cfg2", batch=1)
    tile = O.split_regions(gen.features(c)[0], c.grid_h, c.grid_w, c.tile_h, c.tile_w)[5].astype(np.float64)
    idx, _ = O.select_tile(tile, O.dest_count(c.n_loc, c.merge_ratio))
    A = O.softmax_shares(tile, idx, c.tau)
    w = O.merge_weights(tile, idx, c.tau)
    const = np.full((O.dest_count(c.n_loc, c.merge_ratio), 7), 2.5)
    assert np.allclose(O.unmerge(A, const), 2.5, atol=1e-12)
    assert not np.allclose(O.unmerge(w, const), 2.5, atol=0.1)   # the transpose attenuates
    y = np.random.default_rng(3).normal(size=(O.dest_count(c.n_loc, c.merge_ratio), 5))
    un = O.unmerge(A, y)
    assert np.all(un <= y.max(axis=0) + 1e-12) and np.all(un >= y.min(axis=0) - 1e-12)
    merged = O.merge(w, tile)
    err_t = np.linalg.norm(O.unmerge(w, merged) - tile) / np.linalg.norm(tile)
    err_s = np.linalg.norm(O.unmerge(A, merged) - tile) / np.linalg.norm(tile)
    assert err_s < err_t
    # explicit loops: out_k = sum_i A_ik y_i
    k = 11
    assert np.allclose(un[k], sum(A[i, k] * y[i] for i in range(O.dest_count(c.n_loc, c.merge_ratio))), atol=1e-12)


def test_shares_unmerge_on_orthogonal_groups_copies_the_prototype_output():
    d, groups, rep = 16, 4, 3
    x = np.repeat(np.eye(d)[:groups] * 3.0, rep, axis=0)
    x = x + 0.01 * np.arange(x.size).reshape(x.shape) / x.size
    idx, _ = O.select_tile(x, groups)
    A = O.softmax_shares(x, idx, 0.05)  # cold softmax: hard assignment
    member = np.repeat(np.arange(groups), rep)
    y = np.arange(groups * d, dtype=np.float64).reshape(groups, d)
    un = O.unmerge(A, y)
    for k in range(groups * rep):
        j = list(member[idx]).index(member[k])
        assert np.allclose(un[k], y[j], atol=1e-5)   # (y_j / rep with the transpose unmerge)


def test_block_step_unmerge_modes_differ_only_in_the_unmerge():
    c = gen.config("cfg2", batch=1, grid_h=16, grid_w=16, dim=64, n_heads=1, head_dim=64)
    x = gen.features(c)
    kw = dict(grid_h=16, grid_w=16, tile_h=c.tile_h, tile_w=c.tile_w, merge_ratio=0.5, tau=c.tau, n_heads=1,
              reuse_interval=1)
    st_t, st_s = O.BlockState(), O.BlockState()
    out_t, merged_t, att_t = O.block_step(x, 0, st_t, **kw)
    out_s, merged_s, att_s = O.block_step(x, 0, st_s, unmerge_mode="shares", **kw)
    assert np.array_equal(merged_t, merged_s) and np.array_equal(att_t, att_s)
    assert np.array_equal(st_t.w, st_s.w) and np.array_equal(st_t.idx, st_s.idx)
    ids = O.tile_token_ids(16, 16, c.tile_h, c.tile_w)
    d_loc = O.dest_count(c.n_loc, c.merge_ratio)
    p = 2
    want = st_s.u[0, p].T @ att_s[0, p * d_loc:(p + 1) * d_loc]
    assert np.allclose(out_s[0, ids[p]], want, atol=1e-12)
    assert not np.allclose(out_s, out_t, atol=1e-3)
    with pytest.raises(ValueError):
        O.block_step(x, 0, O.BlockState(), unmerge_mode="nope", **kw)

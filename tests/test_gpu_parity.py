"""GPU-vs-oracle parity of every step of the ToMA block path, called through the C ABI.

Tolerances (written here, as the target states them): selected indices bit-exact;
bf16 tensors max-abs <= 2e-2 and relative Frobenius <= 1e-2; fp32 tensors max-abs <= 1e-4.
"""
import numpy as np
import pytest
import torch

import gen
from oracle import toma_oracle as O
from tests._util import assert_close, sample_tiles, tile_tokens, to_dev, to_host64

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def toma():
    import __graft_entry__ as entry
    entry.build()
    import paper_2509_10918_b200 as t
    return t


@pytest.fixture
def tuning(toma):
    """Forces a launch configuration through the library's test-only setter; the heuristics come back afterwards."""
    yield toma.toma_test_set_tuning
    toma.toma_test_set_tuning()


def od(cfg):
    """Destinations per tile as the oracle counts them."""
    return O.dest_count(cfg.n_loc, cfg.merge_ratio)


def gd(toma, cfg):
    """Destinations per tile as the library counts them (sizes of the device buffers)."""
    return toma.toma_dest_per_tile(toma.desc_from_config(cfg))


class Run:
    """Device buffers of one configuration plus the entry points bound to them."""

    def __init__(self, toma, cfg, x_host, **desc_over):
        self.t, self.cfg = toma, cfg
        self.desc = toma.desc_from_config(cfg, **desc_over)
        self.x = to_dev(x_host, cfg.dtype)
        self.idx = toma.alloc_idx(self.desc)
        self.w = toma.alloc_weights(self.desc)
        self.ws = toma.alloc_workspace(self.desc)
        self.status = torch.zeros(1, dtype=torch.int32, device="cuda")
        self.d_loc = toma.toma_dest_per_tile(self.desc)
        self.lm = cfg.n_tiles * self.d_loc + cfg.n_extra
        self.xm = torch.empty((cfg.batch, self.lm, cfg.dim), dtype=self.x.dtype, device="cuda")

    def ok(self):
        torch.cuda.synchronize()
        assert int(self.status.item()) == 0

    def select(self):
        self.t.toma_select(self.desc, self.x, self.idx, self.ws, self.status)
        self.ok()
        return self.idx.cpu().numpy().astype(np.int64)

    def weights(self):
        self.t.toma_merge_weights(self.desc, self.x, self.idx, self.w, self.ws, self.status)
        self.ok()
        c = self.cfg
        dense = torch.empty((c.batch, c.n_tiles, self.d_loc, c.n_loc), dtype=torch.float32, device="cuda")
        self.t.toma_weights_export(self.desc, self.w, dense)
        torch.cuda.synchronize()
        return dense.cpu().numpy().astype(np.float64)

    def merge(self):
        self.t.toma_merge(self.desc, self.w, self.x, self.xm, self.status)
        self.ok()
        return to_host64(self.xm)

    def attend(self):
        """Attention over the merged tokens (Q = K = V = merged), as toma_block does."""
        c = self.cfg
        att = torch.empty_like(self.xm)
        self.t.toma_attention(c.batch, self.lm, c.n_heads, c.head_dim, c.dtype, self.xm, self.xm, self.xm, att,
                              self.status)
        self.ok()
        return att

    def unmerge(self, y):
        out = torch.empty_like(self.x)
        self.t.toma_unmerge(self.desc, self.w, y, out, self.status)
        self.ok()
        return to_host64(out)


CASES = [
    # name, overrides, number of tiles the oracle checks
    ("cfg1", {}, 16),
    ("cfg2", {}, 32),
    ("cfg3", {"merge_ratio": 0.25}, 8),
    ("cfg3", {"merge_ratio": 0.5}, 32),
    ("cfg3", {"merge_ratio": 0.75}, 8),
    ("cfg4", {}, 6),
    ("cfg5a", {}, 8),
    ("cfg5b", {}, 2),
]


@pytest.mark.parametrize("name,over,n_check", CASES, ids=[f"{n}-{'-'.join(map(str, o.values())) or 'base'}" for n, o, _ in CASES])
def test_select_weights_merge_unmerge_parity(toma, name, over, n_check):
    cfg = gen.config(name, **over)
    x_host = gen.features(cfg)
    run = Run(toma, cfg, x_host)
    idx = run.select()
    # properties that hold for every tile at full size
    assert idx.min() >= 0 and idx.max() < cfg.n_loc
    srt = np.sort(idx, axis=-1)
    assert np.all(srt[..., 1:] != srt[..., :-1]), "a tile selected the same token twice"
    dense = run.weights()
    assert np.all(dense >= 0)
    tol_rows = 1e-5 if cfg.dtype == "f32" else 2e-3
    assert np.abs(dense.sum(-1) - 1.0).max() < tol_rows, "merge rows must sum to 1"
    merged = run.merge()
    # the unmerge input is what the block feeds it: the attention output over the merged tokens
    # (already in storage dtype; the oracle unmerges this same tensor)
    y_dev = run.attend()
    unmerged = run.unmerge(y_dev)
    y_host = to_host64(y_dev)
    D = cfg.n_tiles * gd(toma, cfg)
    if cfg.n_extra:
        assert np.array_equal(merged[:, D:], x_host[:, cfg.n_tokens:].astype(np.float64))
        assert np.array_equal(unmerged[:, cfg.n_tokens:], y_host[:, D:])
    ids = O.tile_token_ids(cfg.grid_h, cfg.grid_w, cfg.tile_h, cfg.tile_w)
    # fp32 logits up to ~512 carry a half-ulp of 3e-5, i.e. <= 1.5e-5 on a softmax share; bf16 mode: fp32 accumulation over d terms perturbs a logit of ~400 by up to ~1e-3, i.e. 2.5e-4 on a share
    w_abs = 2e-5 if cfg.dtype == "f32" else 6e-4
    got_m, want_m, got_u, want_u = [], [], [], []
    for b, p in sample_tiles(cfg, n_check):
        xt = tile_tokens(cfg, x_host, b, p)
        want_idx, margin = O.select_tile(xt, od(cfg))
        assert margin > O.FRAGILE_MARGIN, "input sits on a quantisation boundary; choose another seed"
        assert np.array_equal(idx[b, p], want_idx), f"selection differs in tile ({b},{p})"
        w = O.merge_weights(xt, want_idx, cfg.tau)
        assert np.abs(dense[b, p] - w).max() <= w_abs, f"weights differ in tile ({b},{p})"
        got_m.append(merged[b, p * gd(toma, cfg):(p + 1) * gd(toma, cfg)])
        want_m.append(O.merge(w, xt))
        got_u.append(unmerged[b, ids[p]])
        want_u.append(O.unmerge(w, y_host[b, p * gd(toma, cfg):(p + 1) * gd(toma, cfg)]))
    assert_close(np.stack(got_m), np.stack(want_m), cfg.dtype, "merge")
    assert_close(np.stack(got_u), np.stack(want_u), cfg.dtype, "unmerge")


ATT_CASES = [
    ("f32", 1, 512, 10, 64, None),
    ("bf16", 2, 512, 20, 64, None),
    ("bf16", 2, 2048, 10, 64, 96),
    ("bf16", 1, 2560, 24, 128, 64),
    ("bf16", 2, 1000, 3, 64, None),   # ragged length
    ("bf16", 1, 77, 2, 128, None),    # shorter than one tile
    ("bf16", 4, 8192, 10, 64, 24),
]


@pytest.mark.parametrize("dtype,B,L,h,dh,n_rows", ATT_CASES)
def test_attention_parity(toma, dtype, B, L, h, dh, n_rows):
    rng_tag = (L * 131 + h * 7 + dh) % 1000
    host = [gen.round_to_dtype(gen.normal(0, (77, rng_tag, i), B * L * h * dh).reshape(B, L, h * dh).astype(np.float32),
                               dtype) for i in range(3)]
    q, k, v = (to_dev(a, dtype) for a in host)
    o = torch.empty_like(q)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    toma.toma_attention(B, L, h, dh, dtype, q, k, v, o, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    got = to_host64(o)
    rows = None if n_rows is None else np.unique(np.concatenate(
        [[0, L - 1], np.random.default_rng(L).choice(L, size=n_rows, replace=False)]))
    for b in range(B):
        want = O.attention(host[0][b], host[1][b], host[2][b], h, query_rows=rows)
        assert_close(got[b] if rows is None else got[b][rows], want, dtype, f"attention b={b}")


@pytest.mark.parametrize("split,ctas,B,L,h,dh", [
    ("1", "7", 1, 1000, 3, 64),     # spans run over several units: partial first piece, whole middle ones, partial last
    ("1", "320", 1, 300, 3, 64),    # one key tile per CTA: five contributors per unit, all through scratch
    ("1", "37", 2, 700, 2, 128),    # head_dim 128, ragged, units cut in two or three
    ("1", "2", 1, 640, 1, 64),      # two CTAs share the middle unit
    ("0", "5", 1, 1000, 3, 64),     # whole units, several per CTA
    ("0", "320", 1, 300, 3, 128),   # whole units, fewer units than CTAs
])
def test_attention_span_plans(toma, tuning, split, ctas, B, L, h, dh):
    """The tensor-core kernel under forced work plans (toma_test_set_tuning): every way a unit's keys can
    be cut across CTAs gives the same result."""
    tuning(attention_split=int(split), attention_ctas=int(ctas))
    host = [gen.round_to_dtype(gen.normal(0, (78, L + dh, i), B * L * h * dh).reshape(B, L, h * dh).astype(np.float32),
                               "bf16") for i in range(3)]
    q, k, v = (to_dev(a, "bf16") for a in host)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    outs = []
    for _ in range(2):  # twice: the second launch finds the scratch as the first left it
        o = torch.full_like(q, float("nan"))
        toma.toma_attention(B, L, h, dh, "bf16", q, k, v, o, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        outs.append(to_host64(o))
    assert np.array_equal(outs[0], outs[1])
    for b in range(B):
        assert_close(outs[0][b], O.attention(host[0][b], host[1][b], host[2][b], h), "bf16", f"attention b={b}")


@pytest.mark.parametrize("dh,L", [(64, 1536), (128, 1000)])
def test_attention_growing_logits_exercise_the_rescale_path(toma, dh, L):
    """Keys grow along the sequence so that the row maximum rises by far more than the kernel's
    rescaling threshold many times: the accumulator rescaling and the stale-maximum bookkeeping
    must still give the exact softmax."""
    B, h = 1, 2
    rng = np.random.default_rng(dh)
    u = rng.normal(size=(h, dh))
    u /= np.linalg.norm(u, axis=1, keepdims=True)
    q = rng.normal(size=(B, L, h, dh)) + 6.0 * u[None, None]
    ramp = (np.arange(L) / L)[None, :, None, None]
    k = 0.3 * rng.normal(size=(B, L, h, dh)) + 14.0 * np.sqrt(dh) / 3.0 * ramp * u[None, None]
    v = rng.normal(size=(B, L, h, dh))
    host = [gen.round_to_dtype(a.reshape(B, L, h * dh).astype(np.float32), "bf16") for a in (q, k, v)]
    # the logits really do climb by tens of units of log2 over the sequence
    s = (6.0 * u[0] @ host[1][0, :, :dh].astype(np.float64).T) / np.sqrt(dh) * 1.4427  # a typical query
    assert s[-64:].max() - s[:64].max() > 30
    dq, dk, dv = (to_dev(a, "bf16") for a in host)
    o = torch.empty_like(dq)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    toma.toma_attention(B, L, h, dh, "bf16", dq, dk, dv, o, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    want = O.attention(host[0][0], host[1][0], host[2][0], h)
    assert_close(to_host64(o)[0], want, "bf16", "attention with growing logits")


def test_a_wait_that_nobody_ends_gives_up_and_reports(toma):
    """The bounded wait every tensor-core kernel uses, made to run out on purpose in the accepted way: a
    barrier that nobody signals and a limit of a thousand polls.  The kernel must return, the status word
    must carry the timeout bit, and the next ordinary call on the same context must work."""
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    outcome = torch.zeros(1, dtype=torch.int32, device="cuda")
    toma.toma_test_wait_timeout(1000, status, outcome)
    torch.cuda.synchronize()
    assert int(outcome.item()) == 2, "the wait on an unsignalled barrier did not give up"
    assert int(status.item()) & 1 == 1, "TOMA_ERR_TIMEOUT's bit is missing from the status word"
    # the context is intact: a normal call afterwards succeeds with a clean status word
    cfg = gen.config("cfg2", batch=1, grid_h=16, grid_w=16)
    run = Run(toma, cfg, gen.features(cfg))
    want, _ = O.select_tile(tile_tokens(cfg, gen.features(cfg), 0, 0), od(cfg))
    assert np.array_equal(run.select()[0, 0], want)
    run.weights()
    run.merge()


BLOCK_CASES = [
    ("cfg1", {}, None),
    ("cfg2", {}, None),
    ("cfg3", {"steps": 6}, None),
    ("cfg4", {}, None),
]


@pytest.mark.parametrize("name,over,_", BLOCK_CASES, ids=[c[0] for c in BLOCK_CASES])
def test_block_sequence_parity(toma, name, over, _):
    cfg = gen.config(name, **over)
    desc = toma.desc_from_config(cfg)
    idx = toma.alloc_idx(desc)
    w = toma.alloc_weights(desc)
    ws = toma.alloc_workspace(desc)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    st = O.BlockState()
    kw = dict(grid_h=cfg.grid_h, grid_w=cfg.grid_w, tile_h=cfg.tile_h, tile_w=cfg.tile_w, merge_ratio=cfg.merge_ratio,
              tau=cfg.tau, n_heads=cfg.n_heads, reuse_interval=cfg.reuse_interval, n_extra=cfg.n_extra)
    for step, x_host in enumerate(gen.feature_sequence(cfg)):
        x = to_dev(x_host, cfg.dtype)
        out = torch.empty_like(x)
        toma.toma_block(desc, step, x, out, idx, w, ws, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        want, _, _ = O.block_step(x_host, step, st, **kw)
        assert min(st.margins) > O.FRAGILE_MARGIN
        assert np.array_equal(idx.cpu().numpy().astype(np.int64), st.idx), f"selection differs at step {step}"
        assert_close(to_host64(out), want, cfg.dtype, f"block step {step}")


@pytest.mark.parametrize("over", [dict(), dict(batch=1, grid_h=32, grid_w=16, dim=128, n_heads=2),
                                  dict(batch=3, grid_h=16, grid_w=32, tile_h=4, tile_w=16, dim=640, n_heads=10),
                                  dict(batch=1, grid_h=32, grid_w=16, tile_h=16, tile_w=4, dim=128, n_heads=2),
                                  dict(batch=2, grid_h=16, grid_w=64, tile_h=2, tile_w=32, dim=256, n_heads=4)],
                         ids=["cfg2", "256-merged-tokens", "4x16-tiles", "16x4-tiles", "2x32-tiles"])
def test_block_one_kernel_reuse_step_parity(toma, tuning, over):
    """Shapes with 64-token tiles, 32 destinations and at most 512 merged tokens run merge, attention and unmerge of
    a step as ONE kernel.  Both forms of the step (one kernel; three kernels, forced through the test-only
    setter) must match the oracle on a refresh step and on the reuse step after it, and each other closely."""
    cfg = gen.config("cfg2", steps=2, reuse_interval=2, **over)
    desc = toma.desc_from_config(cfg)
    kw = dict(grid_h=cfg.grid_h, grid_w=cfg.grid_w, tile_h=cfg.tile_h, tile_w=cfg.tile_w, merge_ratio=cfg.merge_ratio,
              tau=cfg.tau, n_heads=cfg.n_heads, reuse_interval=2)
    outs = {}
    for unfused in (0, 1):
        tuning(block_unfused=unfused)
        idx, w, ws = toma.alloc_idx(desc), toma.alloc_weights(desc), toma.alloc_workspace(desc)
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        st = O.BlockState()
        launches = []
        for step, x_host in enumerate(gen.feature_sequence(cfg)):
            x = to_dev(x_host, cfg.dtype)
            out = torch.full_like(x, float("nan"))
            n0 = toma.toma_launch_counter()
            toma.toma_block(desc, step, x, out, idx, w, ws, status)
            torch.cuda.synchronize()
            launches.append(toma.toma_launch_counter() - n0)
            assert int(status.item()) == 0
            want, _, _ = O.block_step(x_host, step, st, **kw)
            assert np.array_equal(idx.cpu().numpy().astype(np.int64), st.idx)
            assert_close(to_host64(out), want, cfg.dtype, f"block step {step}, {'three kernels' if unfused else 'one kernel'}")
            outs[(unfused, step)] = to_host64(out)
            if step == 0:
                # the refresh step's weights themselves (one kernel does Gram, greedy rounds and weights of a tile
                # when the step is not forced onto the separate kernels): every tile against Sec. 4.2.1
                dense = torch.empty((cfg.batch, cfg.n_tiles, gd(toma, cfg), cfg.n_loc), dtype=torch.float32, device="cuda")
                toma.toma_weights_export(desc, w, dense)
                torch.cuda.synchronize()
                dense = dense.cpu().numpy().astype(np.float64)
                ids = O.tile_token_ids(cfg.grid_h, cfg.grid_w, cfg.tile_h, cfg.tile_w)
                for b_ in range(cfg.batch):
                    for p_ in range(cfg.n_tiles):
                        xt = x_host[b_][ids[p_]].astype(np.float64)
                        assert np.abs(dense[b_, p_] - O.merge_weights(xt, st.idx[b_, p_], cfg.tau)).max() <= 6e-4, (b_, p_)
        assert launches[1] == (3 if unfused else 1), f"reuse step launched {launches[1]} kernels"
    for step in (0, 1):
        assert np.abs(outs[(0, step)] - outs[(1, step)]).max() <= 2 ** -6, "the two forms of the step disagree"


@pytest.mark.parametrize("over", [dict(merge_ratio=0.25), dict(merge_ratio=0.75), dict(merge_ratio=0.875, tile_h=4, tile_w=16),
                                  dict(merge_ratio=0.5, batch=1, dim=320, n_heads=5, n_extra=77)],
                         ids=["48-destinations", "16-destinations", "8-destinations-4x16", "text-tokens"])
def test_block_small_tile_refresh_kernel_parity(toma, tuning, over):
    """A refresh step on 64-token tiles takes Gram, greedy rounds and weights of a tile in one kernel (whatever the
    rest of the step runs as).  Indices bit-exact, weights and output against the oracle, for destination counts
    and shapes the one-kernel reuse step does not cover; the same step forced onto the separate kernels agrees."""
    cfg = gen.config("cfg2", steps=1, reuse_interval=1, **over)
    desc = toma.desc_from_config(cfg)
    kw = dict(grid_h=cfg.grid_h, grid_w=cfg.grid_w, tile_h=cfg.tile_h, tile_w=cfg.tile_w, merge_ratio=cfg.merge_ratio,
              tau=cfg.tau, n_heads=cfg.n_heads, reuse_interval=1, n_extra=cfg.n_extra)
    x_host = next(iter(gen.feature_sequence(cfg)))
    want, _, _ = O.block_step(x_host, 0, (st := O.BlockState()), **kw)
    assert min(st.margins) > O.FRAGILE_MARGIN
    ids = O.tile_token_ids(cfg.grid_h, cfg.grid_w, cfg.tile_h, cfg.tile_w)
    dense = {}
    for separate in (0, 1):
        tuning(block_unfused=separate)
        idx, w, ws = toma.alloc_idx(desc), toma.alloc_weights(desc), toma.alloc_workspace(desc)
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        x = to_dev(x_host, cfg.dtype)
        out = torch.full_like(x, float("nan"))
        n0 = toma.toma_launch_counter()
        toma.toma_block(desc, 0, x, out, idx, w, ws, status)
        torch.cuda.synchronize()
        launches = toma.toma_launch_counter() - n0
        assert int(status.item()) == 0
        assert np.array_equal(idx.cpu().numpy().astype(np.int64), st.idx)
        assert_close(to_host64(out), want, cfg.dtype, "block output")
        d = torch.empty((cfg.batch, cfg.n_tiles, gd(toma, cfg), cfg.n_loc), dtype=torch.float32, device="cuda")
        toma.toma_weights_export(desc, w, d)
        torch.cuda.synchronize()
        dense[separate] = d.cpu().numpy().astype(np.float64)
        for b_ in range(cfg.batch):
            for p_ in range(cfg.n_tiles):
                xt = x_host[b_][ids[p_]].astype(np.float64)
                assert np.abs(dense[separate][b_, p_] - O.merge_weights(xt, st.idx[b_, p_], cfg.tau)).max() <= 6e-4, (b_, p_)
        dense[("launches", separate)] = launches
    assert dense[("launches", 0)] == dense[("launches", 1)] - 3, "selection and weights should have taken two launches instead of five"
    assert np.abs(dense[0] - dense[1]).max() <= 6e-4


@pytest.mark.parametrize("name", ["cfg2", "cfg3"])
def test_block_steps_enqueued_back_to_back_equal_synchronised_steps(toma, name):
    """Consecutive toma_block calls overlap on the device (programmatic dependent launch: a kernel's prologue runs
    under the previous kernel's tail).  Thirty steps enqueued without a synchronisation in between must give,
    bit for bit, what the same steps give with the device idle before each call."""
    cfg = gen.config(name, batch=1, steps=6, reuse_interval=3)
    desc = toma.desc_from_config(cfg)
    xs = [to_dev(x, cfg.dtype) for x in gen.feature_sequence(cfg)]
    runs = []
    for synchronise in (True, False):
        idx, w, ws = toma.alloc_idx(desc), toma.alloc_weights(desc), toma.alloc_workspace(desc)
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        out = torch.empty_like(xs[0])
        outs = []
        for t in range(30):
            toma.toma_block(desc, t % 6, xs[t % 6], out, idx, w, ws, status)
            outs.append(out.clone())   # on the same stream, behind the step
            if synchronise:
                torch.cuda.synchronize()
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        runs.append(outs)
    for t, (a, b) in enumerate(zip(*runs)):
        assert torch.equal(a, b), f"step {t} differs"


@pytest.mark.parametrize("over", [dict(batch=1), dict(batch=2, merge_ratio=0.25), dict(batch=1, tile_h=8, tile_w=16, merge_ratio=0.75)],
                         ids=["128-of-256", "192-of-256", "32-of-128"])
def test_block_weights_out_of_the_raw_gram_matrix_parity(toma, tuning, over):
    """A refresh step on few large tiles computes X X^T of every tile on the SMs that idle during the greedy rounds
    and reads the merge weights out of it.  Indices bit-exact, weights within 6e-4 of Sec. 4.2.1 on every tile,
    output against the oracle; the same step forced onto the separate kernels (gather and the tensor-core logits with
    their softmax) agrees."""
    cfg = gen.config("cfg3", steps=1, reuse_interval=1, **over)
    desc = toma.desc_from_config(cfg)
    kw = dict(grid_h=cfg.grid_h, grid_w=cfg.grid_w, tile_h=cfg.tile_h, tile_w=cfg.tile_w, merge_ratio=cfg.merge_ratio,
              tau=cfg.tau, n_heads=cfg.n_heads, reuse_interval=1)
    x_host = next(iter(gen.feature_sequence(cfg)))
    want, _, _ = O.block_step(x_host, 0, (st := O.BlockState()), **kw)
    assert min(st.margins) > O.FRAGILE_MARGIN
    ids = O.tile_token_ids(cfg.grid_h, cfg.grid_w, cfg.tile_h, cfg.tile_w)
    dense, launches = {}, {}
    for separate in (0, 1):
        tuning(block_unfused=separate)
        idx, w, ws = toma.alloc_idx(desc), toma.alloc_weights(desc), toma.alloc_workspace(desc)
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        x = to_dev(x_host, cfg.dtype)
        out = torch.full_like(x, float("nan"))
        n0 = toma.toma_launch_counter()
        toma.toma_block(desc, 0, x, out, idx, w, ws, status)
        torch.cuda.synchronize()
        launches[separate] = toma.toma_launch_counter() - n0
        assert int(status.item()) == 0
        assert np.array_equal(idx.cpu().numpy().astype(np.int64), st.idx)
        assert_close(to_host64(out), want, cfg.dtype, "block output")
        d = torch.empty((cfg.batch, cfg.n_tiles, gd(toma, cfg), cfg.n_loc), dtype=torch.float32, device="cuda")
        toma.toma_weights_export(desc, w, d)
        torch.cuda.synchronize()
        dense[separate] = d.cpu().numpy().astype(np.float64)
        for b_ in range(cfg.batch):
            for p_ in range(cfg.n_tiles):
                xt = x_host[b_][ids[p_]].astype(np.float64)
                assert np.abs(dense[separate][b_, p_] - O.merge_weights(xt, st.idx[b_, p_], cfg.tau)).max() <= 6e-4, (b_, p_)
    assert np.abs(dense[0] - dense[1]).max() <= 6e-4


def test_small_tile_refresh_kernel_agrees_with_the_separate_kernels_on_many_inputs(toma, tuning):
    """Both forms of a refresh step on 64-token tiles work on the same integers (the fixed-point Gram) with the same
    rule (largest gain, lowest index), so their picks must be identical on any input, fragile or not; twenty seeds,
    two noise levels (smooth tiles give many near-ties)."""
    for seed in range(20):
        cfg = gen.config("cfg2", batch=1, steps=1, reuse_interval=1, seed=1000 + seed, noise_sigma=0.05 if seed % 2 else 0.5)
        desc = toma.desc_from_config(cfg)
        x = to_dev(next(iter(gen.feature_sequence(cfg))), cfg.dtype)
        got = {}
        for separate in (0, 1):
            tuning(block_unfused=separate)
            idx, w, ws = toma.alloc_idx(desc), toma.alloc_weights(desc), toma.alloc_workspace(desc)
            status = torch.zeros(1, dtype=torch.int32, device="cuda")
            out = torch.empty_like(x)
            toma.toma_block(desc, 0, x, out, idx, w, ws, status)
            dense = torch.empty((cfg.batch, cfg.n_tiles, gd(toma, cfg), cfg.n_loc), dtype=torch.float32, device="cuda")
            toma.toma_weights_export(desc, w, dense)
            torch.cuda.synchronize()
            assert int(status.item()) == 0
            got[separate] = (idx.cpu().numpy().copy(), dense.cpu().numpy().copy())
        assert np.array_equal(got[0][0], got[1][0]), f"picks differ for seed {seed}"
        assert np.abs(got[0][1] - got[1][1]).max() <= 6e-4, f"weights differ for seed {seed}"


def test_block_separate_weight_schedule_parity(toma):
    """Destinations every 4 steps, weights every 2 (the paper refreshes weights more often than
    destinations): indices stay put at step 2 while the weights follow the drifted features."""
    cfg = gen.config("cfg3", batch=1, steps=5, reuse_interval=4)
    desc = toma.desc_from_config(cfg, weight_reuse_interval=2)
    idx, w, ws = toma.alloc_idx(desc), toma.alloc_weights(desc), toma.alloc_workspace(desc)
    st = O.BlockState()
    kw = dict(grid_h=cfg.grid_h, grid_w=cfg.grid_w, tile_h=cfg.tile_h, tile_w=cfg.tile_w, merge_ratio=cfg.merge_ratio,
              tau=cfg.tau, n_heads=cfg.n_heads, reuse_interval=4, weight_reuse_interval=2)
    for step, x_host in enumerate(gen.feature_sequence(cfg)):
        x = to_dev(x_host, cfg.dtype)
        out = torch.empty_like(x)
        toma.toma_block(desc, step, x, out, idx, w, ws, None)
        torch.cuda.synchronize()
        want, _, _ = O.block_step(x_host, step, st, **kw)
        assert np.array_equal(idx.cpu().numpy().astype(np.int64), st.idx)
        assert_close(to_host64(out), want, cfg.dtype, f"block step {step}")


@pytest.mark.parametrize("streams", [False, True])
def test_block_host_matches_block(toma, streams):
    """toma_block_host (host buffers through the C ABI, copies on the call's streams) returns what
    toma_block returns on the same inputs, with one stream and with separate copy streams."""
    cfg = gen.config("cfg2", batch=1, steps=4, reuse_interval=2)
    desc = toma.desc_from_config(cfg)
    idx, w, ws = toma.alloc_idx(desc), toma.alloc_weights(desc), toma.alloc_workspace(desc)
    idx2, w2, ws2 = toma.alloc_idx(desc), toma.alloc_weights(desc), toma.alloc_workspace(desc)
    s_in = torch.cuda.Stream() if streams else None
    s_out = torch.cuda.Stream() if streams else None
    ev = [torch.cuda.Event() for _ in range(2)] if streams else [None, None]
    for e in ev:
        if e is not None:
            e.record()
    for step, x_host in enumerate(gen.feature_sequence(cfg)):
        xh = torch.from_numpy(x_host).to(torch.bfloat16).pin_memory()
        oh = torch.empty_like(xh).pin_memory()
        x_dev, out_dev = torch.empty_like(xh, device="cuda"), torch.empty_like(xh, device="cuda")
        toma.toma_block_host(desc, step, xh, oh, x_dev, out_dev, idx, w, ws, None, s_in, s_out, ev[0], ev[1])
        x = xh.cuda()
        want = torch.empty_like(x)
        toma.toma_block(desc, step, x, want, idx2, w2, ws2, None)
        torch.cuda.synchronize()
        assert torch.equal(oh, want.cpu())
        assert torch.equal(idx, idx2)


GLOBAL = [
    # grid, tile, dim, heads, dtype: destinations per tile, weights / merge / unmerge over the whole image
    dict(grid_h=32, grid_w=32, tile_h=8, tile_w=8, dim=128, n_heads=2, head_dim=64, dtype="bf16"),
    dict(grid_h=32, grid_w=32, tile_h=8, tile_w=8, dim=128, n_heads=2, head_dim=64, dtype="f32"),
    dict(grid_h=16, grid_w=64, tile_h=4, tile_w=16, dim=64, n_heads=1, head_dim=64, dtype="bf16", merge_ratio=0.75),
    dict(grid_h=16, grid_w=16, tile_h=8, tile_w=8, dim=64, n_heads=1, head_dim=64, dtype="bf16", n_extra=5),
    # 384 channels: a full 320-channel block and a 64-channel one in the tokens-on-M unmerge; 768 destinations
    dict(grid_h=32, grid_w=32, tile_h=16, tile_w=16, dim=384, n_heads=6, head_dim=64, dtype="bf16", merge_ratio=0.25),
]


@pytest.mark.parametrize("over", GLOBAL, ids=[str(i) for i in range(len(GLOBAL))])
def test_global_merge_parity(toma, over):
    """The default ToMA variant (Sec. 5): destinations per tile, then weights, merge and unmerge once over
    all image tokens with the D destinations of the image as one set."""
    cfg = gen.config("cfg2", batch=2, **over)
    x_host = gen.features(cfg)
    run = Run(toma, cfg, x_host, global_merge=True)
    idx = run.select()
    N, D = cfg.n_tokens, cfg.n_tiles * gd(toma, cfg)
    run.t.toma_merge_weights(run.desc, run.x, run.idx, run.w, run.ws, run.status)
    run.ok()
    dense = torch.empty((cfg.batch, 1, D, N), dtype=torch.float32, device="cuda")
    run.t.toma_weights_export(run.desc, run.w, dense)
    torch.cuda.synchronize()
    dense = dense.cpu().numpy().astype(np.float64)
    merged = run.merge()
    y_dev = run.attend()
    unmerged = run.unmerge(y_dev)
    y_host = to_host64(y_dev)
    ids = O.tile_token_ids(cfg.grid_h, cfg.grid_w, cfg.tile_h, cfg.tile_w)
    w_abs = 2e-5 if cfg.dtype == "f32" else 6e-4
    for b in range(cfg.batch):
        for p in range(cfg.n_tiles):
            want_idx, margin = O.select_tile(tile_tokens(cfg, x_host, b, p), od(cfg))
            assert margin > O.FRAGILE_MARGIN
            assert np.array_equal(idx[b, p], want_idx)
        x_img = x_host[b, :N].astype(np.float64)
        w = O.merge_weights(x_img, O.global_destinations(idx[b], ids), cfg.tau)
        assert np.abs(dense[b, 0] - w).max() <= w_abs, "global weights differ"
        assert_close(merged[b, :D], O.merge(w, x_img), cfg.dtype, "global merge")
        assert_close(unmerged[b, :N], O.unmerge(w, y_host[b, :D]), cfg.dtype, "global unmerge")
        if cfg.n_extra:
            assert np.array_equal(merged[b, D:], x_host[b, N:].astype(np.float64))
            assert np.array_equal(unmerged[b, N:], y_host[b, D:])


def test_global_merge_block_parity_at_benchmark_size(toma):
    """toma_block with global merge on the benchmark shape (64x64 tokens, 2048 destinations): a refresh
    step and a reuse step against the oracle."""
    cfg = gen.config("cfg3", batch=1, steps=2, reuse_interval=2)
    desc = toma.desc_from_config(cfg, global_merge=True)
    idx, w, ws = toma.alloc_idx(desc), toma.alloc_weights(desc), toma.alloc_workspace(desc)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    st = O.BlockState()
    kw = dict(grid_h=cfg.grid_h, grid_w=cfg.grid_w, tile_h=cfg.tile_h, tile_w=cfg.tile_w, merge_ratio=cfg.merge_ratio,
              tau=cfg.tau, n_heads=cfg.n_heads, reuse_interval=2, global_merge=True)
    for step, x_host in enumerate(gen.feature_sequence(cfg)):
        x = to_dev(x_host, cfg.dtype)
        out = torch.empty_like(x)
        toma.toma_block(desc, step, x, out, idx, w, ws, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        want, _, _ = O.block_step(x_host, step, st, **kw)
        assert np.array_equal(idx.cpu().numpy().astype(np.int64), st.idx)
        assert_close(to_host64(out), want, cfg.dtype, f"global-merge block step {step}")


SHARES = [
    # name, overrides, global merge
    ("cfg1", {}, False),                                   # fp32, FFMA weights path
    ("cfg2", dict(batch=1), False),                        # 8x8 tiles
    ("cfg3", dict(batch=1), False),                        # the benchmark's tile shape
    ("cfg4", dict(grid_h=32, grid_w=32, n_extra=7), False),  # 3072 channels, 128-wide heads, text tokens
    ("cfg2", dict(batch=2, grid_h=32, grid_w=32, tile_h=8, tile_w=8, dim=128, n_heads=2, head_dim=64), True),
    ("cfg3", dict(batch=1, grid_h=32, grid_w=32, merge_ratio=0.25), True),  # 768 destinations: blocked weights
]


@pytest.mark.parametrize("name,over,global_merge", SHARES, ids=[str(i) for i in range(len(SHARES))])
def test_shares_unmerge_parity(toma, name, over, global_merge):
    """unmerge_mode "shares": toma_unmerge applies A^T, the softmax matrix before row normalisation.  The
    merge side is untouched; the second matrix of the weight buffer is the oracle's A; a constant comes
    back as the same constant (columns of A sum to 1); the unmerged tensor matches the oracle's."""
    cfg = gen.config(name, **over)
    x_host = gen.features(cfg)
    run = Run(toma, cfg, x_host, global_merge=global_merge, unmerge_mode="shares")
    ref = Run(toma, cfg, x_host, global_merge=global_merge)
    assert toma.toma_weights_bytes(run.desc) == 2 * toma.toma_weights_bytes(ref.desc)
    idx = run.select()
    ref.idx.copy_(run.idx)
    N, D = cfg.n_tokens, cfg.n_tiles * gd(toma, cfg)
    shape = (cfg.batch, 1, D, N) if global_merge else (cfg.batch, cfg.n_tiles, gd(toma, cfg), cfg.n_loc)
    for r in (run, ref):
        r.t.toma_merge_weights(r.desc, r.x, r.idx, r.w, r.ws, r.status)
        r.ok()
    nb = toma.toma_weights_bytes(ref.desc)
    assert torch.equal(run.w[:nb], ref.w[:nb]), "the merge matrix must not depend on the unmerge mode"
    dense_u = torch.empty(shape, dtype=torch.float32, device="cuda")
    toma.toma_unmerge_weights_export(run.desc, run.w, dense_u)
    dense_t = torch.empty(shape, dtype=torch.float32, device="cuda")
    toma.toma_unmerge_weights_export(ref.desc, ref.w, dense_t)
    dense_w = torch.empty(shape, dtype=torch.float32, device="cuda")
    toma.toma_weights_export(ref.desc, ref.w, dense_w)
    torch.cuda.synchronize()
    assert torch.equal(dense_t, dense_w), "transpose mode: the unmerge matrix is the merge matrix"
    A = dense_u.cpu().numpy().astype(np.float64)
    assert np.all(A >= 0) and np.abs(A.sum(axis=2) - 1.0).max() < (1e-5 if cfg.dtype == "f32" else 2e-3)
    merged = run.merge()
    assert np.array_equal(merged, ref.merge())
    y_dev = run.attend()
    y_host = to_host64(y_dev)
    unmerged = run.unmerge(y_dev)
    const = torch.full_like(y_dev, 1.5)
    back = run.unmerge(const)
    assert np.abs(back - 1.5).max() <= (1e-5 if cfg.dtype == "f32" else 2 ** -7), "partition of unity"
    ids = O.tile_token_ids(cfg.grid_h, cfg.grid_w, cfg.tile_h, cfg.tile_w)
    w_abs = 2e-5 if cfg.dtype == "f32" else 6e-4
    if global_merge:
        for b in range(cfg.batch):
            x_img = x_host[b, :N].astype(np.float64)
            want = O.softmax_shares(x_img, O.global_destinations(idx[b], ids), cfg.tau)
            assert np.abs(A[b, 0] - want).max() <= w_abs
            assert_close(unmerged[b, :N], O.unmerge(want, y_host[b, :D]), cfg.dtype, "global shares unmerge")
    else:
        got, want_u = [], []
        for b, p in sample_tiles(cfg, 8):
            xt = tile_tokens(cfg, x_host, b, p)
            want = O.softmax_shares(xt, idx[b, p], cfg.tau)
            assert np.abs(A[b, p] - want).max() <= w_abs, f"shares differ in tile ({b},{p})"
            got.append(unmerged[b, ids[p]])
            want_u.append(O.unmerge(want, y_host[b, p * gd(toma, cfg):(p + 1) * gd(toma, cfg)]))
        assert_close(np.stack(got), np.stack(want_u), cfg.dtype, "shares unmerge")
    if cfg.n_extra:
        assert np.array_equal(unmerged[:, N:], y_host[:, D:])


@pytest.mark.parametrize("global_merge", [False, True])
def test_block_with_shares_unmerge_parity(toma, global_merge):
    """toma_block with unmerge_mode "shares" over a refresh, a weights-only and a reuse step."""
    cfg = gen.config("cfg3", batch=1, steps=4, reuse_interval=4, grid_h=32, grid_w=32)
    desc = toma.desc_from_config(cfg, global_merge=global_merge, unmerge_mode="shares", weight_reuse_interval=2)
    idx, w, ws = toma.alloc_idx(desc), toma.alloc_weights(desc), toma.alloc_workspace(desc)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    st = O.BlockState()
    kw = dict(grid_h=cfg.grid_h, grid_w=cfg.grid_w, tile_h=cfg.tile_h, tile_w=cfg.tile_w, merge_ratio=cfg.merge_ratio,
              tau=cfg.tau, n_heads=cfg.n_heads, reuse_interval=4, weight_reuse_interval=2, global_merge=global_merge,
              unmerge_mode="shares")
    for step, x_host in enumerate(gen.feature_sequence(cfg)):
        x = to_dev(x_host, cfg.dtype)
        out = torch.empty_like(x)
        toma.toma_block(desc, step, x, out, idx, w, ws, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        want, _, _ = O.block_step(x_host, step, st, **kw)
        assert np.array_equal(idx.cpu().numpy().astype(np.int64), st.idx)
        assert_close(to_host64(out), want, cfg.dtype, f"shares block step {step}")


@pytest.mark.parametrize("dtype,m,n,k", [
    ("bf16", 4096, 640, 640), ("bf16", 4096, 1920, 640), ("bf16", 1000, 72, 200), ("bf16", 130, 320, 64),
    ("bf16", 128, 328, 640), ("bf16", 2560, 3072, 3072), ("f32", 300, 96, 160),
])
def test_linear_parity(toma, dtype, m, n, k):
    """Projection c = a w through toma_linear: ragged rows, a partial last k-step, partial column blocks."""
    a_host = gen.round_to_dtype(gen.normal(0, (91, m, k), m * k).reshape(m, k).astype(np.float32), dtype)
    w_host = gen.round_to_dtype((gen.normal(0, (92, n, k), k * n).reshape(k, n) / np.sqrt(k)).astype(np.float32), dtype)
    a, w = to_dev(a_host, dtype), to_dev(w_host, dtype)
    c = torch.full((m, n), float("nan"), dtype=a.dtype, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    toma.toma_linear(a, w, c, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    rows = np.unique(np.concatenate([[0, m - 1], np.random.default_rng(m).choice(m, size=min(m, 200), replace=False)]))
    assert not torch.isnan(c).any()
    assert_close(to_host64(c)[rows], O.linear(a_host[rows], w_host), dtype, "linear")


@pytest.mark.parametrize("tile", [0, 1, 2, 3], ids=["128x256", "128x320", "256x256", "128x128"])
@pytest.mark.parametrize("m,n,k", [(300, 328, 200), (129, 1920, 640), (1024, 72, 136), (640, 512, 64)])
def test_linear_every_tile_form(toma, tuning, tile, m, n, k):
    """Each of the projection kernel's four tile forms, forced, on shapes with a ragged last row block (the
    second row block of a 256-row tile partly or wholly past the end), partial column blocks and a partial
    last k-step."""
    tuning(linear_tile=tile + 1)
    a_host = gen.round_to_dtype(gen.normal(0, (191, m, k), m * k).reshape(m, k).astype(np.float32), "bf16")
    w_host = gen.round_to_dtype((gen.normal(0, (192, n, k), k * n).reshape(k, n) / np.sqrt(k)).astype(np.float32), "bf16")
    a, w = to_dev(a_host, "bf16"), to_dev(w_host, "bf16")
    c = torch.full((m, n), float("nan"), dtype=a.dtype, device="cuda")
    guard = torch.full((4096,), 7.0, dtype=a.dtype, device="cuda")  # allocated right after c
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    toma.toma_linear(a, w, c, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert not torch.isnan(c).any()
    assert bool((guard == 7.0).all())
    assert_close(to_host64(c), O.linear(a_host, w_host), "bf16", f"linear, tile form {tile}")


def _proj_weights(cfg, seed=93):
    """Four [d, d] projection matrices N(0, 1/d), rounded to the storage dtype."""
    d = cfg.dim
    return [gen.round_to_dtype((gen.normal(0, (seed, i, d), d * d).reshape(d, d) / np.sqrt(d)).astype(np.float32), cfg.dtype)
            for i in range(4)]


def _storage_rounding(dtype):
    return (lambda t: gen.round_to_dtype(np.asarray(t, dtype=np.float32), dtype).astype(np.float64)) if dtype == "bf16" \
        else (lambda t: np.asarray(t, dtype=np.float32).astype(np.float64))


@pytest.mark.parametrize("name,over", [("cfg2", dict(batch=1)), ("cfg3", dict(batch=1)), ("cfg1", {}),
                                       ("cfg2", dict(batch=1, grid_h=16, grid_w=16, n_extra=9))],
                         ids=["cfg2", "cfg3", "cfg1-f32", "extra-tokens"])
def test_block_with_projections_parity(toma, name, over):
    """toma_block_proj: the wrapped module is the whole attention module (Q/K/V projections, attention, output
    projection) on the merged tokens.  Primary assertion: the plain fp64 chain of the oracle, no rounding
    anywhere.  Secondary (labelled) assertion: the oracle with the storage rounding of the kernels mirrored
    between stages, which isolates arithmetic differences from the six bf16 roundings on the way."""
    cfg = gen.config(name, steps=2, reuse_interval=2, **over)
    desc = toma.desc_from_config(cfg)
    w_host = _proj_weights(cfg)
    w_dev = [to_dev(w, cfg.dtype) for w in w_host]
    idx, w, ws = toma.alloc_idx(desc), toma.alloc_weights(desc), toma.alloc_workspace(desc)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    st, st_mirror = O.BlockState(), O.BlockState()
    kw = dict(grid_h=cfg.grid_h, grid_w=cfg.grid_w, tile_h=cfg.tile_h, tile_w=cfg.tile_w, merge_ratio=cfg.merge_ratio,
              tau=cfg.tau, n_heads=cfg.n_heads, reuse_interval=2, n_extra=cfg.n_extra,
              proj=[x.astype(np.float64) for x in w_host])
    for step, x_host in enumerate(gen.feature_sequence(cfg)):
        x = to_dev(x_host, cfg.dtype)
        out = torch.empty_like(x)
        toma.toma_block_proj(desc, step, x, *w_dev, out, idx, w, ws, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        want, _, _ = O.block_step(x_host, step, st, **kw)
        assert np.array_equal(idx.cpu().numpy().astype(np.int64), st.idx)
        err = assert_close(to_host64(out), want, cfg.dtype, f"block with projections vs the plain fp64 oracle, step {step}")
        mirrored, _, _ = O.block_step(x_host, step, st_mirror, round_fn=_storage_rounding(cfg.dtype), **kw)
        err_m = assert_close(to_host64(out), mirrored, cfg.dtype, f"[secondary: storage rounding mirrored] step {step}")
        print(f"block_proj {name} step {step}: plain max-abs {err[0]:.3g} rel-fro {err[1]:.3g}; mirrored {err_m[0]:.3g} {err_m[1]:.3g}")


@pytest.mark.parametrize("dtype,B,L,h,dh", [("bf16", 2, 1024, 10, 64), ("bf16", 1, 600, 3, 128), ("f32", 1, 200, 2, 64)])
def test_attention_module_with_projections_parity(toma, dtype, B, L, h, dh):
    """toma_attention_proj (the full-token baseline of toma_block_proj) against the oracle."""
    d = h * dh
    cfg = gen.config("cfg2", batch=B, dim=d, n_heads=h, head_dim=dh, dtype=dtype)
    x_host = gen.round_to_dtype(gen.normal(0, (94, L, d), B * L * d).reshape(B, L, d).astype(np.float32), dtype)
    w_host = _proj_weights(cfg, seed=95)
    x, w_dev = to_dev(x_host, dtype), [to_dev(w, dtype) for w in w_host]
    out = torch.empty_like(x)
    ws = torch.empty(toma.toma_attention_proj_workspace_bytes(B, L, h, dh, dtype), dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    toma.toma_attention_proj(B, L, h, dh, dtype, x, *w_dev, out, ws, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    rnd = _storage_rounding(dtype)
    got = to_host64(out)
    for b in range(B):
        q, k, v = (O.linear(x_host[b], w) for w in w_host[:3])
        assert_close(got[b], O.linear(O.attention(q, k, v, h), w_host[3]), dtype, f"attention module vs the plain fp64 chain, b={b}")
        q, k, v = (rnd(O.linear(x_host[b], w)) for w in w_host[:3])
        want = O.linear(rnd(O.attention(q, k, v, h)), w_host[3])
        assert_close(got[b], want, dtype, f"[secondary: storage rounding mirrored] attention module b={b}")


def _mlp_weights(cfg, hidden, seed=97):
    """w1 [d, f] ~ N(0, 1/d) and w2 [f, d] ~ N(0, 1/f), rounded to the storage dtype."""
    d = cfg.dim
    w1 = gen.normal(0, (seed, 1, d, hidden), d * hidden).reshape(d, hidden) / np.sqrt(d)
    w2 = gen.normal(0, (seed, 2, d, hidden), d * hidden).reshape(hidden, d) / np.sqrt(hidden)
    return [gen.round_to_dtype(w.astype(np.float32), cfg.dtype) for w in (w1, w2)]


@pytest.mark.parametrize("dtype,rows,d,f", [("bf16", 2048, 640, 2560), ("bf16", 300, 128, 512), ("bf16", 1000, 64, 40),
                                            ("f32", 130, 64, 96)])
def test_mlp_parity(toma, dtype, rows, d, f):
    """toma_mlp (the full-token baseline of toma_block_mlp): GELU(x w1) w2 against the oracle, which rounds the
    hidden tensor to the storage dtype as the kernels do."""
    cfg = gen.config("cfg2", batch=1, dim=d, n_heads=1, head_dim=d, dtype=dtype)
    x_host = gen.round_to_dtype(gen.normal(0, (98, rows, d), rows * d).reshape(rows, d).astype(np.float32), dtype)
    w_host = _mlp_weights(cfg, f)
    x, w1, w2 = to_dev(x_host, dtype), to_dev(w_host[0], dtype), to_dev(w_host[1], dtype)
    out = torch.empty_like(x)
    ws = torch.empty(toma.toma_mlp_workspace_bytes(rows, d, f, dtype), dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    toma.toma_mlp(rows, d, f, dtype, x, w1, w2, out, ws, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    pick = np.unique(np.concatenate([[0, rows - 1], np.random.default_rng(rows).choice(rows, size=min(rows, 160), replace=False)]))
    assert_close(to_host64(out)[pick], O.mlp(x_host[pick], w_host[0], w_host[1]), dtype, "mlp vs the plain fp64 chain")
    want = O.mlp(x_host[pick], w_host[0], w_host[1], _storage_rounding(dtype))
    assert_close(to_host64(out)[pick], want, dtype, "[secondary: storage rounding mirrored] mlp")
    # the hidden tensor itself: GELU of the first projection, in storage dtype
    hid = ws[: rows * f * (4 if dtype == "f32" else 2)].view(torch.float32 if dtype == "f32" else torch.bfloat16).reshape(rows, f)
    assert_close(to_host64(hid)[pick], O.gelu(O.linear(x_host[pick], w_host[0])), dtype, "mlp hidden")


@pytest.mark.parametrize("name,over,hidden", [("cfg2", dict(batch=1), 5120), ("cfg3", dict(batch=1), 2560), ("cfg1", {}, 320),
                                              ("cfg2", dict(batch=1, grid_h=16, grid_w=16, n_extra=9), 1288)],
                         ids=["cfg2", "cfg3", "cfg1-f32", "extra-tokens"])
def test_block_with_mlp_parity(toma, name, over, hidden):
    """toma_block_mlp: the wrapped module is the MLP on the merged tokens; a refresh step and a reuse step.
    Primary assertion: the plain fp64 chain; secondary (labelled): storage rounding mirrored between stages."""
    cfg = gen.config(name, steps=2, reuse_interval=2, **over)
    desc = toma.desc_from_config(cfg)
    w_host = _mlp_weights(cfg, hidden)
    w1, w2 = (to_dev(w, cfg.dtype) for w in w_host)
    idx, w, ws = toma.alloc_idx(desc), toma.alloc_weights(desc), toma.alloc_workspace(desc)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    st, st_mirror = O.BlockState(), O.BlockState()
    kw = dict(grid_h=cfg.grid_h, grid_w=cfg.grid_w, tile_h=cfg.tile_h, tile_w=cfg.tile_w, merge_ratio=cfg.merge_ratio,
              tau=cfg.tau, n_heads=cfg.n_heads, reuse_interval=2, n_extra=cfg.n_extra,
              mlp_weights=[x.astype(np.float64) for x in w_host])
    for step, x_host in enumerate(gen.feature_sequence(cfg)):
        x = to_dev(x_host, cfg.dtype)
        out = torch.empty_like(x)
        toma.toma_block_mlp(desc, step, x, w1, w2, out, idx, w, ws, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        want, _, _ = O.block_step(x_host, step, st, **kw)
        assert np.array_equal(idx.cpu().numpy().astype(np.int64), st.idx)
        err = assert_close(to_host64(out), want, cfg.dtype, f"block with MLP vs the plain fp64 oracle, step {step}")
        mirrored, _, _ = O.block_step(x_host, step, st_mirror, round_fn=_storage_rounding(cfg.dtype), **kw)
        err_m = assert_close(to_host64(out), mirrored, cfg.dtype, f"[secondary: storage rounding mirrored] step {step}")
        print(f"block_mlp {name} step {step}: plain max-abs {err[0]:.3g} rel-fro {err[1]:.3g}; mirrored {err_m[0]:.3g} {err_m[1]:.3g}")
    # a hidden width beyond four times the model width does not fit the block's workspace
    wide = torch.zeros((cfg.dim, 4 * cfg.dim + 8), dtype=x.dtype, device="cuda")
    with pytest.raises(toma.TomaError):
        toma.toma_block_mlp(desc, 0, x, wide, w2, out, idx, w, ws, status)


def test_block_replays_from_a_cuda_graph(toma):
    """A reuse step and a refresh step captured into CUDA graphs (the calls never allocate or synchronise,
    and their dependent launches are capturable) replay to the same bits as direct calls."""
    cfg = gen.config("cfg3", batch=1, steps=3, reuse_interval=2)
    desc = toma.desc_from_config(cfg)
    xs = [to_dev(x, cfg.dtype) for x in gen.feature_sequence(cfg)]
    idx, w, ws = toma.alloc_idx(desc), toma.alloc_weights(desc), toma.alloc_workspace(desc)
    idx2, w2, ws2 = toma.alloc_idx(desc), toma.alloc_weights(desc), toma.alloc_workspace(desc)
    x_in, out = torch.empty_like(xs[0]), torch.empty_like(xs[0])
    x_in.copy_(xs[0])
    toma.toma_block(desc, 0, x_in, out, idx, w, ws, None)  # first call outside capture (one-time attribute setup)
    toma.toma_block(desc, 1, x_in, out, idx, w, ws, None)
    torch.cuda.synchronize()
    graphs = {}
    for step in (0, 1):
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            toma.toma_block(desc, step, x_in, out, idx, w, ws, None)
        graphs[step] = g
    for t, x in enumerate(xs):
        x_in.copy_(x)
        graphs[t % 2].replay()
        want = torch.empty_like(x)
        toma.toma_block(desc, t, x, want, idx2, w2, ws2, None)
        torch.cuda.synchronize()
        assert torch.equal(out, want), f"graph replay differs at step {t}"
        assert torch.equal(idx, idx2)


def test_stripe_regions_full_size_parity(toma):
    """Stripe regions (Sec. 4.3.1) at the benchmark size: 64x64 tokens cut into stripes of 4 full rows,
    under the schedule the paper settles on (destinations every 10 steps, weights every 5)."""
    cfg = gen.config("cfg3", batch=1, tile_h=4, tile_w=64, steps=7, reuse_interval=10)
    desc = toma.desc_from_config(cfg, weight_reuse_interval=5)
    idx, w, ws = toma.alloc_idx(desc), toma.alloc_weights(desc), toma.alloc_workspace(desc)
    st = O.BlockState()
    kw = dict(grid_h=cfg.grid_h, grid_w=cfg.grid_w, tile_h=4, tile_w=64, merge_ratio=cfg.merge_ratio, tau=cfg.tau,
              n_heads=cfg.n_heads, reuse_interval=10, weight_reuse_interval=5)
    for step, x_host in enumerate(gen.feature_sequence(cfg)):
        x = to_dev(x_host, cfg.dtype)
        out = torch.empty_like(x)
        toma.toma_block(desc, step, x, out, idx, w, ws, None)
        torch.cuda.synchronize()
        if step in (0, 5, 6):  # refresh, weights-only refresh, reuse after it
            want, _, _ = O.block_step(x_host, step, st, **kw)
            assert np.array_equal(idx.cpu().numpy().astype(np.int64), st.idx)
            assert_close(to_host64(out), want, cfg.dtype, f"stripe block step {step}")
        else:  # keep the oracle's state in step without paying for its attention
            assert step % 5 != 0


def test_block_long_sequence_schedule_and_sampled_parity(toma):
    """The 28-step stress sequence: selection may only change on refresh steps, and sampled
    tiles of every refresh match the oracle exactly."""
    cfg = gen.config("cfg5a", batch=1, steps=12)
    desc = toma.desc_from_config(cfg)
    idx = toma.alloc_idx(desc)
    w = toma.alloc_weights(desc)
    ws = toma.alloc_workspace(desc)
    prev = None
    tiles = sample_tiles(cfg, 4)
    for step, x_host in enumerate(gen.feature_sequence(cfg)):
        x = to_dev(x_host, cfg.dtype)
        out = torch.empty_like(x)
        toma.toma_block(desc, step, x, out, idx, w, ws, None)
        torch.cuda.synchronize()
        cur = idx.cpu().numpy().astype(np.int64)
        if step % cfg.reuse_interval == 0:
            for b, p in tiles:
                want, margin = O.select_tile(tile_tokens(cfg, x_host, b, p), od(cfg))
                assert margin > O.FRAGILE_MARGIN
                assert np.array_equal(cur[b, p], want)
        else:
            assert np.array_equal(cur, prev), "selection changed on a reuse step"
        prev = cur
        assert torch.isfinite(out.float()).all()


@pytest.mark.parametrize("name", ["cfg5a", "cfg5b"])
def test_block_output_sampled_parity_at_the_largest_sizes(toma, name):
    """The whole chain merge -> attention over 8192 merged tokens -> unmerge at the stress sizes, element by
    element on sampled tiles, for a refresh step and the reuse step after it.  The oracle cannot run the whole
    batch in reasonable time, so: the destinations of the sampled tiles are checked against the oracle bit for
    bit; weights and merged tokens of every tile of the sampled batch items are computed by the oracle from the
    destinations; the attention is evaluated at the merged rows of the sampled tiles only (all keys); those rows
    are unmerged and compared with the library's output for the tile's tokens."""
    cfg = gen.config(name, steps=2)
    desc = toma.desc_from_config(cfg)
    idx, w, ws = toma.alloc_idx(desc), toma.alloc_weights(desc), toma.alloc_workspace(desc)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    ids = O.tile_token_ids(cfg.grid_h, cfg.grid_w, cfg.tile_h, cfg.tile_w)
    d_loc = od(cfg)
    assert d_loc == gd(toma, cfg)
    sampled = {0: [0, cfg.n_tiles // 2 + 1], cfg.batch - 1: [cfg.n_tiles - 1]}
    weights = {}
    for step, x_host in enumerate(gen.feature_sequence(cfg)):
        x = to_dev(x_host, cfg.dtype)
        out = torch.empty_like(x)
        toma.toma_block(desc, step, x, out, idx, w, ws, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        got_idx = idx.cpu().numpy().astype(np.int64)
        got = to_host64(out)
        for b, tiles in sampled.items():
            xb = x_host[b].astype(np.float64)
            if step == 0:
                for p in tiles:
                    want_idx, margin = O.select_tile(xb[ids[p]], d_loc)
                    assert margin > O.FRAGILE_MARGIN
                    assert np.array_equal(got_idx[b, p], want_idx), f"{name}: selection of tile {p} differs"
                weights[b] = [O.merge_weights(xb[ids[p]], got_idx[b, p], cfg.tau) for p in range(cfg.n_tiles)]
            merged = np.concatenate([O.merge(weights[b][p], xb[ids[p]]) for p in range(cfg.n_tiles)])
            for p in tiles:
                rows = np.arange(p * d_loc, (p + 1) * d_loc)
                att = O.attention(merged, merged, merged, cfg.n_heads, query_rows=rows)
                assert_close(got[b][ids[p]], O.unmerge(weights[b][p], att), cfg.dtype, f"{name} step {step} b={b} tile {p}")


def test_unmerge_does_not_read_the_next_tile(toma):
    """D_loc = 24 (a multiple of 8 but not of 16, the tensor cores' step along destinations) and a NaN planted
    in every tile's successor rows of the unmerge input: a tile's output may depend on its own D_loc rows only."""
    cfg = gen.config("cfg2", batch=1, grid_h=16, grid_w=16, dim=128, n_heads=2, merge_ratio=0.625)
    assert gd(toma, cfg) == 24 and od(cfg) == 24
    x_host = gen.features(cfg)
    run = Run(toma, cfg, x_host)
    idx = run.select()
    wts = run.weights()
    y_host = gen.round_to_dtype(0.25 * gen.normal(0, (41, 24), cfg.n_tiles * 24 * cfg.dim).reshape(1, -1, cfg.dim).astype(np.float32), "bf16")
    ids = O.tile_token_ids(cfg.grid_h, cfg.grid_w, cfg.tile_h, cfg.tile_w)
    for p in range(cfg.n_tiles - 1):
        y = y_host.copy()
        y[0, (p + 1) * 24:(p + 1) * 24 + 8] = np.nan    # the rows a 16-wide step would read past tile p
        got = run.unmerge(to_dev(y, cfg.dtype))
        want = O.unmerge(O.merge_weights(x_host[0][ids[p]], idx[0, p], cfg.tau), y_host[0, p * 24:(p + 1) * 24])
        assert np.isfinite(got[0][ids[p]]).all(), f"tile {p} picked up a value of tile {p + 1}"
        assert_close(got[0][ids[p]], want, cfg.dtype, f"unmerge tile {p}")
        if p >= 2:
            break


def test_identity_weights_round_trip_is_bit_exact(toma):
    for dtype in ("bf16", "f32"):
        cfg = gen.config("cfg2", batch=1, grid_h=16, grid_w=16, dim=128, n_heads=2, merge_ratio=0.0, dtype=dtype)
        assert gd(toma, cfg) == cfg.n_loc
        x_host = gen.features(cfg)
        run = Run(toma, cfg, x_host)
        eye = torch.eye(cfg.n_loc, dtype=torch.float32, device="cuda").repeat(cfg.batch, cfg.n_tiles, 1, 1).contiguous()
        toma.toma_weights_import(run.desc, eye, run.w)
        merged = run.merge()
        ids = O.tile_token_ids(cfg.grid_h, cfg.grid_w, cfg.tile_h, cfg.tile_w)
        assert np.array_equal(merged[0], x_host[0][ids.reshape(-1)].astype(np.float64))
        back = run.unmerge(run.xm)
        assert np.array_equal(back, x_host.astype(np.float64))


EDGE = [
    dict(grid_h=12, grid_w=12, tile_h=6, tile_w=6, dim=64, n_heads=1, merge_ratio=0.5),      # N_loc = 36, not a warp multiple
    dict(grid_h=16, grid_w=32, tile_h=2, tile_w=32, dim=128, n_heads=2, merge_ratio=0.5),    # stripes
    dict(grid_h=16, grid_w=16, tile_h=8, tile_w=16, dim=64, n_heads=1, merge_ratio=0.99),    # one destination per tile
    dict(grid_h=16, grid_w=16, tile_h=16, tile_w=8, dim=72, n_heads=1, head_dim=72, merge_ratio=0.3),  # odd dim, ragged D_loc
    dict(grid_h=8, grid_w=8, tile_h=8, tile_w=8, dim=64, n_heads=1, merge_ratio=0.0),        # keep everything
    dict(grid_h=16, grid_w=16, tile_h=8, tile_w=8, dim=64, n_heads=1, merge_ratio=0.5, n_extra=7),
    dict(grid_h=16, grid_w=16, tile_h=8, tile_w=8, dim=4096, n_heads=32, head_dim=128, merge_ratio=0.5),  # widest supported token
    dict(grid_h=16, grid_w=16, tile_h=8, tile_w=8, dim=16, n_heads=1, head_dim=16, merge_ratio=0.5),     # narrow token
]


@pytest.mark.parametrize("over", EDGE, ids=[str(i) for i in range(len(EDGE))])
@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_edge_shapes(toma, over, dtype):
    cfg = gen.config("cfg2", batch=2, dtype=dtype, **over)
    x_host = gen.features(cfg)
    run = Run(toma, cfg, x_host)
    idx = run.select()
    dense = run.weights()
    merged = run.merge()
    # unmerge input: the merged tokens scaled by 1/4 (exact in both dtypes).  A source token that is
    # split between destinations whose rows carry little mass has unmerge weights summing above 1, and
    # values >= 8 cannot be stored in bf16 within 2e-2 by anyone; the scaling keeps them below that.
    y_dev = (run.xm.float() * 0.25).to(run.xm.dtype)
    unmerged = run.unmerge(y_dev)
    y_host = to_host64(y_dev)
    ids = O.tile_token_ids(cfg.grid_h, cfg.grid_w, cfg.tile_h, cfg.tile_w)
    for b in range(cfg.batch):
        for p in range(cfg.n_tiles):
            xt = tile_tokens(cfg, x_host, b, p)
            want_idx, margin = O.select_tile(xt, od(cfg))
            assert margin > O.FRAGILE_MARGIN
            assert np.array_equal(idx[b, p], want_idx)
            w = O.merge_weights(xt, want_idx, cfg.tau)
            assert np.abs(dense[b, p] - w).max() <= (2e-5 if dtype == "f32" else 6e-4)
            sl = slice(p * gd(toma, cfg), (p + 1) * gd(toma, cfg))
            assert_close(merged[b, sl], O.merge(w, xt), dtype, "merge")
            assert_close(unmerged[b, ids[p]], O.unmerge(w, y_host[b, sl]), dtype, "unmerge")


def test_degenerate_inputs_identical_and_zero_tokens(toma):
    cfg = gen.config("cfg2", batch=1, grid_h=8, grid_w=16, tile_h=8, tile_w=8, dim=64, n_heads=1)
    x_host = np.zeros((1, 128, 64), dtype=np.float32)
    x_host[0, :, :] = np.linspace(-1, 1, 64, dtype=np.float32)[None, :]   # all tokens identical
    ids = O.tile_token_ids(8, 16, 8, 8)
    x_host[0, ids[1][5]] = 0.0                                             # one zero-norm token in tile 1
    x_host = gen.round_to_dtype(x_host, "bf16")
    run = Run(toma, cfg, x_host)
    idx = run.select()
    assert list(idx[0, 0]) == list(range(32))                              # ties resolve to the lowest index
    for p in range(2):
        want, _ = O.select_tile(tile_tokens(cfg, x_host, 0, p), od(cfg))
        assert np.array_equal(idx[0, p], want)
    # the same through a refresh step of toma_block, which runs selection and weights of 64-token tiles as one
    # kernel with a one-warp greedy: the same picks, weights against Sec. 4.2.1, finite output
    desc = toma.desc_from_config(cfg)
    idx_b, w_b, ws_b = toma.alloc_idx(desc), toma.alloc_weights(desc), toma.alloc_workspace(desc)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    x = to_dev(x_host, cfg.dtype)
    out = torch.full_like(x, float("nan"))
    toma.toma_block(desc, 0, x, out, idx_b, w_b, ws_b, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert np.array_equal(idx_b.cpu().numpy().astype(np.int64), idx)
    dense = torch.empty((1, 2, 32, 64), dtype=torch.float32, device="cuda")
    toma.toma_weights_export(desc, w_b, dense)
    torch.cuda.synchronize()
    for p in range(2):
        want_w = O.merge_weights(tile_tokens(cfg, x_host, 0, p), idx[0, p], cfg.tau)
        assert np.abs(dense[0, p].cpu().numpy().astype(np.float64) - want_w).max() <= 6e-4
    assert torch.isfinite(out.float()).all()


def test_results_are_deterministic(toma):
    cfg = gen.config("cfg3", batch=1)
    x_host = gen.features(cfg)
    a = Run(toma, cfg, x_host)
    b = Run(toma, cfg, x_host)
    ia, ib = a.select(), b.select()
    assert np.array_equal(ia, ib)
    wa, wb = a.weights(), b.weights()
    assert np.array_equal(wa, wb)
    assert np.array_equal(a.merge(), b.merge())

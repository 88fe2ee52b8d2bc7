"""CPU oracle for the ToMA per-block token-reduction path (TEST INFRASTRUCTURE).

A plain, slow, fp64 restatement of what the paper defines, step by step, with
no blocking, fusion or reordering.  It exists only so tests, the smoke check
and the benchmark's CPU-baseline leg can compare the CUDA path against it.  It
shares no code with the CUDA path and the product never calls it.

Every function names the passage of the paper it follows.  Where the paper is
silent or ambiguous the reading taken is stated in the docstring.

Parity status: the functions below are pinned by brute-force enumeration,
closed forms and invariants (see tests/test_oracle_*.py).  The paper prints no
worked numeric example, so the *values* selected/merged on the benchmark
configs are pinned only through those properties.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import List, Optional, Tuple

import numpy as np

# ----------------------------------------------------------------------------
# Region split (Algorithm 3, "Split into local regions"; Sec. 4.3.1 tile-shaped
# regions)
# ----------------------------------------------------------------------------


def tile_token_ids(grid_h: int, grid_w: int, tile_h: int, tile_w: int) -> np.ndarray:
    """int64 [P, N_loc]: global token id of local slot l in tile p.

    Token n = y*W + x belongs to tile p = (y // th) * (W // tw) + (x // tw) and
    has local index l = (y % th) * tw + (x % tw).  Regions must be equal sized
    (Algorithm 3 requires N_loc * P = N).
    """
    if grid_h % tile_h or grid_w % tile_w:
        raise ValueError("tiles must divide the grid")
    ids = np.arange(grid_h * grid_w, dtype=np.int64).reshape(grid_h // tile_h, tile_h, grid_w // tile_w, tile_w)
    return ids.transpose(0, 2, 1, 3).reshape(-1, tile_h * tile_w)


def split_regions(x: np.ndarray, grid_h: int, grid_w: int, tile_h: int, tile_w: int) -> np.ndarray:
    """[N, d] -> [P, N_loc, d] (Algorithm 3: X.reshape(B*P, N_loc, d) for 2-D tiles)."""
    return x[tile_token_ids(grid_h, grid_w, tile_h, tile_w)]


def dest_count(n_loc: int, merge_ratio: float) -> int:
    """Destinations per region.  `merge_ratio` is the fraction of tokens REMOVED
    (the reading under which the paper's tables get faster as the ratio grows,
    App. F: D = (1 - r) N)."""
    # half-way cases round up; the ratio is taken at float32 precision like the C descriptor field
    d_loc = n_loc - int(np.floor(float(np.float32(merge_ratio)) * n_loc + 0.5))
    if d_loc < 1 or d_loc > n_loc:
        raise ValueError("merge ratio leaves no destination")
    return d_loc


# ----------------------------------------------------------------------------
# Facility location (Eq. 2) and greedy selection (Algorithms 1 and 2)
# ----------------------------------------------------------------------------


def facility_location(S: np.ndarray, subset) -> float:
    """f_FL(D) = sum_i max_{j in D} S_ij  (Eq. 2).  f(empty set) is taken as 0."""
    subset = list(subset)
    if not subset:
        return 0
    return S[:, subset].max(axis=1).sum()


def cosine_similarity(x: np.ndarray) -> np.ndarray:
    """S_ij = cos(X_i, X_j) in fp64 (Sec. 4.1) -- the *definition*, used to
    report how faithful the fixed-point similarity below is."""
    x = np.asarray(x, dtype=np.float64)
    n = np.sqrt((x * x).sum(axis=1))
    xn = x / np.maximum(n, 1e-30)[:, None]
    return xn @ xn.T


# Fixed-point cosine similarity -------------------------------------------------
#
# The paper fixes no precision for S, and a floating-point greedy is not
# reproducible across implementations: the facility-location gain has exact
# structural ties, so rounding order decides picks and one flip cascades.  The
# reading taken here makes the similarity an exact integer quantity:
#
#   n_i   = sqrt(sum_c x_ic^2)                               (fp64)
#   k_ic  = rint(x_ic * (COS_SCALE*4096 / max(n_i, 1e-30)))  (fp64, ties-to-even)
#   k_ic <- k_ic rounded to 8 significant bits (ties-to-even), so that
#           k_ic * 2^-12 is exactly representable in bf16
#   K_ij  = sum_c k_ic k_jc                                  (exact integer, < 2^24)
#   S_q   = rint(K_ij / 4096) for i != j  (ties-to-even), units of 2^-12
#   S_q[i][i] = rint(COS_SCALE^2 * 4096) = 4014 for every i
#
# COS_SCALE = 0.99 keeps every |K_ij| below 2^24 for d <= 4096, so an fp32
# accumulation of the bf16 values in ANY order reproduces K_ij exactly.

COS_SCALE = 0.99
Q_ONE = 4096
DIAG_Q = 4014  # rint(0.99^2 * 4096)
FRAGILE_MARGIN = 2.0 ** -30


def _round_to_8_significant_bits(k: np.ndarray) -> np.ndarray:
    a = np.abs(k).astype(np.int64)
    nbits = np.where(a > 0, np.frexp(a.astype(np.float64))[1], 0).astype(np.int64)
    sh = np.maximum(nbits - 8, 0)
    q = a >> sh
    rem = a - (q << sh)
    half = (np.int64(1) << sh) >> 1
    up = (rem > half) | ((rem == half) & (sh > 0) & ((q & 1) == 1))
    q = q + up.astype(np.int64)
    return np.sign(k).astype(np.int64) * (q << sh)


def quantise_tokens(x: np.ndarray) -> Tuple[np.ndarray, float]:
    """int64 [n, d] integer directions k (units 2^-12) and the smallest distance
    of any rint argument from a half-integer (a margin below FRAGILE_MARGIN
    means a different fp64 summation order could flip a rounding)."""
    x = np.asarray(x, dtype=np.float64)
    norm = np.sqrt((x * x).sum(axis=1))
    scale = (COS_SCALE * 4096.0) / np.maximum(norm, 1e-30)
    arg = x * scale[:, None]
    margin = float(np.abs(np.abs(arg - np.floor(arg)) - 0.5).min()) if arg.size else 1.0
    k = np.rint(arg).astype(np.int64)
    return _round_to_8_significant_bits(k), margin


def round_gram(K: np.ndarray) -> np.ndarray:
    """rint(K / 4096) with ties to even, in integer arithmetic: the step that turns the exact integer
    Gram entries K_ij (units of 2^-24) into the similarities S_q (units of 2^-12)."""
    K = np.asarray(K, dtype=np.int64)
    q = K >> 12            # floor(K / 4096)
    rem = K - (q << 12)    # in [0, 4096)
    up = (rem > 2048) | ((rem == 2048) & ((q & 1) == 1))
    return (q + up).astype(np.int32)


def pinned_similarity(x: np.ndarray) -> Tuple[np.ndarray, float]:
    """int32 [n, n] fixed-point cosine similarity S_q (units of 2^-12) of one
    region, plus the quantisation margin (see quantise_tokens)."""
    k, margin = quantise_tokens(x)
    K = k @ k.T  # exact in int64
    if np.abs(K).max(initial=0) >= (1 << 24):
        raise ValueError("Gram entry does not fit 24 bits; input outside the supported range")
    S = round_gram(K)
    np.fill_diagonal(S, DIAG_Q)
    return S, margin


def greedy_select(S: np.ndarray, n_select: int) -> np.ndarray:
    """Greedy facility-location selection (Algorithm 2), in pick order.

    * first pick: argmax_i sum_j S_ij;  m <- S[t1]
    * then n_select-1 rounds: g_i = sum_j max(0, S_ij - m_j) for unselected i;
      pick argmax;  m <- max(m, S[t])
    Already selected indices are excluded from the argmax explicitly (the
    algorithm's "argmax over i not in d"); ties go to the lowest index.
    """
    S = np.asarray(S)
    n = S.shape[0]
    if not (1 <= n_select <= n):
        raise ValueError("n_select out of range")
    acc = np.int64 if np.issubdtype(S.dtype, np.integer) else np.float64
    selected = np.zeros(n, dtype=bool)
    picks = np.empty(n_select, dtype=np.int64)
    t = int(np.argmax(S.sum(axis=1, dtype=acc)))  # np.argmax returns the first maximum
    picks[0] = t
    selected[t] = True
    m = S[t].astype(acc).copy()
    for r in range(1, n_select):
        gain = np.maximum(S.astype(acc) - m[None, :], 0).sum(axis=1)
        cand = np.flatnonzero(~selected)
        t = int(cand[np.argmax(gain[cand])])
        picks[r] = t
        selected[t] = True
        m = np.maximum(m, S[t].astype(acc))
    return picks


def select_tile(x_tile: np.ndarray, d_loc: int) -> Tuple[np.ndarray, float]:
    """Destinations of one region from its tokens [N_loc, d]: fixed-point
    similarity then Algorithm 2.  Returns (local indices in pick order, margin)."""
    S, margin = pinned_similarity(x_tile)
    return greedy_select(S, d_loc), margin


def select_tile_definition(x_tile: np.ndarray, d_loc: int) -> np.ndarray:
    """Algorithm 2 on the fp64 cosine matrix (fidelity reporting only)."""
    return greedy_select(cosine_similarity(x_tile), d_loc)


# ----------------------------------------------------------------------------
# Merge weights, merge, unmerge (Sec. 4.2.1, 4.2.2; Algorithm 3 steps 2 and 3)
# ----------------------------------------------------------------------------


def softmax_shares(x_tile: np.ndarray, idx: np.ndarray, tau: float) -> np.ndarray:
    """A [D_loc, N_loc] for one region: the softmax of Sec. 4.2.1 before its rows are normalised.

    logits  L_ik = <X[idx_i], X_k> / (tau * sqrt(d));  A_ik = softmax over the destination axis i,
    separately for every source token k, so every column of A sums to 1.
    """
    x = np.asarray(x_tile, dtype=np.float64)
    d = x.shape[1]
    dest = x[np.asarray(idx, dtype=np.int64)]
    L = (dest @ x.T) / (tau * np.sqrt(float(d)))
    L = L - L.max(axis=0, keepdims=True)
    E = np.exp(L)
    return E / E.sum(axis=0, keepdims=True)


def merge_weights(x_tile: np.ndarray, idx: np.ndarray, tau: float) -> np.ndarray:
    """A~ [D_loc, N_loc] for one region.

    logits  L_ik = <X[idx_i], X_k> / (tau * sqrt(d))   (SDPA scaling of Eq. 1,
                   raw un-normalised features; Sec. 4.2.1)
    A_ik    = softmax over the DESTINATION axis i, separately for every source
              token k (the paper's "column-wise" softmax: a token is split into
              shares that sum to 1)
    A~_ik   = A_ik / sum_k' A_ik'  (row normalisation; Algorithm 3, A / A.sum(-1))
    """
    A = softmax_shares(x_tile, idx, tau)
    Z = A.sum(axis=1, keepdims=True)
    return A / Z


def merge(w: np.ndarray, x_tile: np.ndarray) -> np.ndarray:
    """X_merged = A~ X  (Sec. 4.2.1)."""
    return np.asarray(w, dtype=np.float64) @ np.asarray(x_tile, dtype=np.float64)


def unmerge(w: np.ndarray, y_tile: np.ndarray) -> np.ndarray:
    """X'_unmerged = A~^T X'  (Sec. 4.2.2, transpose unmerge).

    Passing the column-stochastic A of softmax_shares instead of A~ gives the "shares" variant: every
    source token receives the convex combination sum_i A_ik X'_i of the destinations' outputs."""
    return np.asarray(w, dtype=np.float64).T @ np.asarray(y_tile, dtype=np.float64)


# ----------------------------------------------------------------------------
# Attention over the merged tokens (Eq. 1 with tau = 1, per head)
# ----------------------------------------------------------------------------


def linear(a: np.ndarray, w: np.ndarray) -> np.ndarray:
    """Projection c = a w (the Q/K/V and output maps of the wrapped attention module; App. C's 4 d^2 N
    term): a [m, k], w [k, n] -> [m, n], fp64."""
    return np.asarray(a, dtype=np.float64) @ np.asarray(w, dtype=np.float64)


_erf = np.vectorize(math.erf, otypes=[np.float64])


def gelu(v: np.ndarray) -> np.ndarray:
    """GELU(v) = v * Phi(v) with the exact standard normal distribution function
    Phi(v) = (1 + erf(v / sqrt 2)) / 2: the activation of the wrapped MLP."""
    v = np.asarray(v, dtype=np.float64)
    return 0.5 * v * (1.0 + _erf(v / math.sqrt(2.0)))


def mlp(x: np.ndarray, w1: np.ndarray, w2: np.ndarray, round_fn=None) -> np.ndarray:
    """The MLP as the wrapped module F (Sec. 4.2.2, "Attention/MLP"): GELU(x w1) w2, no biases.
    round_fn, if given, mirrors the storage rounding of the hidden tensor and of the result."""
    rnd = (lambda t: t) if round_fn is None else round_fn
    return rnd(linear(rnd(gelu(linear(x, w1))), w2))


def attention(q: np.ndarray, k: np.ndarray, v: np.ndarray, n_heads: int,
              query_rows: Optional[np.ndarray] = None) -> np.ndarray:
    """Multi-head softmax(Q K^T / sqrt(dh)) V for one batch item.

    q, k, v: [L, n_heads*dh] with head h in columns [h*dh, (h+1)*dh).
    `query_rows` restricts the computation to some query positions.
    """
    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    if query_rows is not None:
        q = q[query_rows]
    dh = q.shape[1] // n_heads
    out = np.empty((q.shape[0], v.shape[1]), dtype=np.float64)
    for h in range(n_heads):
        sl = slice(h * dh, (h + 1) * dh)
        s = (q[:, sl] @ k[:, sl].T) / np.sqrt(float(dh))
        s = s - s.max(axis=1, keepdims=True)
        p = np.exp(s)
        p = p / p.sum(axis=1, keepdims=True)
        out[:, sl] = p @ v[:, sl]
    return out


# ----------------------------------------------------------------------------
# The whole block with pattern reuse (Algorithm 3; Sec. 4.3.2)
# ----------------------------------------------------------------------------


def global_destinations(idx_tiles: np.ndarray, ids: np.ndarray) -> np.ndarray:
    """Image-level token ids of the destinations chosen per tile: idx_tiles [P, D_loc] holds tile-local
    picks, ids [P, N_loc] the image token of every tile slot; the result [P * D_loc] is tile-major, pick
    order inside a tile (the order of the merged rows)."""
    return np.concatenate([ids[p][np.asarray(idx_tiles[p], dtype=np.int64)] for p in range(ids.shape[0])])


@dataclass
class BlockState:
    """Cached selection and weights of one batch (what Sec. 4.3.2 reuses)."""
    idx: Optional[np.ndarray] = None      # [B, P, D_loc] local indices, pick order
    w: Optional[np.ndarray] = None        # [B, P, D_loc, N_loc]
    u: Optional[np.ndarray] = None        # matrix the unmerge applies (w itself, or the shares A), same shape
    margins: List[float] = field(default_factory=list)


def block_step(x: np.ndarray, step: int, state: BlockState, *, grid_h: int, grid_w: int,
               tile_h: int, tile_w: int, merge_ratio: float, tau: float, n_heads: int,
               reuse_interval: int, n_extra: int = 0, round_fn=None, weight_reuse_interval: int = 0,
               global_merge: bool = False, proj=None, unmerge_mode: str = "transpose", mlp_weights=None):
    """One ToMA-wrapped attention call (Algorithm 3) on x [B, N + n_extra, d].

    Selection and weights are recomputed when step % reuse_interval == 0 and
    reused otherwise (Sec. 4.3.2).  With weight_reuse_interval > 0 the weights alone are also
    recomputed when step % weight_reuse_interval == 0, from the current x at the cached
    destinations (the paper's schedule: destinations every 10 steps, weights every 5).  Merged tokens are ordered tile-major, pick
    order inside a tile; the n_extra trailing tokens are not merged and join the
    attention after the merged image tokens.  The core module F is the attention
    core with Q = K = V = merged tokens.

    With global_merge (the paper's default variant, Sec. 5 "ToMA Variants": destinations chosen per
    tile, merge over the whole image) the D destinations of an image, in the same tile-major pick
    order, form one destination set and Sec. 4.2's weights, merge and unmerge are applied once to all
    N image tokens; state.w is then [B, 1, D, N].

    With proj = (wq, wk, wv, wo), each [d, d] as [in, out], the wrapped module is the whole attention
    module: attention(X_m wq, X_m wk, X_m wv) wo (Algorithm 3 applies F to the merged tokens; App. C's
    4 d^2 N term).  round_fn is then also applied to q, k, v and to the projected output.

    With mlp_weights = (w1 [d, f], w2 [f, d]) the wrapped module is the MLP GELU(X_m w1) w2 instead of
    attention; round_fn is then applied to the hidden tensor and to the MLP's output.

    unmerge_mode "transpose" applies A~^T (Algorithm 3); "shares" applies A^T, the softmax matrix
    before row normalisation (columns sum to 1).

    `round_fn`, if given, is applied to the merged and to the attended tensor; it
    lets a test mirror the storage rounding between stages.  Returns
    (out [B, N + n_extra, d], merged [B, D + n_extra, d], attended (same shape)).
    """
    x = np.asarray(x, dtype=np.float64)
    B, n_all, d = x.shape
    N = grid_h * grid_w
    ids = tile_token_ids(grid_h, grid_w, tile_h, tile_w)
    P, n_loc = ids.shape
    d_loc = dest_count(n_loc, merge_ratio)
    D = P * d_loc
    refresh_sel = step % reuse_interval == 0 or state.idx is None
    refresh_w = refresh_sel or (weight_reuse_interval > 0 and step % weight_reuse_interval == 0)
    if refresh_sel:
        state.idx = np.empty((B, P, d_loc), dtype=np.int64)
        for b in range(B):
            for p in range(P):
                state.idx[b, p], mg = select_tile(x[b, ids[p]], d_loc)
                state.margins.append(mg)
    if unmerge_mode not in ("transpose", "shares"):
        raise ValueError(unmerge_mode)
    if refresh_w and global_merge:
        state.w = np.empty((B, 1, D, N), dtype=np.float64)
        state.u = np.empty_like(state.w)
        for b in range(B):
            state.u[b, 0] = softmax_shares(x[b, :N], global_destinations(state.idx[b], ids), tau)
            state.w[b, 0] = state.u[b, 0] / state.u[b, 0].sum(axis=1, keepdims=True)
    elif refresh_w:
        state.w = np.empty((B, P, d_loc, n_loc), dtype=np.float64)
        state.u = np.empty_like(state.w)
        for b in range(B):
            for p in range(P):
                state.u[b, p] = softmax_shares(x[b, ids[p]], state.idx[b, p], tau)
                state.w[b, p] = state.u[b, p] / state.u[b, p].sum(axis=1, keepdims=True)
    u = state.w if unmerge_mode == "transpose" else state.u
    merged = np.empty((B, D + n_extra, d), dtype=np.float64)
    for b in range(B):
        if global_merge:
            merged[b, :D] = merge(state.w[b, 0], x[b, :N])
        else:
            for p in range(P):
                merged[b, p * d_loc:(p + 1) * d_loc] = merge(state.w[b, p], x[b, ids[p]])
        merged[b, D:] = x[b, N:]
    if round_fn is not None:
        merged = round_fn(merged)
    rnd = (lambda t: t) if round_fn is None else round_fn
    attended = np.empty_like(merged)
    for b in range(B):
        if mlp_weights is not None:
            attended[b] = mlp(merged[b], mlp_weights[0], mlp_weights[1], round_fn)
        elif proj is None:
            attended[b] = attention(merged[b], merged[b], merged[b], n_heads)
        else:
            q, k, v = (rnd(linear(merged[b], w)) for w in proj[:3])
            attended[b] = rnd(linear(rnd(attention(q, k, v, n_heads)), proj[3]))
    if round_fn is not None and proj is None and mlp_weights is None:
        attended = round_fn(attended)
    out = np.empty((B, n_all, d), dtype=np.float64)
    for b in range(B):
        if global_merge:
            out[b, :N] = unmerge(u[b, 0], attended[b, :D])
        else:
            for p in range(P):
                out[b, ids[p]] = unmerge(u[b, p], attended[b, p * d_loc:(p + 1) * d_loc])
        out[b, N:] = attended[b, D:]
    return out, merged, attended


# ----------------------------------------------------------------------------
# Cost model (App. C), in multiplications as the paper counts them
# ----------------------------------------------------------------------------


def cost_base(N: int, d: int) -> float:
    """C_base = 4 d^2 N + 2 d N^2 (App. C, baseline self-attention block)."""
    return 4.0 * d * d * N + 2.0 * d * N * N


def cost_toma_global(N: int, d: int, keep: float) -> float:
    """C_total(r) = 4 d^2 r N + 2 d r^2 N^2 + N^2 d + 3 r N^2 d (App. C), r = D/N kept."""
    return 4.0 * d * d * keep * N + 2.0 * d * keep * keep * N * N + float(N) * N * d + 3.0 * keep * N * N * d


def overhead_tiled(N: int, d: int, keep: float, n_tiles: int) -> float:
    """Selection + weights + merge + unmerge when all four run inside P equal
    regions: each region costs N_loc^2 d + 3 (keep N_loc) N_loc d, and there are P of them."""
    n_loc = N / n_tiles
    return n_tiles * (n_loc * n_loc * d + 3.0 * keep * n_loc * n_loc * d)

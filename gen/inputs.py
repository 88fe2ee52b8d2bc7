"""Deterministic synthetic token tensors shaped like SDXL / Flux hidden states.

Recipe (stands in for real hidden states, which need model weights):

* image tokens: a coarse lattice of i.i.d. N(0,1) vectors, one node every 8
  tokens in each spatial direction, bilinearly interpolated to the H x W grid
  (unit coefficient), plus i.i.d. per-token noise N(0, sigma^2).  With
  sigma = 0.3 neighbouring tokens have cosine similarity of about 0.8.
* text tokens (DiT joint attention): i.i.d. N(0,1), appended after the image
  tokens.
* step sequences: X_{t+1} = X_t + drift * N(0,1), state kept in fp32 and
  rounded to the storage dtype at every step.

Random numbers come from a counter-based generator: splitmix64 of
(stream key, counter) followed by Box-Muller, so any element of any tensor is
a pure function of (seed, config name, batch item, step, tensor tag, index).

bf16 tensors are carried on the host as uint16 bit patterns (numpy has no
bf16); `bf16_bits_to_f32` widens them exactly.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import Dict, Iterator, Tuple

import numpy as np

_MASK = np.uint64(0xFFFFFFFFFFFFFFFF)


def _splitmix64(x: np.ndarray) -> np.ndarray:
    """One splitmix64 output per 64-bit input (vectorised, wrap-around math)."""
    with np.errstate(over="ignore"):
        z = (x + np.uint64(0x9E3779B97F4A7C15)) & _MASK
        z = ((z ^ (z >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)) & _MASK
        z = ((z ^ (z >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)) & _MASK
        return z ^ (z >> np.uint64(31))


def _stream_key(seed: int, *tags: int) -> np.uint64:
    k = np.array([seed & 0xFFFFFFFFFFFFFFFF], dtype=np.uint64)
    for t in tags:
        k = _splitmix64(k ^ np.uint64((t * 0xD6E8FEB86659FD93) & 0xFFFFFFFFFFFFFFFF))
    return k[0]


def normal(seed: int, tags: Tuple[int, ...], count: int) -> np.ndarray:
    """`count` standard normal float64 draws of the stream named by (seed, tags)."""
    key = _stream_key(seed, *tags)
    n_pairs = (count + 1) // 2
    ctr = np.arange(2 * n_pairs, dtype=np.uint64)
    with np.errstate(over="ignore"):
        bits = _splitmix64((key + ctr * np.uint64(0x2545F4914F6CDD1D)) & _MASK)
    # 53-bit uniforms in (0, 1]
    u = ((bits >> np.uint64(11)).astype(np.float64) + 1.0) * (1.0 / 9007199254740992.0)
    u1, u2 = u[0::2], u[1::2]
    r = np.sqrt(-2.0 * np.log(u1))
    out = np.empty(2 * n_pairs, dtype=np.float64)
    out[0::2] = r * np.cos(2.0 * np.pi * u2)
    out[1::2] = r * np.sin(2.0 * np.pi * u2)
    return out[:count]


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bf16 (round-to-nearest-even); returns uint16 bit patterns."""
    b = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounding = np.uint32(0x7FFF) + ((b >> np.uint32(16)) & np.uint32(1))
    return ((b + rounding) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def round_to_dtype(x: np.ndarray, dtype: str) -> np.ndarray:
    """Values of `x` after one rounding to the storage dtype, returned as float32."""
    x = np.asarray(x, dtype=np.float32)
    if dtype == "bf16":
        return bf16_bits_to_f32(f32_to_bf16_bits(x))
    if dtype == "f32":
        return x
    raise ValueError(dtype)


@dataclass(frozen=True)
class TomaConfig:
    name: str
    batch: int
    grid_h: int
    grid_w: int
    dim: int
    dtype: str            # "bf16" | "f32"
    tile_h: int
    tile_w: int
    merge_ratio: float    # fraction of tokens removed
    n_heads: int
    head_dim: int
    tau: float = 0.1
    n_extra: int = 0      # trailing text tokens that are never merged
    noise_sigma: float = 0.3
    steps: int = 1
    reuse_interval: int = 1
    drift_sigma: float = 0.05
    seed: int = 0
    tag: int = 0          # distinguishes configs in the random streams

    @property
    def n_tokens(self) -> int:
        return self.grid_h * self.grid_w

    @property
    def n_loc(self) -> int:
        return self.tile_h * self.tile_w

    @property
    def n_tiles(self) -> int:
        return (self.grid_h // self.tile_h) * (self.grid_w // self.tile_w)

    def with_(self, **kw) -> "TomaConfig":
        return replace(self, **kw)


CONFIGS: Dict[str, TomaConfig] = {
    # tiny correctness instance
    "cfg1": TomaConfig("cfg1", 1, 32, 32, 640, "f32", 8, 8, 0.5, 10, 64, noise_sigma=1.0, tag=1),
    # SDXL-like mid-resolution block (CFG pair)
    "cfg2": TomaConfig("cfg2", 2, 32, 32, 1280, "bf16", 8, 8, 0.5, 20, 64, tag=2),
    # SDXL-like high-resolution block, 10 steps, reuse 5
    "cfg3": TomaConfig("cfg3", 2, 64, 64, 640, "bf16", 16, 16, 0.5, 10, 64, steps=10, reuse_interval=5, tag=3),
    # Flux-like joint attention block with 512 text tokens
    "cfg4": TomaConfig("cfg4", 1, 64, 64, 3072, "bf16", 16, 16, 0.5, 24, 128, n_extra=512, tag=4),
    # scaling stress, two tile sizes
    "cfg5a": TomaConfig("cfg5a", 4, 128, 128, 640, "bf16", 16, 16, 0.5, 10, 64, steps=28, reuse_interval=5, tag=5),
    "cfg5b": TomaConfig("cfg5b", 4, 128, 128, 640, "bf16", 32, 32, 0.5, 10, 64, steps=28, reuse_interval=5, tag=5),
}


def config(name: str, **overrides) -> TomaConfig:
    c = CONFIGS[name]
    return c.with_(**overrides) if overrides else c


_LATTICE = 8
_T_FIELD, _T_NOISE, _T_TEXT, _T_DRIFT = 11, 12, 13, 14


def _image_tokens(cfg: TomaConfig, b: int) -> np.ndarray:
    """float32 [H*W, d]: bilinear low-frequency field + per-token noise."""
    H, W, d = cfg.grid_h, cfg.grid_w, cfg.dim
    gh, gw = H // _LATTICE + 2, W // _LATTICE + 2
    lat = normal(cfg.seed, (cfg.tag, b, 0, _T_FIELD), gh * gw * d).reshape(gh, gw, d)
    ys = np.arange(H, dtype=np.float64) / _LATTICE
    xs = np.arange(W, dtype=np.float64) / _LATTICE
    y0 = np.floor(ys).astype(np.int64)
    x0 = np.floor(xs).astype(np.int64)
    fy = (ys - y0)[:, None, None]
    fx = (xs - x0)[None, :, None]
    a = lat[y0][:, x0]
    b_ = lat[y0][:, x0 + 1]
    c = lat[y0 + 1][:, x0]
    e = lat[y0 + 1][:, x0 + 1]
    fld = (1 - fy) * ((1 - fx) * a + fx * b_) + fy * ((1 - fx) * c + fx * e)
    noise = normal(cfg.seed, (cfg.tag, b, 0, _T_NOISE), H * W * d).reshape(H, W, d)
    return (fld + cfg.noise_sigma * noise).reshape(H * W, d).astype(np.float32)


def _state0(cfg: TomaConfig) -> np.ndarray:
    """float32 [B, N + n_extra, d] un-rounded state at step 0."""
    out = np.empty((cfg.batch, cfg.n_tokens + cfg.n_extra, cfg.dim), dtype=np.float32)
    for b in range(cfg.batch):
        out[b, : cfg.n_tokens] = _image_tokens(cfg, b)
        if cfg.n_extra:
            out[b, cfg.n_tokens:] = normal(
                cfg.seed, (cfg.tag, b, 0, _T_TEXT), cfg.n_extra * cfg.dim
            ).reshape(cfg.n_extra, cfg.dim).astype(np.float32)
    return out


def feature_sequence(cfg: TomaConfig, steps: int | None = None) -> Iterator[np.ndarray]:
    """Yields, per step, float32 [B, N + n_extra, d] already rounded to cfg.dtype."""
    steps = cfg.steps if steps is None else steps
    state = _state0(cfg)
    for t in range(steps):
        if t > 0:
            for b in range(cfg.batch):
                state[b] += (cfg.drift_sigma * normal(
                    cfg.seed, (cfg.tag, b, t, _T_DRIFT), state[b].size
                ).reshape(state[b].shape)).astype(np.float32)
        yield round_to_dtype(state, cfg.dtype)


def features(cfg: TomaConfig, step: int = 0) -> np.ndarray:
    """float32 [B, N + n_extra, d] at `step`, already rounded to cfg.dtype."""
    x = None
    for x in feature_sequence(cfg, step + 1):
        pass
    return x


def neighbour_cosine(cfg: TomaConfig, x: np.ndarray) -> float:
    """Mean cosine between horizontally adjacent image tokens (a recorded statistic)."""
    H, W = cfg.grid_h, cfg.grid_w
    g = np.asarray(x[0, : H * W], dtype=np.float64).reshape(H, W, -1)
    a, b = g[:, :-1], g[:, 1:]
    num = (a * b).sum(-1)
    den = np.sqrt((a * a).sum(-1) * (b * b).sum(-1))
    return float((num / den).mean())

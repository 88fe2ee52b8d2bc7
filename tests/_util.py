"""Helpers shared by the GPU parity tests (marshalling between numpy inputs and torch tensors)."""
import numpy as np
import torch

import gen
from oracle import toma_oracle as O

BF16_MAX_ABS, BF16_REL_FRO, F32_MAX_ABS = 2e-2, 1e-2, 1e-4


def to_dev(x_host: np.ndarray, dtype: str) -> torch.Tensor:
    t = torch.from_numpy(np.ascontiguousarray(x_host, dtype=np.float32)).cuda()
    return t if dtype == "f32" else t.to(torch.bfloat16)


def to_host64(t: torch.Tensor) -> np.ndarray:
    return t.detach().float().cpu().numpy().astype(np.float64)


def assert_close(got: np.ndarray, want: np.ndarray, dtype: str, what: str):
    err = np.abs(got - want)
    max_abs = float(err.max()) if err.size else 0.0
    fro = float(np.linalg.norm(got - want) / max(np.linalg.norm(want), 1e-30))
    if dtype == "f32":
        assert max_abs <= F32_MAX_ABS, f"{what}: max-abs {max_abs:.3g} > {F32_MAX_ABS}"
    else:
        assert max_abs <= BF16_MAX_ABS, f"{what}: max-abs {max_abs:.3g} > {BF16_MAX_ABS}"
        assert fro <= BF16_REL_FRO, f"{what}: rel-Frobenius {fro:.3g} > {BF16_REL_FRO}"
    return max_abs, fro


def sample_tiles(cfg, count: int, seed: int = 0):
    """(b, p) pairs: all tiles if few, else a seeded sample that always includes the first and last."""
    pairs = [(b, p) for b in range(cfg.batch) for p in range(cfg.n_tiles)]
    if len(pairs) <= count:
        return pairs
    rng = np.random.default_rng(seed)
    pick = set(rng.choice(len(pairs), size=count - 2, replace=False).tolist()) | {0, len(pairs) - 1}
    return [pairs[i] for i in sorted(pick)]


def tile_tokens(cfg, x_host: np.ndarray, b: int, p: int) -> np.ndarray:
    ids = O.tile_token_ids(cfg.grid_h, cfg.grid_w, cfg.tile_h, cfg.tile_w)
    return x_host[b, ids[p]]

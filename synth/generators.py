"""Seeded tensor generators (see package docstring).  numpy only."""
from __future__ import annotations

import concurrent.futures
import os
import zlib
from dataclasses import dataclass

import numpy as np

# Base seed per workload family (paper id * 10 + workload index).
CONFIG_SEEDS = {
    "block_s2": 2503025081,
    "forward_xl2": 2503025082,
    "ddim50_xl2": 2503025083,
    "ddim100_xl2_512": 2503025084,
    "gemm_sweep": 2503025085,
}


@dataclass(frozen=True)
class DiTConfig:
    """Shape of a class-conditional DiT (the model family of Experimental Settings)."""

    hidden: int          # D
    heads: int           # H
    mlp: int             # MLP width
    depth: int           # number of blocks
    grid: int            # tokens per image side (latent side / patch)
    patch: int = 2
    channels: int = 4    # latent channels C
    num_classes: int = 1000
    freq_dim: int = 256  # sinusoidal timestep feature width

    @property
    def tokens(self) -> int:
        return self.grid * self.grid

    @property
    def head_dim(self) -> int:
        return self.hidden // self.heads

    @property
    def latent_side(self) -> int:
        return self.grid * self.patch

    @property
    def patch_dim(self) -> int:
        return self.patch * self.patch * self.channels

    @property
    def out_dim(self) -> int:  # final linear width: patch*patch*(2C) (noise + learned sigma)
        return self.patch * self.patch * 2 * self.channels


DIT_S2_BLOCK = DiTConfig(hidden=384, heads=6, mlp=1536, depth=1, grid=16)
DIT_XL2 = DiTConfig(hidden=1152, heads=16, mlp=4608, depth=28, grid=16)
DIT_XL2_512 = DiTConfig(hidden=1152, heads=16, mlp=4608, depth=28, grid=32)
# A small model with the awkward XL head width (72) for tests that run in seconds.
DIT_TINY = DiTConfig(hidden=144, heads=2, mlp=576, depth=3, grid=8)


def stream(seed: int, name: str) -> np.random.Generator:
    """Independent generator for one named tensor."""
    key = (int(seed) & 0xFFFFFFFFFFFFFFFF, zlib.crc32(name.encode()))
    return np.random.Generator(np.random.Philox(key=np.array(key, dtype=np.uint64)))


def normal(seed: int, name: str, shape, std: float = 1.0, mean: float = 0.0) -> np.ndarray:
    g = stream(seed, name)
    x = g.standard_normal(size=shape, dtype=np.float32)
    if std != 1.0:
        x *= np.float32(std)
    if mean != 0.0:
        x += np.float32(mean)
    return x


def uniform_int(seed: int, name: str, shape, low: int, high: int) -> np.ndarray:
    """Integers uniform in [low, high)."""
    g = stream(seed, name)
    return g.integers(low, high, size=shape, dtype=np.int64).astype(np.int32)


_W_STD = 0.02


def block_weights(seed: int, cfg: DiTConfig, index: int) -> dict:
    """fp32 parameters of one DiT block; every linear is [out_features, in_features]."""
    D, F = cfg.hidden, cfg.mlp
    p = f"blk{index}."
    return {
        "w_ada": normal(seed, p + "w_ada", (6 * D, D), _W_STD),
        "b_ada": normal(seed, p + "b_ada", (6 * D,), _W_STD),
        "w_qkv": normal(seed, p + "w_qkv", (3 * D, D), _W_STD),
        "b_qkv": normal(seed, p + "b_qkv", (3 * D,), _W_STD),
        "w_proj": normal(seed, p + "w_proj", (D, D), _W_STD),
        "b_proj": normal(seed, p + "b_proj", (D,), _W_STD),
        "w_fc1": normal(seed, p + "w_fc1", (F, D), _W_STD),
        "b_fc1": normal(seed, p + "b_fc1", (F,), _W_STD),
        "w_fc2": normal(seed, p + "w_fc2", (D, F), _W_STD),
        "b_fc2": normal(seed, p + "b_fc2", (D,), _W_STD),
    }


def pos_embed_table(cfg: DiTConfig) -> np.ndarray:
    """Fixed 2-D sine/cosine position table [tokens, hidden], fp32 (an input, not learned)."""
    D, g = cfg.hidden, cfg.grid
    q = D // 4
    omega = 1.0 / (10000.0 ** (np.arange(q, dtype=np.float64) / q))
    ys, xs = np.meshgrid(np.arange(g, dtype=np.float64), np.arange(g, dtype=np.float64), indexing="ij")

    def emb(pos):
        a = pos.reshape(-1)[:, None] * omega[None, :]
        return np.concatenate([np.sin(a), np.cos(a)], axis=1)

    table = np.concatenate([emb(xs), emb(ys)], axis=1)
    out = np.zeros((g * g, D), dtype=np.float32)
    out[:, : table.shape[1]] = table.astype(np.float32)
    return out


def model_weights(seed: int, cfg: DiTConfig) -> dict:
    """fp32 parameters of a whole DiT: embedders, `depth` blocks, final layer."""
    D = cfg.hidden
    w = {
        "w_patch": normal(seed, "w_patch", (D, cfg.patch_dim), _W_STD),
        "b_patch": normal(seed, "b_patch", (D,), _W_STD),
        "pos": pos_embed_table(cfg),
        "w_t1": normal(seed, "w_t1", (D, cfg.freq_dim), _W_STD),
        "b_t1": normal(seed, "b_t1", (D,), _W_STD),
        "w_t2": normal(seed, "w_t2", (D, D), _W_STD),
        "b_t2": normal(seed, "b_t2", (D,), _W_STD),
        # row num_classes is the "no class" embedding used by classifier-free guidance
        "y_table": normal(seed, "y_table", (cfg.num_classes + 1, D), _W_STD),
        "w_ada_f": normal(seed, "w_ada_f", (2 * D, D), _W_STD),
        "b_ada_f": normal(seed, "b_ada_f", (2 * D,), _W_STD),
        "w_out": normal(seed, "w_out", (cfg.out_dim, D), _W_STD),
        "b_out": normal(seed, "b_out", (cfg.out_dim,), _W_STD),
    }
    # every tensor has its own stream, so blocks can be drawn concurrently with identical results
    with concurrent.futures.ThreadPoolExecutor(max_workers=min(16, os.cpu_count() or 1)) as ex:
        w["blocks"] = list(ex.map(lambda i: block_weights(seed, cfg, i), range(cfg.depth)))
    return w


def outlier_activations(seed: int, name: str, M: int, K: int, frac: float = 0.01, gain: float = 20.0) -> np.ndarray:
    """N(0,1) activations [M,K] with a seeded `frac` of the K channels scaled by `gain`."""
    x = normal(seed, name, (M, K))
    g = stream(seed, name + ".outliers")
    n_out = max(1, int(round(frac * K)))
    cols = g.choice(K, size=n_out, replace=False)
    x[:, cols] *= np.float32(gain)
    return x

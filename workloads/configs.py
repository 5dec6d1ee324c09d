"""Workload recipes: shapes, splits, node counts, seeds and seeded input generators.

Orientation follows the paper (Section II-B): a column of X is one sample, W is
N1 x N0, X is N0 x B, all row-major.  Every generator draws with
``numpy.random.default_rng(seed)`` in FP64 and casts to FP32, so that the CPU
oracle and the CUDA library receive bit-identical FP32 inputs.

Nothing here computes any quantity of the coding method; the node counts P are
plain constants (tests check them against the thresholds the oracle derives).
"""

from __future__ import annotations

from dataclasses import dataclass, replace
from typing import List, Tuple

import numpy as np

BASE_SEED = 181110751


@dataclass(frozen=True)
class CodedMatmulConfig:
    """One coded product S = W X (Problem 1 of the paper)."""

    name: str
    N1: int            # rows of W
    N0: int            # columns of W = rows of X
    B: int             # columns of X (mini-batch)
    m: int             # row blocks of W
    n: int             # column blocks of W = row blocks of X
    d: int             # column blocks of X
    P: int             # number of simulated worker nodes
    w_dist: str        # "uniform" (U[-1,1]) or "gauss" (N(0, 1/N0))
    x_dist: str        # "uniform" (U[-1,1]) or "gauss" (N(0, 1))
    seed: int
    inject: str        # "none" | "bitflip" | "additive"
    inject_count: int = 0      # bitflip: number of distinct corrupted nodes
    inject_prob: float = 0.0   # additive: per-node corruption probability
    inject_seeds: Tuple[int, ...] = ()


@dataclass(frozen=True)
class MLPConfig:
    """Coded training step of a ReLU multi-layer perceptron with softmax cross-entropy."""

    name: str
    widths: Tuple[int, ...]    # N_0, N_1, ..., N_L
    B: int
    m: int
    n: int
    d1: int
    d2: int
    P: int
    lr: float
    n_classes: int
    inject_prob: float
    seed: int
    steps: int = 1


@dataclass(frozen=True)
class AutoencoderConfig:
    """Coded training of a one-hidden-layer sparse autoencoder (sigmoid encoder, linear decoder)."""

    name: str
    n_visible: int
    n_hidden: int
    B: int
    m: int
    n: int
    d1: int
    d2: int
    P: int
    lr: float
    rho: float
    beta: float
    inject_prob: float
    seed: int
    steps: int = 10


CONFIG_1_TINY = CodedMatmulConfig(
    name="cfg1_tiny_matmul_64", N1=64, N0=64, B=64, m=2, n=2, d=2, P=11,
    w_dist="uniform", x_dist="uniform", seed=BASE_SEED + 1, inject="none")

CONFIG_2_MATVEC = CodedMatmulConfig(
    name="cfg2_matvec_4096", N1=4096, N0=4096, B=1, m=4, n=2, d=1, P=13,
    w_dist="gauss", x_dist="gauss", seed=BASE_SEED + 2, inject="bitflip",
    inject_count=2, inject_seeds=(BASE_SEED + 20,))

CONFIG_3_MATMUL = CodedMatmulConfig(
    name="cfg3_matmul_8192x8192x512", N1=8192, N0=8192, B=512, m=2, n=4, d=2, P=25,
    w_dist="gauss", x_dist="gauss", seed=BASE_SEED + 3, inject="additive",
    inject_prob=0.1,
    inject_seeds=tuple(BASE_SEED + 30 + s for s in range(8)))

CONFIG_4_MLP = MLPConfig(
    name="cfg4_mlp_4096x3_10", widths=(4096, 4096, 4096, 4096, 10), B=256,
    m=2, n=2, d1=1, d2=1, P=10, lr=0.01, n_classes=10, inject_prob=0.05,
    seed=BASE_SEED + 4, steps=1)

CONFIG_5_AUTOENCODER = AutoencoderConfig(
    name="cfg5_sparse_autoencoder_1024_8192", n_visible=1024, n_hidden=8192, B=1024,
    m=4, n=4, d1=1, d2=1, P=36, lr=0.01, rho=0.05, beta=3.0, inject_prob=0.05,
    seed=BASE_SEED + 5, steps=10)


def _draw(rng: np.random.Generator, dist: str, shape, fan_in: int) -> np.ndarray:
    if dist == "uniform":
        a = rng.uniform(-1.0, 1.0, size=shape)
    elif dist == "gauss":
        a = rng.standard_normal(size=shape)
    elif dist == "gauss_fan":
        a = rng.standard_normal(size=shape) / np.sqrt(float(fan_in))
    else:
        raise ValueError(f"unknown distribution {dist!r}")
    return np.ascontiguousarray(a.astype(np.float32))


def matmul_inputs(cfg: CodedMatmulConfig) -> Tuple[np.ndarray, np.ndarray]:
    """W (N1 x N0) and X (N0 x B), FP32, drawn as the config says."""
    rng = np.random.default_rng(cfg.seed)
    w_dist = "gauss_fan" if cfg.w_dist == "gauss" else cfg.w_dist
    W = _draw(rng, w_dist, (cfg.N1, cfg.N0), cfg.N0)
    X = _draw(rng, cfg.x_dist, (cfg.N0, cfg.B), cfg.N0)
    return W, X


def mlp_inputs(cfg: MLPConfig) -> Tuple[List[np.ndarray], np.ndarray, np.ndarray]:
    """Weights W^l ~ N(0, 2/fan_in), inputs X^1 ~ N(0,1) (N_0 x B), labels uniform over classes."""
    rng = np.random.default_rng(cfg.seed)
    Ws = []
    for l in range(len(cfg.widths) - 1):
        fan_in, fan_out = cfg.widths[l], cfg.widths[l + 1]
        w = rng.standard_normal(size=(fan_out, fan_in)) * np.sqrt(2.0 / fan_in)
        Ws.append(np.ascontiguousarray(w.astype(np.float32)))
    X1 = np.ascontiguousarray(rng.standard_normal(size=(cfg.widths[0], cfg.B)).astype(np.float32))
    labels = rng.integers(0, cfg.n_classes, size=cfg.B).astype(np.int32)
    return Ws, X1, labels


def autoencoder_inputs(cfg: AutoencoderConfig) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """Encoder W1 (hidden x visible), decoder W2 (visible x hidden), both N(0, 1/fan_in);
    data X1 (visible x B): U[0,1] entries with 90 % of them zeroed at random."""
    rng = np.random.default_rng(cfg.seed)
    W1 = rng.standard_normal(size=(cfg.n_hidden, cfg.n_visible)) / np.sqrt(float(cfg.n_visible))
    W2 = rng.standard_normal(size=(cfg.n_visible, cfg.n_hidden)) / np.sqrt(float(cfg.n_hidden))
    X = rng.uniform(0.0, 1.0, size=(cfg.n_visible, cfg.B))
    keep = rng.uniform(0.0, 1.0, size=X.shape) >= 0.9
    X = X * keep
    f32 = lambda a: np.ascontiguousarray(a.astype(np.float32))
    return f32(W1), f32(W2), f32(X)


def scaled_down(cfg, factor: int):
    """Same code (splits, P, distributions, seed) on matrices ``factor`` times smaller per side.

    Used by parity tests that need the oracle to finish in seconds.  The mini-batch
    is kept unless it would stop being divisible by the column split."""
    if isinstance(cfg, CodedMatmulConfig):
        B = cfg.B if cfg.B == 1 else max(cfg.d, cfg.B // factor)
        return replace(cfg, name=f"{cfg.name}_div{factor}", N1=cfg.N1 // factor,
                       N0=cfg.N0 // factor, B=B)
    if isinstance(cfg, MLPConfig):
        widths = tuple(max(w // factor, cfg.m * cfg.n) if w > cfg.n_classes else w
                       for w in cfg.widths)
        return replace(cfg, name=f"{cfg.name}_div{factor}", widths=widths,
                       B=max(cfg.d1 * cfg.d2, cfg.B // factor))
    if isinstance(cfg, AutoencoderConfig):
        return replace(cfg, name=f"{cfg.name}_div{factor}", n_visible=cfg.n_visible // factor,
                       n_hidden=cfg.n_hidden // factor, B=max(1, cfg.B // factor))
    raise TypeError(type(cfg))

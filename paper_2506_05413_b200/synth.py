"""Seeded synthetic inputs for the SmoothRot W4A4 linear layer.

This module only draws random tensors.  It holds none of the method's
arithmetic (no scaling formula, no Hadamard, no quantizer), so that the CUDA
path and the CPU checker can both be fed from it without sharing any logic.

The tensors take the shapes and the value structure of the layers the paper
studies: Gaussian hidden states with a handful of "massive outlier" channels
that fire on a small subset of tokens (Section "Massive Activation Outliers"),
and, for the down-projection, inputs that are products SiLU(gate) * up of a
gated linear unit (Fig. 2).  They stand in for the paper's calibration and
evaluation text and for trained weights, which this repository does not have.

Everything is numpy; fp16 tensors are produced by clamping to the finite fp16
range and rounding once.
"""
from __future__ import annotations

import dataclasses
import math

import numpy as np

FP16_MAX = 65504.0


@dataclasses.dataclass
class LayerCase:
    """One linear layer's worth of synthetic data (all numpy, host memory)."""

    name: str
    X: np.ndarray        # [M, K] fp16 activations (un-smoothed, un-rotated)
    X_calib: np.ndarray  # [T, K] fp16 calibration activations, same law
    W: np.ndarray        # [N, K] fp16 weights, PyTorch layout (Y = X W^T)
    d: np.ndarray        # [K] fp32 entries +1/-1: the random sign diagonal
    alpha: float         # migration strength
    clip_a: float        # activation clip ratio
    clip_w: float        # weight clip ratio
    outlier_channels: np.ndarray
    outlier_tokens: np.ndarray

    @property
    def M(self) -> int:
        return self.X.shape[0]

    @property
    def K(self) -> int:
        return self.X.shape[1]

    @property
    def N(self) -> int:
        return self.W.shape[0]


def _to_fp16(a: np.ndarray) -> np.ndarray:
    return np.clip(a, -FP16_MAX, FP16_MAX).astype(np.float16)


def _normal(rng: np.random.Generator, shape, std: float = 1.0) -> np.ndarray:
    a = rng.standard_normal(shape, dtype=np.float32)
    if std != 1.0:
        a *= np.float32(std)
    return a


def _glu(rng: np.random.Generator, shape) -> np.ndarray:
    g = _normal(rng, shape)
    u = _normal(rng, shape)
    return (g / (1.0 + np.exp(-g))) * u


def sign_vector(rng: np.random.Generator, K: int, period: int | None = None) -> np.ndarray:
    """Random +1/-1 vector of length K; if `period` is given, `period` signs
    are drawn and tiled K/period times."""
    n = K if period is None else period
    base = (rng.integers(0, 2, size=n).astype(np.float32) * 2.0 - 1.0).astype(np.float32)
    if period is None:
        return base
    assert K % period == 0
    return np.tile(base, K // period)


def activations(rng: np.random.Generator, M: int, K: int, *, law: str,
                outlier_channels: np.ndarray, outlier_gain: float,
                outlier_tokens: np.ndarray) -> np.ndarray:
    """[M, K] fp16 activations: `law` is "normal" or "glu"; entries at
    (outlier_tokens x outlier_channels) are multiplied by `outlier_gain`."""
    if law == "normal":
        x = _normal(rng, (M, K))
    elif law == "glu":
        x = _glu(rng, (M, K))
    else:
        raise ValueError(law)
    if len(outlier_tokens) and len(outlier_channels):
        x[np.ix_(outlier_tokens, outlier_channels)] *= np.float32(outlier_gain)
    return _to_fp16(x)


def _token_subset(rng: np.random.Generator, M: int, frac: float) -> np.ndarray:
    n = max(1, math.ceil(frac * M)) if M > 0 else 0
    n = min(n, M)
    return np.sort(rng.choice(M, size=n, replace=False)) if n else np.zeros(0, np.int64)


def make_layer(name: str, *, seed: int, M: int, K: int, N: int, T: int, law: str,
               w_std: float, n_outlier_channels: int, outlier_gain: float,
               outlier_channels=None, outlier_tokens=None, token_frac: float = 0.01,
               sign_period: int | None = None, alpha: float = 0.5,
               clip_a: float = 0.9, clip_w: float = 1.0) -> LayerCase:
    """Draw one layer.  Separate seeded streams feed the outlier pattern, the
    activations, the calibration tokens, the weights and the sign diagonal, so
    that changing M does not change W."""
    ss = np.random.SeedSequence(seed)
    r_pat, r_x, r_cal, r_w, r_d = (np.random.default_rng(s) for s in ss.spawn(5))
    if outlier_channels is None:
        outlier_channels = np.sort(r_pat.choice(K, size=n_outlier_channels, replace=False))
    outlier_channels = np.asarray(outlier_channels, dtype=np.int64)
    if outlier_tokens is None:
        tok = _token_subset(r_pat, M, token_frac)
        tok_cal = _token_subset(r_pat, T, token_frac)
    else:
        tok = np.asarray([t for t in outlier_tokens if t < M], dtype=np.int64)
        tok_cal = np.asarray([t for t in outlier_tokens if t < T], dtype=np.int64)
    X = activations(r_x, M, K, law=law, outlier_channels=outlier_channels,
                    outlier_gain=outlier_gain, outlier_tokens=tok)
    Xc = activations(r_cal, T, K, law=law, outlier_channels=outlier_channels,
                     outlier_gain=outlier_gain, outlier_tokens=tok_cal)
    W = _to_fp16(_normal(r_w, (N, K), w_std))
    d = sign_vector(r_d, K, sign_period)
    return LayerCase(name=name, X=X, X_calib=Xc, W=W, d=d, alpha=alpha, clip_a=clip_a,
                     clip_w=clip_w, outlier_channels=outlier_channels, outlier_tokens=tok)


# ---------------------------------------------------------------------------
# The named workloads.  Index = the seed.
# ---------------------------------------------------------------------------

def config0() -> LayerCase:
    """Tiny layer: 64 tokens x 128 channels, channels 7 and 93 x500 on tokens 0-3."""
    return make_layer("cfg0_tiny", seed=0, M=64, K=128, N=256, T=128, law="normal",
                      w_std=0.02, n_outlier_channels=2, outlier_gain=500.0,
                      outlier_channels=[7, 93], outlier_tokens=[0, 1, 2, 3])


def config1(M: int = 2048, N: int = 6144) -> LayerCase:
    """Fused QKV projection shape: K = 4096, 4 outlier channels x1000 on 1% of tokens."""
    return make_layer("cfg1_qkv", seed=1, M=M, K=4096, N=N, T=512, law="normal",
                      w_std=0.02, n_outlier_channels=4, outlier_gain=1000.0)


def config2(M: int = 2048, N: int = 4096) -> LayerCase:
    """MLP down-projection shape: K = 14336 = 28 * 512, GLU-product inputs with
    2 outlier channels x2000; the sign diagonal repeats with period 512."""
    return make_layer("cfg2_down", seed=2, M=M, K=14336, N=N, T=512, law="glu",
                      w_std=0.01, n_outlier_channels=2, outlier_gain=2000.0,
                      sign_period=512)


def config3(M: int = 8192, N: int = 28672) -> LayerCase:
    """Fused gate/up projection shape (compute-bound GEMM)."""
    return make_layer("cfg3_gateup", seed=3, M=M, K=4096, N=N, T=512, law="normal",
                      w_std=0.02, n_outlier_channels=4, outlier_gain=1000.0)


# (name, N, K) of the distinct linear shapes of one LLaMA-3.1-8B-shaped block.
BLOCK_SHAPES = (
    ("q_o", 4096, 4096),
    ("k_v", 1024, 4096),
    ("gate_up", 14336, 4096),
    ("down", 4096, 14336),
)
SWEEP_M = (1, 4, 16, 128, 512, 2048, 8192)


def config4(shape: str, M: int) -> LayerCase:
    """One point of the token-count sweep over the block's linear shapes."""
    for name, N, K in BLOCK_SHAPES:
        if name == shape:
            break
    else:
        raise KeyError(shape)
    if K == 14336:
        return make_layer(f"cfg4_{shape}_M{M}", seed=4, M=M, K=K, N=N, T=512, law="glu",
                          w_std=0.01, n_outlier_channels=2, outlier_gain=2000.0,
                          sign_period=512)
    return make_layer(f"cfg4_{shape}_M{M}", seed=4, M=M, K=K, N=N, T=512, law="normal",
                      w_std=0.02, n_outlier_channels=4, outlier_gain=1000.0)


def random_codes(seed: int, rows: int, K: int) -> np.ndarray:
    """[rows, K] int8 array of uniformly drawn 4-bit codes in [-8, 7]."""
    rng = np.random.default_rng(seed)
    return rng.integers(-8, 8, size=(rows, K), dtype=np.int8)

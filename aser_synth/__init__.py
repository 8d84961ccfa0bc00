"""Seeded synthetic inputs for an ASER-quantized linear layer.

This module only draws random tensors of the shapes and value distributions of
LLM linear layers (Gaussian activations with a few high-magnitude outlier
channels, small Gaussian weights).  It contains none of the method's arithmetic:
no smoothing formula, no quantizer, no factor construction.  Both the CPU oracle
tests and the CUDA library's tests/bench draw their inputs from here, so both
sides always see byte-identical arrays.

The "stand-in" helpers at the bottom produce a smoothing vector and low-rank
factors that have the right shape, dtype and magnitude but are *not* built by
the method; they exist for throughput measurements, where the values of `s`,
`L_A` and `L_B` do not influence run time.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

BASE_SEED = 24110776


def seed_for(config: int, index: int = 0) -> int:
    """Deterministic seed for workload `config` (1..5) and a sub-index."""
    return BASE_SEED + 1000 * int(config) + int(index)


@dataclass
class LayerInputs:
    """One linear layer's synthetic tensors (all NumPy, host memory)."""

    X: np.ndarray            # [M, K] float16 activations
    W: np.ndarray            # [N, K] float16 weights
    X_cal: np.ndarray        # [T_cal, K] float16 calibration activations
    outlier_idx: np.ndarray  # sorted int64 indices of the seeded outlier channels
    outlier_gain: float
    meta: dict = field(default_factory=dict)


def _gauss_f32(rng: np.random.Generator, shape) -> np.ndarray:
    return rng.standard_normal(shape, dtype=np.float32)


def _apply_outliers(x32: np.ndarray, idx: np.ndarray, gain: float) -> np.ndarray:
    x32[:, idx] *= np.float32(gain)
    return x32


def draw_outlier_channels(rng: np.random.Generator, K: int, n_out: int) -> np.ndarray:
    return np.sort(rng.choice(K, size=n_out, replace=False)).astype(np.int64)


def make_layer(M: int, N: int, K: int, *, seed: int, n_out: int | None = None,
               outlier_gain: float = 30.0, sigma_w: float = 0.02,
               n_cal: int = 512, gated_input: bool = False) -> LayerInputs:
    """Draw X [M,K], W [N,K] and calibration tokens [n_cal,K].

    Activations are N(0,1) rounded to fp16, with `n_out` seeded channels
    multiplied by `outlier_gain` (default n_out = K // 100, i.e. 1 %).
    With `gated_input` the activation is silu(a) * b of two N(0,1) fp16 draws
    (the input of an MLP down projection) before the outlier gain is applied.
    Weights are N(0, sigma_w^2) rounded to fp16.
    """
    rng = np.random.default_rng(seed)
    if n_out is None:
        n_out = max(1, K // 100)
    idx = draw_outlier_channels(rng, K, n_out)

    def draw_act(rows: int) -> np.ndarray:
        if gated_input:
            a = _gauss_f32(rng, (rows, K)).astype(np.float16).astype(np.float32)
            b = _gauss_f32(rng, (rows, K)).astype(np.float16).astype(np.float32)
            x = (a / (1.0 + np.exp(-a))) * b
            x = x.astype(np.float16).astype(np.float32)
        else:
            x = _gauss_f32(rng, (rows, K))
        return _apply_outliers(x, idx, outlier_gain).astype(np.float16)

    X = draw_act(M)
    W = (_gauss_f32(rng, (N, K)) * np.float32(sigma_w)).astype(np.float16)
    X_cal = draw_act(n_cal)
    return LayerInputs(X=X, W=W, X_cal=X_cal, outlier_idx=idx, outlier_gain=outlier_gain,
                       meta=dict(M=M, N=N, K=K, seed=seed, n_out=n_out, sigma_w=sigma_w,
                                 n_cal=n_cal, gated_input=gated_input))


# ----------------------------------------------------------------------------
# Named workloads (shapes and distributions of the five benchmark configurations)
# ----------------------------------------------------------------------------

def config1_tiny() -> tuple[LayerInputs, int]:
    """16 tokens, 512 -> 512, 4 outlier channels x40, 128 calibration tokens, rank 16."""
    return make_layer(16, 512, 512, seed=seed_for(1), n_out=4, outlier_gain=40.0,
                      sigma_w=0.02, n_cal=128), 16


def config2_decode(M: int) -> tuple[LayerInputs, int]:
    """Attention projection 4096 -> 4096 at M in {1, 8} tokens, rank 64."""
    return make_layer(M, 4096, 4096, seed=seed_for(2, M), outlier_gain=30.0,
                      sigma_w=0.02, n_cal=512), 64


def config3_prefill(which: str, M: int = 2048) -> tuple[LayerInputs, int]:
    """MLP projections at M=2048: 'gate_up' 4096 -> 14336, 'down' 14336 -> 4096, rank 64."""
    if which == "gate_up":
        return make_layer(M, 14336, 4096, seed=seed_for(3, 0), outlier_gain=30.0,
                          n_cal=512), 64
    if which == "down":
        return make_layer(M, 4096, 14336, seed=seed_for(3, 1), outlier_gain=30.0,
                          n_cal=512, gated_input=True), 64
    raise ValueError(which)


DECODER_BLOCK_LINEARS = (  # name, K (in features), N (out features)
    ("q", 4096, 4096), ("k", 4096, 1024), ("v", 4096, 1024), ("o", 4096, 4096),
    ("gate", 4096, 14336), ("up", 4096, 14336), ("down", 14336, 4096),
)


def config4_block_layer(name: str, M: int = 4096) -> tuple[LayerInputs, int]:
    """One of the seven linears of a Llama-3-8B-shaped decoder block, rank 128."""
    for i, (nm, K, N) in enumerate(DECODER_BLOCK_LINEARS):
        if nm == name:
            return make_layer(M, N, K, seed=seed_for(4, i), outlier_gain=30.0, n_cal=512), 128
    raise ValueError(name)


def config5_point(M: int, N: int, K: int = 8192) -> LayerInputs:
    """70B-class shapes: outliers x50, weights N(0, 0.015^2)."""
    return make_layer(M, N, K, seed=seed_for(5, (N // 1024) * 10000 + M), outlier_gain=50.0,
                      sigma_w=0.015, n_cal=512)


# ----------------------------------------------------------------------------
# Stand-ins for throughput runs (NOT produced by the method; values are arbitrary)
# ----------------------------------------------------------------------------

def standin_smoothing_vector(K: int, outlier_idx: np.ndarray, value: float = 24.0) -> np.ndarray:
    """A vector that is 1 everywhere and `value` on the outlier channels (fp32)."""
    s = np.ones(K, dtype=np.float32)
    s[outlier_idx] = np.float32(value)
    return s


def standin_factors(N: int, K: int, r: int, *, seed: int,
                    scale_a: float = 0.02, scale_b: float = 0.02) -> tuple[np.ndarray, np.ndarray]:
    """Dense Gaussian fp16 matrices shaped like L_A [r,K] and L_B [N,r]."""
    rng = np.random.default_rng(seed ^ 0x5EED)
    L_A = (_gauss_f32(rng, (r, K)) * np.float32(scale_a)).astype(np.float16)
    L_B = (_gauss_f32(rng, (N, r)) * np.float32(scale_b)).astype(np.float16)
    return L_A, L_B

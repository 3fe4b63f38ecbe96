"""Seeded synthetic inputs for the W4A16 linear layer (shapes and value structure only).

This module is the one place shared by the CUDA path's tests/bench and the CPU oracle's
tests.  It draws random tensors and nothing else: no part of the quantizer, the packing
or the linear layer lives here.  The tensors stand in for the Llama-2 layer weights and
activations that the paper measures on (its checkpoints and calibration text are not
available): fp16 weights ~ N(0, 0.02^2), fp16 activations ~ N(0, 1) in which a seeded 1 %
of the input channels is 20x larger (the activation-outlier structure of Sec. 3.1), and a
128-token calibration batch of the same distribution.

All draws come from a counter-based Philox stream keyed by (seed, tensor id), so any
tensor can be regenerated independently of the others and of the draw order.
"""
from __future__ import annotations

import numpy as np

_T_WEIGHT, _T_X, _T_CALIB, _T_OUTLIER = 1, 2, 3, 4

OUTLIER_FRACTION = 0.01
OUTLIER_GAIN = 20.0
WEIGHT_STD = 0.02
CALIB_TOKENS = 128


def _rng(seed: int, tensor_id: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=int(seed) * 16 + int(tensor_id)))


def _normal_f32(rng: np.random.Generator, shape) -> np.ndarray:
    return rng.standard_normal(size=shape, dtype=np.float32)


def outlier_channels(seed: int, K: int) -> np.ndarray:
    """Sorted indices of the round(1 % * K) input channels that carry 20x activations."""
    n = int(round(OUTLIER_FRACTION * K))
    return np.sort(_rng(seed, _T_OUTLIER).permutation(K)[:n])


def weight(seed: int, N: int, K: int) -> np.ndarray:
    """fp16 [N][K] row-major, ~ N(0, 0.02^2)."""
    rng = _rng(seed, _T_WEIGHT)
    out = np.empty((N, K), dtype=np.float16)
    rows = max(1, (1 << 22) // K)
    for r0 in range(0, N, rows):
        r1 = min(N, r0 + rows)
        out[r0:r1] = (_normal_f32(rng, (r1 - r0, K)) * np.float32(WEIGHT_STD)).astype(np.float16)
    return out


def _activations(rng: np.random.Generator, seed: int, M: int, K: int) -> np.ndarray:
    gain = np.ones(K, dtype=np.float32)
    gain[outlier_channels(seed, K)] = np.float32(OUTLIER_GAIN)
    return (_normal_f32(rng, (M, K)) * gain[None, :]).astype(np.float16)


def activations(seed: int, M: int, K: int) -> np.ndarray:
    """fp16 [M][K] row-major run-time activations x (before the division by s)."""
    return _activations(_rng(seed, _T_X), seed, M, K)


def calibration(seed: int, K: int, tokens: int = CALIB_TOKENS) -> np.ndarray:
    """fp16 [tokens][K]: calibration activations of the same distribution as x."""
    return _activations(_rng(seed, _T_CALIB), seed, tokens, K)


def act_mean_abs(seed: int, K: int, tokens: int = CALIB_TOKENS) -> np.ndarray:
    """fp32 [K]: per-input-channel mean magnitude of the calibration batch (sum in fp64).

    This statistic is an *input* of the library (the s_X of Eq. 5); the power alpha is
    applied by the quantizer itself, not here.
    """
    X = calibration(seed, K, tokens)
    return np.abs(X.astype(np.float64)).mean(axis=0).astype(np.float32)


# Llama-2-shaped linear layers, as (name, K_in, N_out).
LLAMA2_7B_LAYER = (
    ("q_proj", 4096, 4096), ("k_proj", 4096, 4096), ("v_proj", 4096, 4096),
    ("o_proj", 4096, 4096), ("gate_proj", 4096, 11008), ("up_proj", 4096, 11008),
    ("down_proj", 11008, 4096),
)
LLAMA2_13B_MLP = (("up_proj", 5120, 13824), ("down_proj", 13824, 5120))
LLAMA2_70B_MLP = (("up_proj", 8192, 28672), ("down_proj", 28672, 8192))

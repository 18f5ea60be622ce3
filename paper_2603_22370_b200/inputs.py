"""Seeded synthetic inputs shared by the CPU oracle's tests and the CUDA path's
tests and benchmark.  This module holds none of the method's arithmetic: it
only draws tensors with the shapes, value distributions and outlier structure
of the workloads and casts them to their storage dtype.

Every tensor comes from its own child stream of numpy's PCG64, spawned from
SeedSequence(seed) in a fixed order, so any subset can be regenerated alone.
"""
from __future__ import annotations

import numpy as np
import torch


def _streams(seed: int, n: int):
    return [np.random.Generator(np.random.PCG64(s)) for s in np.random.SeedSequence(seed).spawn(n)]


def to_bf16_f32(a: np.ndarray) -> np.ndarray:
    """Cast to BF16 storage (round to nearest even) and return the stored
    values widened back to float32."""
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(torch.bfloat16).to(torch.float32).numpy()


def weights(rng, O: int, K: int, sigma: float = 0.02, outlier_p: float = 0.0, outlier_mul: float = 1.0) -> np.ndarray:
    """sigma * N(0,1), with a Bernoulli(outlier_p) mask of entries multiplied
    by outlier_mul.  float32."""
    W = (sigma * rng.standard_normal((O, K))).astype(np.float32)
    if outlier_p > 0:
        mask = rng.random((O, K)) < outlier_p
        W = np.where(mask, W * np.float32(outlier_mul), W).astype(np.float32)
    return W


def activations_t(rng, T: int, K: int, nu: float = 4.0, n_outlier_ch: int = 16, ch_mul: float = 20.0) -> np.ndarray:
    """Student-t(nu) entries with n_outlier_ch distinct channels scaled by
    ch_mul.  float32."""
    X = rng.standard_t(nu, size=(T, K)).astype(np.float32)
    if n_outlier_ch > 0:
        ch = rng.choice(K, size=n_outlier_ch, replace=False)
        X[:, ch] *= np.float32(ch_mul)
    return X


def hidden_states(rng, T: int, H: int, n_outlier_ch: int = 8, ch_mul: float = 30.0, rms_norm: bool = True) -> np.ndarray:
    """N(0,1) hidden states with outlier channels, each row divided by its
    RMS.  float32."""
    X = rng.standard_normal((T, H)).astype(np.float32)
    if n_outlier_ch > 0:
        ch = rng.choice(H, size=n_outlier_ch, replace=False)
        X[:, ch] *= np.float32(ch_mul)
    if rms_norm:
        X = X / np.sqrt(np.mean(X.astype(np.float64) ** 2, axis=1, keepdims=True)).astype(np.float32)
    return X.astype(np.float32)


def config1(seed: int = 0, O: int = 128, K: int = 256, T: int = 1024):
    """Small parity layer: W float32 0.02*N(0,1) with 1% of entries x8;
    X float32 N(0,1).  Returns (W f32, X f32)."""
    s = _streams(seed, 2)
    W = weights(s[0], O, K, 0.02, 0.01, 8.0)
    X = s[1].standard_normal((T, K)).astype(np.float32)
    return W, X


def config2(seed: int = 0, O: int = 2048, K: int = 8192, T: int = 4096):
    """down_proj-shaped layer: W = bf16(0.02*N(0,1), 0.1% of entries x10);
    X = bf16(Student-t(4), 16 outlier channels x20).  Returned as float32
    arrays holding BF16-representable values."""
    s = _streams(seed, 2)
    W = to_bf16_f32(weights(s[0], O, K, 0.02, 0.001, 10.0))
    X = to_bf16_f32(activations_t(s[1], T, K, 4.0, min(16, K), 20.0))
    return W, X


#: (name, O, K) of the seven linears of one decoder block.
LLAMA32_1B_BLOCK = [("q_proj", 2048, 2048), ("k_proj", 512, 2048), ("v_proj", 512, 2048), ("o_proj", 2048, 2048),
                    ("gate_proj", 8192, 2048), ("up_proj", 8192, 2048), ("down_proj", 2048, 8192)]
QWEN3_1P7B_BLOCK = [("q_proj", 2048, 2048), ("k_proj", 1024, 2048), ("v_proj", 1024, 2048), ("o_proj", 2048, 2048),
                    ("gate_proj", 6144, 2048), ("up_proj", 6144, 2048), ("down_proj", 2048, 6144)]


def block_linear(seed: int, index: int, O: int, K: int, T: int):
    """One linear of a decoder block for the Stage-1 layer-wise workloads:
    W = bf16(0.02*N(0,1)); X = bf16(hidden-state distribution) with K
    channels.  `index` selects the child streams so each linear is
    independent.  Returns float32 arrays holding BF16 values."""
    s = _streams(seed, 2 * (index + 1))
    W = to_bf16_f32(weights(s[2 * index], O, K, 0.02))
    X = to_bf16_f32(hidden_states(s[2 * index + 1], T, K, min(8, K), 30.0, True))
    return W, X

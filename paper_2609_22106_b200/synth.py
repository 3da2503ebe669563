"""Seeded synthetic inputs shaped like the paper's Qwen3 layers.

This module holds none of the method's arithmetic: it only draws weights,
activations, calibration rows and MoE routings, rounds them to bf16 and hands the
same bytes to whoever asks (the CUDA path, the CPU oracle, the benchmark).  bf16
tensors are ``uint16`` numpy arrays holding the raw bit patterns.

Recipes (they stand in for the Qwen3 checkpoints and the calibration corpus the
paper used, which are not available):
  * weights:      N(0, 0.02^2), rounded to bf16;
  * activations:  Student-t(3) per element, times a per-channel lognormal(0, 1)
                  gain, times 30 on 1 % of the channels (drawn without replacement);
                  calibration rows share the gains and outlier channels;
  * tiny config:  N(0, 1) activations with 4 outlier channels times 50;
  * MoE routing:  every token picks 8 distinct experts with Zipf(1.1) popularity
                  (Gumbel top-8 on the log-probabilities), rows sorted by expert.
"""
from __future__ import annotations

import numpy as np


def f32_to_bf16(a: np.ndarray) -> np.ndarray:
    """Round float32 to bf16 (nearest even), returned as uint16 bit patterns."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32).astype(np.uint64)
    rounded = (u + 0x7FFF + ((u >> 16) & 1)) >> 16
    return rounded.astype(np.uint16)


def bf16_to_f32(h: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(h, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32)


def weights(seed: int, N: int, K: int, sigma: float = 0.02) -> np.ndarray:
    rng = np.random.default_rng(seed)
    return f32_to_bf16(rng.standard_normal((N, K), dtype=np.float32) * np.float32(sigma))


class HeavyTailChannels:
    """Per-channel structure shared by a layer's activations and its calibration rows."""

    def __init__(self, seed: int, K: int, outlier_frac: float = 0.01, outlier_gain: float = 30.0):
        rng = np.random.default_rng(seed)
        self.K = K
        self.gain = np.exp(rng.standard_normal(K)).astype(np.float32)
        n_out = int(round(outlier_frac * K))
        self.outliers = np.sort(rng.choice(K, size=n_out, replace=False)).astype(np.int64)
        self.gain[self.outliers] *= np.float32(outlier_gain)

    def rows(self, seed: int, M: int) -> np.ndarray:
        """M rows of Student-t(3) values times the channel gains, as bf16."""
        rng = np.random.default_rng(seed)
        out = np.empty((M, self.K), np.uint16)
        step = max(1, (1 << 22) // self.K)
        for r0 in range(0, M, step):
            r1 = min(M, r0 + step)
            t = rng.standard_t(3.0, size=(r1 - r0, self.K)).astype(np.float32)
            out[r0:r1] = f32_to_bf16(t * self.gain[None, :])
        return out


def tiny_config(seed: int = 0):
    """The tiny single linear: x 16 x 256 N(0,1) with 4 outlier channels x50, W 256 x 256,
    512 calibration rows with the same outlier channels, alpha grid, k = 32."""
    rng = np.random.default_rng(seed)
    M, K, N, T = 16, 256, 256, 512
    outl = np.sort(rng.choice(K, size=4, replace=False))
    gain = np.ones(K, np.float32)
    gain[outl] = 50.0
    x = f32_to_bf16(rng.standard_normal((M, K), dtype=np.float32) * gain[None, :])
    W = f32_to_bf16(rng.standard_normal((N, K), dtype=np.float32) * np.float32(0.02))
    zcal = f32_to_bf16(rng.standard_normal((T, K), dtype=np.float32) * gain[None, :])
    return dict(x=x, W=W, zcal=zcal, alphas=[0.0, 0.25, 0.5, 0.75, 1.0], k=32, outliers=outl)


def layer(config: int, N: int, K: int, M: int, T_cal: int = 512, tag: int = 0):
    """One dense linear layer of a numbered config: weights, M activation rows and T_cal
    calibration rows.  Seeds: 1000*config + 10*tag + {1: x, 2: W, 3: Z_cal, 5: channels}."""
    base = 1000 * config + 10 * tag
    ch = HeavyTailChannels(base + 5, K)
    return dict(
        W=weights(base + 2, N, K),
        x=ch.rows(base + 1, M),
        zcal=ch.rows(base + 3, T_cal),
        channels=ch,
    )


def zipf_routing(seed: int, T: int, E: int = 128, top: int = 8, s: float = 1.1):
    """Top-8 routing with Zipf(s) expert popularity.  Returns (expert_of_row sorted, offsets[E+1],
    token_of_row): rows are grouped by expert, offsets are the group boundaries."""
    rng = np.random.default_rng(seed)
    ranks = np.arange(1, E + 1, dtype=np.float64)
    logp = -s * np.log(ranks)
    expert_of_rank = rng.permutation(E)
    g = rng.gumbel(size=(T, E))
    picks_rank = np.argsort(-(logp[None, :] + g), axis=1)[:, :top]
    picks = expert_of_rank[picks_rank]
    token = np.repeat(np.arange(T), top)
    expert = picks.reshape(-1)
    order = np.argsort(expert, kind="stable")
    expert_sorted = expert[order]
    counts = np.bincount(expert_sorted, minlength=E)
    offsets = np.zeros(E + 1, np.int32)
    offsets[1:] = np.cumsum(counts)
    return expert_sorted.astype(np.int32), offsets, token[order].astype(np.int32)

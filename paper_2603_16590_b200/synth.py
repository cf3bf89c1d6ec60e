"""Seeded synthetic inputs shaped like the paper's LLM / MLLM workloads.

This module only *draws* inputs (activations, weights, transform factors, clip
ratios).  It contains none of the method's arithmetic and is the one module
that both the CUDA path's callers and the CPU oracle's callers may use.

The paper's own workloads are activations of Qwen3-8B / Qwen3-VL-8B on its
calibration and benchmark sets; model weights and datasets are not available,
so the recipes below stand in for them: Gaussian (text) or Student-t(3)
(vision-token) activations with a few outlier channels and outlier tokens,
Gaussian weights, and near-identity random transform factors in place of the
learned ones.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

GROUP = 32


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (nearest even); returns the uint16 bit patterns."""
    b = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = (b + np.uint32(0x7FFF) + ((b >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return r.astype(np.uint16)


def _rng(seed: int, stream: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[seed & 0xFFFFFFFFFFFFFFFF, stream]))


def make_activations(S: int, N: int, seed: int, *, outlier_channel_frac: float = 0.01,
                     outlier_channel_gain: float = 50.0, outlier_row_gain: float = 100.0,
                     vision_rows: int = 0) -> np.ndarray:
    """X [S, N] as bf16 bits.  Rows [0, vision_rows) are Student-t(nu=3) draws
    (heavy-tailed vision tokens); the rest are N(0,1).  max(1, floor(frac*N))
    channels are scaled by `outlier_channel_gain` (on the Gaussian rows only
    when vision rows are present, on all rows otherwise) and round(S/64) rows
    by `outlier_row_gain` (none for S < 32)."""
    g = _rng(seed, 1)
    X = g.standard_normal((S, N), dtype=np.float32)
    if vision_rows > 0:
        z = g.standard_normal((3, vision_rows, N), dtype=np.float32)
        chi = np.sqrt((z * z).sum(axis=0) / 3.0)
        X[:vision_rows] = X[:vision_rows] / chi
    n_ch = max(1, int(outlier_channel_frac * N))
    ch = _rng(seed, 2).permutation(N)[:n_ch]
    X[vision_rows:, ch] *= np.float32(outlier_channel_gain)
    n_rows = int(round(S / 64.0)) if vision_rows == 0 else 0
    if n_rows > 0:
        rows = _rng(seed, 3).permutation(S)[:n_rows]
        X[rows, :] *= np.float32(outlier_row_gain)
    return f32_to_bf16_bits(X)


def make_weight(M: int, N: int, seed: int, std: float = 0.02) -> np.ndarray:
    """W [M, N] ~ N(0, std) as bf16 bits."""
    W = _rng(seed, 4).standard_normal((M, N), dtype=np.float32) * np.float32(std)
    return f32_to_bf16_bits(W)


@dataclass
class Transform:
    """Seeded stand-in for one layer's learned parameters: the two Kronecker
    factors (a leading dimension of 1 means shared by all blocks) and the clip
    ratios.  gr x gr `left` acts on the slow index of a 32-block, gc x gc
    `right` on the contiguous index."""
    n: int
    left: np.ndarray    # [1 or k, gr, gr] float32
    right: np.ndarray   # [1 or k, gc, gc] float32
    clip_lo: np.ndarray | None  # [k] float32 ratios in (0, 1]
    clip_hi: np.ndarray | None

    @property
    def k(self) -> int:
        return self.n // GROUP


def _near_identity(g: np.random.Generator, n: int, max_cond: float) -> np.ndarray:
    # I + 0.1 N(0,1) for the 4 x 4 and 8 x 8 factors of the benchmark configurations; larger factors
    # (the ablation's other sizes) get the noise scaled by sqrt(8 / n) so that its spectral norm,
    # and with it the condition number, stays where the 8 x 8 case has it
    amp = 0.1 * min(1.0, (8.0 / n) ** 0.5)
    while True:
        m = np.eye(n) + amp * g.standard_normal((n, n))
        if np.linalg.cond(m, 2) <= max_cond:
            return m.astype(np.float32)


def make_transform(N: int, seed: int, geometry: str = "baseline", clip: bool = True,
                   identity: bool = False, gr: int = 4, gc: int = 8) -> Transform:
    """geometry "baseline": shared 4x4 left factor, private 8x8 right factors
    (the benchmark configs' "G (x) P_j").  geometry "paper": private 4x4 left
    factors B_j, shared 8x8 right factor A (the paper's default g1=8, g2=4).
    geometry "naive": both private.  Entries are I + 0.1*N(0,1); the shared
    factor is redrawn until its 2-norm condition number is <= 3 and each
    private one until cond(left)*cond(right) <= 10.  gr x gc is the factorisation of
    the 32-block (4 x 8 unless stated; the paper's ablation varies it)."""
    k = N // GROUP
    g = _rng(seed, 5)
    assert gr * gc == GROUP
    if identity:
        left = np.eye(gr, dtype=np.float32)[None]
        right = np.eye(gc, dtype=np.float32)[None]
    elif geometry == "baseline":
        left = _near_identity(g, gr, 3.0)[None]
        cl = np.linalg.cond(left[0].astype(np.float64), 2)
        right = np.stack([_near_identity(g, gc, 10.0 / cl) for _ in range(k)])
    elif geometry == "paper":
        right = _near_identity(g, gc, 3.0)[None]
        cr = np.linalg.cond(right[0].astype(np.float64), 2)
        left = np.stack([_near_identity(g, gr, 10.0 / cr) for _ in range(k)])
    elif geometry == "naive":
        left = np.stack([_near_identity(g, gr, 3.0) for _ in range(k)])
        right = np.stack([_near_identity(g, gc, 10.0 / np.linalg.cond(left[j].astype(np.float64), 2))
                          for j in range(k)])
    else:
        raise ValueError(geometry)
    if clip:
        alpha = _rng(seed, 6).uniform(0.8, 1.0, size=k).astype(np.float32)
        lo, hi = alpha, alpha.copy()
    else:
        lo = hi = None
    return Transform(N, left, right, lo, hi)


# ---- the benchmark configurations ------------------------------------------------
LLAMA8B_PREFILL = [  # (name, N in, M out) at S = 2048 tokens
    ("qkv", 4096, 6144), ("o", 4096, 4096), ("gate_up", 4096, 28672), ("down", 14336, 4096)]
QWEN2VL7B_PREFILL = [  # S = 8192 tokens, 75 % vision rows
    ("qkv", 3584, 4608), ("o", 3584, 3584), ("gate_up", 3584, 37888), ("down", 18944, 3584)]
BASE_SEED = 0xBA7C0000

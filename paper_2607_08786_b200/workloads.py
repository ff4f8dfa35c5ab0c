"""Seeded synthetic inputs shaped like the paper's workloads.

The paper measures on Wanda-pruned OPT/Llama linear layers (Sec. 5); those weights are not
available, so these generators stand in for them: same shapes, ~50 % unstructured density,
LLM-like value scale.  This module holds input generation only -- none of the storage format's
or the kernel's arithmetic -- so that both the library's tests and the CPU oracle's tests can
draw the same inputs from it.

Random streams: ``numpy.random.default_rng([seed, stream])`` with stream 0 = weights,
1 = mask / calibration activations, 2 = X, 3 = per-row scales.  Values are drawn in float32 and
rounded to float16 (round-to-nearest-even).  Masks are applied by *selection*, so a pruned weight
is +0.0, never -0.0.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Iterator

import numpy as np

STREAM_W, STREAM_MASK, STREAM_X, STREAM_SCALE = 0, 1, 2, 3


def _rng(seed: int, stream: int) -> np.random.Generator:
    return np.random.default_rng([seed, stream])


def _normal_f16(rng: np.random.Generator, shape, sigma: float, block_rows: int = 4096) -> np.ndarray:
    out = np.empty(shape, dtype=np.float16)
    for r in range(0, shape[0], block_rows):
        n = min(block_rows, shape[0] - r)
        out[r:r + n] = (rng.standard_normal((n, shape[1]), dtype=np.float32) * np.float32(sigma)).astype(np.float16)
    return out


def weights(seed: int, M: int, K: int, sigma: float = 0.02) -> np.ndarray:
    """fp16 weights ~ N(0, sigma)."""
    return _normal_f16(_rng(seed, STREAM_W), (M, K), sigma)


def weights_row_scaled(seed: int, M: int, K: int, lo: float = 0.005, hi: float = 0.05) -> np.ndarray:
    """Row r ~ N(0, sigma_r) with sigma_r log-uniform in [lo, hi]."""
    rng_s = _rng(seed, STREAM_SCALE)
    sig = np.exp(rng_s.uniform(np.log(lo), np.log(hi), size=M)).astype(np.float32)
    rng = _rng(seed, STREAM_W)
    out = np.empty((M, K), dtype=np.float16)
    for r in range(0, M, 4096):
        n = min(4096, M - r)
        out[r:r + n] = (rng.standard_normal((n, K), dtype=np.float32) * sig[r:r + n, None]).astype(np.float16)
    return out


def activations(seed: int, K: int, N: int) -> np.ndarray:
    """X (K x N) fp16 ~ N(0, 1)."""
    return _normal_f16(_rng(seed, STREAM_X), (K, N), 1.0)


def mask_bernoulli(seed: int, M: int, K: int, keep: float = 0.5) -> np.ndarray:
    """i.i.d. keep-mask."""
    rng = _rng(seed, STREAM_MASK)
    out = np.empty((M, K), dtype=bool)
    for r in range(0, M, 4096):
        n = min(4096, M - r)
        out[r:r + n] = rng.random((n, K), dtype=np.float32) < np.float32(keep)
    return out


def mask_topk_per_row(score: np.ndarray, sparsity: float) -> np.ndarray:
    """Keep the ``K - round(sparsity*K)`` highest scores of each row; ties go to the lower column.

    ``score`` must be non-negative.  Same result as a stable descending sort of each row.
    """
    M, K = score.shape
    keep = K - int(round(sparsity * K))
    out = np.zeros((M, K), dtype=bool)
    if keep <= 0:
        return out
    if keep >= K:
        out[:] = True
        return out
    for r0 in range(0, M, 1024):
        s = score[r0:r0 + 1024]
        thr = np.partition(s, K - keep, axis=1)[:, K - keep][:, None]   # keep-th largest value
        above = s > thr
        need = keep - above.sum(axis=1, keepdims=True)                  # how many ties to take
        tie = s == thr
        take = tie & (np.cumsum(tie, axis=1) <= need)
        out[r0:r0 + 1024] = above | take
    return out


def prune_magnitude(W: np.ndarray, sparsity: float) -> np.ndarray:
    """Per-output-row magnitude pruning on the fp16 values; returns the masked fp16 matrix."""
    mask = mask_topk_per_row(np.abs(W), sparsity)
    return np.where(mask, W, np.float16(0))


def prune_wanda_like(W: np.ndarray, seed: int, sparsity: float = 0.5, calib_rows: int = 128,
                     channel_scales: bool = True) -> np.ndarray:
    """Per-row top-half of the score |w_ik| * ||c_k||_2 over a seeded calibration matrix C.

    ``C`` is ``calib_rows x K``, N(0,1), optionally times a per-channel scale exp(0.5*N(0,1)) so
    that some input channels are outliers (which makes the mask column-correlated).
    """
    K = W.shape[1]
    rng = _rng(seed, STREAM_MASK)
    C = rng.standard_normal((calib_rows, K), dtype=np.float32)
    if channel_scales:
        C *= np.exp(0.5 * rng.standard_normal(K, dtype=np.float32))[None, :]
    norm = np.sqrt((C.astype(np.float64) ** 2).sum(axis=0)).astype(np.float32)
    mask = np.zeros(W.shape, dtype=bool)
    for r0 in range(0, W.shape[0], 2048):
        score = np.abs(W[r0:r0 + 2048].astype(np.float32)) * norm[None, :]
        mask[r0:r0 + 2048] = mask_topk_per_row(score, sparsity)
    return np.where(mask, W, np.float16(0))


@dataclass(frozen=True)
class Case:
    """One SpMM problem: how to draw W, its mask, and X."""
    config: int
    name: str
    M: int
    K: int
    N: int
    seed: int
    sparsity: float = 0.5
    kind: str = "magnitude"      # "bernoulli" | "magnitude" | "row_scaled" | "wanda"

    def make_W(self) -> np.ndarray:
        if self.kind == "bernoulli":
            W = weights(self.seed, self.M, self.K)
            return np.where(mask_bernoulli(self.seed, self.M, self.K, 1.0 - self.sparsity), W, np.float16(0))
        if self.kind == "magnitude":
            return prune_magnitude(weights(self.seed, self.M, self.K), self.sparsity)
        if self.kind == "row_scaled":
            return prune_magnitude(weights_row_scaled(self.seed, self.M, self.K), self.sparsity)
        if self.kind == "wanda":
            return prune_wanda_like(weights(self.seed, self.M, self.K), self.seed, self.sparsity)
        raise ValueError(self.kind)

    def make_X(self) -> np.ndarray:
        return activations(self.seed, self.K, self.N)


CONFIG2_SHAPES = ((5120, 5120), (20480, 5120), (5120, 20480))
CONFIG3_SHAPES = ((4096, 4096), (11008, 4096), (4096, 11008))
CONFIG4_SHAPES = ((9216, 9216), (36864, 9216), (9216, 36864))
CONFIG5_SHAPES = ((21504, 7168), (7168, 7168), (28672, 7168), (7168, 28672))


def config_cases(config: int) -> Iterator[Case]:
    """The five workload configurations (shapes, masks, seeds)."""
    if config == 1:
        yield Case(1, "c1_1024x1024_n8", 1024, 1024, 8, 0, 0.5, "bernoulli")
    elif config == 2:
        for si, (M, K) in enumerate(CONFIG2_SHAPES):
            for N in (8, 16, 32):
                yield Case(2, f"c2_{M}x{K}_n{N}", M, K, N, 2000 + 10 * si, 0.5, "magnitude")
    elif config == 3:
        for si, (M, K) in enumerate(CONFIG3_SHAPES):
            for pi, sp in enumerate((0.4, 0.5, 0.6, 0.7)):
                yield Case(3, f"c3_{M}x{K}_s{int(sp * 100)}_n16", M, K, 16, 3000 + 10 * si + pi, sp, "magnitude")
    elif config == 4:
        for si, (M, K) in enumerate(CONFIG4_SHAPES):
            for N in (8, 32, 64):
                yield Case(4, f"c4_{M}x{K}_n{N}", M, K, N, 4000 + 10 * si, 0.5, "row_scaled")
    elif config == 5:
        for si, (M, K) in enumerate(CONFIG5_SHAPES):
            yield Case(5, f"c5_{M}x{K}_n16", M, K, 16, 5000 + 10 * si, 0.5, "wanda")
    else:
        raise ValueError(f"no config {config}")

"""Seeded synthetic inputs for the LUT-linear hot path.

This module only *makes data*: random weights and activations with the shape and
distribution of the paper's workloads (Gaussian-like weights, activations with a few
outlier channels, Section 3.4 / Section 5 set-up), a SmoothQuant-style smoothing
vector, and a clustered stand-in for the trained model (per-row quantile codebook +
nearest-centroid assignment).  None of the method's own arithmetic (index packing,
activation index assignment, table lookup / accumulation) lives here, so both the CPU
oracle and the CUDA path can be fed from it without sharing any code of the method.

The random numbers come from a counter-based generator written out below
(splitmix64 -> Box-Muller), so a (seed, counter) pair always gives the same value and
tensors do not depend on the RNG of numpy or torch.
"""
from __future__ import annotations

import dataclasses
import numpy as np

BASE_SEED = 250612038

_U64 = np.uint64
_MASK = (1 << 64) - 1


def splitmix64(seed: int, counters: np.ndarray) -> np.ndarray:
    """splitmix64 output function applied to seed + (counter+1)*golden (vectorised, wraps mod 2^64)."""
    with np.errstate(over="ignore"):
        z = (counters.astype(_U64) + _U64(1)) * _U64(0x9E3779B97F4A7C15) + _U64(seed & _MASK)
        z = (z ^ (z >> _U64(30))) * _U64(0xBF58476D1CE4E5B9)
        z = (z ^ (z >> _U64(27))) * _U64(0x94D049BB133111EB)
        z = z ^ (z >> _U64(31))
    return z


def uniform01(seed: int, n: int, offset: int = 0) -> np.ndarray:
    """n doubles in (0, 1], counter-based."""
    c = np.arange(offset, offset + n, dtype=_U64)
    return ((splitmix64(seed, c) >> _U64(11)).astype(np.float64) + 1.0) * (1.0 / 9007199254740992.0)


def normal(seed: int, n: int, chunk: int = 1 << 22) -> np.ndarray:
    """n standard normals (float64) by Box-Muller over counter pairs; element i depends on (seed, i) only."""
    out = np.empty(n + (n & 1), dtype=np.float64)
    half = out.size // 2
    for lo in range(0, half, chunk):
        hi = min(half, lo + chunk)
        u1 = uniform01(seed, hi - lo, 2 * lo)          # counters [2lo, lo+hi): radius
        u2 = uniform01(seed ^ 0x5DEECE66D, hi - lo, 2 * lo)
        r = np.sqrt(-2.0 * np.log(u1))
        t = (2.0 * np.pi) * u2
        out[2 * lo:2 * hi:2] = r * np.cos(t)
        out[2 * lo + 1:2 * hi:2] = r * np.sin(t)
    return out[:n]


def permutation(seed: int, n: int) -> np.ndarray:
    """A seeded permutation of range(n): argsort of counter-based keys (stable)."""
    keys = splitmix64(seed, np.arange(n, dtype=_U64))
    return np.argsort(keys, kind="stable")


def seed_for(config: int, matrix: int, role: int) -> int:
    """role: 0 weights, 1 test tokens, 2 calibration batch, 3 outlier permutation."""
    return BASE_SEED + 1000 * config + 10 * matrix + role


@dataclasses.dataclass
class LayerInputs:
    N: int
    K: int
    bits: int
    C: int
    M: int
    x: np.ndarray          # fp16 [M, K] test tokens
    inv_s: np.ndarray      # fp32 [K]   1 / smoothing factor
    s: np.ndarray          # fp32 [K]   smoothing factor
    codebook: np.ndarray   # fp16 [N, C]
    idx: np.ndarray        # uint8 [N, K] centroid index per weight
    outlier_channels: np.ndarray


def outlier_channels(seed: int, K: int, frac: float) -> np.ndarray:
    n_out = int(np.ceil(frac * K)) if frac > 0 else 0
    return np.sort(permutation(seed, K)[:n_out])


def activations(seed: int, M: int, K: int, channels: np.ndarray, scale: float) -> np.ndarray:
    """fp16 [M, K]: N(0,1) with the given channels multiplied by `scale` (in fp32) before rounding to fp16."""
    x = normal(seed, M * K).astype(np.float32).reshape(M, K)
    if channels.size:
        x[:, channels] *= np.float32(scale)
    return x.astype(np.float16)


def smoothing_vector(calib: np.ndarray, w_absmax: np.ndarray, alpha: float = 0.5) -> np.ndarray:
    """Per-input-channel smoothing s_k = max|x_k|^alpha / max_n|W_nk|^(1-alpha), clamped to [1e-5, 1e5];
    a channel whose activation or weight maximum is zero gets s_k = 1.  float32."""
    ax = np.abs(calib.astype(np.float64)).max(axis=0)
    aw = w_absmax.astype(np.float64)
    s = np.ones_like(ax)
    ok = (ax > 0) & (aw > 0)
    s[ok] = ax[ok] ** alpha / aw[ok] ** (1.0 - alpha)
    return np.clip(s, 1e-5, 1e5).astype(np.float32)


def cluster_rows(Ws: np.ndarray, C: int) -> tuple[np.ndarray, np.ndarray]:
    """Stand-in for a trained clustering: per output row, C fp16 centroids at the row's (i+0.5)/C quantiles
    (sorted[floor((i+0.5)/C*K)]) and, per weight, the index of the nearest centroid (lowest index on ties)."""
    N, K = Ws.shape
    pos = np.floor((np.arange(C) + 0.5) / C * K).astype(np.int64)
    cb = np.empty((N, C), dtype=np.float16)
    idx = np.empty((N, K), dtype=np.uint8)
    step = max(1, (1 << 22) // max(K, 1))
    for lo in range(0, N, step):
        blk = Ws[lo:lo + step].astype(np.float64)
        srt = np.sort(blk, axis=1)
        cbb = srt[:, pos].astype(np.float16)
        cb[lo:lo + step] = cbb
        c64 = cbb.astype(np.float64)
        best = np.abs(blk - c64[:, 0:1])
        bi = np.zeros(blk.shape, dtype=np.uint8)
        for w in range(1, C):
            d = np.abs(blk - c64[:, w:w + 1])
            better = d < best
            bi[better] = w
            best = np.where(better, d, best)
        idx[lo:lo + step] = bi
    return cb, idx


def make_layer(config: int, matrix: int, N: int, K: int, bits: int, M: int, C: int | None = None,
               outlier_frac: float = 0.01, outlier_scale: float = 50.0, calib_tokens: int = 128,
               sigma_w: float = 0.02) -> LayerInputs:
    """Everything one (matrix, M) case needs: weights N(0, sigma_w) -> smoothed by s -> clustered; test tokens
    and a separate calibration batch drawn with the same outlier channels."""
    C = (1 << bits) if C is None else C
    ch = outlier_channels(seed_for(config, matrix, 3), K, outlier_frac)
    x = activations(seed_for(config, matrix, 1), M, K, ch, outlier_scale)
    calib = activations(seed_for(config, matrix, 2), calib_tokens, K, ch, outlier_scale)
    W = (normal(seed_for(config, matrix, 0), N * K) * sigma_w).astype(np.float32).reshape(N, K)
    s = smoothing_vector(calib, np.abs(W).max(axis=0))
    inv_s = (np.float32(1.0) / s).astype(np.float32)
    Ws = W * s[None, :]
    cb, idx = cluster_rows(Ws, C)
    return LayerInputs(N=N, K=K, bits=bits, C=C, M=M, x=x, inv_s=inv_s, s=s, codebook=cb, idx=idx,
                       outlier_channels=ch)


def random_case(seed: int, N: int, K: int, bits: int, M: int, C: int | None = None,
                outlier_frac: float = 0.01, outlier_scale: float = 50.0) -> LayerInputs:
    """A small free-form case for tests (same recipe, arbitrary seed)."""
    return make_layer(config=seed, matrix=0, N=N, K=K, bits=bits, M=M, C=C,
                      outlier_frac=outlier_frac, outlier_scale=outlier_scale)


# Workloads named by the benchmark configurations (shapes of LLaMA projections).
LLAMA7B = [("q", 4096, 4096), ("k", 4096, 4096), ("v", 4096, 4096), ("o", 4096, 4096),
           ("gate", 11008, 4096), ("up", 11008, 4096), ("down", 4096, 11008)]
LLAMA13B = [("q", 5120, 5120), ("k", 5120, 5120), ("v", 5120, 5120), ("o", 5120, 5120),
            ("gate", 13824, 5120), ("up", 13824, 5120), ("down", 5120, 13824)]
LLAMA70B_MLP = [("gate", 28672, 8192), ("up", 28672, 8192), ("down", 8192, 28672)]

CONFIGS = {
    0: dict(name="single-4096-3bit-M1", shapes=[("w", 4096, 4096)], bits=3, Ms=[1], frac=0.01, scale=50.0),
    1: dict(name="llama7b-2bit-M1", shapes=LLAMA7B, bits=2, Ms=[1], frac=0.01, scale=50.0),
    2: dict(name="llama7b-3bit-M4-16", shapes=LLAMA7B, bits=3, Ms=[4, 16], frac=0.01, scale=50.0),
    3: dict(name="llama13b-2bit-M2048", shapes=LLAMA13B, bits=2, Ms=[2048], frac=0.01, scale=50.0),
    4: dict(name="llama70b-mlp-2bit-M1-8", shapes=LLAMA70B_MLP, bits=2, Ms=[1, 8], frac=0.005, scale=100.0),
    # ten centroids per row in 4-bit indices: the paper's 3.3-bit operating point
    5: dict(name="llama7b-4bit-10centroids-M1-16", shapes=LLAMA7B, bits=4, C=10, Ms=[1, 16], frac=0.01, scale=50.0),
}

"""Seeded synthetic inputs shaped like the paper's LLM layers (Section 5, "Workloads").

This module only MAKES inputs: weight matrices, pruning masks, activation vectors and the
threshold that yields a requested activation density.  It contains none of the method's
arithmetic (no encoding, no thresholding decision, no product) and is the one module both
the CUDA path's tests/benchmarks and the CPU oracle's tests draw their inputs from.

Random numbers come from a counter-based generator, so any element can be produced
independently of the others and of the library versions installed:
    u(seed, tag, i) = mix64(mix64(seed * 256 + tag) + (i + 1) * GOLDEN) >> 11, scaled by 2^-53
with mix64 the SplitMix64 output function.
"""
from __future__ import annotations

import os

import numpy as np

_GOLDEN = np.uint64(0x9E3779B97F4A7C15)
_C1 = np.uint64(0xBF58476D1CE4E5B9)
_C2 = np.uint64(0x94D049BB133111EB)
_CHUNK = 1 << 22


def _mix64(z: np.ndarray) -> np.ndarray:
    z = z.astype(np.uint64, copy=True)
    z ^= z >> np.uint64(30)
    z *= _C1
    z ^= z >> np.uint64(27)
    z *= _C2
    z ^= z >> np.uint64(31)
    return z


def _key(seed: int, tag: int) -> np.uint64:
    k = np.array([(int(seed) * 256 + int(tag)) & 0xFFFFFFFFFFFFFFFF], dtype=np.uint64)
    return _mix64(k)[0]


def uniform(seed: int, tag: int, n: int, start: int = 0) -> np.ndarray:
    """n doubles in [0, 1), elements start .. start+n-1 of stream (seed, tag).  Every element depends only on
    its own counter, so large requests are filled chunk by chunk on a few threads (same values either way)."""
    out = np.empty(n, np.float64)
    key = _key(seed, tag)

    def fill(a):
        b = min(n, a + _CHUNK)
        with np.errstate(over="ignore"):
            ctr = np.arange(start + a + 1, start + b + 1, dtype=np.uint64)
            ctr *= _GOLDEN
            ctr += key
            z = _mix64(ctr)
            z >>= np.uint64(11)
        np.multiply(z, 1.0 / 9007199254740992.0, out=out[a:b])

    starts = range(0, n, _CHUNK)
    if n <= 4 * _CHUNK:
        for a in starts:
            fill(a)
    else:
        from concurrent.futures import ThreadPoolExecutor
        with ThreadPoolExecutor(min(16, os.cpu_count() or 1)) as pool:
            list(pool.map(fill, starts))
    return out


def normal(seed: int, tag: int, n: int) -> np.ndarray:
    """Standard normal by Box-Muller on streams tag and tag+1."""
    u1 = uniform(seed, tag, n)
    u2 = uniform(seed, tag + 1, n)
    return np.sqrt(-2.0 * np.log(1.0 - u1)) * np.cos(2.0 * np.pi * u2)     # 1 - u1 is exact


def laplace(seed: int, tag: int, n: int) -> np.ndarray:
    """Laplace(0, 1) by inverse CDF."""
    u = uniform(seed, tag, n) - 0.5
    return -np.sign(u) * np.log(1.0 - 2.0 * np.abs(u))


# ----------------------------------------------------------------------------- weights / masks
def weights(seed: int, M: int, K: int, std: float = 0.02) -> np.ndarray:
    """FP16 M x K row-major weights ~ N(0, std^2)."""
    return (normal(seed, 1, M * K) * std).astype(np.float16).reshape(M, K)


def weights_tiled(seed: int, M: int, K: int, block_cols: int, std: float = 0.02) -> np.ndarray:
    """FP16 M x K weights whose columns repeat a block of `block_cols` columns ~ N(0, std^2) along K.  For the
    largest layers, where drawing every weight would take minutes: which weights are kept comes from the mask,
    which is never repeated, so no two columns hold the same entries."""
    block = weights(seed, M, min(K, block_cols), std)
    reps = -(-K // block.shape[1])
    return np.ascontiguousarray(np.tile(block, (1, reps))[:, :K])


def integer_weights(seed: int, M: int, K: int, amp: int = 3) -> np.ndarray:
    """FP16 weights with small integer values in [-amp, amp] (exactly summable in fp32)."""
    u = uniform(seed, 7, M * K)
    return (np.floor(u * (2 * amp + 1)) - amp).astype(np.float16).reshape(M, K)


def mask_bernoulli(seed: int, M: int, K: int, d_w: float) -> np.ndarray:
    """Uniform-random unstructured mask: each element kept independently with probability d_w."""
    return (uniform(seed, 3, M * K) < d_w).reshape(M, K).astype(np.uint8)


def mask_magnitude(W: np.ndarray, sparsity: float) -> np.ndarray:
    """Per-column magnitude pruning: drop the floor(sparsity * M) smallest |W_ij| of each column.

    Ties go to the lower row index first (stable sort)."""
    M, K = W.shape
    n_drop = int(np.floor(sparsity * M))
    mask = np.ones((M, K), np.uint8)
    if n_drop > 0:
        order = np.argsort(np.abs(W.astype(np.float32)), axis=0, kind="stable")
        np.put_along_axis(mask, order[:n_drop, :], 0, axis=0)
    return mask


def powerlaw_row_probability(M: int, d_w: float) -> np.ndarray:
    """Row-clustered keep probability p_i = min(1, c / (i + 1)) with mean d_w (heavy rows first)."""
    i = np.arange(1, M + 1, dtype=np.float64)
    lo, hi = 0.0, float(M)
    for _ in range(200):
        c = 0.5 * (lo + hi)
        if np.minimum(1.0, c / i).mean() < d_w:
            lo = c
        else:
            hi = c
    return np.minimum(1.0, 0.5 * (lo + hi) / i)


def mask_powerlaw(seed: int, M: int, K: int, d_w: float) -> np.ndarray:
    """Row-clustered mask: element (i, j) kept with probability p_i (power law in the row index)."""
    p = powerlaw_row_probability(M, d_w)
    return (uniform(seed, 5, M * K).reshape(M, K) < p[:, None]).astype(np.uint8)


# ----------------------------------------------------------------------------- activations
def activations(seed: int, K: int, dist: str = "laplace") -> np.ndarray:
    """FP16 activation vector: 'laplace' (Laplace(0,1)), 'normal' (N(0,1)) or
    'swiglu' (SiLU(g) * u of two independent N(0,1) FP16 vectors, the down-projection input)."""
    if dist == "laplace":
        return laplace(seed, 11, K).astype(np.float16)
    if dist == "normal":
        return normal(seed, 13, K).astype(np.float16)
    if dist == "swiglu":
        g = normal(seed, 15, K).astype(np.float16).astype(np.float64)
        u = normal(seed, 17, K).astype(np.float16).astype(np.float64)
        return (g / (1.0 + np.exp(-g)) * u).astype(np.float16)
    raise ValueError(dist)


def integer_activations(seed: int, K: int, amp: int = 4) -> np.ndarray:
    u = uniform(seed, 19, K)
    return (np.floor(u * (2 * amp + 1)) - amp).astype(np.float16)


def threshold_for_density(x: np.ndarray, d_a: float) -> float:
    """tau = the floor((1 - d_a) * K)-th smallest |x| (1-based), 0 if that index is 0.

    With a comparator that keeps only magnitudes strictly above tau, at most a fraction d_a
    of the entries survives (ties at tau are dropped)."""
    K = x.size
    k = int(np.floor((1.0 - d_a) * K))
    if k <= 0:
        return 0.0
    mags = np.sort(np.abs(x.astype(np.float32)))
    return float(mags[k - 1])


def point_seed(config: int, point: int, base: int = 1536) -> int:
    return base * 1000 + 100 * config + point

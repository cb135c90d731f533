"""Seeded synthetic inputs shaped like the paper's workloads (host side, numpy only).

This module holds NO arithmetic of the method: it only draws matrices, labels
and vectors.  The same arrays are handed to the CUDA library and to the CPU
oracle, so both see identical bits.  Generators are ``numpy.random.Generator``
over ``PCG64`` with fixed seeds; nothing is cached on disk.

The paper's experiments (Section 5) use real-sim / rcv1 (sparse text features,
logistic regression) and MNIST.  Those files are not available; the sparse
generators below stand in for the text workloads (Poisson row lengths, Zipf
column popularity, log-normal tf-idf-like values, unit-L2 rows), the dense
ones for small dense problems.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Optional

import numpy as np

DENSE_F32, CSR_F32, DENSE_BF16 = 0, 1, 2
BASE_SEED = 180510111


@dataclass
class HostData:
    format: int
    n: int
    d: int
    values: np.ndarray                   # dense: [n, d] float32 or uint16 (bf16 bits); CSR: [nnz] float32
    labels: np.ndarray                   # [n] float32, +-1
    col_idx: Optional[np.ndarray] = None  # CSR: [nnz] int32
    row_ptr: Optional[np.ndarray] = None  # CSR: [n+1] int64


def rng(k: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(BASE_SEED + k))


def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even conversion of float32 to bfloat16 bit patterns (uint16)."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    bias = ((u >> 16) & 1) + np.uint32(0x7FFF)
    return ((u + bias) >> 16).astype(np.uint16)


def bf16_bits_to_f32(h: np.ndarray) -> np.ndarray:
    return (h.astype(np.uint32) << 16).view(np.float32)


def dense_logistic(n: int, d: int, seed_k: int, flip: float = 0.05, normalise: bool = True) -> HostData:
    """i.i.d. N(0,1) features, rows scaled to unit L2, labels = sign(X w*) with a fraction flipped."""
    g = rng(seed_k)
    X = g.standard_normal((n, d), dtype=np.float32)
    if normalise:
        X /= np.linalg.norm(X, axis=1, keepdims=True).astype(np.float32)
    w = g.standard_normal(d, dtype=np.float32)
    y = np.where(X @ w >= 0, 1.0, -1.0).astype(np.float32)
    y[g.random(n) < flip] *= -1.0
    return HostData(DENSE_F32, n, d, np.ascontiguousarray(X), y)


def dense_bf16_logistic(n: int, d: int, seed_k: int) -> HostData:
    """N(0,1) features rounded to bf16, labels from a seeded N(0,1) teacher (no flips)."""
    g = rng(seed_k)
    bits = np.empty((n, d), np.uint16)
    w = g.standard_normal(d, dtype=np.float32) / np.float32(np.sqrt(d))
    score = np.empty(n, np.float32)
    step = max(1, (1 << 24) // d)
    for r in range(0, n, step):
        blk = g.standard_normal((min(step, n - r), d), dtype=np.float32)
        bits[r:r + blk.shape[0]] = f32_to_bf16_bits(blk)
        score[r:r + blk.shape[0]] = bf16_bits_to_f32(bits[r:r + blk.shape[0]]) @ w
    y = np.where(score >= 0, 1.0, -1.0).astype(np.float32)
    return HostData(DENSE_BF16, n, d, bits, y)


def sparse_logistic(n: int, d: int, mean_nnz: float, zipf_a: float, seed_k: int) -> HostData:
    """CSR rows with max(1, Poisson(mean_nnz)) draws of Zipf(zipf_a)-popular columns (rank -> id by a
    fixed permutation, duplicates inside a row merged), log-normal(0,1) values, unit-L2 rows, and
    balanced +-1 labels from a seeded teacher thresholded at the median score."""
    g = rng(seed_k)
    cnt = np.maximum(1, g.poisson(mean_nnz, n)).astype(np.int64)
    total = int(cnt.sum())
    wts = np.arange(1, d + 1, dtype=np.float64) ** (-zipf_a)
    cdf = np.cumsum(wts); cdf /= cdf[-1]
    rank = np.searchsorted(cdf, g.random(total), side="right").clip(0, d - 1)
    perm = g.permutation(d)
    col = perm[rank].astype(np.int64)
    row = np.repeat(np.arange(n, dtype=np.int64), cnt)
    key = np.unique(row * d + col)                         # sorted by (row, col), duplicates merged
    row, col = key // d, (key % d).astype(np.int32)
    val = g.lognormal(0.0, 1.0, key.size).astype(np.float32)
    row_ptr = np.zeros(n + 1, np.int64)
    np.add.at(row_ptr, row + 1, 1)
    row_ptr = np.cumsum(row_ptr)
    sq = np.add.reduceat(val.astype(np.float64) ** 2, row_ptr[:-1])
    val = (val / np.sqrt(sq)[row]).astype(np.float32)
    w = g.standard_normal(d, dtype=np.float32)
    score = np.add.reduceat(val.astype(np.float64) * w[col], row_ptr[:-1])
    y = np.where(score >= np.median(score), 1.0, -1.0).astype(np.float32)
    return HostData(CSR_F32, n, d, val, y, col_idx=col, row_ptr=row_ptr)


def outlier_vectors(M: int, d: int, seed_k: int, frac: float = 1e-3, scale: float = 100.0) -> np.ndarray:
    """[M, d] float32 N(0,1) with a fraction ``frac`` of the entries multiplied by ``scale``."""
    g = rng(seed_k)
    out = np.empty((M, d), np.float32)
    for w in range(M):
        v = g.standard_normal(d, dtype=np.float32)
        k = max(1, int(round(frac * d)))
        v[g.integers(0, d, k)] *= np.float32(scale)
        out[w] = v
    return out


def normal_vector(d: int, seed_k: int, scale: float = 1.0) -> np.ndarray:
    return (rng(seed_k).standard_normal(d, dtype=np.float32) * np.float32(scale)).astype(np.float32)


def image_classification(n: int, n_in: int, classes: int, seed_k: int) -> HostData:
    """Inputs shaped like small grey-scale images (values in [0,1], about 80 % exactly zero, the rest a smooth
    random blob per class plus noise) with the class index as label: stands in for the MNIST subset of Section 5.2."""
    g = rng(seed_k)
    proto = g.random((classes, n_in), dtype=np.float32) ** 4                  # class prototypes, mostly dark
    y = g.integers(0, classes, n)
    X = proto[y] + np.float32(0.15) * g.standard_normal((n, n_in), dtype=np.float32)
    X = np.clip(X, 0.0, 1.0).astype(np.float32)
    X[X < 0.35] = 0.0
    return HostData(DENSE_F32, n, n_in, np.ascontiguousarray(X), y.astype(np.float32))


def mlp_init(n_in: int, hidden: int, classes: int, seed_k: int) -> np.ndarray:
    """Small random weights, zero biases, in the flat layout [W1, b1, W2, b2]."""
    g = rng(seed_k)
    w1 = g.standard_normal((hidden, n_in), dtype=np.float32) * np.float32(1.0 / np.sqrt(n_in))
    w2 = g.standard_normal((classes, hidden), dtype=np.float32) * np.float32(1.0 / np.sqrt(hidden))
    return np.concatenate([w1.ravel(), np.zeros(hidden, np.float32), w2.ravel(), np.zeros(classes, np.float32)]).astype(np.float32)


# ---- the five configurations ---------------------------------------------------------------------------
def config1() -> HostData:
    """Tiny dense L1 logistic regression: n=2,000, d=1,000."""
    return dense_logistic(2000, 1000, 1)


def config2(n: int = 72309, d: int = 20958) -> HostData:
    """Text-classification-shaped CSR: Poisson(52) row lengths, Zipf(1.1) columns."""
    return sparse_logistic(n, d, 52.0, 1.1, 2)


def config3(n: int = 200000, d: int = 1 << 20) -> HostData:
    """Wide sparse CSR: Poisson(100) row lengths, Zipf(1.2) columns."""
    return sparse_logistic(n, d, 100.0, 1.2, 3)


def config4(n: int = 65536, d: int = 4096) -> HostData:
    """Dense bf16 features for the tensor-core path."""
    return dense_bf16_logistic(n, d, 4)


def config_nn(n: int = 10000):
    """MNIST-shaped classification data for the 3-layer network (784-100-10)."""
    return image_classification(n, 784, 10, 8)


def config5(d: int, M: int = 8):
    """Quantiser sweep inputs: M outlier vectors, a model x and a full gradient."""
    return outlier_vectors(M, d, 5), normal_vector(d, 6), normal_vector(d, 7)

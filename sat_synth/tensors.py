"""Seeded dense inputs: features, labels, Glorot-uniform weights.

Every array is drawn from a counter-based generator (Philox) keyed by
(seed, stream tag), so a given (seed, tag, shape) always yields the same values no
matter which other arrays were drawn before it.
"""
from __future__ import annotations

import zlib

import numpy as np


def stream_rng(seed: int, tag: str) -> np.random.Generator:
    """Independent Philox stream for (seed, tag)."""
    key = np.array([np.uint64(seed), np.uint64(zlib.crc32(tag.encode()))], dtype=np.uint64)
    return np.random.Generator(np.random.Philox(key=key))


def normal_features(seed: int, n: int, d: int, tag: str = "features") -> np.ndarray:
    """X ~ N(0, 1), fp32, shape [n, d] (drawn in row chunks to bound peak memory)."""
    rng = stream_rng(seed, tag)
    out = np.empty((n, d), dtype=np.float32)
    step = max(1, (1 << 24) // max(d, 1))
    for lo in range(0, n, step):
        hi = min(n, lo + step)
        out[lo:hi] = rng.standard_normal((hi - lo, d), dtype=np.float32)
    return out


def uniform_labels(seed: int, n: int, n_classes: int, tag: str = "labels") -> np.ndarray:
    """One class id per node, uniform over {0..n_classes-1}, int32."""
    return stream_rng(seed, tag).integers(0, n_classes, size=n, dtype=np.int32)


def bernoulli_labels(seed: int, n: int, n_labels: int, p: float, tag: str = "labels") -> np.ndarray:
    """Independent Bernoulli(p) label matrix, uint8 [n, n_labels]."""
    rng = stream_rng(seed, tag)
    return (rng.random((n, n_labels), dtype=np.float32) < np.float32(p)).astype(np.uint8)


def glorot_uniform(seed: int, fan_in: int, fan_out: int, tag: str) -> np.ndarray:
    """Glorot/Xavier-uniform matrix [fan_in, fan_out], fp32: U(-a, a), a = sqrt(6/(fan_in+fan_out))."""
    a = np.sqrt(6.0 / (fan_in + fan_out))
    rng = stream_rng(seed, tag)
    return ((rng.random((fan_in, fan_out)) * 2.0 - 1.0) * a).astype(np.float32)


# ------------------------------------------------------------------------------------------
# Embedding-like rows that are a function of (seed, tag, row id): any subset of the rows of a very large matrix can be
# produced without producing the matrix (full-size parity tests hand the whole matrix to one side and sampled rows to the
# other).  Rows are picked from a seeded table of non-negative values (what ReLU outputs look like), so this is pure
# indexing: no arithmetic of the method.
# ------------------------------------------------------------------------------------------
_TABLE_ROWS = 8191


def embedding_table(seed: int, d: int, tag: str = "embedding-table", signed: bool = False) -> np.ndarray:
    """[8191, d] fp32: |N(0, 1)| / 2 with about a third of the entries set to zero (signed=True: N(0, 1) / 2, dense)."""
    rng = stream_rng(seed, f"{tag}:{d}:{int(signed)}")
    t = rng.standard_normal((_TABLE_ROWS, d), dtype=np.float32) * np.float32(0.5)
    if signed:
        return t
    t = np.abs(t)
    t[rng.random((_TABLE_ROWS, d), dtype=np.float32) < np.float32(0.33)] = 0.0
    return t


def table_rows(table: np.ndarray, ids, salt: int = 0) -> np.ndarray:
    """Rows of the virtual matrix M[i] = table[(i * 7919 + salt * 104729) mod 8191] for the given row ids i."""
    ids = np.asarray(ids, dtype=np.int64)
    return table[(ids * 7919 + int(salt) * 104729) % _TABLE_ROWS]

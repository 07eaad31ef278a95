"""Seeded synthetic inputs shared by the CPU oracle's tests and the CUDA library's tests/benchmark.

Holds no arithmetic of the training step: only token-id batches and the named
workload shapes.  Token streams are counter-based (a hash of seed, step, batch
row and position), so any slice can be regenerated without state.

Workloads stand in for the pre-training shards the paper trains on (sequence
length 4096, not available offline): uniform ids for the small and the
8B-shaped cases, Zipf(s=1.1) ids elsewhere, with id 0 the most frequent.
"""
from __future__ import annotations

import numpy as np

WEIGHT_SEED = 1234
DATA_SEED = 5678

# name -> model shape, batch shape, token distribution, number of steps, recompute flag
WORKLOADS = {
    "c1_tiny": dict(n_layers=1, d_model=256, n_heads=4, n_kv_heads=4, head_dim=64, d_ffn=688, vocab=1024,
                    batch=2, seq=128, dist="uniform", steps=1, recompute=0),
    "c2_124m": dict(n_layers=12, d_model=768, n_heads=12, n_kv_heads=12, head_dim=64, d_ffn=2048, vocab=32000,
                    batch=8, seq=1024, dist="zipf", steps=10, recompute=0),
    "c3_1b": dict(n_layers=16, d_model=2048, n_heads=16, n_kv_heads=8, head_dim=128, d_ffn=5632, vocab=32000,
                  batch=4, seq=2048, dist="zipf", steps=20, recompute=0),
    "c4_8b_slice": dict(n_layers=8, d_model=4096, n_heads=32, n_kv_heads=8, head_dim=128, d_ffn=14336,
                        vocab=128256, batch=1, seq=4096, dist="uniform", steps=10, recompute=1),
    "c5_1b_long": dict(n_layers=16, d_model=2048, n_heads=16, n_kv_heads=8, head_dim=128, d_ffn=5632, vocab=32000,
                       batch=1, seq=16384, dist="zipf", steps=10, recompute=0),
}

MODEL_KEYS = ("n_layers", "d_model", "n_heads", "n_kv_heads", "head_dim", "d_ffn", "vocab")


def _mix(z: np.ndarray) -> np.ndarray:
    with np.errstate(over="ignore"):
        z = (z + np.uint64(0x9E3779B97F4A7C15)).astype(np.uint64)
        z = (z ^ (z >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)
        z = (z ^ (z >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)
        return z ^ (z >> np.uint64(31))


def uniforms(seed: int, step: int, batch: int, length: int) -> np.ndarray:
    """[batch, length] doubles in [0,1), one per (seed, step, row, position)."""
    with np.errstate(over="ignore"):
        b = np.arange(batch, dtype=np.uint64)[:, None]
        s = np.arange(length, dtype=np.uint64)[None, :]
        key = _mix(np.uint64(seed) ^ (np.uint64(step + 1) * np.uint64(0xA24BAED4963EE407)))
        key = _mix(key ^ (b * np.uint64(0x9FB21C651E98DF25)) ^ (s * np.uint64(0xD6E8FEB86659FD93)))
    return (key >> np.uint64(11)).astype(np.float64) / float(1 << 53)


_zipf_cdf_cache = {}


def zipf_cdf(vocab: int, s: float = 1.1) -> np.ndarray:
    """CDF of P(id = k-1) proportional to k**(-s), k = 1..vocab."""
    key = (vocab, s)
    if key not in _zipf_cdf_cache:
        w = np.arange(1, vocab + 1, dtype=np.float64) ** (-s)
        _zipf_cdf_cache[key] = np.cumsum(w) / np.sum(w)
    return _zipf_cdf_cache[key]


def token_stream(vocab: int, batch: int, length: int, dist: str, seed: int = DATA_SEED, step: int = 0) -> np.ndarray:
    """int32 [batch, length] token ids drawn i.i.d. from `dist` ("uniform" or "zipf")."""
    u = uniforms(seed, step, batch, length)
    if dist == "uniform":
        ids = np.minimum((u * vocab).astype(np.int64), vocab - 1)
    elif dist == "zipf":
        ids = np.minimum(np.searchsorted(zipf_cdf(vocab), u, side="right"), vocab - 1)
    else:
        raise ValueError(dist)
    return ids.astype(np.int32)


def batch(vocab: int, B: int, S: int, dist: str, seed: int = DATA_SEED, step: int = 0):
    """(tokens, labels), both int32 [B, S]: S+1 ids per row, labels are the next token."""
    ids = token_stream(vocab, B, S + 1, dist, seed, step)
    return np.ascontiguousarray(ids[:, :S]), np.ascontiguousarray(ids[:, 1:])


def workload_batch(name: str, step: int = 0, seed: int = DATA_SEED):
    w = WORKLOADS[name]
    return batch(w["vocab"], w["batch"], w["seq"], w["dist"], seed, step)

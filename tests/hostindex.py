"""Test utility: flush (a write batch becomes a sorted run) and compaction (runs are merged) with
numpy on the host -- the LSM steps between put_batch and probe (paper Sec. 2.2). The library does
both on the GPU (lsmkv_flush_batch, lsmkv_merge_runs); the tests use this form to build runs
without going through the code under test.

Keys are uint64 [n, 4] ordered lexicographically as unsigned words; records are 16-byte
entries kept as a numpy structured array or as raw uint8 [n, 16].
"""
from __future__ import annotations

import numpy as np


def sort_order(keys: np.ndarray) -> np.ndarray:
    """Stable ascending order of uint64 [n,4] keys (lexicographic over the 4 words)."""
    keys = np.ascontiguousarray(keys, dtype=np.uint64).reshape(-1, 4)
    return np.lexsort((keys[:, 3], keys[:, 2], keys[:, 1], keys[:, 0]))


def flush(keys: np.ndarray, vals: np.ndarray):
    """Sorted run with unique keys out of a write batch in arrival order; of equal keys the last
    arrival survives (out-of-place update)."""
    keys = np.ascontiguousarray(keys, dtype=np.uint64).reshape(-1, 4)
    if len(keys) == 0:
        return keys.copy(), vals[:0].copy()
    order = sort_order(keys)                      # lexsort is stable: ties stay in arrival order
    k = keys[order]
    last = np.ones(len(k), dtype=bool)
    last[:-1] = np.any(k[1:] != k[:-1], axis=1)   # last element of every group of equal keys
    return np.ascontiguousarray(k[last]), np.ascontiguousarray(vals[order][last])


def merge_runs(runs):
    """One run out of several (newest first): union of keys, newest record wins."""
    if not runs:
        return np.zeros((0, 4), dtype=np.uint64), None
    ks = np.concatenate([k for k, _ in reversed(runs)])    # oldest first, newest arrives last
    vs = np.concatenate([v for _, v in reversed(runs)])
    return flush(ks, vs)

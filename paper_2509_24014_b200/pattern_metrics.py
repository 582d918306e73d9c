"""Host-side comparisons of two CSR block patterns over the same rows (numpy only, no method arithmetic):
how much of a reference pattern another pattern recovers, by count and by score mass."""
from __future__ import annotations

import numpy as np


def _flat_keys(row_ptr: np.ndarray, col_idx: np.ndarray, num_blocks: int) -> np.ndarray:
    rows = np.repeat(np.arange(len(row_ptr) - 1, dtype=np.int64), np.diff(row_ptr).astype(np.int64))
    return rows * num_blocks + col_idx[: int(row_ptr[-1])].astype(np.int64)


def pattern_recall(ref_row_ptr, ref_col_idx, row_ptr, col_idx, num_blocks: int) -> np.ndarray:
    """Per row: the share of the reference row's kept blocks that the other pattern also keeps
    (1.0 for an empty reference row)."""
    n_rows = len(ref_row_ptr) - 1
    if len(row_ptr) - 1 != n_rows:
        raise ValueError("patterns cover different numbers of rows")
    ref = _flat_keys(np.asarray(ref_row_ptr), np.asarray(ref_col_idx), num_blocks)
    oth = _flat_keys(np.asarray(row_ptr), np.asarray(col_idx), num_blocks)
    common = np.intersect1d(ref, oth, assume_unique=True)
    hit = np.bincount(common // num_blocks, minlength=n_rows).astype(np.float64)
    want = np.diff(np.asarray(ref_row_ptr)).astype(np.float64)
    return np.where(want > 0, hit / np.maximum(want, 1.0), 1.0)


def kept_mass(scores: np.ndarray, row_ptr, col_idx) -> np.ndarray:
    """Per row: the sum of the row's scores over its kept blocks. scores: [rows, num_blocks]."""
    row_ptr = np.asarray(row_ptr)
    n_rows, nb = scores.shape
    if len(row_ptr) - 1 != n_rows:
        raise ValueError("scores and pattern cover different numbers of rows")
    keys = _flat_keys(row_ptr, np.asarray(col_idx), nb)
    vals = scores.reshape(-1)[keys].astype(np.float64)
    return np.bincount(keys // nb, weights=vals, minlength=n_rows)

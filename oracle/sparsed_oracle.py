"""CPU oracle for the SparseD attention path (TEST INFRASTRUCTURE, not the product).

A plain, slow, fp64 numpy restatement of what the paper defines, used only by the
tests, the smoke check and the CPU-baseline leg of the benchmark. It shares no code
with the CUDA library and must never be imported by the product package.

What each function follows in the paper:

* ``attn_full``         - Eq. 1 (bidirectional softmax attention, no mask) times V
                          (the "A(Q,K)·V" of the goal statement after Eq. 4).
* ``pooled_scores``     - "Isolated Selection": A' = avgpool(A, block_size), computed one
                          query block at a time as in Algorithm 1's inner loop.
* ``kept_per_region``   - how many blocks "top-rho%" of a region is (reading: ceil).
* ``select_blocks``     - Eq. 5 / Eq. 6: separate top-rho% over prefill and generation key
                          blocks, ranked by A'; result as CSR block lists (Eq. 4's mask).
* ``attn_sparse``       - Eq. 3 with the block mask of Eq. 4, times V.
* ``switch_step`` / ``schedule_mode`` - "Skipping Sparse" and the branch of Algorithm 1.
* ``sparsed_attention`` - Algorithm 1 as a whole for one call.
* ``pooled_qk_scores``  - NOT the paper's scorer: the cheap estimate of A' that pools queries and
                          keys per block before the softmax (the approximate-score family the
                          introduction sets the method against). Kept to measure how much of the
                          exact pattern such an estimate recovers.

Readings where the paper is silent (each listed in the design notes):
pooling is over post-softmax probabilities normalised over the whole row; the number of
kept blocks of a region of n blocks is clamp(ceil(rho*n - 1e-6), 1, n); ties go to the
lower block index; a row's list is stored ascending; steps are 1-based and the switch
step is s = clamp(floor(T*skip + 1e-9), 1, T); with grouped-query attention query head h
reads key/value head h // (Hq // Hkv).

Parity status: pinned by the CPU tests against closed forms, a brute-force
materialised implementation, a library routine and invariants. The paper prints no
worked numeric example, so no pin comes from a printed value. ``pooled_qk_scores`` is pinned
by the two cases in which the estimate is exact (block size 1: a library softmax; inputs
constant inside every block: the exact A').

All tensors are numpy arrays: q [B,Hq,L,D], k and v [B,Hkv,L,D], float64 holding the
exactly widened bf16 inputs.
"""
from __future__ import annotations

import math
from typing import Optional, Sequence, Tuple

import numpy as np

FULL, FULL_AND_SELECT, SPARSE = 0, 1, 2


# --------------------------------------------------------------------------- schedule
def switch_step(total_steps: int, skip: float) -> int:
    """Step (1-based) at which the pattern is selected: the last full-attention step."""
    if total_steps < 1 or not (0.0 <= skip <= 1.0):
        raise ValueError("bad schedule arguments")
    s = int(math.floor(total_steps * skip + 1e-9))
    return min(max(s, 1), total_steps)


def schedule_mode(step: int, total_steps: int, skip: float) -> int:
    """Algorithm 1's branch for a 1-based step: FULL, FULL_AND_SELECT or SPARSE."""
    if not (1 <= step <= total_steps):
        raise ValueError("step out of range")
    s = switch_step(total_steps, skip)
    if step < s:
        return FULL
    if step == s:
        return FULL_AND_SELECT
    return SPARSE


# --------------------------------------------------------------------------- Eq. 1
def _scale(d: int, scale: Optional[float]) -> float:
    return 1.0 / math.sqrt(d) if scale is None else float(scale)


def softmax_rows(qh: np.ndarray, kh: np.ndarray, rows: slice, scale: Optional[float] = None):
    """Eq. 1 for the query rows ``rows`` of one head: (A rows [len(rows), L], LSE rows)."""
    s = (qh[rows] @ kh.T) * _scale(qh.shape[1], scale)
    m = s.max(axis=1, keepdims=True)
    w = np.exp(s - m)
    z = w.sum(axis=1, keepdims=True)
    return w / z, (m + np.log(z))[:, 0]


def head_full_rows(qh: np.ndarray, kh: np.ndarray, vh: np.ndarray, rows: slice,
                   scale: Optional[float] = None):
    """A(Q,K)·V for the query rows ``rows`` of one head. Returns (O rows, LSE rows)."""
    p, lse = softmax_rows(qh, kh, rows, scale)
    return p @ vh, lse


def attn_full(q, k, v, scale: Optional[float] = None, block_rows: int = 128):
    """Returns (O [B,Hq,L,D], LSE [B,Hq,L]) in fp64."""
    B, Hq, L, D = q.shape
    group = Hq // k.shape[1]
    o = np.empty((B, Hq, L, v.shape[3]), dtype=np.float64)
    lse = np.empty((B, Hq, L), dtype=np.float64)
    for b in range(B):
        for h in range(Hq):
            for r0 in range(0, L, block_rows):
                rows = slice(r0, min(L, r0 + block_rows))
                o[b, h, rows], lse[b, h, rows] = head_full_rows(q[b, h], k[b, h // group], v[b, h // group],
                                                                rows, scale)
    return o, lse


# --------------------------------------------------------------------------- avgpool(A)
def head_pooled_row(qh: np.ndarray, kh: np.ndarray, ib: int, block_size: int,
                    scale: Optional[float] = None) -> np.ndarray:
    """One block-row of A' for one head: Algorithm 1's Q' = Q[start:end], avgpool(A(Q',K))."""
    L = kh.shape[0]
    nb = L // block_size
    rows = slice(ib * block_size, (ib + 1) * block_size)
    p, _ = softmax_rows(qh, kh, rows, scale)  # [bs, L], softmax over all L keys
    return p.reshape(block_size, nb, block_size).sum(axis=(0, 2)) / float(block_size * block_size)


def pooled_scores(q, k, block_size: int, scale: Optional[float] = None) -> np.ndarray:
    """A' [B,Hq,nb,nb] in fp64."""
    B, Hq, L, _ = q.shape
    if L % block_size:
        raise ValueError("seq_len must be a multiple of block_size")
    nb = L // block_size
    group = Hq // k.shape[1]
    out = np.empty((B, Hq, nb, nb), dtype=np.float64)
    for b in range(B):
        for h in range(Hq):
            for ib in range(nb):
                out[b, h, ib] = head_pooled_row(q[b, h], k[b, h // group], ib, block_size, scale)
    return out


def pooled_qk_scores(q, k, block_size: int, scale: Optional[float] = None) -> np.ndarray:
    """Estimate of A' [B,Hq,nb,nb] from block means (not in the paper; see the module header).

    Query block i and key block j are replaced by the means of their rows; the estimate of the
    block's pooled probability is softmax_j(scale * mean_q[i] . mean_k[j]) / block_size, which has
    the row sums (1 / block_size) of the exact A' and equals it when every block is constant.
    """
    B, Hq, L, D = q.shape
    if L % block_size:
        raise ValueError("seq_len must be a multiple of block_size")
    nb = L // block_size
    group = Hq // k.shape[1]
    sc = _scale(D, scale)
    out = np.empty((B, Hq, nb, nb), dtype=np.float64)
    for b in range(B):
        for h in range(Hq):
            q_mean = q[b, h].reshape(nb, block_size, D).mean(axis=1)
            k_mean = k[b, h // group].reshape(nb, block_size, D).mean(axis=1)
            z = sc * (q_mean @ k_mean.T)
            z -= z.max(axis=1, keepdims=True)
            e = np.exp(z)
            out[b, h] = e / e.sum(axis=1, keepdims=True) / block_size
    return out


# --------------------------------------------------------------------------- Eq. 5 / Eq. 6
def kept_per_region(n_blocks: int, keep_ratio: float, rounding: str = "ceil") -> int:
    if n_blocks <= 0:
        return 0
    x = keep_ratio * n_blocks
    kk = math.ceil(x - 1e-6) if rounding == "ceil" else math.floor(x + 1e-6)
    return int(min(max(kk, 1), n_blocks))


def select_row(scores_row: np.ndarray, prefill_blocks: int, keep_ratio: float,
               rounding: str = "ceil") -> list:
    """Kept key blocks of one query block: top-k separately over [0,pb) and [pb,nb),
    ranked by (score descending, index ascending); returned ascending."""
    nb = scores_row.shape[0]
    kept = []
    for lo, hi in ((0, prefill_blocks), (prefill_blocks, nb)):
        if hi <= lo:
            continue
        kk = kept_per_region(hi - lo, keep_ratio, rounding)
        order = sorted(range(lo, hi), key=lambda j: (-scores_row[j], j))
        kept.extend(order[:kk])
    return sorted(kept)


def select_blocks(scores: np.ndarray, block_size: int, prefill_len: int, keep_ratio: float,
                  rounding: str = "ceil") -> Tuple[np.ndarray, np.ndarray]:
    """scores [B,Hq,nb,nb] (any float dtype; compared as given) -> CSR (row_ptr, col_idx),
    rows ordered ((b*Hq + h)*nb + ib), int32."""
    if prefill_len % block_size:
        raise ValueError("prefill_len must be a multiple of block_size")
    B, Hq, nb, _ = scores.shape
    pb = prefill_len // block_size
    row_ptr = [0]
    col_idx = []
    for b in range(B):
        for h in range(Hq):
            for ib in range(nb):
                kept = select_row(scores[b, h, ib], pb, keep_ratio, rounding)
                col_idx.extend(kept)
                row_ptr.append(len(col_idx))
    return np.asarray(row_ptr, dtype=np.int32), np.asarray(col_idx, dtype=np.int32)


# --------------------------------------------------------------------------- Eq. 3 / Eq. 4
def head_sparse_rows(qh, kh, vh, ib: int, kept: Sequence[int], block_size: int,
                     scale: Optional[float] = None) -> np.ndarray:
    """Eq. 3 for query block ``ib`` of one head: keys outside the kept blocks get -inf."""
    L = kh.shape[0]
    rows = slice(ib * block_size, (ib + 1) * block_size)
    mask = np.full((L,), -np.inf)
    for jb in kept:
        mask[jb * block_size:(jb + 1) * block_size] = 0.0
    s = (qh[rows] @ kh.T + mask[None, :]) * _scale(qh.shape[1], scale)
    m = s.max(axis=1, keepdims=True)
    w = np.exp(s - m)
    return (w @ vh) / w.sum(axis=1, keepdims=True)


def attn_sparse(q, k, v, row_ptr, col_idx, block_size: int, scale: Optional[float] = None) -> np.ndarray:
    B, Hq, L, _ = q.shape
    nb = L // block_size
    group = Hq // k.shape[1]
    o = np.empty((B, Hq, L, v.shape[3]), dtype=np.float64)
    for b in range(B):
        for h in range(Hq):
            for ib in range(nb):
                r = (b * Hq + h) * nb + ib
                kept = col_idx[row_ptr[r]:row_ptr[r + 1]]
                o[b, h, ib * block_size:(ib + 1) * block_size] = head_sparse_rows(
                    q[b, h], k[b, h // group], v[b, h // group], ib, kept, block_size, scale)
    return o


# --------------------------------------------------------------------------- Algorithm 1
def sparsed_attention(q, k, v, step: int, total_steps: int, keep_ratio: float, skip: float,
                      block_size: int, prefill_len: int = 0, pattern=None):
    """One call of Algorithm 1. Returns (output, pattern); ``pattern`` is (row_ptr, col_idx)
    once selected (at the switch step) and must be passed back in on later steps."""
    mode = schedule_mode(step, total_steps, skip)
    if mode in (FULL, FULL_AND_SELECT):
        out, _ = attn_full(q, k, v)
        if mode == FULL_AND_SELECT:
            pattern = select_blocks(pooled_scores(q, k, block_size), block_size, prefill_len, keep_ratio)
        return out, pattern
    if pattern is None:
        raise ValueError("sparse step before the pattern was selected")
    return attn_sparse(q, k, v, pattern[0], pattern[1], block_size), pattern

"""Brute-force restatement of the SparseD definitions for tiny inputs (TEST INFRASTRUCTURE).

An independent check on ``sparsed_oracle``: it materialises the whole l x l score matrix
of Eq. 1, pools it with explicit loops, ranks blocks with an argsort instead of a keyed
sort, expands the block lists into the token-level mask M_S of Eq. 4 and applies Eq. 3
literally with scalar Python loops. It imports nothing from ``sparsed_oracle``.
Only usable for l up to a few hundred.
"""
from __future__ import annotations

import math

import numpy as np


def score_matrix(qh, kh, mask=None):
    """Eq. 1 (mask None) or Eq. 3 (mask = M_S, entries 0 / -inf), one head, scalar loops."""
    L, D = qh.shape
    Lk = kh.shape[0]
    a = np.zeros((L, Lk))
    for i in range(L):
        logits = []
        for j in range(Lk):
            dot = 0.0
            for d in range(D):
                dot += qh[i, d] * kh[j, d]
            if mask is not None:
                dot += mask[i, j]
            logits.append(dot / math.sqrt(D))
        mx = max(logits)
        e = [math.exp(x - mx) if x != -math.inf else 0.0 for x in logits]
        z = sum(e)
        for j in range(Lk):
            a[i, j] = e[j] / z
    return a


def attend(a, vh):
    L, Lk = a.shape
    out = np.zeros((L, vh.shape[1]))
    for i in range(L):
        for j in range(Lk):
            if a[i, j] != 0.0:
                out[i] += a[i, j] * vh[j]
    return out


def avgpool(a, bs):
    nb_r, nb_c = a.shape[0] // bs, a.shape[1] // bs
    out = np.zeros((nb_r, nb_c))
    for ib in range(nb_r):
        for jb in range(nb_c):
            acc = 0.0
            for i in range(ib * bs, (ib + 1) * bs):
                for j in range(jb * bs, (jb + 1) * bs):
                    acc += a[i, j]
            out[ib, jb] = acc / (bs * bs)
    return out


def topk_region(row, lo, hi, kk):
    """Indices of the kk largest entries of row[lo:hi]; equal scores -> lower index first.
    Uses a stable argsort on the negated scores."""
    seg = -np.asarray(row[lo:hi], dtype=np.float64)
    order = np.argsort(seg, kind="stable")
    return sorted(int(lo + j) for j in order[:kk])


def select(pooled, pb, kk_pre, kk_gen):
    """Per query block: union of the top kk_pre blocks in [0,pb) and top kk_gen in [pb,nb)."""
    nb = pooled.shape[1]
    rows = []
    for ib in range(pooled.shape[0]):
        kept = []
        if pb > 0:
            kept += topk_region(pooled[ib], 0, pb, kk_pre)
        if nb > pb:
            kept += topk_region(pooled[ib], pb, nb, kk_gen)
        rows.append(sorted(kept))
    return rows


def token_mask(rows, bs, L):
    """Eq. 4: M_S[i,j] = 0 if key block j//bs is kept for query block i//bs, else -inf."""
    m = np.full((L, L), -np.inf)
    for i in range(L):
        for j in range(L):
            if (j // bs) in rows[i // bs]:
                m[i, j] = 0.0
    return m

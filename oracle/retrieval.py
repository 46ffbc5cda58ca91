"""Selection step of the top-k retrieval operator (Appendix D) in plain numpy.  TEST INFRASTRUCTURE ONLY.

PARITY UNPINNED as a reading of the paper: Appendix D names the steps but none of the constants (pooling
window and stride, tail length, k, number of anchors, offset window) nor the tie and overflow rules, so all
of them are parameters or choices made here (listed in the design notes).  The mechanics are pinned by
``tests/test_oracle_pins.py`` (brute force on small inputs, constructed best matches, padding, ordering).

Steps, in the paper's order, per batch element and KV head:

1. query summaries from the last ``Lq_last`` queries of the previous segment: the mean over each sliding
   window ``[u*stride, u*stride + window)`` (clipped to the rows present; at least one window) and the mean
   over the last ``tail`` rows; with grouped heads the mean runs over the group's query heads too;
2. dot-product scores of every summary against every pool key;
3. per summary the ``top_k`` best keys (ties: lower position first), deduplicated into one candidate set;
4. anchors: the ``n_anchors`` candidates with the highest score (a candidate's score is its best over the
   summaries; ties: lower position first);
5. window expansion: positions ``anchor - off_lo .. anchor + off_hi`` inside the pool, best anchor first,
   until ``R`` distinct positions are selected; if fewer than ``R`` result, the earliest positions not yet
   selected pad the set to exactly ``R``; the output is sorted ascending.

Floating point decides integers here, so the arithmetic is fixed: fp32, products and sums rounded
separately, sums taken sequentially in index order (head, then row for a summary; dimension for a score).
"""
from __future__ import annotations

import numpy as np

F = np.float32


def n_summaries(Lq_last, window, stride):
    return (max(1, (Lq_last - window) // stride + 1) if Lq_last >= window else 1) + 1


def summaries(Q_last, Hkv, window, stride, tail):
    """[B, Hkv, n_sum, d] fp32 from Q_last [B, Lq_last, Hq, d] (values are exact in fp32)."""
    Q = np.asarray(Q_last, dtype=F)
    B, Lq, Hq, d = Q.shape
    g = Hq // Hkv
    n_w = n_summaries(Lq, window, stride) - 1
    spans = [(u * stride, min(Lq, u * stride + window)) for u in range(n_w)] + [(max(0, Lq - tail), Lq)]
    out = np.zeros((B, Hkv, len(spans), d), dtype=F)
    for m, (r0, r1) in enumerate(spans):
        for c in range(Hkv):
            acc = np.zeros((B, d), dtype=F)
            for r in range(g):
                for row in range(r0, r1):
                    acc = (acc + Q[:, row, c * g + r]).astype(F)
            out[:, c, m] = (acc / F((r1 - r0) * g)).astype(F)
    return out


def scores(summ, K_pool):
    """[B, Hkv, n_sum, P] fp32: sequential sum over the head dimension of separately rounded products."""
    K = np.asarray(K_pool, dtype=F)
    B, P, Hkv, d = K.shape
    out = np.zeros((B, Hkv, summ.shape[2], P), dtype=F)
    for b in range(B):
        for c in range(Hkv):
            for m in range(summ.shape[2]):
                acc = np.zeros(P, dtype=F)
                for e in range(d):
                    acc = (acc + (summ[b, c, m, e] * K[b, :, c, e]).astype(F)).astype(F)
                out[b, c, m] = acc
    return out


def _best(values, positions):
    """Index into `positions` of the highest value; ties go to the lower position."""
    best = 0
    for i in range(1, len(positions)):
        if values[i] > values[best] or (values[i] == values[best] and positions[i] < positions[best]):
            best = i
    return best


def select_from_scores(sc, top_k, n_anchors, off_lo, off_hi, R):
    """Positions [R] (ascending) for one (batch, head) from its scores [n_sum, P]."""
    n_sum, P = sc.shape
    assert R <= P and top_k <= P
    cand = []
    for m in range(n_sum):
        taken = np.zeros(P, bool)
        for _ in range(top_k):
            free = np.flatnonzero(~taken)
            j = int(free[_best(sc[m, free], free)])
            taken[j] = True
            if j not in cand:
                cand.append(j)
    cscore = [sc[:, j].max() for j in cand]
    anchors, pool = [], list(range(len(cand)))
    for _ in range(min(n_anchors, len(cand))):
        i = _best([cscore[q] for q in pool], [cand[q] for q in pool])
        anchors.append(cand[pool.pop(i)])
    chosen = []
    for a in anchors:
        for j in range(a - off_lo, a + off_hi + 1):
            if 0 <= j < P and j not in chosen and len(chosen) < R:
                chosen.append(j)
    j = 0
    while len(chosen) < R:
        if j not in chosen:
            chosen.append(j)
        j += 1
    return np.array(sorted(chosen), dtype=np.int32)


def select(Q_last, K_pool, window, stride, tail, top_k, n_anchors, off_lo, off_hi, R):
    """idx [B, Hkv, R] int32: the whole selection step."""
    K = np.asarray(K_pool)
    B, P, Hkv, _ = K.shape
    sc = scores(summaries(Q_last, Hkv, window, stride, tail), K)
    out = np.zeros((B, Hkv, R), dtype=np.int32)
    for b in range(B):
        for c in range(Hkv):
            out[b, c] = select_from_scores(sc[b, c], top_k, n_anchors, off_lo, off_hi, R)
    return out

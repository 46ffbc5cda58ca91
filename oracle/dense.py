"""Matrix-form fp64 statement of segment-level causal attention (numpy).  TEST INFRASTRUCTURE ONLY.

The same definition as ``seg_attn_oracle.c`` written with explicit ``Lq x Lk`` boolean masks, so
that the two can be checked against each other and against library attention:

* ``visible[p, j] = (j <= p) & ((j >= a[p]) | flag)`` with ``a[p] = max(0, (p // S) * S - T)``
  (own segment causally, the previous segment's last T positions, and - for a flagged KV head -
  everything older; Appendix C, Eqs. "attn" and "ctx"; C_0 empty, Section 3.1); a head of class 2
  reads its own segment only, ``j >= (p // S) * S`` (third case of Eq. "ctx");
* ``diff[p, j] = (j <= p) & (j >= a[p])``: the reads that carry gradient into K/V; older reads
  of a flagged head are stop-gradient (Definition 3.2, Lemma B.1).

Memory is O(Lq*Lk) per head: meant for L up to a few thousand.
"""
from __future__ import annotations

import numpy as np


def masks(Lq, Lk, S, T, flag, q_pos0=0, kv_pos0=0, flagged_tail_is_sg=False):
    p = (q_pos0 + np.arange(Lq))[:, None]
    j = (kv_pos0 + np.arange(Lk))[None, :]
    seg0 = (p // S) * S
    a = np.maximum(0, seg0 - T)
    causal = j <= p
    cls = int(flag)  # head class: 0 local, 1 past access, 2 own segment only
    lo_vis = {0: a, 1: np.zeros_like(a), 2: seg0}[cls]
    visible = causal & (j >= lo_vis)
    lo_diff = seg0 if (cls == 2 or (cls == 1 and flagged_tail_is_sg)) else a
    diff = causal & (j >= lo_diff)
    return visible, diff


def fwd(Q, K, V, S, T, head_past_mask=None, scale=None, q_pos0=0, kv_pos0=0):
    Q, K, V = (np.asarray(x, dtype=np.float64) for x in (Q, K, V))
    B, Lq, Hq, d = Q.shape
    _, Lk, Hkv, _ = K.shape
    g = Hq // Hkv
    scale = 1.0 / np.sqrt(d) if scale is None else scale
    flags = np.zeros(Hkv, int) if head_past_mask is None else np.asarray(head_past_mask).astype(int)
    O = np.zeros_like(Q)
    LSE = np.full((B, Hq, Lq), -np.inf)
    for h in range(Hq):
        c = h // g
        vis, _ = masks(Lq, Lk, S, T, flags[c], q_pos0, kv_pos0)
        for b in range(B):
            s = scale * (Q[b, :, h] @ K[b, :, c].T)
            s = np.where(vis, s, -np.inf)
            m = s.max(axis=1, keepdims=True)
            e = np.exp(s - m)
            z = e.sum(axis=1, keepdims=True)
            O[b, :, h] = (e / z) @ V[b, :, c]
            LSE[b, h] = (m + np.log(z))[:, 0]
    return O, LSE


def bwd(Q, K, V, dO, S, T, head_past_mask=None, scale=None, q_pos0=0, kv_pos0=0, flagged_tail_is_sg=False):
    Q, K, V, dO = (np.asarray(x, dtype=np.float64) for x in (Q, K, V, dO))
    B, Lq, Hq, d = Q.shape
    _, Lk, Hkv, _ = K.shape
    g = Hq // Hkv
    scale = 1.0 / np.sqrt(d) if scale is None else scale
    flags = np.zeros(Hkv, int) if head_past_mask is None else np.asarray(head_past_mask).astype(int)
    dQ, dK, dV = np.zeros_like(Q), np.zeros_like(K), np.zeros_like(V)
    for h in range(Hq):
        c = h // g
        vis, dif = masks(Lq, Lk, S, T, flags[c], q_pos0, kv_pos0, flagged_tail_is_sg)
        for b in range(B):
            s = np.where(vis, scale * (Q[b, :, h] @ K[b, :, c].T), -np.inf)
            m = s.max(axis=1, keepdims=True)
            e = np.exp(s - m)
            P = e / e.sum(axis=1, keepdims=True)
            o = P @ V[b, :, c]
            D = (dO[b, :, h] * o).sum(axis=1, keepdims=True)
            dP = dO[b, :, h] @ V[b, :, c].T
            dS = P * (dP - D)
            dQ[b, :, h] = scale * (dS @ K[b, :, c])
            dK[b, :, c] += scale * ((dS * dif).T @ Q[b, :, h])
            dV[b, :, c] += (P * dif).T @ dO[b, :, h]
    return dQ, dK, dV

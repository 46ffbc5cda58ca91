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


def masks(Lq, Lk, S, T, flag, q_pos0=0, kv_pos0=0, flagged_tail_is_sg=False, seg_starts=None):
    p = (q_pos0 + np.arange(Lq))[:, None]
    j = (kv_pos0 + np.arange(Lk))[None, :]
    if seg_starts is None:
        seg0 = (p // S) * S
        a = np.maximum(0, seg0 - T)
    else:
        # segments of given lengths: the tail is the last min(T, length) positions of the previous segment
        st = np.asarray(seg_starts)
        i = np.searchsorted(st, p, side="right") - 1
        seg0 = st[i]
        prev0 = np.where(i > 0, st[np.maximum(i - 1, 0)], 0)
        a = np.maximum(prev0, seg0 - T)
    causal = j <= p
    cls = int(flag)  # head class: 0 local, 1 past access, 2 own segment only
    lo_vis = {0: a, 1: np.zeros_like(a), 2: seg0}[cls]
    visible = causal & (j >= lo_vis)
    lo_diff = seg0 if (cls == 2 or (cls == 1 and flagged_tail_is_sg)) else a
    diff = causal & (j >= lo_diff)
    return visible, diff


def fwd(Q, K, V, S, T, head_past_mask=None, scale=None, q_pos0=0, kv_pos0=0, seg_starts=None):
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
        vis, _ = masks(Lq, Lk, S, T, flags[c], q_pos0, kv_pos0, seg_starts=seg_starts)
        for b in range(B):
            s = scale * (Q[b, :, h] @ K[b, :, c].T)
            s = np.where(vis, s, -np.inf)
            m = s.max(axis=1, keepdims=True)
            e = np.exp(s - m)
            z = e.sum(axis=1, keepdims=True)
            O[b, :, h] = (e / z) @ V[b, :, c]
            LSE[b, h] = (m + np.log(z))[:, 0]
    return O, LSE


def bwd(Q, K, V, dO, S, T, head_past_mask=None, scale=None, q_pos0=0, kv_pos0=0, flagged_tail_is_sg=False,
        seg_starts=None):
    Q, K, V, dO = (np.asarray(x, dtype=np.float64) for x in (Q, K, V, dO))
    B, Lq, Hq, d = Q.shape
    _, Lk, Hkv, _ = K.shape
    g = Hq // Hkv
    scale = 1.0 / np.sqrt(d) if scale is None else scale
    flags = np.zeros(Hkv, int) if head_past_mask is None else np.asarray(head_past_mask).astype(int)
    dQ, dK, dV = np.zeros_like(Q), np.zeros_like(K), np.zeros_like(V)
    for h in range(Hq):
        c = h // g
        vis, dif = masks(Lq, Lk, S, T, flags[c], q_pos0, kv_pos0, flagged_tail_is_sg, seg_starts)
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


def retrieved_context(K_pool, V_pool, idx, K_seg, V_seg):
    """Keys and values a head with a retrieved prefix attends over: ``[K_ret ; K_i]`` with
    ``K_ret[b, r, c] = K_pool[b, idx[b, c, r], c]`` (Appendix C, Eq. "ctx", first case).  Shapes:
    pools ``[B, P, Hkv, d]``, ``idx [B, Hkv, R]``, segment ``[B, Lseg, Hkv, d]`` -> ``[B, R + Lseg, Hkv, d]``."""
    K_pool, V_pool, K_seg, V_seg = (np.asarray(x) for x in (K_pool, V_pool, K_seg, V_seg))
    idx = np.asarray(idx)
    B, Hkv, R = idx.shape
    out = []
    for pool, seg in ((K_pool, K_seg), (V_pool, V_seg)):
        ctx = np.empty((B, R + seg.shape[1], Hkv, pool.shape[3]), dtype=pool.dtype)
        for b in range(B):
            for c in range(Hkv):
                for r in range(R):
                    ctx[b, r, c] = pool[b, idx[b, c, r], c]
        ctx[:, R:] = seg
        out.append(ctx)
    return out[0], out[1]


def retrieved_attention(Q_seg, K_pool, V_pool, idx, K_seg, V_seg, dO=None, scale=None):
    """Attention of one segment over ``[retrieved prefix ; own segment]``: every prefix row visible, the
    segment causal (Appendix C, Eq. "attn"); the prefix is stop-gradient (Definition 3.2, Lemma B.1).
    Returns (O, LSE) or, with dO, (O, LSE, dQ, dK_seg, dV_seg)."""
    Kc, Vc = retrieved_context(K_pool, V_pool, idx, K_seg, V_seg)
    Q = np.asarray(Q_seg, dtype=np.float64)
    Kc, Vc = Kc.astype(np.float64), Vc.astype(np.float64)
    B, L, Hq, d = Q.shape
    Hkv, R = Kc.shape[2], Kc.shape[1] - L
    g = Hq // Hkv
    scale = 1.0 / np.sqrt(d) if scale is None else scale
    vis = np.concatenate([np.ones((L, R), bool), np.tril(np.ones((L, L), bool))], axis=1)
    O, LSE = np.zeros_like(Q), np.zeros((B, Hq, L))
    dQ = np.zeros_like(Q)
    dK, dV = np.zeros((B, L, Hkv, d)), np.zeros((B, L, Hkv, d))
    for b in range(B):
        for h in range(Hq):
            c = h // g
            s = np.where(vis, scale * (Q[b, :, h] @ Kc[b, :, c].T), -np.inf)
            m = s.max(axis=1, keepdims=True)
            e = np.exp(s - m)
            z = e.sum(axis=1, keepdims=True)
            P = e / z
            O[b, :, h] = P @ Vc[b, :, c]
            LSE[b, h] = (m + np.log(z))[:, 0]
            if dO is not None:
                go = np.asarray(dO, dtype=np.float64)[b, :, h]
                dP = go @ Vc[b, :, c].T
                dS = P * (dP - (go * O[b, :, h]).sum(axis=1, keepdims=True))
                dQ[b, :, h] = scale * dS @ Kc[b, :, c]
                dK[b, :, c] += scale * dS[:, R:].T @ Q[b, :, h]   # the segment's own keys only
                dV[b, :, c] += P[:, R:].T @ go
    return (O, LSE) if dO is None else (O, LSE, dQ, dK, dV)

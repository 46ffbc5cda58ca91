"""Pins for the fp64 oracle: each test ties it to something fixed outside the oracle itself -
library attention and autograd (torch CPU, fp64), closed forms, finite differences, the
paper's cost model and its gradient-reach statements.  No GPU is used here."""
import os

import numpy as np
import pytest
import torch
import torch.nn.functional as F

import oracle
from oracle import dense
from oracle import retrieval
from oracle import rope

RNG = np.random.default_rng(7)
TOL = 1e-10


def rand(B, L, Hq, Hkv, d, rng=RNG):
    return (rng.standard_normal((B, L, Hq, d)), rng.standard_normal((B, L, Hkv, d)),
            rng.standard_normal((B, L, Hkv, d)), rng.standard_normal((B, L, Hq, d)))


def t64(a, grad=False):
    return torch.tensor(a, dtype=torch.float64, requires_grad=grad)


def sdpa_causal(Q, K, V, dO):
    """Textbook full causal attention and its gradients from the library (fp64), with GQA expansion."""
    q, k, v = t64(Q, True), t64(K, True), t64(V, True)
    g = Q.shape[2] // K.shape[2]
    kk = k.repeat_interleave(g, dim=2)
    vv = v.repeat_interleave(g, dim=2)
    o = F.scaled_dot_product_attention(q.transpose(1, 2), kk.transpose(1, 2), vv.transpose(1, 2), is_causal=True)
    o = o.transpose(1, 2)
    (o * t64(dO)).sum().backward()
    s = torch.einsum("blhd,bmhd->bhlm", q, kk) / np.sqrt(Q.shape[3])
    L = Q.shape[1]
    s = s.masked_fill(~torch.ones(L, L, dtype=torch.bool).tril(), float("-inf"))
    lse = torch.logsumexp(s, dim=-1)
    return o.detach().numpy(), lse.detach().numpy(), q.grad.numpy(), k.grad.numpy(), v.grad.numpy()


# ---- forward / backward: S >= L is textbook causal attention --------------------------------
@pytest.mark.parametrize("S,T", [(64, 0), (64, 64), (200, 17)])
def test_single_segment_equals_library_causal_attention(S, T):
    Q, K, V, dO = rand(2, 64, 4, 2, 16)
    o, lse, gq, gk, gv = sdpa_causal(Q, K, V, dO)
    O, LSE = oracle.fwd(Q, K, V, S, T)
    dQ, dK, dV = oracle.bwd(Q, K, V, dO, S, T)
    for a, b in ((O, o), (LSE, lse), (dQ, gq), (dK, gk), (dV, gv)):
        np.testing.assert_allclose(a, b, rtol=0, atol=TOL)


def test_no_tail_no_flags_is_block_diagonal():
    S, L = 24, 96
    Q, K, V, dO = rand(1, L, 2, 2, 8)
    O, LSE = oracle.fwd(Q, K, V, S, 0)
    dQ, dK, dV = oracle.bwd(Q, K, V, dO, S, 0)
    for i in range(L // S):
        sl = slice(i * S, (i + 1) * S)
        o, lse, gq, gk, gv = sdpa_causal(Q[:, sl], K[:, sl], V[:, sl], dO[:, sl])
        np.testing.assert_allclose(O[:, sl], o, atol=TOL)
        np.testing.assert_allclose(LSE[:, :, sl], lse, atol=TOL)
        np.testing.assert_allclose(dQ[:, sl], gq, atol=TOL)
        np.testing.assert_allclose(dK[:, sl], gk, atol=TOL)
        np.testing.assert_allclose(dV[:, sl], gv, atol=TOL)


@pytest.mark.parametrize("S,T", [(16, 0), (16, 5), (32, 32), (7, 3)])
def test_all_heads_flagged_forward_is_full_causal(S, T):
    Q, K, V, dO = rand(1, 80, 4, 2, 8)
    o, lse, gq, _, _ = sdpa_causal(Q, K, V, dO)
    O, LSE = oracle.fwd(Q, K, V, S, T, head_past_mask=[1, 1])
    np.testing.assert_allclose(O, o, atol=TOL)
    np.testing.assert_allclose(LSE, lse, atol=TOL)
    # stop-gradient cuts K/V only: dQ is the full-causal dQ
    dQ, _, _ = oracle.bwd(Q, K, V, dO, S, T, head_past_mask=[1, 1])
    np.testing.assert_allclose(dQ, gq, atol=TOL)


# ---- the paper's segment recurrence, built with library ops and autograd -----------------------
def test_own_segment_only_heads_are_block_diagonal_for_any_tail():
    # A head of class 2 never reads the carried tail: for any T it equals T = 0, i.e. independent
    # causal attention per segment (Appendix C, Eq. "ctx", third case), in values and gradients.
    S, L, T = 24, 96, 11
    Q, K, V, dO = rand(1, L, 4, 2, 8)
    O, LSE = oracle.fwd(Q, K, V, S, T, head_past_mask=[2, 0])
    dQ, dK, dV = oracle.bwd(Q, K, V, dO, S, T, head_past_mask=[2, 0])
    hq, c = slice(0, 2), slice(0, 1)
    for i in range(L // S):
        sl = slice(i * S, (i + 1) * S)
        o, lse, gq, gk, gv = sdpa_causal(Q[:, sl, hq], K[:, sl, c], V[:, sl, c], dO[:, sl, hq])
        np.testing.assert_allclose(O[:, sl, hq], o, atol=TOL)
        np.testing.assert_allclose(LSE[:, hq, sl], lse, atol=TOL)
        np.testing.assert_allclose(dQ[:, sl, hq], gq, atol=TOL)
        np.testing.assert_allclose(dK[:, sl, c], gk, atol=TOL)
        np.testing.assert_allclose(dV[:, sl, c], gv, atol=TOL)
    # the local head beside it is untouched by its neighbour's class
    O0, _ = oracle.fwd(Q, K, V, S, T, head_past_mask=[0, 0])
    np.testing.assert_array_equal(O[:, :, 2:], O0[:, :, 2:])
    # and the dense statement of the definition agrees
    d2 = dense.bwd(Q, K, V, dO, S, T, head_past_mask=[2, 0])
    for a, b in zip((dQ, dK, dV), d2):
        np.testing.assert_allclose(a, b, atol=TOL)
    np.testing.assert_allclose(dense.fwd(Q, K, V, S, T, head_past_mask=[2, 0])[0], O, atol=TOL)


def recurrence_autograd(Q, K, V, dO, S, T, flags, flagged_tail_is_sg=False, detach_before=0, seg_starts=None):
    """For every segment i and head: context = [sg(older past) if flagged ; tail of segment i-1 ;
    own segment], every prefix position visible and the own segment causal (Appendix C), run
    through library attention; stop-gradient realised with .detach() (Definition 3.2)."""
    q, k0, v0 = t64(Q, True), t64(K, True), t64(V, True)
    # keys before detach_before enter as constants (the boundary state of a truncated chain)
    X = detach_before
    k = torch.cat([k0[:, :X].detach(), k0[:, X:]], dim=1)
    v = torch.cat([v0[:, :X].detach(), v0[:, X:]], dim=1)
    B, L, Hq, d = Q.shape
    Hkv = K.shape[2]
    g = Hq // Hkv
    outs = torch.zeros(B, L, Hq, d, dtype=torch.float64)
    lses = torch.zeros(B, Hq, L, dtype=torch.float64)
    pieces = []
    bounds = list(range(0, L, S)) if seg_starts is None else [b for b in seg_starts if b < L]
    for i, s0 in enumerate(bounds):
        s1 = bounds[i + 1] if i + 1 < len(bounds) else L
        a = max(bounds[i - 1] if i > 0 else 0, s0 - T)   # the tail is at most the whole previous segment
        for h in range(Hq):
            c = h // g
            ks, vs = [], []
            if flags[c] == 1 and a > 0:
                ks.append(k[:, :a, c].detach())
                vs.append(v[:, :a, c].detach())
            if flags[c] != 2 and s0 > a:      # class 2: the own segment is the whole context
                kt, vt = k[:, a:s0, c], v[:, a:s0, c]
                if flags[c] == 1 and flagged_tail_is_sg:
                    kt, vt = kt.detach(), vt.detach()
                ks.append(kt)
                vs.append(vt)
            ks.append(k[:, s0:s1, c])
            vs.append(v[:, s0:s1, c])
            kc, vc = torch.cat(ks, dim=1), torch.cat(vs, dim=1)
            P = kc.shape[1] - (s1 - s0)
            m = torch.ones(s1 - s0, kc.shape[1], dtype=torch.bool)
            m[:, P:] = torch.ones(s1 - s0, s1 - s0, dtype=torch.bool).tril()
            o = F.scaled_dot_product_attention(q[:, s0:s1, h].unsqueeze(1), kc.unsqueeze(1), vc.unsqueeze(1),
                                               attn_mask=m).squeeze(1)
            pieces.append((o * t64(dO[:, s0:s1, h])).sum())
            outs[:, s0:s1, h] = o.detach()
            sc = torch.einsum("bld,bmd->blm", q[:, s0:s1, h], kc) / np.sqrt(d)
            lses[:, h, s0:s1] = torch.logsumexp(sc.masked_fill(~m, float("-inf")), dim=-1).detach()
    torch.stack(pieces).sum().backward()
    return outs.numpy(), lses.numpy(), q.grad.numpy(), k0.grad.numpy(), v0.grad.numpy()


@pytest.mark.parametrize("L,S,T,flags,variant", [
    (96, 32, 8, [0, 1], False),
    (96, 32, 32, [1, 0], False),
    (100, 32, 8, [0, 1], False),      # ragged last segment
    (90, 30, 7, [1, 1], False),
    (96, 32, 8, [0, 1], True),        # flagged heads' tail reads stop-gradient too
    (64, 16, 0, [0, 0], False),
    (96, 32, 8, [2, 0], False),       # an own-segment-only head beside a local one
    (100, 32, 8, [1, 2], False),      # ... beside a past-access one, ragged last segment
    (96, 32, 32, [2, 2], True),
])
def test_segment_recurrence_with_autograd(L, S, T, flags, variant):
    Q, K, V, dO = rand(2, L, 4, 2, 8)
    o, lse, gq, gk, gv = recurrence_autograd(Q, K, V, dO, S, T, flags, variant)
    O, LSE = oracle.fwd(Q, K, V, S, T, head_past_mask=flags)
    dQ, dK, dV = oracle.bwd(Q, K, V, dO, S, T, head_past_mask=flags, flagged_tail_is_sg=variant)
    np.testing.assert_allclose(O, o, atol=TOL)
    np.testing.assert_allclose(LSE, lse, atol=TOL)
    np.testing.assert_allclose(dQ, gq, atol=TOL)
    np.testing.assert_allclose(dK, gk, atol=TOL)
    np.testing.assert_allclose(dV, gv, atol=TOL)
    if not variant:
        d2 = dense.bwd(Q, K, V, dO, S, T, head_past_mask=flags)
        for a, b in zip((dQ, dK, dV), d2):
            np.testing.assert_allclose(a, b, atol=TOL)


@pytest.mark.parametrize("L,S,T,flags,X", [
    (96, 32, 8, [0, 1], 32),      # the window's differentiable part starts at segment 1
    (96, 32, 8, [0, 1], 64),
    (100, 32, 32, [2, 0], 40),    # a boundary inside a segment, ragged end
    (96, 32, 8, [1, 1], 96),      # everything detached: no K/V gradient at all
])
def test_detached_prefix_equals_autograd_with_constant_keys(L, S, T, flags, X):
    Q, K, V, dO = rand(2, L, 4, 2, 8)
    o, lse, gq, gk, gv = recurrence_autograd(Q, K, V, dO, S, T, flags, detach_before=X)
    dQ, dK, dV = oracle.bwd(Q, K, V, dO, S, T, head_past_mask=flags, detach_before=X)
    np.testing.assert_allclose(dQ, gq, atol=TOL)
    np.testing.assert_allclose(dK, gk, atol=TOL)
    np.testing.assert_allclose(dV, gv, atol=TOL)
    assert not dK[:, :X].any() and not dV[:, :X].any()
    # dQ does not depend on where K/V are cut
    np.testing.assert_array_equal(dQ, oracle.bwd(Q, K, V, dO, S, T, head_past_mask=flags)[0])


def test_windows_with_detached_incoming_state_compose_to_depth_one_truncation():
    # Truncation depth 1 over one layer: the loss of segment i sends gradient into the K/V of segments
    # i-1 (its tail) and i only.  Summing, over windows [i-1, i] whose incoming state is detached, the
    # gradients of the window's LAST segment loss gives the gradient of the whole untruncated call,
    # because one attention layer has no longer state chain than one transition.
    L, S, T = 128, 32, 8
    Q, K, V, dO = rand(1, L, 2, 2, 8)
    full = oracle.bwd(Q, K, V, dO, S, T)
    acc = [np.zeros_like(a) for a in full]
    for i in range(L // S):
        lo = max(0, i - 1) * S
        sl = slice(lo, (i + 1) * S)
        dOw = dO[:, sl].copy()
        dOw[:, :i * S - lo] = 0.0                      # only segment i's loss term
        g = oracle.bwd(Q[:, sl], K[:, sl], V[:, sl], dOw, S, T, q_pos0=lo, kv_pos0=lo, detach_before=lo)
        for a, b in zip(acc, g):
            a[:, sl] += b
    for a, b in zip(acc, full):
        np.testing.assert_allclose(a, b, atol=TOL)


# ---- segments of given lengths m_i (Section 3.1) ----------------------------------------------------
@pytest.mark.parametrize("L,starts,T,flags,variant", [
    (96, [0, 20, 50, 51, 80], 8, [0, 1], False),       # a one-token segment, a tail longer than its segment
    (100, [0, 33, 66], 40, [2, 0], False),              # T larger than every segment: the tail is the whole previous one
    (90, [0, 10, 30, 60], 7, [1, 1], True),
    (64, [0], 5, [0, 0], False),                        # one open-ended segment: plain causal
])
def test_segments_of_given_lengths_with_autograd(L, starts, T, flags, variant):
    Q, K, V, dO = rand(2, L, 4, 2, 8)
    o, lse, gq, gk, gv = recurrence_autograd(Q, K, V, dO, None, T, flags, variant, seg_starts=starts)
    O, LSE = oracle.fwd(Q, K, V, 1, T, head_past_mask=flags, seg_starts=starts)
    dQ, dK, dV = oracle.bwd(Q, K, V, dO, 1, T, head_past_mask=flags, flagged_tail_is_sg=variant, seg_starts=starts)
    for a, b in ((O, o), (LSE, lse), (dQ, gq), (dK, gk), (dV, gv)):
        np.testing.assert_allclose(a, b, atol=TOL)
    if not variant:
        d2 = dense.bwd(Q, K, V, dO, 1, T, head_past_mask=flags, seg_starts=starts)
        for a, b in zip((dQ, dK, dV), d2):
            np.testing.assert_allclose(a, b, atol=TOL)
        np.testing.assert_allclose(dense.fwd(Q, K, V, 1, T, head_past_mask=flags, seg_starts=starts)[0], O, atol=TOL)


def test_equal_given_lengths_are_the_constant_length_case():
    L, S, T = 100, 32, 9
    Q, K, V, dO = rand(1, L, 2, 2, 8)
    starts = list(range(0, L, S))
    a = oracle.fwd(Q, K, V, S, T, [0, 1]) + oracle.bwd(Q, K, V, dO, S, T, [0, 1])
    b = oracle.fwd(Q, K, V, 1, T, [0, 1], seg_starts=starts) + oracle.bwd(Q, K, V, dO, 1, T, [0, 1], seg_starts=starts)
    for x, y in zip(a, b):
        np.testing.assert_array_equal(x, y)
    assert oracle.count_pairs(1, L, 2, 2, S, T, [0, 1]) == oracle.count_pairs(1, L, 2, 2, 1, T, [0, 1], seg_starts=starts)


# ---- retrieved prefix: [K_ret ; K_i] -------------------------------------------------------------
def test_retrieving_every_older_position_is_the_dense_past_access_head():
    # with the index list naming all positions before the segment, the retrieved context is the context of a
    # past-access head of the dense reading; its own-segment gradients are those of that head too
    L, S = 96, 32
    Q, K, V, dO = rand(2, L, 4, 2, 8)
    O, LSE = oracle.fwd(Q, K, V, S, 0, head_past_mask=[1, 1])
    for i in range(1, L // S):
        sl = slice(i * S, (i + 1) * S)
        idx = np.broadcast_to(np.arange(i * S, dtype=np.int32), (2, 2, i * S))
        dOw = np.zeros_like(dO)
        dOw[:, sl] = dO[:, sl]
        _, dK, dV = oracle.bwd(Q, K, V, dOw, S, 0, head_past_mask=[1, 1])
        dQ = oracle.bwd(Q, K, V, dOw, S, 0, head_past_mask=[1, 1])[0]
        o, lse, gq, gk, gv = dense.retrieved_attention(Q[:, sl], K, V, idx, K[:, sl], V[:, sl], dO[:, sl])
        np.testing.assert_allclose(o, O[:, sl], atol=TOL)
        np.testing.assert_allclose(lse, LSE[:, :, sl], atol=TOL)
        np.testing.assert_allclose(gq, dQ[:, sl], atol=TOL)
        np.testing.assert_allclose(gk, dK[:, sl], atol=TOL)     # T = 0: only the own segment is differentiable
        np.testing.assert_allclose(gv, dV[:, sl], atol=TOL)


def test_retrieved_prefix_is_order_free_and_matches_library_attention():
    rng = np.random.default_rng(3)
    Q, Kp, Vp, dO = rand(1, 40, 2, 2, 8, rng)
    Ks, Vs = rng.standard_normal((1, 12, 2, 8)), rng.standard_normal((1, 12, 2, 8))
    Qs, dOs = Q[:, :12], dO[:, :12]
    idx = np.stack([rng.choice(40, size=9, replace=False) for _ in range(2)])[None].astype(np.int32)
    Kc, Vc = dense.retrieved_context(Kp, Vp, idx, Ks, Vs)
    for c in range(2):
        np.testing.assert_array_equal(Kc[0, :9, c], Kp[0, idx[0, c], c])
        np.testing.assert_array_equal(Vc[0, 9:, c], Vs[0, :, c])
    o1, l1 = dense.retrieved_attention(Qs, Kp, Vp, idx, Ks, Vs)
    o2, l2 = dense.retrieved_attention(Qs, Kp, Vp, idx[:, :, ::-1], Ks, Vs)   # softmax does not see the order
    np.testing.assert_allclose(o1, o2, atol=TOL)
    np.testing.assert_allclose(l1, l2, atol=TOL)
    # library attention over the same context with the same mask, prefix detached
    q = t64(Qs, True)
    ks, vs = t64(Ks, True), t64(Vs, True)
    kc = torch.cat([t64(Kc[:, :9]), ks], dim=1)
    vc = torch.cat([t64(Vc[:, :9]), vs], dim=1)
    m = torch.cat([torch.ones(12, 9, dtype=torch.bool), torch.ones(12, 12, dtype=torch.bool).tril()], dim=1)
    o = F.scaled_dot_product_attention(q.transpose(1, 2), kc.transpose(1, 2), vc.transpose(1, 2), attn_mask=m).transpose(1, 2)
    (o * t64(dOs)).sum().backward()
    o3, _, gq, gk, gv = dense.retrieved_attention(Qs, Kp, Vp, idx, Ks, Vs, dOs)
    np.testing.assert_allclose(o3, o.detach().numpy(), atol=TOL)
    np.testing.assert_allclose(gq, q.grad.numpy(), atol=TOL)
    np.testing.assert_allclose(gk, ks.grad.numpy(), atol=TOL)
    np.testing.assert_allclose(gv, vs.grad.numpy(), atol=TOL)


# ---- selection step of the retrieval operator (Appendix D): mechanics ------------------------------
def _select_by_sorting(Q, K, Hkv, window, stride, tail, top_k, n_anchors, off_lo, off_hi, R):
    """The same steps from fp64 scores and library sorting (valid when no two scores tie)."""
    B, Lq, Hq, d = Q.shape
    g, P = Hq // Hkv, K.shape[1]
    n_w = max(1, (Lq - window) // stride + 1) if Lq >= window else 1
    spans = [(u * stride, min(Lq, u * stride + window)) for u in range(n_w)] + [(max(0, Lq - tail), Lq)]
    out = np.zeros((B, Hkv, R), dtype=np.int32)
    for b in range(B):
        for c in range(Hkv):
            summ = np.stack([Q[b, r0:r1, c * g:(c + 1) * g].astype(np.float64).mean(axis=(0, 1)) for r0, r1 in spans])
            sc = summ @ K[b, :, c].astype(np.float64).T
            cand = sorted(set(np.argsort(-sc, axis=1)[:, :top_k].ravel().tolist()))
            anchors = sorted(cand, key=lambda j: -sc[:, j].max())[:n_anchors]
            chosen = []
            for a in anchors:
                for j in range(a - off_lo, a + off_hi + 1):
                    if 0 <= j < P and j not in chosen and len(chosen) < R:
                        chosen.append(j)
            chosen += [j for j in range(P) if j not in chosen][:R - len(chosen)]
            out[b, c] = sorted(chosen)
    return out


@pytest.mark.parametrize("Lq,window,stride,tail,top_k,n_anchors,off_lo,off_hi,R", [
    (24, 8, 4, 4, 5, 3, 2, 2, 32),
    (64, 16, 16, 8, 8, 4, 4, 3, 40),
    (5, 8, 4, 4, 3, 2, 0, 0, 7),          # fewer rows than one window; windows of one position
    (32, 8, 8, 32, 6, 6, 10, 10, 16),     # R smaller than the windows: best anchors first
])
def test_retrieval_selection_against_sorting_and_its_invariants(Lq, window, stride, tail, top_k, n_anchors, off_lo, off_hi, R):
    rng = np.random.default_rng(Lq + R)
    Q = rng.standard_normal((2, Lq, 4, 8)).astype(np.float32)
    K = rng.standard_normal((2, 300, 2, 8)).astype(np.float32)
    idx = retrieval.select(Q, K, window, stride, tail, top_k, n_anchors, off_lo, off_hi, R)
    assert idx.shape == (2, 2, R) and idx.dtype == np.int32
    assert (np.diff(idx, axis=2) > 0).all() and idx.min() >= 0 and idx.max() < 300     # sorted, distinct, in range
    np.testing.assert_array_equal(idx, _select_by_sorting(Q, K, 2, window, stride, tail, top_k, n_anchors, off_lo, off_hi, R))
    sc = retrieval.scores(retrieval.summaries(Q, 2, window, stride, tail), K)
    ref = np.einsum("bcme,bpce->bcmp", retrieval.summaries(Q, 2, window, stride, tail).astype(np.float64), K.astype(np.float64))
    assert np.abs(sc - ref).max() < 1e-5


def test_retrieval_summaries_written_out_by_hand():
    # Appendix D "Query construction": sliding-window means plus the mean of the last rows.  Rows q_r = (r, r^2),
    # so every expected mean below is worked out by hand, not by the span formula.
    q = lambda n: np.array([[r, r * r] for r in range(n)], dtype=np.float32).reshape(1, n, 1, 2)
    # 8 rows, window 4, stride 2, tail 2: windows [0,4) [2,6) [4,8), tail rows 6..7
    assert retrieval.n_summaries(8, 4, 2) == 4
    np.testing.assert_array_equal(retrieval.summaries(q(8), 1, 4, 2, 2)[0, 0],
                                  np.array([[1.5, 3.5], [3.5, 13.5], [5.5, 31.5], [6.5, 42.5]], dtype=np.float32))
    # 7 rows: a window must lie inside the rows present, so row 6 enters through the tail summary only
    assert retrieval.n_summaries(7, 4, 2) == 3
    np.testing.assert_array_equal(retrieval.summaries(q(7), 1, 4, 2, 2)[0, 0],
                                  np.array([[1.5, 3.5], [3.5, 13.5], [5.5, 30.5]], dtype=np.float32))
    # fewer rows than one window: a single window over what is there (rows 0..2), tail rows 1..2
    assert retrieval.n_summaries(3, 4, 2) == 2
    np.testing.assert_allclose(retrieval.summaries(q(3), 1, 4, 2, 2)[0, 0],
                               np.array([[1.0, 5.0 / 3.0], [1.5, 2.5]]), rtol=1e-6)
    # a tail longer than the rows present is all rows; stride = window gives disjoint windows
    np.testing.assert_array_equal(retrieval.summaries(q(4), 1, 2, 2, 9)[0, 0],
                                  np.array([[0.5, 0.5], [2.5, 6.5], [1.5, 3.5]], dtype=np.float32))
    # grouped heads: the mean runs over the group's query heads too.  Head 0 rows (r, r^2), head 1 rows (10 + r, 0)
    Q = np.zeros((1, 4, 2, 2), dtype=np.float32)
    Q[0, :, 0] = q(4)[0, :, 0]
    Q[0, :, 1, 0] = 10 + np.arange(4)
    np.testing.assert_array_equal(retrieval.summaries(Q, 1, 4, 4, 1)[0, 0],
                                  np.array([[6.5, 1.75], [8.0, 4.5]], dtype=np.float32))
    # two KV heads of one query head each keep their rows apart
    out = retrieval.summaries(Q, 2, 4, 4, 1)
    np.testing.assert_array_equal(out[0, 0], np.array([[1.5, 3.5], [3.0, 9.0]], dtype=np.float32))
    np.testing.assert_array_equal(out[0, 1], np.array([[11.5, 0.0], [13.0, 0.0]], dtype=np.float32))


def test_retrieval_selection_against_sorting_at_a_pool_of_thousands():
    rng = np.random.default_rng(77)
    Q = rng.standard_normal((1, 48, 4, 16)).astype(np.float32)
    K = rng.standard_normal((1, 3000, 2, 16)).astype(np.float32)
    args = (16, 8, 8, 6, 5, 7, 8, 96)
    np.testing.assert_array_equal(retrieval.select(Q, K, *args), _select_by_sorting(Q, K, 2, *args))


def test_retrieval_selection_finds_a_planted_key_and_pads_with_the_earliest():
    rng = np.random.default_rng(5)
    Q = rng.standard_normal((1, 16, 2, 8)).astype(np.float32)
    K = (0.01 * rng.standard_normal((1, 500, 1, 8))).astype(np.float32)
    tail_mean = Q[0, -4:].mean(axis=(0, 1))
    K[0, 321, 0] = 50.0 * tail_mean                    # by far the best match of the tail summary
    idx = retrieval.select(Q, K, 8, 8, 4, 1, 1, 3, 2, 12)[0, 0]
    assert set(range(318, 324)) <= set(idx.tolist())   # the anchor's window
    assert idx[:6].tolist() == [0, 1, 2, 3, 4, 5]      # and the earliest positions as padding
    # ties go to the lower position: all keys equal -> the first positions win everything
    Kc = np.ones((1, 50, 1, 8), dtype=np.float32)
    assert retrieval.select(Q, Kc, 8, 8, 4, 3, 2, 0, 1, 6)[0, 0].tolist() == [0, 1, 2, 3, 4, 5]


# ---- RoPE re-indexing for prefix concatenation (Section 3.4, Appendix E) -----------------------------
def test_rope_is_a_complex_rotation_of_the_half_split_pairs():
    rng = np.random.default_rng(3)
    d, base = 16, 10000.0
    x = rng.standard_normal((2, 9, 3, d))
    pos = np.array([0, 1, 2, 5, 17, 100, 1000, 4095, 70000])
    y = rope.rotate(x, pos, base)
    # z_i = x_i + 1j x_{i+d/2} multiplied by exp(1j pos base^(-2i/d)), written out with numpy's complex type
    z = x[..., : d // 2] + 1j * x[..., d // 2:]
    w = np.exp(1j * pos[:, None] * base ** (-2.0 * np.arange(d // 2) / d))[:, None, :]
    zz = z * w
    np.testing.assert_allclose(y, np.concatenate([zz.real, zz.imag], axis=-1), atol=1e-12)
    # the library form x cos + rotate_half(x) sin, with torch
    t = torch.tensor(x)
    ang = torch.tensor(pos, dtype=torch.float64)[:, None] * torch.pow(torch.tensor(base, dtype=torch.float64),
                                                                       -torch.arange(0, d, 2, dtype=torch.float64) / d)
    emb = torch.cat([ang, ang], dim=-1)[:, None, :]
    rot_half = torch.cat([-t[..., d // 2:], t[..., : d // 2]], dim=-1)
    np.testing.assert_allclose(y, (t * emb.cos() + rot_half * emb.sin()).numpy(), atol=1e-12)
    np.testing.assert_array_equal(y[:, 0], x[:, 0])                                   # position 0: identity
    np.testing.assert_allclose(np.linalg.norm(y, axis=-1), np.linalg.norm(x, axis=-1), rtol=1e-12)
    np.testing.assert_allclose(rope.rotate(y, pos, base, inverse=True), x, atol=1e-12)  # the transpose undoes it
    # the first pair turns by pos radians (frequency 1), the last by pos * base^(-(d-2)/d)
    e0 = np.zeros((1, 1, 1, d)); e0[..., 0] = 1.0
    r = rope.rotate(e0, [2.0], base)[0, 0, 0]
    assert abs(r[0] - np.cos(2.0)) < 1e-15 and abs(r[d // 2] - np.sin(2.0)) < 1e-15
    el = np.zeros((1, 1, 1, d)); el[..., d // 2 - 1] = 1.0
    r = rope.rotate(el, [3.0], base)[0, 0, 0]
    assert abs(r[d - 1] - np.sin(3.0 * base ** (-(d - 2.0) / d))) < 1e-15


def test_rope_scores_depend_on_the_position_difference_only():
    rng = np.random.default_rng(4)
    q, k = rng.standard_normal((1, 1, 1, 32)), rng.standard_normal((1, 1, 1, 32))
    for a, b in ((5, 3), (900, 17), (0, 40), (123, 123)):
        lhs = (rope.rotate(q, [a]) * rope.rotate(k, [b])).sum()
        rhs = (q * rope.rotate(k, [b - a])).sum()
        assert abs(lhs - rhs) < 1e-11
        assert abs(lhs - (rope.rotate(q, [a + 1000]) * rope.rotate(k, [b + 1000])).sum()) < 1e-10


def test_reindexed_prefix_of_the_preceding_rows_is_attention_under_global_positions():
    # Appendix E: re-indexing "is equivalent to treating the prefix as preceding context under standard RoPE".
    # Retrieve exactly the R rows in front of the segment, in order: positions 0..R-1 and R..R+m-1 differ from
    # the global ones s-R..s+m-1 by a constant, so the attention must equal library attention over those rows
    # with every tensor rotated at its global position.
    rng = np.random.default_rng(6)
    B, Hq, Hkv, d, s, R, m = 2, 4, 2, 16, 40, 12, 9
    Q = rng.standard_normal((B, s + m, Hq, d))
    K = rng.standard_normal((B, s + m, Hkv, d))
    V = rng.standard_normal((B, s + m, Hkv, d))
    idx = np.broadcast_to(np.arange(s - R, s, dtype=np.int32), (B, Hkv, R)).copy()
    Kc, Vc, Qr = rope.reindexed_context(K[:, :s], V[:, :s], idx, K[:, s:], V[:, s:], Q[:, s:])
    # the attention over the rotated context: prefix rows all visible, the segment causal
    sc = 1.0 / np.sqrt(d)
    g = Hq // Hkv
    vis = np.concatenate([np.ones((m, R), bool), np.tril(np.ones((m, m), bool))], axis=1)
    pos = np.arange(s - R, s + m)
    Kg, Qg = rope.rotate(K[:, s - R:], pos), rope.rotate(Q[:, s:], pos[R:])
    for b in range(B):
        for h in range(Hq):
            c = h // g
            a1 = np.where(vis, sc * Qr[b, :, h] @ Kc[b, :, c].T, -np.inf)
            a2 = np.where(vis, sc * Qg[b, :, h] @ Kg[b, :, c].T, -np.inf)
            np.testing.assert_allclose(a1, a2, atol=1e-10)
            p1 = torch.softmax(torch.tensor(a1), dim=-1).numpy()
            np.testing.assert_allclose(p1 @ Vc[b, :, c], torch.softmax(torch.tensor(a2), dim=-1).numpy() @ V[b, s - R:, c], atol=1e-10)
    np.testing.assert_array_equal(Vc[:, R:], V[:, s:])                                  # values are not rotated
    np.testing.assert_array_equal(Vc[:, :R], V[:, s - R:s])
    # an arbitrary (non-contiguous, per-head) selection: each retrieved key is rotated by its slot, not its origin
    idx2 = np.stack([np.stack([np.sort(rng.choice(s, R, replace=False)) for _ in range(Hkv)]) for _ in range(B)]).astype(np.int32)
    Kc2, _, _ = rope.reindexed_context(K[:, :s], V[:, :s], idx2, K[:, s:], V[:, s:], Q[:, s:])
    for r in (0, 5, R - 1):
        np.testing.assert_allclose(Kc2[1, r, 1], rope.rotate(K[1:2, idx2[1, 1, r]:idx2[1, 1, r] + 1, 1:2], [r])[0, 0, 0], atol=1e-12)


# ---- closed form: zero keys => uniform attention over the visible set ---------------------------
def test_zero_keys_closed_form_counts_the_context():
    B, L, Hq, Hkv, d, S, T = 1, 120, 2, 2, 4, 40, 10
    Q, K, V, _ = rand(B, L, Hq, Hkv, d)
    K[:] = 0.0
    O, LSE = oracle.fwd(Q, K, V, S, T, head_past_mask=[0, 1])
    for p in range(L):
        i, t = divmod(p, S)
        n_local = t + 1 + (T if i > 0 else 0)          # S + M context of the cost model, Section 3.5
        lo = p + 1 - n_local
        assert abs(LSE[0, 0, p] - np.log(n_local)) < 1e-12
        assert abs(LSE[0, 1, p] - np.log(p + 1)) < 1e-12
        np.testing.assert_allclose(O[0, p, 0], V[0, lo:p + 1, 0].mean(axis=0), atol=1e-12)
        np.testing.assert_allclose(O[0, p, 1], V[0, :p + 1, 1].mean(axis=0), atol=1e-12)


def test_context_size_golden():
    path = os.path.join(os.path.dirname(__file__), "golden", "context_size.txt")
    rows = [tuple(int(x) for x in ln.split()) for ln in open(path) if ln.strip() and not ln.startswith("#")]
    assert rows
    for S, M, i, t, n in rows:
        L = (i + 1) * S
        Q = np.zeros((1, L, 1, 1))
        O, LSE = oracle.fwd(Q, Q, Q, S, M)
        assert abs(np.exp(LSE[0, 0, i * S + t]) - n) < 1e-6


# ---- finite differences with the stop-gradient semantics -----------------------------------------
def fd_objective(Q, K, V, Kbar, Vbar, dO, S, T, flags):
    """<O, dO> where every stop-gradient read takes its key/value from the constant copies
    Kbar/Vbar (sg = identity forward, constant backward).  Built from oracle.fwd alone, one
    segment at a time through its position offsets."""
    L = Q.shape[1]
    tot = 0.0
    for i in range((L + S - 1) // S):
        s0, s1 = i * S, min(L, (i + 1) * S)
        a = max(0, s0 - T)
        Km = np.concatenate([Kbar[:, :a], K[:, a:s1]], axis=1)
        Vm = np.concatenate([Vbar[:, :a], V[:, a:s1]], axis=1)
        O, _ = oracle.fwd(Q[:, s0:s1], Km, Vm, S, T, head_past_mask=flags, q_pos0=s0)
        tot += float((O * dO[:, s0:s1]).sum())
    return tot


def test_gradients_match_central_finite_differences():
    rng = np.random.default_rng(3)
    B, L, Hq, Hkv, d, S, T = 1, 48, 2, 2, 4, 16, 5
    flags = [1, 0]
    Q, K, V, dO = rand(B, L, Hq, Hkv, d, rng)
    dQ, dK, dV = oracle.bwd(Q, K, V, dO, S, T, head_past_mask=flags)
    eps = 1e-5
    for name, X, G in (("Q", Q, dQ), ("K", K, dK), ("V", V, dV)):
        idxs = [tuple(rng.integers(0, n) for n in X.shape) for _ in range(40)]
        # make sure tail, non-tail and first-segment positions of both heads are probed
        for pos in (0, S - T - 1, S - T, S - 1, S, 2 * S - 1, L - 1):
            for hh in range(X.shape[2]):
                idxs.append((0, pos, hh, int(rng.integers(0, d))))
        for idx in idxs:
            args = {"Q": Q, "K": K, "V": V}
            Xp, Xm = X.copy(), X.copy()
            Xp[idx] += eps
            Xm[idx] -= eps
            ap, am = dict(args), dict(args)
            ap[name], am[name] = Xp, Xm
            fp = fd_objective(ap["Q"], ap["K"], ap["V"], K, V, dO, S, T, flags)
            fm = fd_objective(am["Q"], am["K"], am["V"], K, V, dO, S, T, flags)
            fd = (fp - fm) / (2 * eps)
            assert abs(fd - G[idx]) <= 1e-6 * max(1.0, abs(fd)), (name, idx, fd, G[idx])


# ---- gradient reach: the tail is the only differentiable cross-segment state -------------------
def test_loss_on_one_segment_reaches_only_that_segment_and_previous_tail():
    B, L, Hq, Hkv, d, S, T = 1, 128, 4, 2, 8, 32, 8
    Q, K, V, dO = rand(B, L, Hq, Hkv, d)
    dO[:, :2 * S] = 0.0
    dO[:, 3 * S:] = 0.0                      # loss on the third segment only
    for flags in ([0, 0], [1, 0], [1, 1]):
        dQ, dK, dV = oracle.bwd(Q, K, V, dO, S, T, head_past_mask=flags)
        for G in (dK, dV):
            assert np.all(G[:, :2 * S - T] == 0.0)       # exactly zero before the tail of segment 2
            assert np.all(G[:, 3 * S:] == 0.0)
            assert np.abs(G[:, 2 * S - T:3 * S]).min() > 0.0
        assert np.all(dQ[:, :2 * S] == 0.0) and np.all(dQ[:, 3 * S:] == 0.0)


def test_flag_changes_dq_but_not_the_reach_of_dk_dv():
    B, L, Hq, Hkv, d, S, T = 1, 96, 2, 1, 8, 32, 8
    Q, K, V, dO = rand(B, L, Hq, Hkv, d)
    dQ0, dK0, dV0 = oracle.bwd(Q, K, V, dO, S, T, head_past_mask=[0])
    dQ1, dK1, dV1 = oracle.bwd(Q, K, V, dO, S, T, head_past_mask=[1])
    assert np.abs(dQ1[:, S:] - dQ0[:, S:]).max() > 1e-6          # sg keys do feed dQ
    np.testing.assert_allclose(dQ1[:, :S], dQ0[:, :S], atol=TOL)  # first segment: nothing older to read
    # a key outside the tail of segment 0 still gets nothing from segment 1 or 2 queries:
    dO2 = dO.copy()
    dO2[:, :S] = 0.0
    _, dK2, dV2 = oracle.bwd(Q, K, V, dO2, S, T, head_past_mask=[1])
    assert np.all(dK2[:, :S - T] == 0.0) and np.all(dV2[:, :S - T] == 0.0)


def test_unflagged_output_ignores_keys_before_the_tail():
    B, L, Hq, Hkv, d, S, T = 1, 96, 2, 2, 8, 32, 8
    Q, K, V, _ = rand(B, L, Hq, Hkv, d)
    O, LSE = oracle.fwd(Q, K, V, S, T, head_past_mask=[0, 1])
    K2, V2 = K.copy(), V.copy()
    K2[:, :2 * S - T] += 3.0
    V2[:, :2 * S - T] -= 2.0
    O2, LSE2 = oracle.fwd(Q, K2, V2, S, T, head_past_mask=[0, 1])
    assert np.array_equal(O[:, 2 * S:, 0], O2[:, 2 * S:, 0]) and np.array_equal(LSE[:, 0, 2 * S:], LSE2[:, 0, 2 * S:])
    assert np.abs(O[:, 2 * S:, 1] - O2[:, 2 * S:, 1]).max() > 1e-3   # the flagged head does read them


# ---- cost model: pair counts --------------------------------------------------------------------
@pytest.mark.parametrize("L,S,T", [(2048, 512, 128), (4096, 1024, 1024), (1536, 512, 0)])
def test_pair_counts_match_closed_forms(L, S, T):
    N = L // S
    local = N * S * (S + 1) // 2 + (N - 1) * S * T
    full = L * (L + 1) // 2
    nv, nd = oracle.count_pairs(2, L, 4, 2, S, T, head_past_mask=[0, 1])
    assert nv == 2 * 2 * (local + full) and nd == 2 * 4 * local
    nv, nd = oracle.count_pairs(1, L, 4, 4, S, T)
    assert nv == nd == 4 * local
    own = N * S * (S + 1) // 2                       # class 2: the causal triangle of each segment
    nv, nd = oracle.count_pairs(1, L, 4, 2, S, T, head_past_mask=[2, 1])
    assert nv == 2 * (own + full) and nd == 2 * (own + local)


def test_benchmark_pair_counts():
    # visible pairs of the benchmark configurations, recomputed from the closed forms
    assert oracle.count_pairs(1, 2048, 4, 4, 512, 128)[0] == 2887680
    nv, nd = oracle.count_pairs(2, 16384, 32, 8, 2048, 512, head_past_mask=[0, 0, 1, 0, 1, 0, 0, 0])
    local = 8 * 2048 * 2049 // 2 + 7 * 2048 * 512
    assert nv == 2 * (24 * local + 8 * (16384 * 16385 // 2)) == 3305635840
    assert nd == 2 * 32 * local


@pytest.mark.parametrize("q0,L,k0,Lk", [(10, 9, 4, 15), (0, 20, 0, 20), (14, 5, 0, 19), (21, 7, 30, 4)])
def test_pair_counts_of_a_window_match_enumeration(q0, L, k0, Lk):
    # a window of queries at q0 against keys at k0: counted pair by pair from the mask's definition
    S, T, classes = 7, 3, [0, 1]
    nv = nd = 0
    for cls in classes:
        for p in range(q0, q0 + L):
            a = max(0, (p // S) * S - T)
            for j in range(max(k0, 0), k0 + Lk):
                if j <= p and (j >= a or cls == 1):
                    nv += 1
                    nd += j >= a
    assert oracle.count_pairs(1, L, 2, 2, S, T, classes, Lk=Lk, q_pos0=q0, kv_pos0=k0) == (nv, nd)


# ---- the two statements of the definition agree; streamed == one-shot ---------------------------
def test_c_oracle_matches_dense_form_on_configuration_1():
    import workloads
    w = workloads.CONFIGS[0]
    x = workloads.make_inputs(w)
    Q, K, V, dO = (workloads.to_f64(x[k]) for k in ("Q", "K", "V", "dO"))
    O, LSE = oracle.fwd(Q, K, V, w.S, w.T, x["mask"])
    O2, LSE2 = dense.fwd(Q, K, V, w.S, w.T, x["mask"])
    np.testing.assert_allclose(O, O2, atol=1e-12)
    np.testing.assert_allclose(LSE, LSE2, atol=1e-12)
    g1 = oracle.bwd(Q, K, V, dO, w.S, w.T, x["mask"])
    g2 = dense.bwd(Q, K, V, dO, w.S, w.T, x["mask"])
    for a, b in zip(g1, g2):
        np.testing.assert_allclose(a, b, atol=1e-11)


def test_streamed_segments_equal_one_shot_forward():
    B, L, Hq, Hkv, d, S, T = 1, 128, 4, 2, 8, 32, 8
    flags = [0, 1]
    Q, K, V, _ = rand(B, L, Hq, Hkv, d)
    O, LSE = oracle.fwd(Q, K, V, S, T, head_past_mask=flags)
    for i in range(L // S):
        s0, s1 = i * S, (i + 1) * S
        # flagged head: whole history; the other head would need only [s0-T, s1) - pass that window
        Oi, LSEi = oracle.fwd(Q[:, s0:s1], K[:, :s1], V[:, :s1], S, T, head_past_mask=flags, q_pos0=s0)
        np.testing.assert_array_equal(Oi, O[:, s0:s1])
        np.testing.assert_array_equal(LSEi, LSE[:, :, s0:s1])
        a = max(0, s0 - T)
        Ow, _ = oracle.fwd(Q[:, s0:s1, :2], K[:, a:s1, :1], V[:, a:s1, :1], S, T, q_pos0=s0, kv_pos0=a)
        np.testing.assert_array_equal(Ow, O[:, s0:s1, :2])


def test_invalid_configurations_are_rejected():
    Q, K, V, _ = rand(1, 8, 2, 2, 4)
    with pytest.raises(ValueError):
        oracle.fwd(Q, K, V, 4, 5)          # tail longer than a segment
    with pytest.raises(ValueError):
        oracle.fwd(Q, K, V, 0, 0)

"""GPU parity: the CUDA path, called through the C ABI, against the fp64 oracle on the same
seeded inputs - element by element on small and mid-size cases, on oracle-computable
sub-problems at the full benchmark sizes."""
import os

import numpy as np
import pytest
import torch

import oracle
import workloads
import paper_2605_11744_b200 as sa
from util import (TOL_GRAD, assert_fwd_close, assert_grads_close, f64, group_slices, oracle_last_rows, oracle_rows,
                  oracle_window, rand_inputs, rel_l2)

pytestmark = pytest.mark.gpu

SMALL = [
    # B, L, Hq, Hkv, d, S, T, mask
    (1, 128, 1, 1, 128, 128, 0, [0]),                 # one tile
    (1, 384, 2, 1, 128, 128, 128, [0]),               # tail = whole previous segment
    (1, 1024, 4, 2, 128, 256, 128, [0, 1]),           # GQA, mixed flags
    (2, 700, 4, 2, 128, 200, 72, [1, 0]),             # nothing aligned to the 128 tile, ragged end
    (1, 1000, 2, 2, 128, 1000, 0, [0, 0]),            # S >= L: plain causal
    (1, 640, 2, 1, 128, 128, 0, [0]),                 # T = 0: block diagonal
    (1, 640, 2, 2, 128, 64, 64, [1, 1]),              # segments shorter than a tile, all flagged
    (1, 333, 2, 2, 64, 100, 100, [0, 1]),             # d = 64, ragged
    (1, 130, 1, 1, 64, 7, 3, [0]),                    # tiny segments
    (3, 1, 2, 1, 128, 4, 2, [1]),                     # a single query row
]


@pytest.mark.parametrize("B,L,Hq,Hkv,d,S,T,mask", SMALL)
def test_small_cases_match_oracle_elementwise(B, L, Hq, Hkv, d, S, T, mask):
    Q, K, V, dO = rand_inputs(B, L, Hq, Hkv, d, seed=L + S)
    O, LSE = sa.seg_attn_fwd(Q, K, V, S, T, mask)
    dQ, dK, dV = sa.seg_attn_bwd(Q, K, V, O, LSE, dO, S, T, mask)
    sa.poll_status()
    Oo, LSEo = oracle.fwd(f64(Q), f64(K), f64(V), S, T, mask)
    ref = oracle.bwd(f64(Q), f64(K), f64(V), f64(dO), S, T, mask)
    assert_fwd_close(O, LSE, Oo, LSEo, "fwd")
    assert_grads_close((dQ, dK, dV), ref, "bwd")


@pytest.mark.parametrize("B,L,Hq,Hkv,d,S,T,mask", [
    (1, 1024, 4, 2, 128, 256, 128, [2, 0]),           # own-segment-only beside local
    (2, 700, 6, 3, 128, 200, 72, [1, 2, 0]),          # all three classes, nothing aligned, ragged end
    (1, 1152, 4, 4, 128, 384, 128, [2, 2, 1, 0]),     # segments of three tiles
    (1, 333, 2, 2, 64, 100, 100, [2, 2]),             # d = 64, every head own-only
    (1, 640, 2, 2, 128, 64, 64, [2, 1]),              # segments shorter than a tile
])
@pytest.mark.parametrize("tail_sg", [False, True])
def test_head_classes_local_past_and_own_segment_only(B, L, Hq, Hkv, d, S, T, mask, tail_sg):
    # the three contexts of Eq. "ctx": [tail ; own], [past ; own] and own alone, chosen per KV head
    Q, K, V, dO = rand_inputs(B, L, Hq, Hkv, d, seed=L + S + T)
    O, LSE = sa.seg_attn_fwd(Q, K, V, S, T, mask)
    dQ, dK, dV = sa.seg_attn_bwd(Q, K, V, O, LSE, dO, S, T, mask, flagged_tail_is_sg=tail_sg)
    sa.poll_status()
    Oo, LSEo = oracle.fwd(f64(Q), f64(K), f64(V), S, T, mask)
    ref = oracle.bwd(f64(Q), f64(K), f64(V), f64(dO), S, T, mask, flagged_tail_is_sg=tail_sg)
    assert_fwd_close(O, LSE, Oo, LSEo, "fwd")
    assert_grads_close((dQ, dK, dV), ref, "bwd")
    # an own-segment-only head never reads the tail: T does not matter for it, to the bit
    O0, LSE0 = sa.seg_attn_fwd(Q, K, V, S, 0, mask)
    g = Hq // Hkv
    for c, cls in enumerate(mask):
        if cls == 2:
            assert torch.equal(O[:, :, c * g:(c + 1) * g], O0[:, :, c * g:(c + 1) * g])


@pytest.mark.parametrize("B,L,Hq,Hkv,d,S,T,mask,X", [
    (1, 1024, 4, 2, 128, 256, 128, [0, 1], 256),      # boundary on a segment and a tile
    (2, 700, 4, 2, 128, 200, 72, [1, 0], 400),        # boundary inside a tile
    (1, 1152, 6, 3, 128, 384, 128, [2, 1, 0], 500),   # boundary inside a segment, all head classes
    (1, 333, 2, 2, 64, 100, 100, [0, 1], 333),        # everything detached
    (1, 640, 2, 1, 128, 128, 64, [0], 0),             # none
])
def test_detached_prefix_gets_no_gradient(B, L, Hq, Hkv, d, S, T, mask, X):
    # keys before detach_before are constants of the window (the boundary state of a truncated chain)
    Q, K, V, dO = rand_inputs(B, L, Hq, Hkv, d, seed=L + X)
    O, LSE = sa.seg_attn_fwd(Q, K, V, S, T, mask)
    dQ, dK, dV = sa.seg_attn_bwd(Q, K, V, O, LSE, dO, S, T, mask, detach_before=X)
    sa.poll_status()
    ref = oracle.bwd(f64(Q), f64(K), f64(V), f64(dO), S, T, mask, detach_before=X)
    assert_grads_close((dQ, dK, dV), ref, "detached prefix")
    assert not dK[:, :X].any() and not dV[:, :X].any()
    dQ0, _, _ = sa.seg_attn_bwd(Q, K, V, O, LSE, dO, S, T, mask)
    assert torch.equal(dQ, dQ0)


def test_window_of_two_segments_with_detached_incoming_tail():
    # one step of depth-one truncation: queries of segments i-1 and i, keys from the tail of segment i-2 on;
    # that tail is read (forward) but receives nothing
    B, L, Hq, Hkv, d, S, T = 1, 1024, 4, 2, 128, 256, 128
    Q, K, V, dO = rand_inputs(B, L, Hq, Hkv, d, seed=5)
    lo, k0 = 2 * S, 2 * S - T
    Qw, dOw = Q[:, lo:lo + 2 * S].contiguous(), dO[:, lo:lo + 2 * S].contiguous()
    Kw, Vw = K[:, k0:lo + 2 * S].contiguous(), V[:, k0:lo + 2 * S].contiguous()
    Ow, LSEw = sa.seg_attn_fwd(Qw, Kw, Vw, S, T, [0, 0], q_pos0=lo, kv_pos0=k0)
    g = sa.seg_attn_bwd(Qw, Kw, Vw, Ow, LSEw, dOw, S, T, [0, 0], q_pos0=lo, kv_pos0=k0, detach_before=lo)
    sa.poll_status()
    ref = oracle.bwd(f64(Qw), f64(Kw), f64(Vw), f64(dOw), S, T, [0, 0], q_pos0=lo, kv_pos0=k0, detach_before=lo)
    assert_grads_close(g, ref, "window")
    assert not g[1][:, :T].any() and not g[2][:, :T].any()


@pytest.mark.parametrize("B,L,Hq,Hkv,d,S,T,mask", [
    (1, 1024, 4, 2, 128, 256, 128, [0, 1]),
    (2, 700, 4, 2, 128, 200, 72, [1, 0]),
    (1, 640, 2, 2, 128, 64, 64, [1, 1]),
    (1, 333, 2, 2, 64, 100, 100, [0, 1]),
])
def test_flagged_heads_reading_the_tail_forward_only(B, L, Hq, Hkv, d, S, T, mask):
    # the literal reading of Eq. "ctx": only unflagged (local) heads send gradient through the carried tail
    Q, K, V, dO = rand_inputs(B, L, Hq, Hkv, d, seed=L + T)
    O, LSE = sa.seg_attn_fwd(Q, K, V, S, T, mask)
    dQ, dK, dV = sa.seg_attn_bwd(Q, K, V, O, LSE, dO, S, T, mask, flagged_tail_is_sg=True)
    sa.poll_status()
    ref = oracle.bwd(f64(Q), f64(K), f64(V), f64(dO), S, T, mask, flagged_tail_is_sg=True)
    assert_grads_close((dQ, dK, dV), ref, "flagged tail sg")
    # it differs from the default reading exactly on the flagged heads' K/V gradients
    dQ0, dK0, dV0 = sa.seg_attn_bwd(Q, K, V, O, LSE, dO, S, T, mask)
    assert torch.equal(dQ, dQ0)
    for c, f in enumerate(mask):
        same = torch.equal(dK[:, :, c], dK0[:, :, c]) and torch.equal(dV[:, :, c], dV0[:, :, c])
        assert same == (f != 1 or T == 0)


def test_window_of_queries_with_position_offsets():
    # queries of segments 2..3 only (q_pos0 = 2 S) against all keys up to their end: forward and backward
    # equal the oracle's for the same window; this is the call shape of a windowed training step
    B, L, Hq, Hkv, d, S, T = 1, 1024, 4, 2, 128, 256, 128
    Q, K, V, dO = rand_inputs(B, L, Hq, Hkv, d, seed=17)
    mask = [1, 0]
    q0, q1 = 2 * S, 4 * S
    Qw, dOw, Kw, Vw = Q[:, q0:q1].contiguous(), dO[:, q0:q1].contiguous(), K[:, :q1].contiguous(), V[:, :q1].contiguous()
    O, LSE = sa.seg_attn_fwd(Qw, Kw, Vw, S, T, mask, q_pos0=q0)
    dQ, dK, dV = sa.seg_attn_bwd(Qw, Kw, Vw, O, LSE, dOw, S, T, mask, q_pos0=q0)
    sa.poll_status()
    Oo, LSEo = oracle.fwd(f64(Qw), f64(Kw), f64(Vw), S, T, mask, q_pos0=q0)
    ref = oracle.bwd(f64(Qw), f64(Kw), f64(Vw), f64(dOw), S, T, mask, q_pos0=q0)
    assert_fwd_close(O, LSE, Oo, LSEo, "window")
    assert_grads_close((dQ, dK, dV), ref, "window")
    # keys before the tail of segment 1 get gradient from no query of the window
    assert torch.count_nonzero(dK[:, :q0 - T]) == 0 and torch.count_nonzero(dV[:, :q0 - T]) == 0
    # the forward of the window equals the rows of the whole-sequence forward, bit for bit (same tiles)
    O_all, LSE_all = sa.seg_attn_fwd(Q, K, V, S, T, mask)
    assert torch.equal(O, O_all[:, q0:q1]) and torch.equal(LSE, LSE_all[:, :, q0:q1])


def test_configuration_1_in_full():
    w = workloads.CONFIGS[0]
    x = workloads.make_inputs(w)
    Q, K, V, dO = (x[k].cuda() for k in ("Q", "K", "V", "dO"))
    O, LSE = sa.seg_attn_fwd(Q, K, V, w.S, w.T, x["mask"], w.sm_scale)
    grads = sa.seg_attn_bwd(Q, K, V, O, LSE, dO, w.S, w.T, x["mask"], w.sm_scale)
    sa.poll_status()
    Oo, LSEo = oracle.fwd(f64(Q), f64(K), f64(V), w.S, w.T, x["mask"])
    ref = oracle.bwd(f64(Q), f64(K), f64(V), f64(dO), w.S, w.T, x["mask"])
    assert_fwd_close(O, LSE, Oo, LSEo, w.name)
    assert_grads_close(grads, ref, w.name)


def test_structural_zeros_and_reproducibility():
    # loss on the third segment only: dK/dV are exactly zero before the tail of segment 2 and after segment 3
    B, L, Hq, Hkv, d, S, T = 1, 1024, 4, 2, 128, 256, 128
    Q, K, V, dO = rand_inputs(B, L, Hq, Hkv, d, seed=5)
    dO[:, :2 * S] = 0
    dO[:, 3 * S:] = 0
    mask = [1, 0]
    O, LSE = sa.seg_attn_fwd(Q, K, V, S, T, mask)
    dQ, dK, dV = sa.seg_attn_bwd(Q, K, V, O, LSE, dO, S, T, mask)
    for G in (dK, dV):
        assert torch.count_nonzero(G[:, :2 * S - T]) == 0
        assert torch.count_nonzero(G[:, 3 * S:]) == 0
        assert torch.count_nonzero(G[:, 2 * S - T:3 * S]) > 0
    assert torch.count_nonzero(dQ[:, :2 * S]) == 0 and torch.count_nonzero(dQ[:, 3 * S:]) == 0
    # no atomics anywhere: a second run gives the same bits
    O2, LSE2 = sa.seg_attn_fwd(Q, K, V, S, T, mask)
    dQ2, dK2, dV2 = sa.seg_attn_bwd(Q, K, V, O2, LSE2, dO, S, T, mask)
    for a, b in ((O, O2), (LSE, LSE2), (dQ, dQ2), (dK, dK2), (dV, dV2)):
        assert torch.equal(a, b)


def test_unflagged_heads_ignore_everything_before_the_tail():
    B, L, Hq, Hkv, d, S, T = 1, 1024, 2, 2, 128, 256, 128
    Q, K, V, _ = rand_inputs(B, L, Hq, Hkv, d, seed=9)
    O, LSE = sa.seg_attn_fwd(Q, K, V, S, T, [0, 1])
    K2, V2 = K.clone(), V.clone()
    K2[:, :2 * S - T, 0] = float("nan")  # never staged for the unflagged head's later segments
    V2[:, :2 * S - T, 0] = float("nan")
    K2[:, :2 * S - T, 1] += 3.0
    V2[:, :2 * S - T, 1] -= 2.0
    O2, LSE2 = sa.seg_attn_fwd(Q, K2, V2, S, T, [0, 1])
    assert torch.equal(O[:, 2 * S:, 0], O2[:, 2 * S:, 0]) and torch.equal(LSE[:, 0, 2 * S:], LSE2[:, 0, 2 * S:])
    assert (O[:, 2 * S:, 1].float() - O2[:, 2 * S:, 1].float()).abs().max() > 1e-2   # the flagged head does read them


def test_outputs_outside_the_problem_are_untouched_and_strides_respected():
    # O, dQ, dK, dV live inside larger poisoned buffers (head and position padding)
    B, L, Hq, Hkv, d, S, T = 2, 300, 2, 1, 128, 128, 64
    Q, K, V, dO = rand_inputs(B, L, Hq, Hkv, d, seed=11)

    def padded(t):
        big = torch.full((t.shape[0], t.shape[1] + 3, t.shape[2] + 1, t.shape[3]), float("nan"),
                         dtype=t.dtype, device=t.device)
        view = big[:, :t.shape[1], :t.shape[2]]
        view.copy_(t)
        return big, view

    _, Qv = padded(Q)
    _, Kv = padded(K)
    _, Vv = padded(V)
    Obig, Ov = padded(torch.zeros_like(Q))
    Obig.fill_(float("nan"))
    O, LSE = sa.seg_attn_fwd(Qv, Kv, Vv, S, T, [1], out=Ov)
    Oo, LSEo = oracle.fwd(f64(Q), f64(K), f64(V), S, T, [1])
    assert_fwd_close(Ov, LSE, Oo, LSEo, "strided")
    assert torch.isnan(Obig[:, L:]).all() and torch.isnan(Obig[:, :, Hq:]).all()


def test_empty_and_degenerate_shapes():
    mk = lambda *s: torch.zeros(*s, dtype=torch.bfloat16, device="cuda")
    # no batch, no rows: nothing to do, no error
    for B, L in ((0, 128), (2, 0)):
        O, LSE = sa.seg_attn_fwd(mk(B, L, 2, 128), mk(B, L, 1, 128), mk(B, L, 1, 128), 64, 16, [0])
        dQ, dK, dV = sa.seg_attn_bwd(mk(B, L, 2, 128), mk(B, L, 1, 128), mk(B, L, 1, 128), O, LSE,
                                     mk(B, L, 2, 128), 64, 16, [0])
        assert O.numel() == 0 and dK.numel() == 0
    # keys that do not reach the queries: rows without any visible key give O = 0, LSE = -inf, zero gradients
    Q, K, V, dO = rand_inputs(1, 256, 2, 1, 128, seed=3, Lk=100)
    O, LSE = sa.seg_attn_fwd(Q, K, V, 64, 16, [0])
    dQ, dK, dV = sa.seg_attn_bwd(Q, K, V, O, LSE, dO, 64, 16, [0])
    sa.poll_status()
    Oo, LSEo = oracle.fwd(f64(Q), f64(K), f64(V), 64, 16, [0])
    ref = oracle.bwd(f64(Q), f64(K), f64(V), f64(dO), 64, 16, [0])
    assert_fwd_close(O, LSE, Oo, LSEo, "short kv")
    assert torch.isinf(LSE[:, :, 128:]).all() and torch.count_nonzero(O[:, 128:]) == 0
    assert_grads_close((dQ, dK, dV), ref, "short kv")
    assert torch.count_nonzero(dQ[:, 128:]) == 0


def test_more_work_items_per_block_than_the_item_ring_holds_with_keyless_items_among_them():
    # 1536 work items (about ten per persistent block, more than the ring of decoded items between the scheduling
    # warp and the other roles holds), of which the later query tiles of the local head have no key in reach
    # (the keys end half way): those items carry no tiles and are written as zeros / -inf between items that do
    B, L, Lk, Hq, Hkv, d, S, T, mask = 2, 6144, 3000, 16, 2, 128, 256, 128, [0, 1]
    Q, K, V, dO = rand_inputs(B, L, Hq, Hkv, d, seed=11, Lk=Lk)
    O, LSE = sa.seg_attn_fwd(Q, K, V, S, T, mask)
    dQ, dK, dV = sa.seg_attn_bwd(Q, K, V, O, LSE, dO, S, T, mask)
    sa.poll_status()
    Oo, LSEo = oracle.fwd(f64(Q), f64(K), f64(V), S, T, mask)
    ref = oracle.bwd(f64(Q), f64(K), f64(V), f64(dO), S, T, mask)
    assert_fwd_close(O, LSE, Oo, LSEo, "many items")
    assert_grads_close((dQ, dK, dV), ref, "many items")
    g = Hq // Hkv
    assert torch.isinf(LSE[:, :g, 3328:]).all() and torch.count_nonzero(O[:, 3328:, :g]) == 0   # local head: tail start >= 3000
    assert torch.isfinite(LSE[:, g:]).all()                                                       # past-access head


@pytest.mark.parametrize("B,L,Hq,Hkv,d,starts,T,mask,X", [
    (1, 1024, 4, 2, 128, [0, 200, 456, 457, 800], 100, [0, 1], 0),        # a one-token segment; tails longer than it
    (2, 700, 6, 3, 128, [0, 128, 256, 384, 512], 128, [2, 1, 0], 300),    # tile-aligned; a detached prefix
    (1, 900, 2, 2, 64, [0, 33, 66, 500], 300, [0, 0], 0),                 # T longer than the short segments
    (1, 640, 2, 1, 128, [0], 64, [0], 0),                                 # one open-ended segment: plain causal
    (1, 1500, 2, 2, 128, [0, 700, 1400], 256, [1, 2], 0),                 # long segments, several tiles each
])
@pytest.mark.parametrize("tail_sg", [False, True])
def test_segments_of_given_lengths(B, L, Hq, Hkv, d, starts, T, mask, X, tail_sg):
    # segments of lengths m_i instead of the constant S; the carried tail of a short segment is all of it
    Q, K, V, dO = rand_inputs(B, L, Hq, Hkv, d, seed=L + T)
    O, LSE = sa.seg_attn_fwd(Q, K, V, 1, T, mask, seg_starts=starts)
    dQ, dK, dV = sa.seg_attn_bwd(Q, K, V, O, LSE, dO, 1, T, mask, flagged_tail_is_sg=tail_sg, detach_before=X,
                                 seg_starts=starts)
    sa.poll_status()
    Oo, LSEo = oracle.fwd(f64(Q), f64(K), f64(V), 1, T, mask, seg_starts=starts)
    ref = oracle.bwd(f64(Q), f64(K), f64(V), f64(dO), 1, T, mask, flagged_tail_is_sg=tail_sg, detach_before=X,
                     seg_starts=starts)
    assert_fwd_close(O, LSE, Oo, LSEo, "fwd")
    assert_grads_close((dQ, dK, dV), ref, "bwd")


def test_equal_given_lengths_are_the_constant_length_path_to_the_bit():
    B, L, Hq, Hkv, d, S, T, mask = 1, 1000, 4, 2, 128, 256, 100, [0, 1]
    Q, K, V, dO = rand_inputs(B, L, Hq, Hkv, d, seed=11)
    starts = list(range(0, L, S))
    O, LSE = sa.seg_attn_fwd(Q, K, V, S, T, mask)
    O2, LSE2 = sa.seg_attn_fwd(Q, K, V, 1, T, mask, seg_starts=starts)
    assert torch.equal(O, O2) and torch.equal(LSE, LSE2)
    g1 = sa.seg_attn_bwd(Q, K, V, O, LSE, dO, S, T, mask)
    g2 = sa.seg_attn_bwd(Q, K, V, O, LSE, dO, 1, T, mask, seg_starts=starts)
    assert torch.equal(g1[0], g2[0])
    assert (g1[1].float() - g2[1].float()).abs().max() <= 2e-2     # the dK/dV pass walks its tiles in another order


def _random_case(rng):
    d = int(rng.choice([64, 128]))
    Hkv = int(rng.integers(1, 4))
    g = int(rng.choice([1, 2, 4]))
    S = int(rng.choice([int(rng.integers(1, 40)), int(rng.integers(40, 300)), 128, 256, int(rng.integers(300, 700))]))
    T = int(rng.integers(0, S + 1)) if rng.random() < 0.8 else int(rng.choice([0, S]))
    Lq = int(rng.integers(1, 900))
    q0 = int(rng.integers(0, 4 * S + 1)) if rng.random() < 0.5 else 0
    # keys from somewhere at or before the first query's tail (sometimes before position 0, sometimes too late)
    k0 = q0 - int(rng.integers(0, 2 * S + 50)) if rng.random() < 0.8 else q0 + int(rng.integers(1, 100))
    Lk = max(1, q0 + Lq - k0 - (int(rng.integers(0, 200)) if rng.random() < 0.3 else 0))
    mask = [int(rng.integers(0, 3)) for _ in range(Hkv)]
    X = int(rng.integers(0, q0 + Lq + 1)) if rng.random() < 0.4 else 0
    starts = None
    if rng.random() < 0.35:   # segments of given lengths instead of the constant S
        cuts = np.unique(rng.integers(1, q0 + Lq + 1, size=int(rng.integers(0, 7))))
        starts = [0] + [int(c) for c in cuts]
    return dict(B=int(rng.integers(1, 3)), Lq=Lq, Lk=Lk, Hq=Hkv * g, Hkv=Hkv, d=d, S=S, T=T, q0=q0, k0=k0, mask=mask,
                X=X, tail_sg=bool(rng.random() < 0.3), starts=starts)


@pytest.mark.parametrize("seed", range(int(os.environ.get("SEGATTN_FUZZ_SEEDS", "64"))))   # more seeds for a soak run
def test_random_shapes_offsets_classes_and_boundaries(seed):
    # seeded random problems over everything the interface takes at once: ragged sizes, position offsets on
    # both sides (keys starting before position 0 or after the first query), head classes, the paper-literal
    # flag, a detached prefix and segments of given lengths
    c = _random_case(np.random.default_rng(1000 + seed))
    Q, K, V, dO = rand_inputs(c["B"], c["Lq"], c["Hq"], c["Hkv"], c["d"], seed=seed, Lk=c["Lk"])
    kw = dict(q_pos0=c["q0"], kv_pos0=c["k0"], seg_starts=c["starts"])
    O, LSE = sa.seg_attn_fwd(Q, K, V, c["S"], c["T"], c["mask"], **kw)
    dQ, dK, dV = sa.seg_attn_bwd(Q, K, V, O, LSE, dO, c["S"], c["T"], c["mask"], flagged_tail_is_sg=c["tail_sg"],
                                 detach_before=c["X"], **kw)
    sa.poll_status()
    Oo, LSEo = oracle.fwd(f64(Q), f64(K), f64(V), c["S"], c["T"], c["mask"], **kw)
    ref = oracle.bwd(f64(Q), f64(K), f64(V), f64(dO), c["S"], c["T"], c["mask"], flagged_tail_is_sg=c["tail_sg"],
                     detach_before=c["X"], **kw)
    assert_fwd_close(O, LSE, Oo, LSEo, "fwd %r" % c)
    assert_grads_close((dQ, dK, dV), ref, "bwd %r" % c)


def test_limits_of_the_interface():
    # 64 KV heads (the most the head table holds), all three classes, one query head each
    Hkv = 64
    mask = [(c * 7) % 3 for c in range(Hkv)]
    Q, K, V, dO = rand_inputs(1, 300, Hkv, Hkv, 64, seed=64)
    O, LSE = sa.seg_attn_fwd(Q, K, V, 100, 40, mask)
    dQ, dK, dV = sa.seg_attn_bwd(Q, K, V, O, LSE, dO, 100, 40, mask)
    sa.poll_status()
    Oo, LSEo = oracle.fwd(f64(Q), f64(K), f64(V), 100, 40, mask)
    ref = oracle.bwd(f64(Q), f64(K), f64(V), f64(dO), 100, 40, mask)
    assert_fwd_close(O, LSE, Oo, LSEo, "64 KV heads")
    assert_grads_close((dQ, dK, dV), ref, "64 KV heads")
    with pytest.raises(sa.SegAttnError):
        sa.seg_attn_fwd(*rand_inputs(1, 128, 65, 65, 64, seed=1)[:3], 64, 0, [0] * 65)
    # positions near the top of the supported range (q_pos0 + Lq <= 2^30 - 1): the segment arithmetic
    # must not wrap; keys start one tail before the window
    S, T, L = 4096, 512, 512
    q0 = (1 << 30) - 1 - L
    q0 -= q0 % 128
    k0 = q0 - (q0 % S) - T          # from the tail of the previous segment on
    Lk = q0 + L - k0
    Q, K, V, dO = rand_inputs(1, L, 2, 2, 128, seed=30, Lk=Lk)
    mask = [0, 2]
    O, LSE = sa.seg_attn_fwd(Q, K, V, S, T, mask, q_pos0=q0, kv_pos0=k0)
    dQ, dK, dV = sa.seg_attn_bwd(Q, K, V, O, LSE, dO, S, T, mask, q_pos0=q0, kv_pos0=k0)
    sa.poll_status()
    Oo, LSEo = oracle.fwd(f64(Q), f64(K), f64(V), S, T, mask, q_pos0=q0, kv_pos0=k0)
    ref = oracle.bwd(f64(Q), f64(K), f64(V), f64(dO), S, T, mask, q_pos0=q0, kv_pos0=k0)
    assert_fwd_close(O, LSE, Oo, LSEo, "high positions")
    assert_grads_close((dQ, dK, dV), ref, "high positions")
    with pytest.raises(sa.SegAttnError):
        sa.seg_attn_fwd(Q, K, V, S, T, mask, q_pos0=(1 << 30), kv_pos0=k0)


def test_invalid_arguments_are_rejected_before_launch():
    Q, K, V, dO = rand_inputs(1, 128, 2, 1, 128)
    with pytest.raises(sa.SegAttnError) as e:
        sa.seg_attn_fwd(Q, K, V, 64, 65, [0])                      # T > S
    assert e.value.status == 1
    with pytest.raises(sa.SegAttnError):
        sa.seg_attn_fwd(Q[..., :96].contiguous(), K[..., :96].contiguous(), V[..., :96].contiguous(), 64, 0, [0])
    O, LSE = sa.seg_attn_fwd(Q, K, V, 64, 16, [0])
    with pytest.raises(sa.SegAttnError) as e:
        sa.seg_attn_bwd(Q, K, V, O, LSE, dO, 64, 16, [0], workspace=torch.empty(256, dtype=torch.uint8, device="cuda"))
    assert e.value.status == 5                                      # workspace too small


def _check_window(w, ref, b, c, hq, O, LSE, grads, what):
    rows = ref["rows"]
    assert_fwd_close(O[b:b + 1, rows, hq], LSE[b:b + 1, hq, rows], ref["O"], ref["LSE"], what)
    if grads is not None:
        dQ, dK, dV = grads
        keys = ref["keys"]
        assert_grads_close((dQ[b:b + 1, rows, hq], dK[b:b + 1, keys, c:c + 1], dV[b:b + 1, keys, c:c + 1]),
                           (ref["dQ"], ref["dK"], ref["dV"]), what)


def _full_size_check(w, late_rows=24, windows=((1, 2),), last_rows=0):
    """The benchmark's launch configuration at full size against the oracle on sub-problems it can compute: per
    KV group (one past-access, one not) the windows of whole segments listed in `windows` as (first segment,
    number of segments; negative = counted from the end; a pair of pairs = (past-access group, other group)),
    the last `last_rows` rows with the last key tiles, and rows sampled from the last segment."""
    x = workloads.make_inputs(w, device="cuda")
    O, LSE = sa.seg_attn_fwd(x["Q"], x["K"], x["V"], w.S, w.T, x["mask"], w.sm_scale)
    grads = None
    if w.backward:
        grads = sa.seg_attn_bwd(x["Q"], x["K"], x["V"], O, LSE, x["dO"], w.S, w.T, x["mask"], w.sm_scale)
    sa.poll_status()
    g = w.Hq // w.Hkv
    b = w.B - 1
    n_seg_total = (w.L + w.S - 1) // w.S
    rng = np.random.default_rng(w.seed + 1)
    for c, hq in group_slices(x["mask"], g):
        for win in windows:
            if isinstance(win[0], tuple):
                win = win[0] if int(x["mask"][c]) == 1 else win[1]
            seg_lo, n_seg = win
            if seg_lo < 0:
                seg_lo += n_seg_total
            ref = oracle_window(x, w, b, c, hq, seg_lo, n_seg)
            _check_window(w, ref, b, c, hq, O, LSE, grads, "%s segments %d..%d kv%d" % (w.name, seg_lo, seg_lo + n_seg - 1, c))
        if last_rows:
            ref = oracle_last_rows(x, w, b, c, hq, last_rows)
            _check_window(w, ref, b, c, hq, O, LSE, grads, "%s last %d rows kv%d" % (w.name, last_rows, c))
        # rows sampled from the last segment, where a flagged head's visible range is longest
        last0 = (w.L - 1) // w.S * w.S
        ps = sorted(set(int(p) for p in rng.integers(last0, w.L, size=late_rows)) | {w.L - 1, last0})
        num = den = 0.0
        for p, Oo, LSEo, dQo in oracle_rows(x, w, b, c, hq, ps):
            assert_fwd_close(O[b:b + 1, p:p + 1, hq], LSE[b:b + 1, hq, p:p + 1], Oo, LSEo, "%s row %d" % (w.name, p))
            if dQo is not None:
                num += float(((f64(grads[0][b:b + 1, p:p + 1, hq]) - dQo) ** 2).sum())
                den += float((dQo ** 2).sum())
        if grads is not None:
            assert (num / den) ** 0.5 <= TOL_GRAD, "%s late rows dQ" % w.name


def test_configuration_2_full_size_sampled():
    # an early window and the last two segments (every key of which has all its readers inside the window)
    _full_size_check(workloads.CONFIGS[1], windows=((1, 2), (-2, 2)))


def test_configuration_3_full_size_sampled_with_outlier_keys():
    # late window: the last two segments for the local group, the last segment for the past-access group
    # (its rows read 32K keys each)
    _full_size_check(workloads.CONFIGS[2], late_rows=12, windows=((1, 2), ((-1, 1), (-2, 2))))


@pytest.mark.parametrize("S,T,frac", [(1024, 256, 0.25), (4096, 4096, 0.0), (16384, 1024, 1.0)])
def test_configuration_5_sweep_points_sampled(S, T, frac):
    w = workloads.CONFIGS[4].with_(S=S, T=T, past_frac=frac, name="cfg5_S%d_T%d_f%g" % (S, T, frac))
    # (one segment of 16384 rows is as much as the oracle does in about a minute)
    _full_size_check(w, late_rows=6, windows=((1, 2) if S <= 4096 else (0, 1),))


@pytest.mark.parametrize("w", workloads.sweep(), ids=lambda w: w.name)
def test_configuration_5_every_sweep_point(w):
    # all 24 points: the last 136 rows of the sequence (the last key tile and a ragged piece of the one before,
    # with complete dK/dV) and sampled rows of the last segment
    _full_size_check(w, late_rows=4, windows=(), last_rows=136)


def test_host_buffer_step_matches_device_path():
    w = workloads.CONFIGS[0]
    x = workloads.make_inputs(w)
    outs = sa.seg_attn_step_host(x["Q"], x["K"], x["V"], x["dO"], w.S, w.T, x["mask"], w.sm_scale)
    Q, K, V, dO = (x[k].cuda() for k in ("Q", "K", "V", "dO"))
    O, LSE = sa.seg_attn_fwd(Q, K, V, w.S, w.T, x["mask"], w.sm_scale)
    dQ, dK, dV = sa.seg_attn_bwd(Q, K, V, O, LSE, dO, w.S, w.T, x["mask"], w.sm_scale)
    for k, t in (("O", O), ("LSE", LSE), ("dQ", dQ), ("dK", dK), ("dV", dV)):
        assert torch.equal(outs[k], t.cpu()), k


@pytest.mark.parametrize("B", [2, 6])
def test_host_buffer_step_in_overlapped_chunks(B):
    # the host-buffer step cuts the batch into chunks (here of unequal size for B = 6) whose copies and
    # kernels overlap on separate streams: the results are those of one launch over the whole batch
    L, Hq, Hkv, d, S, T, mask = 640, 4, 2, 128, 256, 128, [1, 0]
    Q, K, V, dO = rand_inputs(B, L, Hq, Hkv, d, seed=B, device="cpu")
    for forward_only in (False, True):
        outs = sa.seg_attn_step_host(Q, K, V, None if forward_only else dO, S, T, mask)
        Qd, Kd, Vd, dOd = (t.cuda() for t in (Q, K, V, dO))
        O, LSE = sa.seg_attn_fwd(Qd, Kd, Vd, S, T, mask)
        assert torch.equal(outs["O"], O.cpu()) and torch.equal(outs["LSE"], LSE.cpu())
        if not forward_only:
            dQ, dK, dV = sa.seg_attn_bwd(Qd, Kd, Vd, O, LSE, dOd, S, T, mask)
            for k, t in (("dQ", dQ), ("dK", dK), ("dV", dV)):
                assert torch.equal(outs[k], t.cpu()), k


@pytest.mark.parametrize("B,Hq,Hkv,mask", [
    (1, 8, 8, [0, 1, 2, 0, 1, 0, 0, 1]),     # eight chunks of one KV head each
    (2, 6, 3, [1, 0, 2]),                    # three head ranges per batch element
    (1, 10, 5, [0, 0, 1, 0, 2]),             # five ranges of one head, two query heads each
    (3, 4, 2, [0, 1]),                       # 3 x 2 chunks
])
def test_host_buffer_step_in_chunks_of_kv_heads(B, Hq, Hkv, mask):
    # a batch smaller than the number of chunks is cut along the KV heads: every (batch element, KV head) is an
    # independent problem, so the results are those of one launch over everything, bit for bit
    L, d, S, T = 512, 128, 256, 128
    Q, K, V, dO = rand_inputs(B, L, Hq, Hkv, d, seed=B + Hkv, device="cpu")
    outs = sa.seg_attn_step_host(Q, K, V, dO, S, T, mask)
    Qd, Kd, Vd, dOd = (t.cuda() for t in (Q, K, V, dO))
    O, LSE = sa.seg_attn_fwd(Qd, Kd, Vd, S, T, mask)
    dQ, dK, dV = sa.seg_attn_bwd(Qd, Kd, Vd, O, LSE, dOd, S, T, mask)
    for k, t in (("O", O), ("LSE", LSE), ("dQ", dQ), ("dK", dK), ("dV", dV)):
        assert torch.equal(outs[k], t.cpu()), k


def test_a_training_step_captured_in_a_cuda_graph_replays_on_new_data():
    # nothing in the entry points synchronises, allocates or depends on host state at run time, so a
    # forward + backward can be captured once and replayed (the launch-bound small shapes gain from it)
    B, L, Hq, Hkv, d, S, T, mask = 1, 512, 4, 2, 128, 128, 64, [0, 1]
    Q, K, V, dO = rand_inputs(B, L, Hq, Hkv, d, seed=21)
    O = torch.empty_like(Q)
    LSE = torch.empty(B, Hq, L, dtype=torch.float32, device="cuda")
    ws = torch.empty(max(256, B * Hq * L * 4 + 256), dtype=torch.uint8, device="cuda")
    sa.seg_attn_fwd(Q, K, V, S, T, mask, out=O, lse=LSE)          # warm-up outside the capture (function attributes)
    sa.seg_attn_bwd(Q, K, V, O, LSE, dO, S, T, mask, workspace=ws)
    torch.cuda.synchronize()
    stream = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(stream):
        with torch.cuda.graph(graph, stream=stream):
            sa.seg_attn_fwd(Q, K, V, S, T, mask, out=O, lse=LSE, stream=stream)
            grads = sa.seg_attn_bwd(Q, K, V, O, LSE, dO, S, T, mask, workspace=ws, stream=stream)
    for seed in (22, 23):
        Q2, K2, V2, dO2 = rand_inputs(B, L, Hq, Hkv, d, seed=seed)
        for dst, src in ((Q, Q2), (K, K2), (V, V2), (dO, dO2)):
            dst.copy_(src)
        graph.replay()
        torch.cuda.synchronize()
        sa.poll_status()
        O_e, LSE_e = sa.seg_attn_fwd(Q2, K2, V2, S, T, mask)
        g_e = sa.seg_attn_bwd(Q2, K2, V2, O_e, LSE_e, dO2, S, T, mask)
        assert torch.equal(O, O_e) and torch.equal(LSE, LSE_e)
        for a, b in zip(grads, g_e):
            assert torch.equal(a, b)


def test_a_bounded_wait_that_runs_out_is_reported_and_the_context_survives():
    # a wait on a barrier nothing signals gives up after its limit and sets the status word: no hang, no fault
    sa.poll_status()
    sa.selftest_wait_timeout()
    with pytest.raises(sa.SegAttnError) as e:
        sa.poll_status()
    assert e.value.status == 4
    assert sa.lib().seg_attn_last_cuda_error() == (4 << 8) | 99
    sa.poll_status()   # the word was cleared
    Q, K, V, dO = rand_inputs(1, 256, 2, 1, 128, seed=2)
    O, LSE = sa.seg_attn_fwd(Q, K, V, 128, 64, [0])
    Oo, LSEo = oracle.fwd(f64(Q), f64(K), f64(V), 128, 64, [0])
    assert_fwd_close(O, LSE, Oo, LSEo, "after a timeout")


def test_launch_log_on_request():
    # SEGATTN_LOG=1: one line per launch on stderr with the shapes and the size of the schedule
    import subprocess
    import sys
    code = ("import torch, paper_2605_11744_b200 as sa\n"
            "mk = lambda H: torch.zeros(1, 256, H, 128, dtype=torch.bfloat16, device='cuda')\n"
            "Q, K, V = mk(2), mk(1), mk(1)\n"
            "O, LSE = sa.seg_attn_fwd(Q, K, V, 128, 64, [1])\n"
            "sa.seg_attn_bwd(Q, K, V, O, LSE, Q, 128, 64, [1])\n"
            "sa.poll_status()\n")
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    r = subprocess.run([sys.executable, "-c", code], env=dict(os.environ, SEGATTN_LOG="1", PYTHONPATH=root), capture_output=True,
                       text=True, timeout=300)
    assert r.returncode == 0, r.stderr
    assert "[segattn] fwd: B=1 Lq=256 kv_len=256 Hq=2 Hkv=1 d=128 S=128 T=64" in r.stderr and "items=4 grid=4" in r.stderr
    assert "[segattn] bwd dQ pass:" in r.stderr and "[segattn] bwd dK/dV pass: key tiles=2" in r.stderr
    quiet = subprocess.run([sys.executable, "-c", code], env=dict(os.environ, PYTHONPATH=root, SEGATTN_LOG="0"),
                           capture_output=True, text=True, timeout=300)
    assert quiet.returncode == 0 and "[segattn]" not in quiet.stderr

"""Streamed prefill on the GPU: equals the one-shot forward (the forward identity between
segment-by-segment and whole-sequence execution) and the oracle."""
import numpy as np
import pytest
import torch

import oracle
import workloads
import paper_2605_11744_b200 as sa
from util import assert_fwd_close, f64, group_slices, oracle_rows, rand_inputs

pytestmark = pytest.mark.gpu


def run_streamed(Q, K, V, S, T, mask, scale=None):
    B, L, Hq, d = Q.shape
    Hkv = K.shape[2]
    pf = sa.Prefill(B, S, T, Hq, Hkv, d, L, mask, scale)
    O = torch.empty_like(Q)
    LSE = torch.empty(B, Hq, L, dtype=torch.float32, device=Q.device)
    for i in range(L // S):
        sl = slice(i * S, (i + 1) * S)
        o, l = pf.step(Q[:, sl].contiguous(), K[:, sl].contiguous(), V[:, sl].contiguous())
        O[:, sl] = o
        LSE[:, :, sl] = l
    sa.poll_status()
    state = pf.state_bytes
    pf.close()
    return O, LSE, state


@pytest.mark.parametrize("B,L,Hq,Hkv,d,S,T,mask", [
    (1, 1024, 4, 2, 128, 256, 128, [0, 1]),
    (2, 768, 4, 4, 128, 256, 0, [1, 0, 0, 1]),
    (1, 800, 2, 2, 64, 200, 72, [0, 1]),        # tiles of the window do not line up with the one-shot tiles
    (1, 512, 2, 2, 128, 128, 128, [0, 0]),
    (1, 512, 2, 1, 128, 128, 64, [1]),
    (1, 1024, 4, 4, 128, 256, 128, [2, 1, 0, 2]),   # all three head classes; own-only heads ignore the window's tail
])
def test_streamed_equals_one_shot_and_oracle(B, L, Hq, Hkv, d, S, T, mask):
    Q, K, V, _ = rand_inputs(B, L, Hq, Hkv, d, seed=L + T)
    O1, LSE1 = sa.seg_attn_fwd(Q, K, V, S, T, mask)
    O2, LSE2, _ = run_streamed(Q, K, V, S, T, mask)
    Oo, LSEo = oracle.fwd(f64(Q), f64(K), f64(V), S, T, mask)
    assert_fwd_close(O2, LSE2, Oo, LSEo, "streamed")
    if S % 128 == 0 and T % 128 == 0:
        # same tiles in the same order: the two paths agree to the bit
        assert torch.equal(O1, O2) and torch.equal(LSE1, LSE2)
    else:
        assert (O1.float() - O2.float()).abs().max() <= 2e-2


def test_reset_and_reuse():
    Q, K, V, _ = rand_inputs(1, 512, 2, 2, 128, seed=1)
    pf = sa.Prefill(1, 128, 128, 2, 2, 128, 512, [0, 1])
    outs = []
    for rep in range(2):
        o = [pf.step(Q[:, i * 128:(i + 1) * 128].contiguous(), K[:, i * 128:(i + 1) * 128].contiguous(),
                     V[:, i * 128:(i + 1) * 128].contiguous())[0] for i in range(4)]
        outs.append(torch.cat(o, dim=1))
        with pytest.raises(sa.SegAttnError):
            pf.step(Q[:, :128].contiguous(), K[:, :128].contiguous(), V[:, :128].contiguous())   # pool is full
        pf.reset()
    assert torch.equal(outs[0], outs[1])
    pf.close()


def test_configuration_4_streamed_at_full_size_sampled():
    w = workloads.CONFIGS[3]
    x = workloads.make_inputs(w, device="cuda")
    torch.cuda.synchronize()
    O, LSE, state = run_streamed(x["Q"], x["K"], x["V"], w.S, w.T, x["mask"], w.sm_scale)
    # persistent state: the flagged heads' whole history plus the other heads' tail + segment window
    nf = int(x["mask"].sum())
    expect = 2 * w.B * nf * w.L * w.d * 2 + 2 * w.B * (w.Hkv - nf) * (w.S + w.T) * w.d * 2
    assert state == expect
    O1, LSE1 = sa.seg_attn_fwd(x["Q"], x["K"], x["V"], w.S, w.T, x["mask"], w.sm_scale)
    assert torch.equal(O, O1) and torch.equal(LSE, LSE1)
    g = w.Hq // w.Hkv
    rng = np.random.default_rng(4)
    for c, hq in group_slices(x["mask"], g):
        ps = sorted(set(int(p) for p in rng.integers(0, w.L, size=10)) | {0, w.S - 1, w.S, w.L - 1})
        for p, Oo, LSEo, _ in oracle_rows(x, w, 0, c, hq, ps):
            assert_fwd_close(O[:, p:p + 1, hq], LSE[:, hq, p:p + 1], Oo, LSEo, "cfg4 row %d kv%d" % (p, c))


@pytest.mark.parametrize("B,L,Hq,Hkv,d,S,T,mask", [
    (1, 1024, 4, 2, 128, 256, 128, [0, 1]),
    (2, 768, 4, 4, 128, 256, 0, [1, 0, 0, 1]),
    (1, 800, 2, 2, 64, 200, 72, [0, 1]),
    (1, 1024, 6, 3, 128, 256, 256, [2, 1, 0]),     # all head classes, tail = whole previous segment
    (1, 512, 2, 1, 128, 128, 64, [1]),             # past-access heads only
])
def test_streamed_backward_sums_to_the_one_shot_backward(B, L, Hq, Hkv, d, S, T, mask):
    # segment by segment: forward, then the backward of that segment's loss term; the key/value gradients of
    # [previous tail ; segment] added up over the segments are those of the whole-sequence backward (one
    # attention layer has no longer state chain than one transition), and every term matches the oracle
    from util import assert_grads_close
    Q, K, V, dO = rand_inputs(B, L, Hq, Hkv, d, seed=L + S)
    pf = sa.Prefill(B, S, T, Hq, Hkv, d, L, mask)
    dQ = torch.empty_like(Q)
    dK = torch.zeros(B, L, Hkv, d, dtype=torch.float32, device="cuda")
    dV = torch.zeros_like(dK)
    Qf, Kf, Vf, dOf = f64(Q), f64(K), f64(V), f64(dO)
    for i in range(L // S):
        sl = slice(i * S, (i + 1) * S)
        q, do = Q[:, sl].contiguous(), dO[:, sl].contiguous()
        o, lse = pf.step(q, K[:, sl].contiguous(), V[:, sl].contiguous())
        gq, gk, gv = pf.step_bwd(q, o, lse, do)
        sa.poll_status()
        dQ[:, sl] = gq
        lo = i * S - T
        cut = max(0, -lo)
        assert not gk[:, :cut].any() and not gv[:, :cut].any()
        dK[:, lo + cut:(i + 1) * S] += gk[:, cut:].float()
        dV[:, lo + cut:(i + 1) * S] += gv[:, cut:].float()
        if i in (0, 1, L // S - 1):
            # this segment's term against the oracle: the loss of segment i alone, whole sequence up to its end
            hi = (i + 1) * S
            dOw = np.zeros_like(dOf[:, :hi])
            dOw[:, sl] = dOf[:, sl]
            rq, rk, rv = oracle.bwd(Qf[:, :hi], Kf[:, :hi], Vf[:, :hi], dOw, S, T, mask)
            assert not rk[:, :lo + cut].any()          # nothing older than the tail receives gradient
            assert_grads_close((gq, gk[:, cut:], gv[:, cut:]), (rq[:, sl], rk[:, lo + cut:], rv[:, lo + cut:]), "segment %d" % i)
    pf.close()
    O1, LSE1 = sa.seg_attn_fwd(Q, K, V, S, T, mask)
    ref = oracle.bwd(Qf, Kf, Vf, dOf, S, T, mask)
    assert_grads_close((dQ, dK, dV), ref, "sum over segments")


def test_streamed_backward_needs_a_stepped_segment_and_a_workspace():
    pf = sa.Prefill(1, 128, 64, 2, 1, 128, 256, [0])
    q = torch.zeros(1, 128, 2, 128, dtype=torch.bfloat16, device="cuda")
    lse = torch.zeros(1, 2, 128, dtype=torch.float32, device="cuda")
    with pytest.raises(sa.SegAttnError):
        pf.step_bwd(q, q, lse, q)            # nothing stepped yet
    k = torch.zeros(1, 128, 1, 128, dtype=torch.bfloat16, device="cuda")
    o, lse = pf.step(q, k, k)
    pf._bwd_ws = torch.empty(256, dtype=torch.uint8, device="cuda")   # too small and kept: the call must refuse it
    need = int(sa.lib().seg_prefill_bwd_workspace_bytes(pf._h))
    assert need > 256
    import ctypes
    st = sa.lib().seg_prefill_step_bwd(pf._h, q.data_ptr(), o.data_ptr(), lse.data_ptr(), q.data_ptr(), q.data_ptr(),
                                       k.data_ptr(), k.data_ptr(), ctypes.c_void_p(pf._bwd_ws.data_ptr()), 256, None)
    assert st == 5
    pf._bwd_ws = None
    dq, dk, dv = pf.step_bwd(q, o, lse, q)   # zero cotangent: zero gradients
    sa.poll_status()
    assert not dq.any() and not dk.any() and not dv.any() and dk.shape == (1, 192, 1, 128)
    pf.close()


@pytest.mark.parametrize("seed", range(12))
def test_streamed_forward_and_backward_on_random_problems(seed):
    # seeded random segment lengths, tails, head classes and group sizes through the streamed driver:
    # forward against the oracle, per-segment backward summed against the whole-sequence oracle backward
    from util import assert_grads_close
    rng = np.random.default_rng(500 + seed)
    d = int(rng.choice([64, 128]))
    Hkv = int(rng.integers(1, 4))
    g = int(rng.choice([1, 2]))
    S = int(rng.choice([int(rng.integers(1, 60)), 128, int(rng.integers(60, 300))]))
    T = int(rng.integers(0, S + 1))
    n_seg = int(rng.integers(1, 5))
    B, L, Hq = int(rng.integers(1, 3)), S * n_seg, Hkv * g
    mask = [int(rng.integers(0, 3)) for _ in range(Hkv)]
    Q, K, V, dO = rand_inputs(B, L, Hq, Hkv, d, seed=seed)
    pf = sa.Prefill(B, S, T, Hq, Hkv, d, L, mask)
    O = torch.empty_like(Q)
    LSE = torch.empty(B, Hq, L, dtype=torch.float32, device="cuda")
    dQ = torch.empty_like(Q)
    dK = torch.zeros(B, L, Hkv, d, dtype=torch.float32, device="cuda")
    dV = torch.zeros_like(dK)
    for i in range(n_seg):
        sl = slice(i * S, (i + 1) * S)
        q, do = Q[:, sl].contiguous(), dO[:, sl].contiguous()
        o, lse = pf.step(q, K[:, sl].contiguous(), V[:, sl].contiguous())
        gq, gk, gv = pf.step_bwd(q, o, lse, do)
        O[:, sl], LSE[:, :, sl], dQ[:, sl] = o, lse, gq
        lo = i * S - T
        cut = max(0, -lo)
        dK[:, lo + cut:(i + 1) * S] += gk[:, cut:].float()
        dV[:, lo + cut:(i + 1) * S] += gv[:, cut:].float()
    sa.poll_status()
    pf.close()
    what = "S=%d T=%d n=%d mask=%r d=%d g=%d" % (S, T, n_seg, mask, d, g)
    Oo, LSEo = oracle.fwd(f64(Q), f64(K), f64(V), S, T, mask)
    assert_fwd_close(O, LSE, Oo, LSEo, what)
    assert_grads_close((dQ, dK, dV), oracle.bwd(f64(Q), f64(K), f64(V), f64(dO), S, T, mask), what)


def run_streamed_lengths(Q, K, V, S, T, mask, lengths):
    """Segments of the given lengths (each <= S) through the streamed driver."""
    B, L, Hq, d = Q.shape
    pf = sa.Prefill(B, S, T, Hq, K.shape[2], d, L, mask)
    O = torch.empty_like(Q)
    LSE = torch.empty(B, Hq, L, dtype=torch.float32, device=Q.device)
    bufs = [torch.empty(B, S, t.shape[2], d, dtype=torch.bfloat16, device="cuda") for t in (Q, K, V)]
    s0 = 0
    for m in lengths:
        views = []
        for buf, t in zip(bufs, (Q, K, V)):
            buf[:, :m] = t[:, s0:s0 + m]
            views.append(buf[:, :m])
        o, l = pf.step(*views)
        O[:, s0:s0 + m] = o
        LSE[:, :, s0:s0 + m] = l
        s0 += m
    assert s0 == L
    sa.poll_status()
    pf.close()
    return O, LSE


@pytest.mark.parametrize("B,Hq,Hkv,d,S,T,mask,lengths", [
    (1, 4, 2, 128, 256, 128, [0, 1], [256, 256, 256, 100]),            # a shorter last segment
    (2, 4, 2, 128, 256, 128, [0, 1], [256, 128, 256, 128, 256]),       # unequal lengths, everything on tile boundaries
    (1, 2, 2, 128, 300, 100, [0, 1], [300, 37, 1, 250, 300, 64]),      # nothing aligned; a one-token segment;
                                                                       # segments shorter than the tail
    (1, 6, 3, 64, 200, 200, [2, 1, 0], [64, 200, 150, 3, 199]),        # d = 64, all head classes, T = S
    (1, 2, 1, 128, 128, 0, [0], [128, 5, 128]),                        # no tail
])
def test_streamed_segments_of_unequal_lengths(B, Hq, Hkv, d, S, T, mask, lengths):
    # Section 3.1: segments of lengths m_i.  The streamed driver fed those lengths step by step gives the rows of the
    # whole-sequence forward over the same segment starts (and the oracle's).
    L = sum(lengths)
    starts = [0] + list(np.cumsum(lengths)[:-1])
    Q, K, V, _ = rand_inputs(B, L, Hq, Hkv, d, seed=L + S)
    O2, LSE2 = run_streamed_lengths(Q, K, V, S, T, mask, lengths)
    Oo, LSEo = oracle.fwd(f64(Q), f64(K), f64(V), 1, T, mask, seg_starts=starts)
    assert_fwd_close(O2, LSE2, Oo, LSEo, "streamed, unequal lengths")
    O1, LSE1 = sa.seg_attn_fwd(Q, K, V, 1, T, mask, seg_starts=starts)
    if all(m % 128 == 0 for m in lengths) and T % 128 == 0:
        assert torch.equal(O1, O2) and torch.equal(LSE1, LSE2)     # same tiles in the same order
    else:
        assert (O1.float() - O2.float()).abs().max() <= 2e-2


@pytest.mark.parametrize("B,Hq,Hkv,d,S,T,mask,lengths", [
    (1, 4, 2, 128, 256, 128, [0, 1], [256, 256, 100]),                 # a shorter last segment
    (2, 4, 2, 128, 256, 128, [0, 1], [256, 128, 256, 128]),            # unequal lengths on tile boundaries, two batch elements
    (1, 2, 2, 128, 300, 100, [0, 1], [300, 37, 1, 250, 64]),           # nothing aligned; segments shorter than the tail
    (1, 6, 3, 64, 200, 200, [2, 1, 0], [64, 200, 150, 3]),             # d = 64, all head classes, T = S
])
def test_streamed_backward_over_segments_of_unequal_lengths(B, Hq, Hkv, d, S, T, mask, lengths):
    # The backward of each streamed step, for segments of lengths m_i: every term against the oracle (loss of that
    # segment alone over the same segment starts), and the terms added up against the whole-sequence backward.
    from util import assert_grads_close
    L = sum(lengths)
    starts = [0] + [int(v) for v in np.cumsum(lengths)[:-1]]
    Q, K, V, dO = rand_inputs(B, L, Hq, Hkv, d, seed=L + S + 7)
    Qf, Kf, Vf, dOf = f64(Q), f64(K), f64(V), f64(dO)
    pf = sa.Prefill(B, S, T, Hq, Hkv, d, L, mask)
    dQ = torch.empty_like(Q)
    dK = torch.zeros(B, L, Hkv, d, dtype=torch.float32, device="cuda")
    dV = torch.zeros_like(dK)
    bufs = [torch.empty(B, S, t.shape[2], d, dtype=torch.bfloat16, device="cuda") for t in (Q, K, V, dO)]
    s0 = 0
    for i, m in enumerate(lengths):
        views = []
        for buf, t in zip(bufs, (Q, K, V, dO)):
            buf[:, :m] = t[:, s0:s0 + m]
            views.append(buf[:, :m])
        q, k, v, do = views
        o, lse = pf.step(q, k, v)
        gq, gk, gv = pf.step_bwd(q, o, lse, do)
        sa.poll_status()
        assert gq.shape == (B, m, Hq, d) and gk.shape == (B, T + S, Hkv, d)
        dQ[:, s0:s0 + m] = gq
        lo = s0 - T                      # global position of row 0 of gk / gv
        cut = max(0, -lo)
        assert not gk[:, :cut].any() and not gv[:, :cut].any()            # rows before position 0
        assert not gk[:, T + m:].any() and not gv[:, T + m:].any()        # rows after a shorter segment
        dK[:, lo + cut:s0 + m] += gk[:, cut:T + m].float()
        dV[:, lo + cut:s0 + m] += gv[:, cut:T + m].float()
        # this segment's term against the oracle: the loss of segment i alone, sequence up to its end
        hi = s0 + m
        dOw = np.zeros_like(dOf[:, :hi])
        dOw[:, s0:hi] = dOf[:, s0:hi]
        rq, rk, rv = oracle.bwd(Qf[:, :hi], Kf[:, :hi], Vf[:, :hi], dOw, 1, T, mask, seg_starts=starts[:i + 1])
        assert not rk[:, :lo + cut].any()          # nothing in front of the T rows before the segment receives gradient
        assert_grads_close((gq, gk[:, cut:T + m], gv[:, cut:T + m]), (rq[:, s0:hi], rk[:, lo + cut:], rv[:, lo + cut:]),
                           "segment %d" % i)
        s0 += m
    pf.close()
    ref = oracle.bwd(Qf, Kf, Vf, dOf, 1, T, mask, seg_starts=starts)
    assert_grads_close((dQ, dK, dV), ref, "sum over segments of unequal lengths")


def test_streamed_driver_refuses_oversized_segments():
    B, Hq, Hkv, d, S, T = 1, 2, 1, 128, 128, 64
    Q, K, V, dO = rand_inputs(B, 256, Hq, Hkv, d, seed=4)
    pf = sa.Prefill(B, S, T, Hq, Hkv, d, 256, [0])
    o, l = pf.step(Q[:, :100], K[:, :100], V[:, :100])
    with pytest.raises(ValueError):
        pf.step(Q[:, :200], K[:, :200], V[:, :200])     # longer than S
    h = pf._h
    assert sa.lib().seg_prefill_step_len(h, 0, 4096, 4096, 4096, 4096, 4096, None) == 1
    assert sa.lib().seg_prefill_step_len(h, S + 1, 4096, 4096, 4096, 4096, 4096, None) == 1
    pf.close()

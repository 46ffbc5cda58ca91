"""Attention over a retrieved prefix on the GPU: the gather is exact, and the existing forward and
backward on the gathered context match the oracle's [K_ret ; K_i] attention."""
import numpy as np
import pytest
import torch

from oracle import dense
from oracle import retrieval
import paper_2605_11744_b200 as sa
from util import assert_fwd_close, assert_grads_close, f64

pytestmark = pytest.mark.gpu


def bits(t):
    return t.contiguous().view(torch.int16).cpu().numpy()


def make(B, P, Hq, Hkv, d, R, Lseg, seed, pool_layout="blhd"):
    g = torch.Generator().manual_seed(seed)
    mk = lambda *s: torch.randn(*s, generator=g).bfloat16().cuda()
    if pool_layout == "blhd":
        Kp, Vp = mk(B, P, Hkv, d), mk(B, P, Hkv, d)
    else:  # the layout of a per-head pool, [B][Hkv][P][d], seen as [B, P, Hkv, d]
        Kp, Vp = mk(B, Hkv, P, d).permute(0, 2, 1, 3), mk(B, Hkv, P, d).permute(0, 2, 1, 3)
    idx = torch.randint(0, P, (B, Hkv, R), generator=g, dtype=torch.int32).cuda()
    return Kp, Vp, idx, mk(B, Lseg, Hkv, d), mk(B, Lseg, Hkv, d), mk(B, Lseg, Hq, d), mk(B, Lseg, Hq, d)


@pytest.mark.parametrize("B,P,Hq,Hkv,d,R,Lseg,layout", [
    (1, 2048, 4, 2, 128, 512, 512, "blhd"),     # R = 512 as in the paper's setting, several tiles
    (2, 1000, 4, 4, 128, 300, 200, "bhld"),     # nothing aligned to a tile; pool stored per head
    (1, 700, 2, 1, 64, 129, 77, "blhd"),        # d = 64, ragged
    (2, 64, 2, 2, 128, 0, 256, "blhd"),         # nothing retrieved: plain causal attention of the segment
    (1, 512, 2, 2, 128, 256, 1, "bhld"),        # a single query row
])
def test_retrieved_prefix_attention_matches_oracle(B, P, Hq, Hkv, d, R, Lseg, layout):
    Kp, Vp, idx, Ks, Vs, Q, dO = make(B, P, Hq, Hkv, d, R, Lseg, seed=P + R, pool_layout=layout)
    Kc, Vc = sa.gather_context(Kp, Vp, idx, Ks, Vs)
    sa.poll_status()
    # index work: bit-exact against the oracle's gather
    Kc_ref, Vc_ref = dense.retrieved_context(bits(Kp), bits(Vp), idx.cpu().numpy(), bits(Ks), bits(Vs))
    assert np.array_equal(bits(Kc), Kc_ref) and np.array_equal(bits(Vc), Vc_ref)
    # the attention is the library's forward / backward on the context: queries at positions R.., one
    # segment, and the retrieved rows detached
    S = max(1, R + Lseg)
    mask = [0] * Hkv
    O, LSE = sa.seg_attn_fwd(Q, Kc, Vc, S, 0, mask, q_pos0=R, kv_pos0=0)
    dQ, dK, dV = sa.seg_attn_bwd(Q, Kc, Vc, O, LSE, dO, S, 0, mask, q_pos0=R, kv_pos0=0, detach_before=R)
    sa.poll_status()
    Oo, LSEo, gq, gk, gv = dense.retrieved_attention(f64(Q), f64(Kp), f64(Vp), idx.cpu().numpy(), f64(Ks), f64(Vs), f64(dO))
    assert_fwd_close(O, LSE, Oo, LSEo, "retrieved prefix")
    assert_grads_close((dQ, dK[:, R:], dV[:, R:]), (gq, gk, gv), "retrieved prefix")
    assert not dK[:, :R].any() and not dV[:, :R].any()


def test_an_index_out_of_range_is_reported_and_not_read():
    Kp, Vp, idx, Ks, Vs, _, _ = make(1, 100, 2, 2, 128, 16, 8, seed=9)
    idx[0, 1, 3] = 100
    idx[0, 0, 5] = -1
    Kc, Vc = sa.gather_context(Kp, Vp, idx, Ks, Vs)
    with pytest.raises(sa.SegAttnError) as e:
        sa.poll_status()
    assert e.value.status == 1
    sa.poll_status()   # cleared
    assert not Kc[0, 3, 1].any() and not Vc[0, 5, 0].any()
    ok = idx.clone()
    ok[0, 1, 3] = 0
    ok[0, 0, 5] = 0
    Kc2, _ = sa.gather_context(Kp, Vp, ok, Ks, Vs)
    sa.poll_status()
    keep = torch.ones(16 + 8, 2, dtype=torch.bool)
    keep[3, 1] = keep[5, 0] = False
    assert torch.equal(Kc[0][keep.cuda()], Kc2[0][keep.cuda()])
    with pytest.raises(sa.SegAttnError):
        sa.gather_context(Kp[:, :, :, :100], Vp[:, :, :, :100], idx, Ks[:, :, :, :100], Vs[:, :, :, :100])   # d = 100


@pytest.mark.parametrize("B,P,Hq,Hkv,d,Lq,window,stride,tail,top_k,n_anchors,off_lo,off_hi,R,layout", [
    (1, 3000, 4, 2, 128, 48, 16, 8, 8, 16, 8, 32, 31, 512, "blhd"),    # R = 512, L_q = 48 as in the paper's range
    (2, 777, 4, 4, 128, 24, 8, 4, 4, 5, 3, 2, 2, 64, "bhld"),          # nothing aligned; pool stored per head
    (1, 300, 2, 1, 64, 5, 8, 4, 4, 3, 2, 0, 0, 7, "blhd"),             # fewer rows than a window; d = 64
    (1, 260, 2, 2, 128, 32, 8, 8, 32, 6, 6, 10, 10, 16, "blhd"),       # R smaller than the windows
    (1, 64, 2, 2, 128, 60, 4, 4, 4, 60, 4, 1, 1, 64, "blhd"),          # 16 summaries, R = P: everything is retrieved
])
def test_retrieval_selection_is_bit_exact(B, P, Hq, Hkv, d, Lq, window, stride, tail, top_k, n_anchors, off_lo, off_hi, R, layout):
    g = torch.Generator().manual_seed(P + R)
    mk = lambda *s: torch.randn(*s, generator=g).bfloat16().cuda()
    Q_last = mk(B, Lq, Hq, d)
    Kp = mk(B, P, Hkv, d) if layout == "blhd" else mk(B, Hkv, P, d).permute(0, 2, 1, 3)
    idx = sa.retrieval_select(Q_last, Kp, window, stride, tail, top_k, n_anchors, off_lo, off_hi, R)
    sa.poll_status()
    ref = retrieval.select(Q_last.float().cpu().numpy(), Kp.float().cpu().numpy(), window, stride, tail, top_k, n_anchors,
                           off_lo, off_hi, R)
    assert np.array_equal(idx.cpu().numpy(), ref)


def test_retrieve_gather_attend_end_to_end():
    # the long-range channel of one segment: select R positions from the pool, gather them, attend over
    # [retrieved ; own segment]; every stage against its oracle
    B, P, Hq, Hkv, d, S, R = 1, 2048, 4, 2, 128, 256, 512
    Kp, Vp, _, Ks, Vs, Q, dO = make(B, P, Hq, Hkv, d, 8, S, seed=77)
    Q_prev = torch.randn(B, 48, Hq, d, generator=torch.Generator().manual_seed(78)).bfloat16().cuda()
    idx = sa.retrieval_select(Q_prev, Kp, 16, 8, 8, 16, 8, 32, 31, R)
    ref_idx = retrieval.select(Q_prev.float().cpu().numpy(), Kp.float().cpu().numpy(), 16, 8, 8, 16, 8, 32, 31, R)
    assert np.array_equal(idx.cpu().numpy(), ref_idx)
    Kc, Vc = sa.gather_context(Kp, Vp, idx, Ks, Vs)
    O, LSE = sa.seg_attn_fwd(Q, Kc, Vc, R + S, 0, [0] * Hkv, q_pos0=R, kv_pos0=0)
    dQ, dK, dV = sa.seg_attn_bwd(Q, Kc, Vc, O, LSE, dO, R + S, 0, [0] * Hkv, q_pos0=R, kv_pos0=0, detach_before=R)
    sa.poll_status()
    Oo, LSEo, gq, gk, gv = dense.retrieved_attention(f64(Q), f64(Kp), f64(Vp), ref_idx, f64(Ks), f64(Vs), f64(dO))
    assert_fwd_close(O, LSE, Oo, LSEo, "end to end")
    assert_grads_close((dQ, dK[:, R:], dV[:, R:]), (gq, gk, gv), "end to end")


def test_retrieval_selection_rejects_what_it_cannot_hold():
    Q_last = torch.zeros(1, 8, 2, 128, dtype=torch.bfloat16, device="cuda")
    Kp = torch.zeros(1, 100, 1, 128, dtype=torch.bfloat16, device="cuda")
    for kw in (dict(R=101), dict(top_k=101), dict(top_k=0), dict(off_lo=-1), dict(stride=0)):
        a = dict(window=8, stride=4, tail=4, top_k=4, n_anchors=2, off_lo=1, off_hi=1, R=16)
        a.update(kw)
        with pytest.raises(sa.SegAttnError):
            sa.retrieval_select(Q_last, Kp, **a)
    many = torch.zeros(1, 40, 2, 128, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(sa.SegAttnError):       # 41 summaries
        sa.retrieval_select(many, Kp, 1, 1, 4, 4, 2, 1, 1, 16)


@pytest.mark.parametrize("seed", range(16))
def test_retrieval_selection_on_random_parameters(seed):
    rng = np.random.default_rng(900 + seed)
    d = int(rng.choice([64, 128]))
    Hkv = int(rng.integers(1, 4))
    Hq = Hkv * int(rng.choice([1, 2, 4]))
    P = int(rng.integers(20, 1500))
    Lq = int(rng.integers(1, 70))
    window = int(rng.integers(1, 20))
    stride = int(rng.integers(max(1, (Lq + 13) // 14), 24))       # at most 15 windows
    tail = int(rng.integers(1, 16))
    n_sum = retrieval.n_summaries(Lq, window, stride)
    top_k = int(rng.integers(1, min(P, 1024 // n_sum) + 1))
    R = int(rng.integers(1, min(P, 600) + 1))
    a = dict(window=window, stride=stride, tail=tail, top_k=top_k, n_anchors=int(rng.integers(1, 12)),
             off_lo=int(rng.integers(0, 40)), off_hi=int(rng.integers(0, 40)), R=R)
    g = torch.Generator().manual_seed(seed)
    # coarse values make equal scores likely: the tie rule is exercised too
    coarse = seed % 3 == 0
    mk = lambda *s: (torch.randint(-2, 3, s, generator=g).float() if coarse else torch.randn(*s, generator=g)).bfloat16().cuda()
    Q_last, Kp = mk(1, Lq, Hq, d), mk(1, P, Hkv, d)
    idx = sa.retrieval_select(Q_last, Kp, **a)
    sa.poll_status()
    ref = retrieval.select(Q_last.float().cpu().numpy(), Kp.float().cpu().numpy(), **a)
    assert np.array_equal(idx.cpu().numpy(), ref), a

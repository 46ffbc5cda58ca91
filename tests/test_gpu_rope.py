"""RoPE re-indexing on the GPU (Section 3.4, Appendix E) against the fp64 oracle: the table, the rotation
and its transpose, the gather that rotates retrieved keys by their slot, and the long-range channel of one
segment end to end (select, gather + rotate, attend, rotate the gradients back)."""
import numpy as np
import pytest
import torch

from oracle import dense
from oracle import retrieval
from oracle import rope
import paper_2605_11744_b200 as sa
from util import assert_fwd_close, assert_grads_close, f64

pytestmark = pytest.mark.gpu

BF16_HALF_ULP = 2.0 ** -8     # rounding to bf16 moves a value by at most 2^-9 of its magnitude; twice that is allowed


def close_to_rounded(got, want, slack):
    """got (bf16 from fp32 arithmetic) against want (fp64): one bf16 rounding plus fp32 round-off `slack`."""
    err = np.abs(f64(got) - want)
    assert (err <= BF16_HALF_ULP * np.abs(want) + slack).all(), float((err - BF16_HALF_ULP * np.abs(want)).max())


@pytest.mark.parametrize("d,n_pos,base", [(128, 4608, 10000.0), (64, 1000, 500000.0)])
def test_table_holds_the_cosines_and_sines_of_the_angles(d, n_pos, base):
    t = sa.rope_table(n_pos, d, base).cpu().numpy().astype(np.float64)
    a = rope.angles(np.arange(n_pos), d, base)
    assert np.abs(t[..., 0] - np.cos(a)).max() <= 1e-7 and np.abs(t[..., 1] - np.sin(a)).max() <= 1e-7
    assert (t[0, :, 0] == 1.0).all() and (t[0, :, 1] == 0.0).all()


@pytest.mark.parametrize("B,L,H,d,pos0", [(2, 300, 4, 128, 0), (1, 129, 3, 64, 512), (1, 77, 2, 128, 130000)])
def test_rotation_and_its_transpose(B, L, H, d, pos0):
    g = torch.Generator().manual_seed(L + pos0)
    # a strided view: heads padded, as a slice of a fused QKV projection would be
    big = torch.randn(B, L, H + 1, d, generator=g).bfloat16().cuda()
    X = big[:, :, :H]
    table = sa.rope_table(pos0 + L, d)
    Y = sa.rope_apply(X, table, pos0=pos0)
    sa.poll_status()
    want = rope.rotate(f64(X), pos0 + np.arange(L))
    slack = 1e-6 * (np.abs(f64(X)[..., : d // 2]) + np.abs(f64(X)[..., d // 2:]))
    close_to_rounded(Y, want, np.concatenate([slack, slack], axis=-1))
    # the transpose against the oracle's, and back to where it started within two roundings
    Z = sa.rope_apply(Y, table, pos0=pos0, inverse=True)
    close_to_rounded(Z, rope.rotate(f64(Y), pos0 + np.arange(L), inverse=True), 1e-5)
    assert np.abs(f64(Z) - f64(X)).max() <= 2 * BF16_HALF_ULP * np.abs(f64(X)).max()
    # in place
    Xc = X.contiguous()
    sa.rope_apply(Xc, table, pos0=pos0, out=Xc)
    assert torch.equal(Xc, Y)
    with pytest.raises(sa.SegAttnError):
        sa.rope_apply(X, table, pos0=pos0 + 1)       # the table does not reach the last position


def make(B, P, Hq, Hkv, d, R, Lseg, seed, layout="blhd"):
    g = torch.Generator().manual_seed(seed)
    mk = lambda *s: torch.randn(*s, generator=g).bfloat16().cuda()
    if layout == "blhd":
        Kp, Vp = mk(B, P, Hkv, d), mk(B, P, Hkv, d)
    else:
        Kp, Vp = mk(B, Hkv, P, d).permute(0, 2, 1, 3), mk(B, Hkv, P, d).permute(0, 2, 1, 3)
    idx = torch.randint(0, P, (B, Hkv, R), generator=g, dtype=torch.int32).cuda()
    return Kp, Vp, idx, mk(B, Lseg, Hkv, d), mk(B, Lseg, Hkv, d), mk(B, Lseg, Hq, d), mk(B, Lseg, Hq, d)


def oracle_long_range_step(Q, Kp, Vp, idx, Ks, Vs, dO, base=10000.0):
    """The oracle's long-range channel of one segment with re-indexed RoPE: rotated tensors kept in bf16 (as the
    library keeps them), attention and its gradients in fp64, gradients rotated back."""
    R, m = idx.shape[2], Ks.shape[1]
    Kc, Vc, Qr = rope.reindexed_context(f64(Kp), f64(Vp), idx, f64(Ks), f64(Vs), f64(Q), base)
    Kc, Qr = rope.round_bf16(Kc), rope.round_bf16(Qr)
    ar = np.broadcast_to(np.arange(R, dtype=np.int32), idx.shape)
    O, LSE, gq, gk, gv = dense.retrieved_attention(Qr, Kc[:, :R], Vc[:, :R], ar, Kc[:, R:], Vc[:, R:], f64(dO))
    pos = R + np.arange(m)
    return Kc, Vc, Qr, O, LSE, rope.rotate(gq, pos, base, inverse=True), rope.rotate(gk, pos, base, inverse=True), gv


@pytest.mark.parametrize("B,P,Hq,Hkv,d,R,Lseg,layout", [
    (1, 2048, 4, 2, 128, 512, 512, "blhd"),     # R = 512 as in the paper's setting
    (2, 1000, 4, 4, 128, 300, 200, "bhld"),     # nothing aligned to a tile; pool stored per head
    (1, 700, 2, 1, 64, 129, 77, "blhd"),        # d = 64, ragged
    (2, 64, 2, 2, 128, 0, 256, "blhd"),         # nothing retrieved: the segment alone, positions 0..m-1
])
def test_reindexed_long_range_channel_matches_oracle(B, P, Hq, Hkv, d, R, Lseg, layout):
    Kp, Vp, idx, Ks, Vs, Q, dO = make(B, P, Hq, Hkv, d, R, Lseg, seed=P + R + 1, layout=layout)
    table = sa.rope_table(R + Lseg, d)
    Kc, Vc = sa.gather_context_rope(Kp, Vp, idx, Ks, Vs, table)
    Qr = sa.rope_apply(Q, table, pos0=R)
    sa.poll_status()
    Kc_o, Vc_o, Qr_o, Oo, LSEo, gq, gk, gv = oracle_long_range_step(Q, Kp, Vp, idx.cpu().numpy(), Ks, Vs, dO)
    # values: index work, bit-exact; keys and queries: one bf16 rounding of the fp64 rotation (the oracle's own
    # rounded copy can differ from the library's by one bf16 step where fp32 and fp64 round apart)
    assert np.array_equal(f64(Vc), Vc_o)
    assert np.abs(f64(Kc) - Kc_o).max() <= 2 * BF16_HALF_ULP * max(1.0, np.abs(Kc_o).max())
    assert np.abs(f64(Qr) - Qr_o).max() <= 2 * BF16_HALF_ULP * np.abs(Qr_o).max()
    assert (f64(Kc) != Kc_o).mean() < 0.01
    S = max(1, R + Lseg)
    mask = [0] * Hkv
    O, LSE = sa.seg_attn_fwd(Qr, Kc, Vc, S, 0, mask, q_pos0=R, kv_pos0=0)
    dQr, dKc, dVc = sa.seg_attn_bwd(Qr, Kc, Vc, O, LSE, dO, S, 0, mask, q_pos0=R, kv_pos0=0, detach_before=R)
    dQ = sa.rope_apply(dQr, table, pos0=R, inverse=True)
    dK = sa.rope_apply(dKc[:, R:], table, pos0=R, inverse=True)
    sa.poll_status()
    assert_fwd_close(O, LSE, Oo, LSEo, "re-indexed long-range channel")
    assert_grads_close((dQ, dK, dVc[:, R:]), (gq, gk, gv), "re-indexed long-range channel")
    assert not dKc[:, :R].any() and not dVc[:, :R].any()


def test_gather_with_rotation_reports_an_index_out_of_range():
    Kp, Vp, idx, Ks, Vs, _, _ = make(1, 100, 2, 2, 128, 16, 8, seed=9)
    table = sa.rope_table(24, 128)
    idx[0, 1, 3] = 100
    Kc, Vc = sa.gather_context_rope(Kp, Vp, idx, Ks, Vs, table)
    with pytest.raises(sa.SegAttnError) as e:
        sa.poll_status()
    assert e.value.status == 1
    sa.poll_status()
    assert not Kc[0, 3, 1].any() and not Vc[0, 3, 1].any()
    with pytest.raises(sa.SegAttnError):
        sa.gather_context_rope(Kp, Vp, idx, Ks, Vs, table[:23])     # table shorter than R + Lseg


def test_select_gather_rotate_attend_end_to_end():
    B, P, Hq, Hkv, d, S, R = 1, 2048, 4, 2, 128, 256, 512
    Kp, Vp, _, Ks, Vs, Q, dO = make(B, P, Hq, Hkv, d, 8, S, seed=79)
    Q_prev = torch.randn(B, 48, Hq, d, generator=torch.Generator().manual_seed(80)).bfloat16().cuda()
    idx = sa.retrieval_select(Q_prev, Kp, 16, 8, 8, 16, 8, 32, 31, R)
    ref_idx = retrieval.select(Q_prev.float().cpu().numpy(), Kp.float().cpu().numpy(), 16, 8, 8, 16, 8, 32, 31, R)
    assert np.array_equal(idx.cpu().numpy(), ref_idx)
    table = sa.rope_table(R + S, d)
    Kc, Vc = sa.gather_context_rope(Kp, Vp, idx, Ks, Vs, table)
    Qr = sa.rope_apply(Q, table, pos0=R)
    O, LSE = sa.seg_attn_fwd(Qr, Kc, Vc, R + S, 0, [0] * Hkv, q_pos0=R, kv_pos0=0)
    dQr, dKc, dVc = sa.seg_attn_bwd(Qr, Kc, Vc, O, LSE, dO, R + S, 0, [0] * Hkv, q_pos0=R, kv_pos0=0, detach_before=R)
    dQ = sa.rope_apply(dQr, table, pos0=R, inverse=True)
    dK = sa.rope_apply(dKc[:, R:], table, pos0=R, inverse=True)
    sa.poll_status()
    _, _, _, Oo, LSEo, gq, gk, gv = oracle_long_range_step(Q, Kp, Vp, ref_idx, Ks, Vs, dO)
    assert_fwd_close(O, LSE, Oo, LSEo, "end to end with re-indexing")
    assert_grads_close((dQ, dK, dVc[:, R:]), (gq, gk, gv), "end to end with re-indexing")

"""Rotary position embedding with the re-indexed positions of a prefix concatenation, in numpy fp64.
TEST INFRASTRUCTURE ONLY.

Section 3.4 "RoPE Re-indexing for Prefix Concatenation" and Appendix E: when a prefix of P key/value rows
(the carried tail, P = M, or the retrieved rows, P = R) is put in front of a segment of m rows, the prefix
keys are rotated with positions 0 .. P-1 and the segment's queries and keys with positions P .. P+m-1;
values are not rotated.

"Standard RoPE" is taken as the rotation of the pairs (x[i], x[i + d/2]), i < d/2, by the angle
pos * base^(-2i/d) (the half-split pairing of the LLaMA family the paper fine-tunes; the paper does not name
a pairing or a base, so both are this repository's reading, base a parameter with the usual 10000):

    y[i]       = x[i] cos a_i - x[i + d/2] sin a_i
    y[i + d/2] = x[i] sin a_i + x[i + d/2] cos a_i,        a_i = pos * base^(-2i/d)

Pins (tests/test_oracle_pins.py): the same rotation as a complex multiplication, the library's
rotate-half form, position 0 = identity, norm preservation, the relative-position identity
<R_a q, R_b k> = <q, R_{b-a} k>, and re-indexed attention over the rows immediately before a segment
equal to attention under global positions.
"""
from __future__ import annotations

import numpy as np


def angles(positions, d, base=10000.0):
    """[len(positions), d/2] rotation angles."""
    i = np.arange(d // 2, dtype=np.float64)
    inv_freq = np.power(float(base), -2.0 * i / d)
    return np.asarray(positions, dtype=np.float64)[:, None] * inv_freq[None, :]


def rotate(x, positions, base=10000.0, inverse=False):
    """Rotate x [..., L, H, d] (row l at position positions[l]); inverse=True rotates back (the transpose of the
    rotation, which is also the map a gradient with respect to the rotated tensor goes through)."""
    x = np.asarray(x, dtype=np.float64)
    d = x.shape[-1]
    a = angles(positions, d, base)
    if inverse:
        a = -a
    c, s = np.cos(a)[:, None, :], np.sin(a)[:, None, :]      # [L, 1, d/2]
    lo, hi = x[..., : d // 2], x[..., d // 2:]
    return np.concatenate([lo * c - hi * s, lo * s + hi * c], axis=-1)


def reindexed_context(K_pool, V_pool, idx, K_seg, V_seg, Q_seg, base=10000.0):
    """[K_ret ; K_i] with re-indexed rotations, V plain, and the rotated segment queries.
    K_pool, V_pool [B, P, Hkv, d] unrotated; idx [B, Hkv, R]; K_seg, V_seg [B, m, Hkv, d]; Q_seg [B, m, Hq, d].
    Returns K_ctx, V_ctx [B, R + m, Hkv, d] and Q_rot [B, m, Hq, d]."""
    K_pool, V_pool = np.asarray(K_pool, np.float64), np.asarray(V_pool, np.float64)
    K_seg, V_seg, Q_seg = (np.asarray(t, np.float64) for t in (K_seg, V_seg, Q_seg))
    B, m, Hkv, d = K_seg.shape
    R = idx.shape[2]
    K_ctx = np.zeros((B, R + m, Hkv, d))
    V_ctx = np.zeros((B, R + m, Hkv, d))
    for b in range(B):
        for c in range(Hkv):
            K_ctx[b, :R, c] = K_pool[b, idx[b, c], c]
            V_ctx[b, :R, c] = V_pool[b, idx[b, c], c]
    K_ctx[:, R:], V_ctx[:, R:] = K_seg, V_seg
    K_ctx = rotate(K_ctx, np.arange(R + m), base)            # prefix 0..R-1, segment R..R+m-1
    Q_rot = rotate(Q_seg, R + np.arange(m), base)
    return K_ctx, V_ctx, Q_rot


def round_bf16(x):
    """x rounded to bfloat16 (nearest even) and widened again: the precision in which rotated tensors are kept."""
    import torch
    return torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).to(torch.bfloat16).to(torch.float64).numpy()

"""Helpers shared by the GPU parity tests: tolerances and oracle sub-problems."""
import numpy as np
import torch

import oracle
import workloads

# Tolerances of the parity gate: bf16 inputs, fp32 accumulation.
TOL_O = 2e-2      # max |O - O_oracle|
TOL_LSE = 1e-3    # max |LSE - LSE_oracle|
TOL_GRAD = 5e-2   # relative L2 of each gradient


def f64(t):
    return workloads.to_f64(t)


def rel_l2(a, b):
    a, b = np.asarray(a, dtype=np.float64), np.asarray(b, dtype=np.float64)
    n = np.linalg.norm(b)
    return float(np.linalg.norm(a - b) / n) if n > 0 else float(np.linalg.norm(a - b))


def rand_inputs(B, L, Hq, Hkv, d, seed=0, Lk=None, device="cuda"):
    g = torch.Generator().manual_seed(seed)
    Lk = L if Lk is None else Lk
    mk = lambda *s: torch.randn(*s, generator=g).bfloat16().to(device)
    return mk(B, L, Hq, d), mk(B, Lk, Hkv, d), mk(B, Lk, Hkv, d), mk(B, L, Hq, d)


def assert_fwd_close(O, LSE, Oo, LSEo, what=""):
    eo = np.abs(f64(O) - Oo).max() if Oo.size else 0.0
    fin = np.isfinite(LSEo)
    el = np.abs(f64(LSE)[fin] - LSEo[fin]).max() if fin.any() else 0.0
    assert np.array_equal(np.isfinite(f64(LSE)), fin), what + ": LSE finiteness differs"
    assert eo <= TOL_O, "%s: O max-abs error %.3e" % (what, eo)
    assert el <= TOL_LSE, "%s: LSE max-abs error %.3e" % (what, el)


# Row-level gate beside the whole-tensor one.  A gradient row is a sum of terms whose factors P and dS were
# rounded to bf16 (relative error <= 2^-9 each, independent), accumulated in fp32 and rounded to bf16 once
# more: the row's error is about 2^-9 * sqrt(sum of squared terms), i.e. 2^-9 times the row norm times the
# row's cancellation factor.  For rows of at least typical norm that factor is O(1..10), which is what the
# whole-tensor tolerance already assumes, so such rows are held to the same TOL_GRAD one by one.  Rows of
# smaller norm (strong cancellation, where no relative bound holds even for a correct kernel) are held to
# the absolute error a row of typical norm may have.  One wrong row of typical norm has error ~ its norm,
# twenty times this bound, while it moves the whole-tensor figure by only ~1/sqrt(rows).
def row_errors(a, b):
    """Per-row error of gradient a against reference b over the last dimension, divided by
    max(row norm, RMS row norm of the tensor)."""
    a, b = np.asarray(a, dtype=np.float64), np.asarray(b, dtype=np.float64)
    if b.size == 0:
        return np.zeros(0)
    rn = np.linalg.norm(b.reshape(-1, b.shape[-1]), axis=1)
    en = np.linalg.norm((a - b).reshape(-1, b.shape[-1]), axis=1)
    rms = float(np.sqrt(np.mean(rn ** 2)))
    if rms == 0.0:
        return en
    return en / np.maximum(rn, rms)


def assert_grads_close(grads, ref, what=""):
    for name, a, b in zip(("dQ", "dK", "dV"), grads, ref):
        a = f64(a) if torch.is_tensor(a) else a
        e = rel_l2(a, b)
        assert e <= TOL_GRAD, "%s: %s relative L2 error %.3e" % (what, name, e)
        re = row_errors(a, b)
        if re.size:
            k = int(re.argmax())
            assert re[k] <= TOL_GRAD, "%s: %s row %d (flattened) error %.3e of max(row norm, RMS row norm)" % (what, name, k, re[k])


def group_slices(mask, g):
    """One flagged and one unflagged KV head (if present) with their query-head ranges."""
    out = []
    for want in (1, 0):
        idx = [c for c in range(len(mask)) if int(mask[c] != 0) == want]
        if idx:
            c = idx[len(idx) // 2]
            out.append((c, slice(c * g, (c + 1) * g)))
    return out


def oracle_window(x, w, b, c, hq, seg_lo, n_seg=2):
    """Oracle forward + backward for batch b, KV head c (query heads hq) on the queries of
    segments [seg_lo, seg_lo + n_seg) against every key before the window's end.  `keys` is the range whose
    dK/dV are complete: the window's keys without the last T of them (the tail the next segment also reads),
    or all of them when the window ends the sequence."""
    S = w.S
    r0, r1 = seg_lo * S, min(w.L, (seg_lo + n_seg) * S)
    Q = f64(x["Q"][b:b + 1, r0:r1, hq])
    K = f64(x["K"][b:b + 1, :r1, c:c + 1])
    V = f64(x["V"][b:b + 1, :r1, c:c + 1])
    m = [int(x["mask"][c])]
    O, LSE = oracle.fwd(Q, K, V, S, w.T, m, scale=w.sm_scale, q_pos0=r0)
    out = {"rows": slice(r0, r1), "O": O, "LSE": LSE}
    if "dO" in x:
        dO = f64(x["dO"][b:b + 1, r0:r1, hq])
        dQ, dK, dV = oracle.bwd(Q, K, V, dO, S, w.T, m, scale=w.sm_scale, q_pos0=r0)
        k1 = r1 if r1 == w.L else r1 - w.T
        out.update(dQ=dQ, dK=dK[:, r0:k1], dV=dV[:, r0:k1], keys=slice(r0, k1))
    return out


def oracle_last_rows(x, w, b, c, hq, n_rows):
    """Oracle forward + backward for the last n_rows query rows (all query heads hq of KV head c) against the
    keys they can see.  Nothing reads the last keys after them, so dK/dV of keys [L - n_rows, L) are complete:
    the last key tiles of the dK/dV grid."""
    r0 = w.L - n_rows
    k0 = 0 if int(x["mask"][c]) == 1 else max(0, (r0 // w.S) * w.S - w.T)
    Q = f64(x["Q"][b:b + 1, r0:, hq])
    K = f64(x["K"][b:b + 1, k0:, c:c + 1])
    V = f64(x["V"][b:b + 1, k0:, c:c + 1])
    m = [int(x["mask"][c])]
    O, LSE = oracle.fwd(Q, K, V, w.S, w.T, m, scale=w.sm_scale, q_pos0=r0, kv_pos0=k0)
    out = {"rows": slice(r0, w.L), "O": O, "LSE": LSE}
    if "dO" in x:
        dO = f64(x["dO"][b:b + 1, r0:, hq])
        dQ, dK, dV = oracle.bwd(Q, K, V, dO, w.S, w.T, m, scale=w.sm_scale, q_pos0=r0, kv_pos0=k0)
        out.update(dQ=dQ, dK=dK[:, r0 - k0:], dV=dV[:, r0 - k0:], keys=slice(r0, w.L))
    return out


def oracle_rows(x, w, b, c, hq, rows):
    """Oracle forward (and dQ) for single query rows, one call per row."""
    outs = []
    for p in rows:
        Q = f64(x["Q"][b:b + 1, p:p + 1, hq])
        K = f64(x["K"][b:b + 1, :p + 1, c:c + 1])
        V = f64(x["V"][b:b + 1, :p + 1, c:c + 1])
        m = [int(x["mask"][c])]
        O, LSE = oracle.fwd(Q, K, V, w.S, w.T, m, scale=w.sm_scale, q_pos0=p)
        dQ = None
        if "dO" in x:
            dO = f64(x["dO"][b:b + 1, p:p + 1, hq])
            dQ, _, _ = oracle.bwd(Q, K, V, dO, w.S, w.T, m, scale=w.sm_scale, q_pos0=p)
        outs.append((p, O, LSE, dQ))
    return outs

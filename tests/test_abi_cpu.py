"""CPU-side checks of the boundary: the library loads without a GPU, exports every symbol the
header declares, validates arguments before touching a device, and its pair counter agrees
with the oracle's enumeration of the mask."""
import ctypes
import os
import re

import numpy as np
import pytest

import oracle
import workloads
import paper_2605_11744_b200 as sa
from paper_2605_11744_b200.binding import Params

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "seg_attn.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(seg_(?:attn|prefill|retrieval|rope)_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = declared_symbols()
    assert "seg_attn_fwd" in names and "seg_attn_bwd" in names and "seg_prefill_step" in names
    L = sa.lib()
    for n in names:
        assert hasattr(L, n), n


def test_status_strings():
    L = sa.lib()
    assert L.seg_attn_status_string(0) == b"ok"
    for s in range(1, 6):
        assert len(L.seg_attn_status_string(s)) > 3


def _params(**kw):
    p = Params()
    base = dict(B=1, Lq=256, kv_len=256, Hq=4, Hkv=2, d=128, S=64, T=16, q_pos0=0, kv_pos0=0, sm_scale=0.1)
    base.update(kw)
    for k, v in base.items():
        setattr(p, k, v)
    for name, H in (("q_stride", base["Hq"]), ("o_stride", base["Hq"]), ("k_stride", base["Hkv"]), ("v_stride", base["Hkv"])):
        L = base["Lq"] if name[0] in "qo" else base["kv_len"]
        setattr(p, name, (ctypes.c_int64 * 3)(L * H * base["d"], H * base["d"], base["d"]))
    return p


@pytest.mark.parametrize("bad", [dict(T=65), dict(S=0), dict(d=96), dict(Hq=3), dict(Hkv=128, Hq=128), dict(B=-1),
                                 dict(sm_scale=0.0), dict(q_pos0=-1)])
def test_invalid_params_rejected_on_the_host(bad):
    p = _params(**bad)
    m = np.zeros(128, dtype=np.uint8)
    L = sa.lib()
    dummy = ctypes.c_void_p(4096)
    assert L.seg_attn_fwd(ctypes.byref(p), dummy, dummy, dummy, m.ctypes.data, dummy, dummy, None, 0, None) == 1
    assert L.seg_attn_workspace_bytes(ctypes.byref(p), 1) == 0
    assert L.seg_attn_count_pairs(ctypes.byref(p), m.ctypes.data, None, None, None) == 1


def test_null_and_misaligned_pointers_rejected():
    p = _params()
    m = np.zeros(2, dtype=np.uint8)
    L = sa.lib()
    ok = ctypes.c_void_p(4096)
    assert L.seg_attn_fwd(ctypes.byref(p), None, ok, ok, m.ctypes.data, ok, ok, None, 0, None) == 1
    assert L.seg_attn_fwd(ctypes.byref(p), ctypes.c_void_p(4100), ok, ok, m.ctypes.data, ok, ok, None, 0, None) == 1
    assert L.seg_attn_fwd(ctypes.byref(p), ok, ok, ok, None, ok, ok, None, 0, None) == 1
    p2 = _params()
    p2.k_stride = (ctypes.c_int64 * 3)(256 * 2 * 128, 2 * 128 + 4, 128)      # not a multiple of 8 elements
    assert L.seg_attn_fwd(ctypes.byref(p2), ok, ok, ok, m.ctypes.data, ok, ok, None, 0, None) == 1
    # backward without (enough) workspace
    assert L.seg_attn_bwd(ctypes.byref(p), ok, ok, ok, ok, ok, ok, m.ctypes.data, ok, ok, ok, None, 0, None) == 5
    assert L.seg_attn_bwd(ctypes.byref(p), ok, ok, ok, ok, ok, ok, m.ctypes.data, ok, ok, ok, ok, 16, None) == 5


def test_workspace_sizes():
    p = _params(B=2, Lq=1000, Hq=4)
    assert sa.workspace_bytes(p, False) == 0
    assert sa.workspace_bytes(p, True) == (2 * 4 * 1000 * 4 + 255) // 256 * 256
    assert sa.lib().seg_attn_host_arena_bytes(ctypes.byref(p)) > 0


def test_no_device_means_an_error_not_a_fallback():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    p = _params()
    m = np.zeros(2, dtype=np.uint8)
    ok = ctypes.c_void_p(4096)
    L = sa.lib()
    st = L.seg_attn_fwd(ctypes.byref(p), ok, ok, ok, m.ctypes.data, ok, ok, None, 0, None)
    assert st in (2, 3)      # unsupported device / CUDA error: never a silent CPU path
    # the retrieval entry points refuse the same way, before any launch
    stride = (ctypes.c_int64 * 3)(256 * 2 * 128, 2 * 128, 128)
    st = L.seg_attn_gather_context(1, 2, 128, 8, 16, 256, ok, ok, stride, ok, ok, stride, ok, ok, ok, None)
    assert st in (2, 3)
    r = sa.binding.RetrievalParams(Lq_last=16, window=8, stride=4, tail=4, top_k=4, n_anchors=2, off_lo=1, off_hi=1, R=16)
    L.seg_retrieval_workspace_bytes.restype = ctypes.c_size_t
    need = L.seg_retrieval_workspace_bytes(1, 4, 2, 128, 256, ctypes.byref(r))
    assert need > 0
    st = L.seg_retrieval_select(1, 4, 2, 128, 256, ok, ok, stride, ctypes.byref(r), ok, ctypes.c_void_p(1 << 20),
                                ctypes.c_size_t(need), None)
    assert st in (2, 3)


@pytest.mark.parametrize("B,L,Hq,Hkv,S,T,mask", [
    (1, 2048, 4, 4, 512, 128, [0, 0, 0, 0]),
    (2, 1000, 4, 2, 200, 72, [1, 0]),
    (1, 777, 2, 2, 64, 64, [0, 1]),
    (1, 300, 2, 1, 7, 0, [0]),
    (2, 1000, 4, 2, 200, 72, [2, 1]),       # an own-segment-only head beside a past-access one
    (1, 777, 3, 3, 64, 64, [2, 0, 1]),      # all three head classes
])
def test_pair_counter_matches_oracle_enumeration(B, L, Hq, Hkv, S, T, mask):
    nv, nd, tiles = sa.count_pairs(B, L, Hq, Hkv, 128, S, T, mask)
    assert (nv, nd) == oracle.count_pairs(B, L, Hq, Hkv, S, T, mask)
    assert tiles * 128 * 128 >= nv
    # the reading in which flagged heads read the carried tail forward-only too: fewer differentiable pairs
    nv2, nd2, _ = sa.count_pairs(B, L, Hq, Hkv, 128, S, T, mask, flagged_tail_is_sg=True)
    assert (nv2, nd2) == oracle.count_pairs(B, L, Hq, Hkv, S, T, mask, flagged_tail_is_sg=True)
    assert nv2 == nv and nd2 <= nd


def test_pair_counter_with_a_detached_prefix():
    for X in (0, 200, 300, 1000):
        nv, nd, _ = sa.count_pairs(2, 1000, 4, 2, 128, 200, 72, [1, 0], detach_before=X)
        assert (nv, nd) == oracle.count_pairs(2, 1000, 4, 2, 200, 72, [1, 0], detach_before=X)
    with pytest.raises(sa.SegAttnError):
        sa.count_pairs(1, 256, 2, 2, 128, 64, 16, [0, 0], detach_before=-1)


@pytest.mark.parametrize("S", [1, 2, 3, 7, 100, 127, 128, 1000, 4096, 12345, 65537])
def test_segment_arithmetic_for_many_segment_lengths(S):
    # the library divides positions by S through a launch-time reciprocal: check it against the oracle's
    # plain division, at low positions and near the top of the supported range
    T = min(S, 5)
    for L in (1, 257, 3000):
        nv, nd, _ = sa.count_pairs(1, L, 2, 2, 128, S, T, [0, 2])
        assert (nv, nd) == oracle.count_pairs(1, L, 2, 2, S, T, [0, 2])
    # high positions: a window of 300 queries whose keys start one tail before it, against the same
    # window moved down by a whole number of segments (the mask only depends on positions modulo S)
    q0 = ((1 << 30) - 1 - 300) // S * S
    lo = max(0, q0 - T)
    hi = sa.count_pairs(1, 300, 2, 2, 128, S, T, [0, 2], kv_len=300 + q0 - lo, q_pos0=q0, kv_pos0=lo)
    q1 = min(q0, 5 * S)
    lo1 = max(0, q1 - T)
    ref = sa.count_pairs(1, 300, 2, 2, 128, S, T, [0, 2], kv_len=300 + q1 - lo1, q_pos0=q1, kv_pos0=lo1)
    assert hi[:2] == ref[:2]


@pytest.mark.parametrize("starts,T", [([0, 20, 50, 51, 300, 700], 8), ([0, 128, 256, 384], 128), ([0], 5),
                                      ([0, 33, 66], 40), ([0, 1, 2, 3, 500], 2)])
def test_pair_counter_with_segments_of_given_lengths(starts, T):
    for mask in ([0, 1], [2, 0]):
        for X in (0, 60):
            nv, nd, _ = sa.count_pairs(2, 900, 4, 2, 128, 1, T, mask, seg_starts=starts, detach_before=X)
            assert (nv, nd) == oracle.count_pairs(2, 900, 4, 2, 1, T, mask, seg_starts=starts, detach_before=X)
    # equal lengths are the constant-length case
    S = 128
    eq = list(range(0, 900, S))
    assert sa.count_pairs(1, 900, 2, 2, 128, S, 40, [0, 1]) == sa.count_pairs(1, 900, 2, 2, 128, 1, 40, [0, 1], seg_starts=eq)
    for bad in ([1, 5], [0, 5, 5], [0, 9, 3], list(range(257))):
        with pytest.raises(sa.SegAttnError):
            sa.count_pairs(1, 64, 2, 2, 128, 1, 4, [0, 0], seg_starts=bad)


def test_unknown_head_class_is_rejected():
    with pytest.raises(sa.SegAttnError):
        sa.count_pairs(1, 256, 2, 2, 128, 64, 16, [0, 3])


def test_benchmark_configuration_counts():
    for w, want in ((workloads.CONFIGS[0], 2887680), (workloads.CONFIGS[1], 3305635840),
                    (workloads.CONFIGS[2], 10133962752), (workloads.CONFIGS[3], 87646273536)):
        m = workloads.head_past_mask(w.Hkv, w.past_frac, w.seed)
        assert sa.count_pairs(w.B, w.L, w.Hq, w.Hkv, w.d, w.S, w.T, m)[0] == want


def test_prefill_state_size_and_validation():
    pf_params = _params(B=1, Lq=128, kv_len=1024, S=128, T=64, Hq=4, Hkv=2)
    m = np.array([1, 0], dtype=np.uint8)
    L = sa.lib()
    n = L.seg_prefill_state_bytes(ctypes.byref(pf_params), m.ctypes.data)
    assert n == 2 * (1 * 1 * 1024 * 128 * 2) + 2 * (1 * 1 * (128 + 64) * 128 * 2)
    bad = _params(B=1, Lq=64, kv_len=1024, S=128, T=64)
    assert L.seg_prefill_state_bytes(ctypes.byref(bad), m.ctypes.data) == 0
    h = ctypes.c_void_p()
    assert L.seg_prefill_create(ctypes.byref(pf_params), m.ctypes.data, None, 0, ctypes.byref(h)) == 5

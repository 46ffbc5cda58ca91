"""fp64 CPU oracle for segment-level causal attention.  TEST INFRASTRUCTURE ONLY.

Two independent statements of the same definition live here:

* ``seg_attn_oracle.c``  - row-by-row C (OpenMP), the oracle proper (``fwd``, ``bwd``,
  ``count_pairs`` below are thin ctypes wrappers around it);
* ``dense.py``           - the matrix form in numpy with explicit L x L masks, for L <= ~4K.

Nothing on the product path may import this package: only ``tests/``, the smoke check and
the CPU-baseline leg of the benchmark do.  It shares no code with the CUDA library.
Inputs and outputs are numpy float64 arrays, Q/O/dO/dQ ``[B, Lq, Hq, d]``,
K/V/dK/dV ``[B, Lk, Hkv, d]``, LSE ``[B, Hq, Lq]``.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "seg_attn_oracle.c")
_LIB = os.path.join(_HERE, "_build", "libsegattn_oracle.so")
_lib = None


class _Cfg(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in
                ("B", "Lq", "Lk", "Hq", "Hkv", "d", "S", "T", "q_pos0", "kv_pos0", "flagged_tail_is_sg", "detach_before")] + \
               [("scale", ctypes.c_double), ("seg_starts", ctypes.c_void_p), ("n_segs", ctypes.c_int32)]


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (OpenMP) if the shared object is missing or stale."""
    os.makedirs(os.path.dirname(_LIB), exist_ok=True)
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".%d.tmp" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        dp = ctypes.POINTER(ctypes.c_double)
        u8 = ctypes.POINTER(ctypes.c_uint8)
        cp = ctypes.POINTER(_Cfg)
        lib.oracle_seg_attn_fwd.argtypes = [cp, dp, dp, dp, u8, dp, dp]
        lib.oracle_seg_attn_bwd.argtypes = [cp, dp, dp, dp, dp, u8, dp, dp, dp]
        lib.oracle_count_pairs.argtypes = [cp, u8, ctypes.POINTER(ctypes.c_int64), ctypes.POINTER(ctypes.c_int64)]
        lib.oracle_num_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


def _f64(a):
    return np.ascontiguousarray(a, dtype=np.float64)


def _ptr(a):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def _with_starts(cfg, seg_starts):
    """Attach variable segment starts (kept alive on the struct) or leave the constant length S."""
    if seg_starts is not None:
        st = np.ascontiguousarray(np.asarray(seg_starts), dtype=np.int32)
        cfg._starts = st
        cfg.seg_starts = st.ctypes.data
        cfg.n_segs = int(st.size)
    return cfg


def _cfg(Q, K, S, T, scale, q_pos0, kv_pos0, flagged_tail_is_sg, detach_before=0):
    B, Lq, Hq, d = Q.shape
    Bk, Lk, Hkv, dk = K.shape
    assert B == Bk and d == dk and Hq % Hkv == 0
    if scale is None:
        scale = 1.0 / np.sqrt(d)
    return _Cfg(B, Lq, Lk, Hq, Hkv, d, S, T, q_pos0, kv_pos0, int(bool(flagged_tail_is_sg)), int(detach_before), float(scale))


def _mask(head_past_mask, Hkv):
    m = np.zeros(Hkv, dtype=np.uint8) if head_past_mask is None else \
        np.ascontiguousarray(np.asarray(head_past_mask), dtype=np.uint8)  # head class: 0 local, 1 past, 2 own only
    assert m.shape == (Hkv,) and int(m.max(initial=0)) <= 2
    return m


def fwd(Q, K, V, S, T, head_past_mask=None, scale=None, q_pos0=0, kv_pos0=0, flagged_tail_is_sg=False, seg_starts=None):
    """O ``[B,Lq,Hq,d]`` and natural-log LSE ``[B,Hq,Lq]`` of the scaled scores over visible keys."""
    Q, K, V = _f64(Q), _f64(K), _f64(V)
    cfg = _with_starts(_cfg(Q, K, S, T, scale, q_pos0, kv_pos0, flagged_tail_is_sg), seg_starts)
    m = _mask(head_past_mask, cfg.Hkv)
    O = np.empty_like(Q)
    LSE = np.empty((cfg.B, cfg.Hq, cfg.Lq), dtype=np.float64)
    rc = _load().oracle_seg_attn_fwd(ctypes.byref(cfg), _ptr(Q), _ptr(K), _ptr(V),
                                     m.ctypes.data_as(ctypes.POINTER(ctypes.c_uint8)), _ptr(O), _ptr(LSE))
    if rc:
        raise ValueError("oracle_seg_attn_fwd: invalid configuration (rc=%d)" % rc)
    return O, LSE


def bwd(Q, K, V, dO, S, T, head_past_mask=None, scale=None, q_pos0=0, kv_pos0=0, flagged_tail_is_sg=False,
        detach_before=0, seg_starts=None):
    """dQ, dK, dV for the cotangent dO; dK/dV hold only what the queries passed in contribute.  Keys at
    global positions below ``detach_before`` are read forward-only (a window with a detached incoming state)."""
    Q, K, V, dO = _f64(Q), _f64(K), _f64(V), _f64(dO)
    cfg = _with_starts(_cfg(Q, K, S, T, scale, q_pos0, kv_pos0, flagged_tail_is_sg, detach_before), seg_starts)
    m = _mask(head_past_mask, cfg.Hkv)
    dQ, dK, dV = np.empty_like(Q), np.empty_like(K), np.empty_like(V)
    rc = _load().oracle_seg_attn_bwd(ctypes.byref(cfg), _ptr(Q), _ptr(K), _ptr(V), _ptr(dO),
                                     m.ctypes.data_as(ctypes.POINTER(ctypes.c_uint8)),
                                     _ptr(dQ), _ptr(dK), _ptr(dV))
    if rc:
        raise ValueError("oracle_seg_attn_bwd: invalid configuration (rc=%d)" % rc)
    return dQ, dK, dV


def count_pairs(B, L, Hq, Hkv, S, T, head_past_mask=None, flagged_tail_is_sg=False, detach_before=0, seg_starts=None,
                Lk=None, q_pos0=0, kv_pos0=0):
    """(visible, differentiable) query-key pair counts by enumerating the mask row by row.  ``L`` query rows
    starting at global position ``q_pos0`` against ``Lk`` key rows (default ``L``) starting at ``kv_pos0``."""
    Lk = L if Lk is None else Lk
    cfg = _with_starts(_Cfg(B, L, Lk, Hq, Hkv, 1, S, T, q_pos0, kv_pos0, int(bool(flagged_tail_is_sg)), int(detach_before), 1.0),
                       seg_starts)
    m = _mask(head_past_mask, Hkv)
    nv, nd = ctypes.c_int64(), ctypes.c_int64()
    rc = _load().oracle_count_pairs(ctypes.byref(cfg), m.ctypes.data_as(ctypes.POINTER(ctypes.c_uint8)),
                                    ctypes.byref(nv), ctypes.byref(nd))
    if rc:
        raise ValueError("oracle_count_pairs: invalid configuration")
    return nv.value, nd.value


def num_threads() -> int:
    return int(_load().oracle_num_threads())

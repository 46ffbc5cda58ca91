"""ctypes binding with the same names as the C ABI in ``include/seg_attn.h``.

Argument marshalling only: pointers, strides and the stream are taken from torch tensors and
handed to the library.  There is no fallback: if ``libsegattn.so`` is missing the import fails.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libsegattn.so")


class SegAttnError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = lib().seg_attn_status_string(status).decode()
        extra = " (cuda/driver code %d)" % lib().seg_attn_last_cuda_error() if status in (3, 4) else ""
        super().__init__("%s: %s%s" % (where, msg, extra))


class Params(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in ("B", "Lq", "kv_len", "Hq", "Hkv", "d", "S", "T", "q_pos0", "kv_pos0")] + \
               [("sm_scale", ctypes.c_float), ("flags", ctypes.c_int32), ("detach_before", ctypes.c_int32),
                ("q_stride", ctypes.c_int64 * 3), ("k_stride", ctypes.c_int64 * 3),
                ("v_stride", ctypes.c_int64 * 3), ("o_stride", ctypes.c_int64 * 3),
                ("seg_starts", ctypes.c_void_p), ("n_segs", ctypes.c_int32)]


_lib = None


def lib():
    """The loaded C-ABI library.  Raises if it has not been built (no CPU or eager fallback exists)."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise ImportError("libsegattn.so is not built: run `python -m paper_2605_11744_b200.build` "
                              "(or __graft_entry__.build()); there is no fallback path")
        L = ctypes.CDLL(_LIB_PATH)
        vp, u8p, fp = ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p
        pp = ctypes.POINTER(Params)
        L.seg_attn_workspace_bytes.restype = ctypes.c_size_t
        L.seg_attn_workspace_bytes.argtypes = [pp, ctypes.c_int]
        L.seg_attn_fwd.argtypes = [pp, vp, vp, vp, u8p, vp, fp, vp, ctypes.c_size_t, vp]
        L.seg_attn_bwd.argtypes = [pp, vp, vp, vp, vp, fp, vp, u8p, vp, vp, vp, vp, ctypes.c_size_t, vp]
        L.seg_attn_bwd_static.argtypes = [pp, vp, vp, vp, vp, fp, vp, u8p, vp, vp, vp, vp]
        L.seg_prefill_state_bytes.restype = ctypes.c_size_t
        L.seg_prefill_state_bytes.argtypes = [pp, u8p]
        L.seg_prefill_create.argtypes = [pp, u8p, vp, ctypes.c_size_t, ctypes.POINTER(vp)]
        L.seg_prefill_step.argtypes = [vp, vp, vp, vp, vp, fp, vp]
        L.seg_prefill_step_len.argtypes = [vp, ctypes.c_int32, vp, vp, vp, vp, fp, vp]
        L.seg_prefill_bwd_workspace_bytes.restype = ctypes.c_size_t
        L.seg_prefill_bwd_workspace_bytes.argtypes = [vp]
        L.seg_prefill_step_bwd.argtypes = [vp, vp, vp, fp, vp, vp, vp, vp, vp, ctypes.c_size_t, vp]
        L.seg_retrieval_workspace_bytes.restype = ctypes.c_size_t
        L.seg_retrieval_workspace_bytes.argtypes = [ctypes.c_int32] * 5 + [vp]
        L.seg_retrieval_select.argtypes = [ctypes.c_int32] * 5 + [vp, vp, ctypes.POINTER(ctypes.c_int64), vp, vp, vp,
                                                                  ctypes.c_size_t, vp]
        i64p = ctypes.POINTER(ctypes.c_int64)
        L.seg_rope_table_bytes.restype = ctypes.c_size_t
        L.seg_rope_table_bytes.argtypes = [ctypes.c_int32, ctypes.c_int32]
        L.seg_rope_table.argtypes = [ctypes.c_int32, ctypes.c_int32, ctypes.c_double, vp, vp]
        L.seg_rope_apply.argtypes = [ctypes.c_int32] * 4 + [vp, i64p, vp, i64p, ctypes.c_int32, ctypes.c_int32, vp,
                                                            ctypes.c_int32, vp]
        L.seg_attn_gather_context_rope.argtypes = [ctypes.c_int32] * 6 + [vp, vp, i64p, vp, vp, i64p, vp, vp, vp, vp,
                                                                          ctypes.c_int32, vp]
        L.seg_prefill_reset.argtypes = [vp]
        L.seg_prefill_destroy.argtypes = [vp]
        L.seg_prefill_destroy.restype = None
        L.seg_attn_host_arena_bytes.restype = ctypes.c_size_t
        L.seg_attn_host_arena_bytes.argtypes = [pp]
        L.seg_attn_step_host.argtypes = [pp, vp, vp, vp, vp, u8p, vp, fp, vp, vp, vp, vp, ctypes.c_size_t, vp]
        L.seg_attn_profile_kernels.argtypes = [pp, vp, vp, vp, vp, fp, vp, u8p, vp, vp, vp, vp, ctypes.c_size_t,
                                               ctypes.c_int, ctypes.POINTER(ctypes.c_float * 4), vp]
        L.seg_attn_poll_status.argtypes = [vp]
        L.seg_attn_gather_context.argtypes = [ctypes.c_int32] * 6 + [vp, vp, ctypes.POINTER(ctypes.c_int64), vp, vp,
                                                                     ctypes.POINTER(ctypes.c_int64), vp, vp, vp, vp]
        L.seg_attn_selftest_wait_timeout.argtypes = [vp]
        L.seg_attn_status_string.restype = ctypes.c_char_p
        L.seg_attn_status_string.argtypes = [ctypes.c_int]
        L.seg_attn_last_cuda_error.restype = ctypes.c_int
        L.seg_attn_launch_count.restype = ctypes.c_int64
        L.seg_attn_count_pairs.argtypes = [pp, u8p] + [ctypes.POINTER(ctypes.c_int64)] * 3
        _lib = L
    return _lib


def _check(status: int, where: str):
    if status != 0:
        raise SegAttnError(status, where)


def _mask_arr(head_past_mask, Hkv: int) -> np.ndarray:
    # one head class per KV head (booleans count as 0 / 1); the library rejects values above HEAD_OWN
    m = np.zeros(Hkv, dtype=np.uint8) if head_past_mask is None else \
        np.ascontiguousarray(np.asarray(head_past_mask), dtype=np.uint8)
    if m.shape != (Hkv,):
        raise ValueError("head_past_mask must have Hkv entries")
    return m


def _strides3(t: torch.Tensor):
    if t.dim() != 4 or (t.shape[3] > 1 and t.stride(3) != 1):
        raise ValueError("expected a [B, L, H, d] tensor with a contiguous last dimension")
    return (ctypes.c_int64 * 3)(t.stride(0), t.stride(1), t.stride(2))


FLAG_FLAGGED_TAIL_SG = 1   # SEGATTN_FLAG_FLAGGED_TAIL_SG of the C header
HEAD_LOCAL, HEAD_PAST, HEAD_OWN = 0, 1, 2   # SEGATTN_HEAD_* of the C header: entries of head_past_mask


def set_seg_starts(p: "Params", seg_starts) -> None:
    """Segments of given lengths: `seg_starts` (ascending, first 0) replaces the constant length S."""
    if seg_starts is not None:
        arr = np.ascontiguousarray(np.asarray(seg_starts), dtype=np.int32)
        p._seg_starts = arr          # keeps the host array alive as long as the parameter block
        p.seg_starts = arr.ctypes.data
        p.n_segs = int(arr.size)


def params_for(Q, K, V, O, S: int, T: int, sm_scale: Optional[float] = None, q_pos0: int = 0,
               kv_pos0: int = 0, flagged_tail_is_sg: bool = False, detach_before: int = 0, seg_starts=None) -> Params:
    """seg_attn_params for [B, L, H, d] tensors (only shapes and strides are read)."""
    B, Lq, Hq, d = Q.shape
    kv_len, Hkv = K.shape[1], K.shape[2]
    p = Params()
    p.B, p.Lq, p.kv_len, p.Hq, p.Hkv, p.d = B, Lq, kv_len, Hq, Hkv, d
    p.S, p.T, p.q_pos0, p.kv_pos0 = S, T, q_pos0, kv_pos0
    p.flags = FLAG_FLAGGED_TAIL_SG if flagged_tail_is_sg else 0
    p.detach_before = detach_before
    set_seg_starts(p, seg_starts)
    p.sm_scale = float(sm_scale if sm_scale is not None else d ** -0.5)
    p.q_stride, p.k_stride, p.v_stride, p.o_stride = _strides3(Q), _strides3(K), _strides3(V), _strides3(O)
    return p


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None or t.numel() == 0 else ctypes.c_void_p(t.data_ptr())


def _stream(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def _need_cuda_bf16(*ts):
    for t in ts:
        if t.device.type != "cuda" or t.dtype != torch.bfloat16:
            raise ValueError("tensors must be bf16 CUDA tensors")


def workspace_bytes(p: Params, is_bwd: bool) -> int:
    return int(lib().seg_attn_workspace_bytes(ctypes.byref(p), int(is_bwd)))


def seg_attn_fwd(Q, K, V, S: int, T: int, head_past_mask=None, sm_scale=None, q_pos0=0, kv_pos0=0,
                 out=None, lse=None, stream=None, seg_starts=None):
    """O [B,Lq,Hq,d] bf16 and LSE [B,Hq,Lq] fp32 (natural log) - one call of the C entry point `seg_attn_fwd`."""
    _need_cuda_bf16(Q, K, V)
    O = torch.empty_like(Q) if out is None else out
    LSE = torch.empty((Q.shape[0], Q.shape[2], Q.shape[1]), dtype=torch.float32, device=Q.device) if lse is None else lse
    p = params_for(Q, K, V, O, S, T, sm_scale, q_pos0, kv_pos0, seg_starts=seg_starts)
    m = _mask_arr(head_past_mask, p.Hkv)
    _check(lib().seg_attn_fwd(ctypes.byref(p), _ptr(Q), _ptr(K), _ptr(V), m.ctypes.data, _ptr(O), _ptr(LSE),
                              None, 0, _stream(stream)), "seg_attn_fwd")
    return O, LSE


def seg_attn_bwd(Q, K, V, O, LSE, dO, S: int, T: int, head_past_mask=None, sm_scale=None, q_pos0=0, kv_pos0=0,
                 workspace: Optional[torch.Tensor] = None, stream=None, flagged_tail_is_sg: bool = False,
                 detach_before: int = 0, seg_starts=None):
    """dQ, dK, dV (bf16) - one call of the C entry point `seg_attn_bwd`.  `flagged_tail_is_sg` selects the
    reading in which flagged heads read the carried tail forward-only as well; keys at global positions
    below `detach_before` are read forward-only (a window of segments whose incoming state is a constant)."""
    _need_cuda_bf16(Q, K, V, O, dO)
    if dO.stride() != O.stride():
        raise ValueError("dO must have the strides of O")
    dQ, dK, dV = torch.empty_like(Q), torch.empty_like(K), torch.empty_like(V)
    if dQ.stride() != Q.stride() or dK.stride() != K.stride() or dV.stride() != V.stride():
        raise ValueError("Q, K, V must be dense (non-overlapping) tensors")
    p = params_for(Q, K, V, O, S, T, sm_scale, q_pos0, kv_pos0, flagged_tail_is_sg, detach_before, seg_starts)
    m = _mask_arr(head_past_mask, p.Hkv)
    need = workspace_bytes(p, True)
    ws = torch.empty(max(need, 256), dtype=torch.uint8, device=Q.device) if workspace is None else workspace
    _check(lib().seg_attn_bwd(ctypes.byref(p), _ptr(Q), _ptr(K), _ptr(V), _ptr(O), _ptr(LSE), _ptr(dO),
                              m.ctypes.data, _ptr(dQ), _ptr(dK), _ptr(dV), ctypes.c_void_p(ws.data_ptr()),
                              ws.numel(), _stream(stream)), "seg_attn_bwd")
    return dQ, dK, dV


STATIC_MAX_ROWS = 1 << 20   # SEG_ATTN_STATIC_MAX_ROWS of the C header


def seg_attn_bwd_static(Q, K, V, O, LSE, dO, S: int, T: int, head_past_mask=None, sm_scale=None, q_pos0=0,
                        kv_pos0=0, out=None, stream=None):
    """dQ, dK, dV through the C entry point `seg_attn_bwd_static`: the backward for callers that cannot
    allocate device memory where it runs.  No workspace is passed and none is allocated - the row dots
    live in a fixed 4 MiB array inside the library, so B*Hq*Lq must not exceed STATIC_MAX_ROWS (larger
    problems raise SegAttnError, status 6).  Pass `out=(dQ, dK, dV)` to supply the gradient buffers too;
    otherwise they are the only tensors this wrapper creates.  Calls share the array: do not let two of
    them overlap on the GPU, and make the first call on a device outside any stream capture."""
    _need_cuda_bf16(Q, K, V, O, dO)
    if dO.stride() != O.stride():
        raise ValueError("dO must have the strides of O")
    dQ, dK, dV = (torch.empty_like(Q), torch.empty_like(K), torch.empty_like(V)) if out is None else out
    if dQ.stride() != Q.stride() or dK.stride() != K.stride() or dV.stride() != V.stride():
        raise ValueError("gradients must have the strides of Q, K, V")
    p = params_for(Q, K, V, O, S, T, sm_scale, q_pos0, kv_pos0)
    m = _mask_arr(head_past_mask, p.Hkv)
    _check(lib().seg_attn_bwd_static(ctypes.byref(p), _ptr(Q), _ptr(K), _ptr(V), _ptr(O), _ptr(LSE), _ptr(dO),
                                     m.ctypes.data, _ptr(dQ), _ptr(dK), _ptr(dV), _stream(stream)),
           "seg_attn_bwd_static")
    return dQ, dK, dV


def seg_attn_step_host(Q, K, V, dO, S: int, T: int, head_past_mask=None, sm_scale=None,
                       arena: Optional[torch.Tensor] = None, outs=None, stream=None):
    """Forward (+ backward if dO is given) with HOST bf16 tensors in, HOST tensors out, through the
    C entry point `seg_attn_step_host`; copies both ways happen inside the call."""
    for t in (Q, K, V) + ((dO,) if dO is not None else ()):
        if t.device.type != "cpu" or t.dtype != torch.bfloat16 or not t.is_contiguous():
            raise ValueError("host entry point takes contiguous bf16 CPU tensors")
    p = params_for(Q, K, V, Q, S, T, sm_scale)
    m = _mask_arr(head_past_mask, p.Hkv)
    need = int(lib().seg_attn_host_arena_bytes(ctypes.byref(p)))
    if arena is None:
        arena = torch.empty(need, dtype=torch.uint8, device="cuda")
    if outs is None:
        pin = torch.cuda.is_available()
        mk = lambda like: torch.empty(like.shape, dtype=like.dtype, pin_memory=pin)
        outs = {"O": mk(Q), "LSE": torch.empty((p.B, p.Hq, p.Lq), dtype=torch.float32, pin_memory=pin)}
        if dO is not None:
            outs.update(dQ=mk(Q), dK=mk(K), dV=mk(V))
    g = lambda k: _ptr(outs.get(k))
    _check(lib().seg_attn_step_host(ctypes.byref(p), _ptr(Q), _ptr(K), _ptr(V), _ptr(dO), m.ctypes.data,
                                    g("O"), g("LSE"), g("dQ"), g("dK"), g("dV"),
                                    ctypes.c_void_p(arena.data_ptr()), arena.numel(), _stream(stream)),
           "seg_attn_step_host")
    return outs


def gather_context(K_pool, V_pool, idx, K_seg, V_seg, stream=None):
    """[retrieved rows ; segment rows] for K and V - the C entry point `seg_attn_gather_context`.
    K_pool, V_pool [B, P, Hkv, d]; idx int32 [B, Hkv, R] (device); K_seg, V_seg [B, Lseg, Hkv, d]."""
    _need_cuda_bf16(K_pool, V_pool, K_seg, V_seg)
    if idx.dtype != torch.int32 or not idx.is_cuda or not idx.is_contiguous():
        raise ValueError("idx must be a contiguous int32 CUDA tensor")
    B, P, Hkv, d = K_pool.shape
    R, Lseg = idx.shape[2], K_seg.shape[1]
    if idx.shape[:2] != (B, Hkv) or K_seg.shape[0] != B or K_seg.shape[2:] != (Hkv, d):
        raise ValueError("shapes do not fit")
    if V_pool.stride() != K_pool.stride() or V_seg.stride() != K_seg.stride():
        raise ValueError("K and V must share strides")
    K_ctx = torch.empty((B, R + Lseg, Hkv, d), dtype=torch.bfloat16, device=K_pool.device)
    V_ctx = torch.empty_like(K_ctx)
    _check(lib().seg_attn_gather_context(B, Hkv, d, R, Lseg, P, _ptr(K_pool), _ptr(V_pool), _strides3(K_pool),
                                         _ptr(K_seg), _ptr(V_seg), _strides3(K_seg), _ptr(idx), _ptr(K_ctx),
                                         _ptr(V_ctx), _stream(stream)), "seg_attn_gather_context")
    return K_ctx, V_ctx


def rope_table(n_pos: int, d: int, base: float = 10000.0, device="cuda", stream=None) -> torch.Tensor:
    """fp32 [n_pos, d/2, 2] = (cos, sin) of pos * base^(-2i/d) - the C entry point `seg_rope_table`."""
    need = int(lib().seg_rope_table_bytes(n_pos, d))
    if need == 0 and n_pos != 0:
        raise SegAttnError(1, "seg_rope_table_bytes")
    table = torch.empty((n_pos, d // 2, 2), dtype=torch.float32, device=device)
    _check(lib().seg_rope_table(n_pos, d, float(base), _ptr(table), _stream(stream)), "seg_rope_table")
    return table


def rope_apply(X, table, pos0: int = 0, inverse: bool = False, out=None, stream=None):
    """Row r of X [B, L, H, d] rotated by position pos0 + r (back, with inverse) - the C entry point `seg_rope_apply`."""
    _need_cuda_bf16(X)
    Y = torch.empty_like(X) if out is None else out
    B, L, H, d = X.shape
    _check(lib().seg_rope_apply(B, L, H, d, _ptr(X), _strides3(X), _ptr(Y), _strides3(Y), pos0, int(bool(inverse)),
                                _ptr(table), table.shape[0], _stream(stream)), "seg_rope_apply")
    return Y


def gather_context_rope(K_pool, V_pool, idx, K_seg, V_seg, table, stream=None):
    """[retrieved rows ; segment rows] with the keys rotated at their re-indexed positions (retrieved row r at r,
    segment row t at R + t) and the values copied - the C entry point `seg_attn_gather_context_rope`."""
    _need_cuda_bf16(K_pool, V_pool, K_seg, V_seg)
    if idx.dtype != torch.int32 or not idx.is_cuda or not idx.is_contiguous():
        raise ValueError("idx must be a contiguous int32 CUDA tensor")
    B, P, Hkv, d = K_pool.shape
    R, Lseg = idx.shape[2], K_seg.shape[1]
    if idx.shape[:2] != (B, Hkv) or K_seg.shape[0] != B or K_seg.shape[2:] != (Hkv, d):
        raise ValueError("shapes do not fit")
    if V_pool.stride() != K_pool.stride() or V_seg.stride() != K_seg.stride():
        raise ValueError("K and V must share strides")
    K_ctx = torch.empty((B, R + Lseg, Hkv, d), dtype=torch.bfloat16, device=K_pool.device)
    V_ctx = torch.empty_like(K_ctx)
    _check(lib().seg_attn_gather_context_rope(B, Hkv, d, R, Lseg, P, _ptr(K_pool), _ptr(V_pool), _strides3(K_pool),
                                              _ptr(K_seg), _ptr(V_seg), _strides3(K_seg), _ptr(idx), _ptr(K_ctx),
                                              _ptr(V_ctx), _ptr(table), table.shape[0], _stream(stream)),
           "seg_attn_gather_context_rope")
    return K_ctx, V_ctx


class RetrievalParams(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in ("Lq_last", "window", "stride", "tail", "top_k", "n_anchors", "off_lo",
                                               "off_hi", "R")]


def retrieval_select(Q_last, K_pool, window, stride, tail, top_k, n_anchors, off_lo, off_hi, R, stream=None):
    """idx int32 [B, Hkv, R]: the positions a head retrieves from the pool - the C entry point
    `seg_retrieval_select`.  Q_last [B, Lq_last, Hq, d] contiguous, K_pool [B, P, Hkv, d]."""
    _need_cuda_bf16(Q_last, K_pool)
    if not Q_last.is_contiguous():
        raise ValueError("Q_last must be contiguous")
    B, Lq, Hq, d = Q_last.shape
    P, Hkv = K_pool.shape[1], K_pool.shape[2]
    r = RetrievalParams(Lq, window, stride, tail, top_k, n_anchors, off_lo, off_hi, R)
    need = int(lib().seg_retrieval_workspace_bytes(B, Hq, Hkv, d, P, ctypes.byref(r)))
    if need == 0:
        raise SegAttnError(1, "seg_retrieval_workspace_bytes")
    ws = torch.empty(need, dtype=torch.uint8, device=Q_last.device)
    idx = torch.empty((B, Hkv, R), dtype=torch.int32, device=Q_last.device)
    _check(lib().seg_retrieval_select(B, Hq, Hkv, d, P, _ptr(Q_last), _ptr(K_pool), _strides3(K_pool), ctypes.byref(r),
                                      _ptr(idx), ctypes.c_void_p(ws.data_ptr()), ws.numel(), _stream(stream)),
           "seg_retrieval_select")
    return idx


def profile_kernels(Q, K, V, dO, S: int, T: int, head_past_mask=None, sm_scale=None, iters: int = 5, stream=None):
    """Average milliseconds per launch of (forward, row dots, dQ pass, dK/dV pass), each timed on its own
    with CUDA events on the launching stream by the C entry point `seg_attn_profile_kernels`."""
    _need_cuda_bf16(Q, K, V, dO)
    O = torch.empty_like(Q)
    LSE = torch.empty((Q.shape[0], Q.shape[2], Q.shape[1]), dtype=torch.float32, device=Q.device)
    dQ, dK, dV = torch.empty_like(Q), torch.empty_like(K), torch.empty_like(V)
    p = params_for(Q, K, V, O, S, T, sm_scale)
    m = _mask_arr(head_past_mask, p.Hkv)
    ws = torch.empty(max(workspace_bytes(p, True), 256), dtype=torch.uint8, device=Q.device)
    ms = (ctypes.c_float * 4)()
    _check(lib().seg_attn_profile_kernels(ctypes.byref(p), _ptr(Q), _ptr(K), _ptr(V), _ptr(O), _ptr(LSE), _ptr(dO),
                                          m.ctypes.data, _ptr(dQ), _ptr(dK), _ptr(dV), ctypes.c_void_p(ws.data_ptr()),
                                          ws.numel(), iters, ctypes.byref(ms), _stream(stream)),
           "seg_attn_profile_kernels")
    return {"fwd": ms[0], "rowdot": ms[1], "dq": ms[2], "dkv": ms[3]}


class Prefill:
    """Streamed, memory-bounded prefill: wraps seg_prefill_create/step/reset/destroy.  The persistent
    state (the flagged heads' key/value pool and the other heads' tail) lives in one torch buffer."""

    def __init__(self, B, S, T, Hq, Hkv, d, max_len, head_past_mask=None, sm_scale=None, device="cuda"):
        p = Params()
        p.B, p.Lq, p.kv_len, p.Hq, p.Hkv, p.d, p.S, p.T = B, S, max_len, Hq, Hkv, d, S, T
        p.sm_scale = float(sm_scale if sm_scale is not None else d ** -0.5)
        p.q_stride = p.o_stride = (ctypes.c_int64 * 3)(S * Hq * d, Hq * d, d)
        p.k_stride = p.v_stride = (ctypes.c_int64 * 3)(S * Hkv * d, Hkv * d, d)
        self.params = p
        self.mask = _mask_arr(head_past_mask, Hkv)
        self.state_bytes = int(lib().seg_prefill_state_bytes(ctypes.byref(p), self.mask.ctypes.data))
        self.state = torch.empty(max(self.state_bytes, 256), dtype=torch.uint8, device=device)
        h = ctypes.c_void_p()
        _check(lib().seg_prefill_create(ctypes.byref(p), self.mask.ctypes.data, ctypes.c_void_p(self.state.data_ptr()),
                                        self.state.numel(), ctypes.byref(h)), "seg_prefill_create")
        self._h = h

    def step(self, Qseg, Kseg, Vseg, out=None, lse=None, stream=None):
        """The next segment: [B, Lseg, H, d] tensors with Lseg <= S (a view of a [B, S, H, d] buffer when B > 1, so
        that batch elements keep the strides given at creation) - `seg_prefill_step` / `seg_prefill_step_len`."""
        _need_cuda_bf16(Qseg, Kseg, Vseg)
        p = self.params
        Lseg = Qseg.shape[1]

        def fits(t, H):
            return (t.dim() == 4 and t.shape[0] == p.B and t.shape[1] == Lseg and t.shape[2] == H and t.shape[3] == p.d and
                    t.stride(3) == 1 and t.stride(2) == p.d and t.stride(1) == H * p.d and
                    (p.B == 1 or t.stride(0) == p.S * H * p.d))
        if not (1 <= Lseg <= p.S and fits(Qseg, p.Hq) and fits(Kseg, p.Hkv) and fits(Vseg, p.Hkv)):
            raise ValueError("segment tensors must be [B, Lseg <= S, H, d] with the strides of a contiguous [B, S, H, d]")
        if out is None:
            out = torch.empty((p.B, p.S, p.Hq, p.d), dtype=torch.bfloat16, device=Qseg.device)[:, :Lseg]
        if not fits(out, p.Hq):
            raise ValueError("out must be laid out like the query segment")
        LSE = torch.empty((p.B, p.Hq, Lseg), dtype=torch.float32, device=Qseg.device) if lse is None else lse
        if Lseg == p.S:
            _check(lib().seg_prefill_step(self._h, _ptr(Qseg), _ptr(Kseg), _ptr(Vseg), _ptr(out), _ptr(LSE),
                                          _stream(stream)), "seg_prefill_step")
        else:
            _check(lib().seg_prefill_step_len(self._h, Lseg, _ptr(Qseg), _ptr(Kseg), _ptr(Vseg), _ptr(out), _ptr(LSE),
                                              _stream(stream)), "seg_prefill_step_len")
        return out, LSE

    def step_bwd(self, Qseg, Oseg, LSEseg, dOseg, stream=None):
        """Backward of the segment stepped last: dQ [B,Lseg,Hq,d] and dK, dV [B,T+S,Hkv,d] for the key/value rows
        [T positions in front of the segment ; segment ; zeros] - the C entry point `seg_prefill_step_bwd`."""
        _need_cuda_bf16(Qseg, Oseg, dOseg)
        p = self.params
        Lseg = Qseg.shape[1]
        for t in (Qseg, Oseg, dOseg):
            if not (t.dim() == 4 and tuple(t.shape) == (p.B, Lseg, p.Hq, p.d) and t.stride(3) == 1 and t.stride(2) == p.d and
                    t.stride(1) == p.Hq * p.d and (p.B == 1 or t.stride(0) == p.S * p.Hq * p.d)):
                raise ValueError("segment tensors must be [B, Lseg, Hq, d] with the strides of a contiguous [B, S, Hq, d]")
        dQ = torch.empty((p.B, p.S, p.Hq, p.d), dtype=torch.bfloat16, device=Qseg.device)[:, :Lseg]
        dK = torch.empty((p.B, p.T + p.S, p.Hkv, p.d), dtype=torch.bfloat16, device=Qseg.device)
        dV = torch.empty_like(dK)
        need = int(lib().seg_prefill_bwd_workspace_bytes(self._h))
        if getattr(self, "_bwd_ws", None) is None or self._bwd_ws.numel() < need:
            self._bwd_ws = torch.empty(max(need, 256), dtype=torch.uint8, device=Qseg.device)
        _check(lib().seg_prefill_step_bwd(self._h, _ptr(Qseg), _ptr(Oseg), _ptr(LSEseg), _ptr(dOseg), _ptr(dQ), _ptr(dK),
                                          _ptr(dV), ctypes.c_void_p(self._bwd_ws.data_ptr()), self._bwd_ws.numel(),
                                          _stream(stream)), "seg_prefill_step_bwd")
        return dQ, dK, dV

    def reset(self):
        _check(lib().seg_prefill_reset(self._h), "seg_prefill_reset")

    def close(self):
        if getattr(self, "_h", None):
            lib().seg_prefill_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def poll_status(stream=None):
    _check(lib().seg_attn_poll_status(_stream(stream)), "seg_attn_poll_status")


def selftest_wait_timeout(stream=None):
    """Enqueue the kernel whose bounded wait runs out (C entry point `seg_attn_selftest_wait_timeout`);
    the next `poll_status` raises SegAttnError with status 4."""
    _check(lib().seg_attn_selftest_wait_timeout(_stream(stream)), "seg_attn_selftest_wait_timeout")


def launch_count() -> int:
    return int(lib().seg_attn_launch_count())


def count_pairs(B, Lq, Hq, Hkv, d, S, T, head_past_mask=None, kv_len=None, q_pos0=0, kv_pos0=0,
                flagged_tail_is_sg: bool = False, detach_before: int = 0, seg_starts=None):
    """(visible pairs, differentiable pairs, 128x128 forward tiles visited), summed over batch and query heads."""
    p = Params()
    p.B, p.Lq, p.kv_len, p.Hq, p.Hkv, p.d, p.S, p.T = B, Lq, Lq if kv_len is None else kv_len, Hq, Hkv, d, S, T
    p.q_pos0, p.kv_pos0, p.sm_scale = q_pos0, kv_pos0, 1.0
    p.flags = FLAG_FLAGGED_TAIL_SG if flagged_tail_is_sg else 0
    p.detach_before = detach_before
    set_seg_starts(p, seg_starts)
    m = _mask_arr(head_past_mask, Hkv)
    a, b, c = ctypes.c_int64(), ctypes.c_int64(), ctypes.c_int64()
    _check(lib().seg_attn_count_pairs(ctypes.byref(p), m.ctypes.data, ctypes.byref(a), ctypes.byref(b),
                                      ctypes.byref(c)), "seg_attn_count_pairs")
    return a.value, b.value, c.value

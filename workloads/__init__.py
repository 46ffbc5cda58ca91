"""Seeded synthetic inputs shaped like the paper's long-context workloads.

This module holds NO attention arithmetic: it only draws tensors and head flags.  Both the
CUDA path's tests/benchmark and the CPU oracle's tests take their inputs from here, so the
two sides see identical bits.

Shapes follow the paper's experimental set-up (32 query heads, head dimension 128, segment
length in the thousands, a carried tail of a few hundred positions, contexts from 4K to 128K
tokens; Appendix F "Implementation details") and the five benchmark configurations of this
repository.  All values are drawn N(0,1) in fp32 and rounded to bf16; the softmax scale
1/sqrt(d) is passed to the attention call, not folded into the data.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Dict, Optional

import numpy as np
import torch


@dataclass(frozen=True)
class Workload:
    name: str
    B: int
    L: int
    Hq: int
    Hkv: int
    d: int
    S: int
    T: int
    past_frac: float = 0.0      # fraction of KV heads flagged for stop-gradient access to older KV
    outlier_frac: float = 0.0   # fraction of (batch, position, KV head) key rows redrawn with outlier_std
    outlier_std: float = 5.0
    seed: int = 0
    backward: bool = True
    streamed: bool = False

    @property
    def sm_scale(self) -> float:
        return 1.0 / float(np.sqrt(self.d))

    def with_(self, **kw) -> "Workload":
        return replace(self, **kw)


# The five configurations (index = configuration number - 1).  Configuration 5 is a sweep;
# `sweep()` expands it.
CONFIGS = (
    Workload("cfg1_tiny", B=1, L=2048, Hq=4, Hkv=4, d=64, S=512, T=128, past_frac=0.0, seed=0),
    Workload("cfg2_gqa16k", B=2, L=16384, Hq=32, Hkv=8, d=128, S=2048, T=512, past_frac=0.25, seed=0),
    Workload("cfg3_outlier32k", B=1, L=32768, Hq=32, Hkv=8, d=128, S=4096, T=1024, past_frac=0.5,
             outlier_frac=0.01, outlier_std=5.0, seed=0),
    Workload("cfg4_prefill128k", B=1, L=131072, Hq=32, Hkv=8, d=128, S=8192, T=2048, past_frac=0.25,
             seed=0, backward=False, streamed=True),
    Workload("cfg5_sweep64k", B=1, L=65536, Hq=64, Hkv=8, d=128, S=4096, T=1024, past_frac=0.25, seed=0),
)


def sweep():
    """Configuration 5: S x T (T <= S) x past fraction, 24 workloads."""
    out = []
    for S in (1024, 4096, 16384):
        for T in (256, 1024, 4096):
            if T > S:
                continue
            for frac in (0.0, 0.25, 1.0):
                out.append(CONFIGS[4].with_(name="cfg5_S%d_T%d_f%g" % (S, T, frac), S=S, T=T, past_frac=frac))
    return out


def head_past_mask(Hkv: int, frac: float, seed: int) -> np.ndarray:
    """u8[Hkv]; round(frac*Hkv) heads picked by a seeded permutation (an arbitrary, not contiguous, subset)."""
    n = int(round(frac * Hkv))
    m = np.zeros(Hkv, dtype=np.uint8)
    if n > 0:
        m[np.sort(np.random.default_rng(seed).permutation(Hkv)[:n])] = 1
    return m


def _normal_bf16(shape, gen: torch.Generator, device, std: float = 1.0, chunk_rows: int = 1 << 14):
    """N(0, std^2) drawn in fp32 and rounded to bf16, generated in slabs along dim 1 to bound memory."""
    out = torch.empty(shape, dtype=torch.bfloat16, device=device)
    L = shape[1]
    for r0 in range(0, L, chunk_rows):
        r1 = min(L, r0 + chunk_rows)
        slab = torch.randn((shape[0], r1 - r0) + tuple(shape[2:]), generator=gen, device=device, dtype=torch.float32)
        if std != 1.0:
            slab *= std
        out[:, r0:r1] = slab.to(torch.bfloat16)
    return out


def make_inputs(w: Workload, device: str = "cpu", with_dO: Optional[bool] = None,
                rows: Optional[slice] = None) -> Dict[str, object]:
    """Q ``[B,L,Hq,d]``, K, V ``[B,L,Hkv,d]`` (and dO like Q) as bf16 tensors on `device`, plus the
    head flag array.  The draw depends only on (workload, device type); `rows` is not a way to
    subsample (the whole tensor is always drawn)."""
    dev = torch.device(device)
    gen = torch.Generator(device=dev)
    gen.manual_seed(1000003 * w.seed + 12345)
    Q = _normal_bf16((w.B, w.L, w.Hq, w.d), gen, dev)
    K = _normal_bf16((w.B, w.L, w.Hkv, w.d), gen, dev)
    V = _normal_bf16((w.B, w.L, w.Hkv, w.d), gen, dev)
    if w.outlier_frac > 0:
        sel = torch.rand((w.B, w.L, w.Hkv), generator=gen, device=dev) < w.outlier_frac
        big = _normal_bf16((w.B, w.L, w.Hkv, w.d), gen, dev, std=w.outlier_std)
        K = torch.where(sel[..., None], big, K)
        del big
    out = {"Q": Q, "K": K, "V": V, "mask": head_past_mask(w.Hkv, w.past_frac, w.seed)}
    if w.backward if with_dO is None else with_dO:
        out["dO"] = _normal_bf16((w.B, w.L, w.Hq, w.d), gen, dev)
    return out


def to_f64(t: torch.Tensor) -> np.ndarray:
    """bf16/fp32 tensor (any device) -> numpy float64 holding exactly the same values."""
    return t.detach().to("cpu", torch.float64).numpy()

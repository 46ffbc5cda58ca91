"""Profiling case for `ncu`: a few forward + backward steps (or streamed-prefill steps) of one workload,
one launch of each kernel per step.  Not the benchmark: nothing is timed here.

    python profile_case.py [--steps 1] [--B 1] [--L 8192] [--S 2048] [--T 512] [--past-frac 0.25] [--Hq 32] [--d 128]
    python profile_case.py --config 3                  # one of the benchmark configurations 1-5
    python profile_case.py --sweep cfg5_S1024_T256_f0  # a point of the configuration-5 sweep
    python profile_case.py --prefill --L 32768 --S 8192 --T 2048   # streamed prefill, L/S steps
    python profile_case.py --retrieval                 # select + gather (+ rotation) at a 128K pool

The default (B = 1, L = 8192) keeps inputs above the 126 MB L2 and far below a GB, the size meant for
captures with many passes; the benchmark-size workloads are for one-pass metrics only.
"""
from __future__ import annotations

import argparse

import torch

import workloads
import paper_2605_11744_b200 as sa


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--steps", type=int, default=1)
    ap.add_argument("--B", type=int, default=1)
    ap.add_argument("--L", type=int, default=8192)
    ap.add_argument("--S", type=int, default=2048)
    ap.add_argument("--T", type=int, default=512)
    ap.add_argument("--Hq", type=int, default=32)
    ap.add_argument("--Hkv", type=int, default=8)
    ap.add_argument("--d", type=int, default=128)
    ap.add_argument("--past-frac", type=float, default=0.25)
    ap.add_argument("--config", type=int, default=0)
    ap.add_argument("--sweep", default="")
    ap.add_argument("--prefill", action="store_true")
    ap.add_argument("--retrieval", action="store_true")
    args = ap.parse_args()
    if args.config:
        w = workloads.CONFIGS[args.config - 1]
    elif args.sweep:
        w = {p.name: p for p in workloads.sweep()}[args.sweep]
    else:
        w = workloads.Workload("profile_case", B=args.B, L=args.L, Hq=args.Hq, Hkv=args.Hkv, d=args.d, S=args.S, T=args.T,
                               past_frac=args.past_frac, seed=0)
    if args.retrieval:
        # the long-range channel of one segment at a 128K pool: select, gather with re-indexed rotation, rotate Q
        B, P, Hq, Hkv, d, S, R = 1, 131072, 8, 2, 128, 4096, 512
        gen = torch.Generator(device="cuda").manual_seed(3)
        mk = lambda *s: torch.randn(*s, device="cuda", generator=gen).bfloat16()
        Kp, Vp, Ks, Vs, Q, Ql = mk(B, P, Hkv, d), mk(B, P, Hkv, d), mk(B, S, Hkv, d), mk(B, S, Hkv, d), mk(B, S, Hq, d), mk(B, 48, Hq, d)
        table = sa.rope_table(R + S, d)
        for _ in range(args.steps):
            idx = sa.retrieval_select(Ql, Kp, 16, 8, 8, 16, 8, 32, 31, R)
            sa.gather_context(Kp, Vp, idx, Ks, Vs)
            sa.gather_context_rope(Kp, Vp, idx, Ks, Vs, table)
            sa.rope_apply(Q, table, pos0=R)
        sa.poll_status()
        print("profile_case ok: retrieval at a pool of %d positions, %d KV heads" % (P, Hkv))
        return
    if args.prefill:
        mask = workloads.head_past_mask(w.Hkv, w.past_frac, w.seed)
        gen = torch.Generator(device="cuda").manual_seed(1)
        mk = lambda H: torch.randn(w.B, w.S, H, w.d, device="cuda", generator=gen).bfloat16()
        q, k, v = mk(w.Hq), mk(w.Hkv), mk(w.Hkv)
        pf = sa.Prefill(w.B, w.S, w.T, w.Hq, w.Hkv, w.d, w.L, mask, w.sm_scale)
        for _ in range(args.steps):
            pf.reset()
            for _i in range(w.L // w.S):
                pf.step(q, k, v)
        sa.poll_status()
        pf.close()
        print("profile_case ok: streamed prefill, %d steps of %d rows" % (w.L // w.S, w.S))
        return
    x = workloads.make_inputs(w, device="cuda")
    for _ in range(args.steps):
        O, LSE = sa.seg_attn_fwd(x["Q"], x["K"], x["V"], w.S, w.T, x["mask"], w.sm_scale)
        if w.backward:
            sa.seg_attn_bwd(x["Q"], x["K"], x["V"], O, LSE, x["dO"], w.S, w.T, x["mask"], w.sm_scale)
    sa.poll_status()
    vis, dif, tiles = sa.count_pairs(w.B, w.L, w.Hq, w.Hkv, w.d, w.S, w.T, x["mask"])
    print("profile_case ok: %s pairs_visible=%d pairs_diff=%d fwd_tiles=%d" % (w.name, vis, dif, tiles))


if __name__ == "__main__":
    main()

"""Small profiling case: one forward + backward step on a mid-size workload whose inputs exceed
the 126 MB L2 but stay well under a GB, meant to be run under `ncu` (one launch of each kernel).

    python -m paper_2605_11744_b200.profile_case [--steps 1] [--L 8192] [--S 2048] [--T 512]
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
    ap.add_argument("--past-frac", type=float, default=0.25)
    args = ap.parse_args()
    w = workloads.Workload("profile_case", B=args.B, L=args.L, Hq=32, Hkv=8, d=128, S=args.S, T=args.T,
                           past_frac=args.past_frac, seed=0)
    x = workloads.make_inputs(w, device="cuda")
    for _ in range(args.steps):
        O, LSE = sa.seg_attn_fwd(x["Q"], x["K"], x["V"], w.S, w.T, x["mask"], w.sm_scale)
        sa.seg_attn_bwd(x["Q"], x["K"], x["V"], O, LSE, x["dO"], w.S, w.T, x["mask"], w.sm_scale)
    sa.poll_status()
    vis, dif, tiles = sa.count_pairs(w.B, w.L, w.Hq, w.Hkv, w.d, w.S, w.T, x["mask"])
    print("profile_case ok: pairs_visible=%d pairs_diff=%d fwd_tiles=%d" % (vis, dif, tiles))


if __name__ == "__main__":
    main()

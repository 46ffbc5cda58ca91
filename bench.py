#!/usr/bin/env python
"""Benchmark of the segment-level attention hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--config I]

One "step" is one pass of the whole training-shape hot path over one batch of synthetic
input: forward (O, LSE), row dots, dQ pass, dK/dV pass.  The metric is attention TFLOP/s over
unmasked work only: fwd 4*d*pairs_visible + bwd 10*d*pairs_diff + 6*d*pairs_sg.  Prints ONE
JSON line on rank 0.  With N > 1 every rank runs an independent replica of the same workload
on its own GPU (the path does not shard; there is no collective on the data path).

`--impl reference` times the fp64 CPU oracle on the host cores on a bounded sample of the same
workload (there is no reference implementation of this paper to install).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import workloads  # noqa: E402

METRIC = "segmented-attention fwd+bwd TFLOP/s (unmasked work only)"
UNIT = "TFLOP/s"

# DRAM traffic per launch (dram__bytes_read.sum + dram__bytes_write.sum) of each kernel on the
# benchmark workload, taken from the ncu captures summarised under profiles/; None = not captured.
NCU_TRAFFIC_BYTES = {
    ("cfg2_gqa16k", "fwd"): 641431168,
    ("cfg2_gqa16k", "dq"): 929728256,
    ("cfg2_gqa16k", "dkv"): 800741376,
    ("cfg3_outlier32k", "fwd"): 828632192,
    ("cfg3_outlier32k", "dq"): 1199171072,
    ("cfg3_outlier32k", "dkv"): 801214208,
    ("cfg5_S1024_T256_f0", "fwd"): 2398129920,
    ("cfg5_S1024_T256_f0", "dq"): 3496404608,
    ("cfg5_S1024_T256_f0", "dkv"): 2771600896,
}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"bf16": float(p["bf16_tflops"]), "bf16_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                "hbm": float(p["hbm_gbs"]), "source": "measured"}
    return {"bf16": 1590.0, "bf16_sustained": 1400.0, "hbm": 6650.0, "source": "fallback"}


def flop_model(w, mask, count_pairs):
    vis, dif, tiles = count_pairs(w.B, w.L, w.Hq, w.Hkv, w.d, w.S, w.T, mask)
    sg = vis - dif
    return {
        "pairs_visible": vis, "pairs_diff": dif, "pairs_sg": sg, "fwd_tiles": tiles,
        "fwd": 4.0 * w.d * vis,
        "bwd": 10.0 * w.d * dif + 6.0 * w.d * sg,
        "dq": 6.0 * w.d * vis,                 # S, dP and dQ products over every visible pair
        "dkv": 4.0 * w.d * dif,                # dK and dV products; the recomputed S^T, dP^T are not counted
        "fwd_issued": 4.0 * w.d * tiles * 128 * 128,
    }


def config_of(w, mask, pairs_visible, pairs_diff, world):
    """The `config` object of the JSON line: the same keys and values for both arms."""
    flops = 4.0 * w.d * pairs_visible
    if w.backward:
        flops += 10.0 * w.d * pairs_diff + 6.0 * w.d * (pairs_visible - pairs_diff)
    return {"workload": w.name, "B": w.B, "L": w.L, "Hq": w.Hq, "Hkv": w.Hkv, "d": w.d, "S": w.S, "T": w.T,
            "past_frac": w.past_frac, "flagged_kv_heads": [int(i) for i in np.nonzero(mask)[0]],
            "passes": "fwd+bwd" if w.backward else "fwd", "l2": "inputs larger than L2 (no flush)",
            "parallelism": "replicas" if world > 1 else "single GPU",
            "pairs_visible": int(pairs_visible), "pairs_diff": int(pairs_diff), "flops_per_step": flops}


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples taken while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, cuda_ordinal):
        # nvidia-smi numbers GPUs physically, CUDA numbers the visible ones: select by UUID so that the
        # samples come from the GPU that is timed
        try:
            self.gpu_id = "GPU-" + str(torch.cuda.get_device_properties(cuda_ordinal).uuid)
        except Exception:
            self.gpu_id = str(cuda_ordinal)
        self.proc = None
        self.file = None

    def start(self):
        try:
            self.file = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
            self.proc = subprocess.Popen(["nvidia-smi", "-i", self.gpu_id, "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=self.file, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.file.flush()
        self.file.seek(0)
        sm, mx, reasons, power = [], [], set(), []
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for ln in self.file.read().splitlines():
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                mx.append(float(f[2]))
                power.append(float(f[3]))
            except ValueError:
                continue
            for name, val in zip(names, f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        try:
            os.unlink(self.file.name)
        except OSError:
            pass
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm),
                       power_w_max=max(power))
        return out


def oracle_sample(w, x, seg_lo=1, n_seg=2):
    """Oracle forward + backward on a bounded sample of the workload: the last batch element, one
    flagged and one unflagged KV head with their query heads, the queries of `n_seg` consecutive
    segments against all earlier keys.  Returns (seconds, algorithmic FLOPs of the sample, cores, text)."""
    import oracle
    g = w.Hq // w.Hkv
    mask = x["mask"]
    picks = []
    for want in (1, 0):
        idx = [c for c in range(w.Hkv) if int(mask[c] != 0) == want]
        if idx:
            picks.append(idx[len(idx) // 2])
    n_seg = max(1, min(n_seg, w.L // w.S))
    seg_lo = min(seg_lo, max(0, w.L // w.S - n_seg))
    r0, r1 = seg_lo * w.S, min(w.L, (seg_lo + n_seg) * w.S)
    b = w.B - 1
    flops, secs = 0.0, 0.0
    for c in picks:
        hq = slice(c * g, (c + 1) * g)
        Q = workloads.to_f64(x["Q"][b:b + 1, r0:r1, hq])
        K = workloads.to_f64(x["K"][b:b + 1, :r1, c:c + 1])
        V = workloads.to_f64(x["V"][b:b + 1, :r1, c:c + 1])
        m = [int(mask[c])]
        vis, dif = oracle.count_pairs(1, r1 - r0, g, 1, w.S, w.T, m, Lk=r1, q_pos0=r0)
        t0 = time.perf_counter()
        oracle.fwd(Q, K, V, w.S, w.T, m, scale=w.sm_scale, q_pos0=r0)
        flops += 4.0 * w.d * vis
        if w.backward:
            dO = workloads.to_f64(x["dO"][b:b + 1, r0:r1, hq])
            oracle.bwd(Q, K, V, dO, w.S, w.T, m, scale=w.sm_scale, q_pos0=r0)
            flops += 10.0 * w.d * dif + 6.0 * w.d * (vis - dif)
        secs += time.perf_counter() - t0
    text = ("batch %d, KV heads %s (one flagged, one not, with their %d query heads each), queries of segments "
            "%d..%d against keys [0,%d), fwd%s" % (b, picks, g, seg_lo, seg_lo + n_seg - 1, r1, "+bwd" if w.backward else ""))
    return secs, flops, oracle.num_threads(), text


def run_reference(args, w):
    """The reference arm: the CPU oracle, as it stands, on a bounded sample per step.  Nothing of the
    CUDA library is imported or loaded in this arm."""
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if rank != 0:
        return
    import oracle
    x = workloads.make_inputs(w)
    times, flops, cores, text = [], 0.0, 1, ""
    for i in range(args.warmup + args.steps):
        s, flops, cores, text = oracle_sample(w, x, n_seg=1 if w.L // w.S < 4 else 2)
        if i >= args.warmup:
            times.append(s)
    total = sum(times)
    val = flops * len(times) / total / 1e12
    vis, dif = oracle.count_pairs(w.B, w.L, w.Hq, w.Hkv, w.S, w.T, x["mask"])
    line = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * total / len(times), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": config_of(w, x["mask"], vis, dif, world),
        "note": "fp64 CPU oracle on host cores; each step is the bounded sample named in cpu_baseline",
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": text},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    assert "paper_2605_11744_b200" not in sys.modules, "the reference arm must not load the CUDA library"
    print(json.dumps(line), flush=True)


def measure_prefill(sa, peaks):
    """Configuration 4: streamed 128K prefill, peak memory and throughput (forward only)."""
    w = workloads.CONFIGS[3]
    mask = workloads.head_past_mask(w.Hkv, w.past_frac, w.seed)
    fm = flop_model(w, mask, sa.count_pairs)
    gen = torch.Generator(device="cuda").manual_seed(1234)
    mk = lambda H: torch.randn(w.B, w.S, H, w.d, device="cuda", dtype=torch.float32, generator=gen).bfloat16()
    O = torch.empty(w.B, w.S, w.Hq, w.d, device="cuda", dtype=torch.bfloat16)
    LSE = torch.empty(w.B, w.Hq, w.S, device="cuda", dtype=torch.float32)
    q, k, v = mk(w.Hq), mk(w.Hkv), mk(w.Hkv)
    step_bytes = sum(t.numel() * t.element_size() for t in (q, k, v, O, LSE))
    torch.cuda.synchronize()
    torch.cuda.empty_cache()
    torch.cuda.reset_peak_memory_stats()
    base = torch.cuda.memory_allocated() - step_bytes     # count the per-step segment buffers, not the RNG scratch
    pf = sa.Prefill(w.B, w.S, w.T, w.Hq, w.Hkv, w.d, w.L, mask, w.sm_scale)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ms = []
    for rep in range(3):
        pf.reset()
        torch.cuda.synchronize()
        e0.record()
        for i in range(w.L // w.S):
            pf.step(q, k, v, out=O, lse=LSE)     # same segment tensors each step: contents do not affect the work
        e1.record()
        torch.cuda.synchronize()
        ms.append(e0.elapsed_time(e1))
    sa.poll_status()
    peak = torch.cuda.max_memory_allocated() - base
    pf.close()
    full = w.B * w.L * (2 * w.Hq + 2 * w.Hkv) * w.d * 2 + w.B * w.Hq * w.L * 4
    t = min(ms) / 1e3
    return {"workload": w.name, "peak_prefill_GB": peak / 1e9, "state_GB": pf.state_bytes / 1e9,
            "full_resident_GB": full / 1e9, "ratio": full / peak, "ms": min(ms),
            "tflops": fm["fwd"] / t / 1e12, "frac_of_bf16_peak": fm["fwd"] / t / 1e12 / peaks["bf16"]}


def measure_retrieval(sa, peaks, P=131072, iters=20):
    """Selection step of the retrieval operator at a 128K pool, two long-range KV heads (configuration 4's), the
    constants of the tests (48 last queries, 7 summaries, top 16 each, 8 anchors, R = 512): HBM-bound, one read
    of the pool keys is the algorithmic traffic."""
    B, Hq, Hkv, d, R = 1, 8, 2, 128, 512
    gen = torch.Generator(device="cuda").manual_seed(7)
    mk = lambda *s: torch.randn(*s, device="cuda", generator=gen).bfloat16()
    Kp, Ql = mk(B, P, Hkv, d), mk(B, 48, Hq, d)
    args = (16, 8, 8, 16, 8, 32, 31, R)
    for _ in range(3):
        sa.retrieval_select(Ql, Kp, *args)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(iters):
        sa.retrieval_select(Ql, Kp, *args)
    e1.record()
    torch.cuda.synchronize()
    sa.poll_status()
    ms = e0.elapsed_time(e1) / iters
    nbytes = B * Hkv * P * d * 2
    gbs = nbytes / (ms / 1e3) / 1e9
    return {"pool_positions": P, "kv_heads": Hkv, "R": R, "ms": ms, "algorithmic_bytes": nbytes, "GBps": gbs,
            "frac_of_hbm": gbs / peaks["hbm"], "bound": "hbm", "launches_per_call": 4}


OTHER_WORKLOADS = ("cfg3_outlier32k", "cfg5_S1024_T256_f0", "cfg5_S4096_T1024_f0.25", "cfg5_S16384_T4096_f1")


def measure_other_workloads(sa, peaks, iters):
    """The larger forward + backward workloads in the same run: per-kernel CUDA-event times with inputs resident
    in HBM, and the whole-step throughput over unmasked work they add up to.  Compact: one entry per workload."""
    by_name = {w.name: w for w in list(workloads.CONFIGS) + workloads.sweep()}
    out = {}
    for name in OTHER_WORKLOADS:
        w = by_name[name]
        x = workloads.make_inputs(w, device="cuda")
        fm = flop_model(w, x["mask"], sa.count_pairs)
        per = sa.profile_kernels(x["Q"], x["K"], x["V"], x["dO"], w.S, w.T, x["mask"], w.sm_scale, iters=iters)
        sa.poll_status()
        ms = per["fwd"] + per["rowdot"] + per["dq"] + per["dkv"]
        tf = (fm["fwd"] + fm["bwd"]) / (ms / 1e3) / 1e12
        out[name] = {"ms_per_step": round(ms, 3), "tflops": round(tf, 1), "frac_of_bf16_peak": round(tf / peaks["bf16"], 3),
                     "flops_per_step": fm["fwd"] + fm["bwd"],
                     "ms": {k: round(per[k], 3) for k in ("fwd", "rowdot", "dq", "dkv")}}
        del x
        torch.cuda.empty_cache()
    return out


def max_over_ranks(value, world, device):
    """The slowest rank's figure (every multi-GPU number is the maximum over ranks).  The only
    collective of a multi-GPU run; it is outside the data path."""
    if world <= 1:
        return float(value)
    import torch.distributed as dist
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_value(flops_per_rank_step, world, seconds_per_step):
    """Whole-job throughput of `world` independent replicas in TFLOP/s."""
    return world * flops_per_rank_step / seconds_per_step / 1e12


def run_ours(args, w):
    import torch.distributed as dist
    import paper_2605_11744_b200 as sa

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the product path has no CPU fallback")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    peaks = load_peaks()
    x = workloads.make_inputs(w, device="cuda")
    mask = x["mask"]
    fm = flop_model(w, mask, sa.count_pairs)
    flops_step = fm["fwd"] + (fm["bwd"] if w.backward else 0.0)
    Q, K, V = x["Q"], x["K"], x["V"]
    dO = x.get("dO")
    O = torch.empty_like(Q)
    LSE = torch.empty(w.B, w.Hq, w.L, dtype=torch.float32, device="cuda")
    p = sa.params_for(Q, K, V, O, w.S, w.T, w.sm_scale)
    ws = torch.empty(max(sa.workspace_bytes(p, True), 256), dtype=torch.uint8, device="cuda")

    def step():
        sa.seg_attn_fwd(Q, K, V, w.S, w.T, mask, w.sm_scale, out=O, lse=LSE)
        if w.backward:
            return sa.seg_attn_bwd(Q, K, V, O, LSE, dO, w.S, w.T, mask, w.sm_scale, workspace=ws)
        return None

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        step()
    sa.poll_status()
    barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    launches0 = sa.launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record()
    for _ in range(args.steps):
        step()
    e1.record()
    barrier()
    ms_total = e0.elapsed_time(e1)
    launches = sa.launch_count() - launches0
    sa.poll_status()
    ms_total = max_over_ranks(ms_total, world, "cuda")

    # end to end through the host-buffer entry point: pinned host tensors in, pinned host tensors out
    host = {k: x[k].cpu().pin_memory() for k in ("Q", "K", "V") + (("dO",) if w.backward else ())}
    arena = torch.empty(int(sa.lib().seg_attn_host_arena_bytes(__import__("ctypes").byref(p))), dtype=torch.uint8,
                        device="cuda")
    outs = sa.seg_attn_step_host(host["Q"], host["K"], host["V"], host.get("dO"), w.S, w.T, mask, w.sm_scale, arena=arena)
    e2e_steps = max(2, min(args.steps, 5))
    barrier()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        sa.seg_attn_step_host(host["Q"], host["K"], host["V"], host.get("dO"), w.S, w.T, mask, w.sm_scale, arena=arena,
                              outs=outs)
    torch.cuda.synchronize()
    e2e_s = time.perf_counter() - t0
    e2e_s = max_over_ranks(e2e_s, world, "cuda")
    h2d = sum(t.numel() * t.element_size() for t in host.values())
    d2h = sum(t.numel() * t.element_size() for t in outs.values())
    clocks = sampler.stop() if rank == 0 else {}
    del host, outs, arena

    line = None
    if rank == 0:
        # per-kernel durations (CUDA events on the launching stream, each kernel on its own)
        per = sa.profile_kernels(Q, K, V, dO if dO is not None else Q, w.S, w.T, mask, w.sm_scale, iters=max(3, min(args.steps, 10)))
        kern_flops = {"fwd": fm["fwd"], "dq": fm["dq"], "dkv": fm["dkv"]}
        share = {k: per[k] for k in ("fwd", "rowdot", "dq", "dkv")}
        dom = max(("fwd", "dq", "dkv"), key=lambda k: per[k])
        achieved = kern_flops[dom] / (per[dom] / 1e3) / 1e12
        hbm_rowdot = (2 * w.B * w.L * w.Hq * w.d * 2 + w.B * w.L * w.Hq * 4) / (per["rowdot"] / 1e3) / 1e9
        roofline = {
            "bound": "tensor", "kernel": {"fwd": "seg_attn_fwd_kernel", "dq": "seg_attn_bwd_dq_kernel",
                                          "dkv": "seg_attn_bwd_dkv_kernel"}[dom],
            "achieved": achieved, "peak": peaks["bf16"], "unit": "TFLOP/s", "frac": achieved / peaks["bf16"],
            "peak_sustained": peaks["bf16_sustained"], "frac_sustained": achieved / peaks["bf16_sustained"],
            "peak_source": peaks["source"], "traffic": NCU_TRAFFIC_BYTES.get((w.name, dom)),
            "ms_per_launch": share,
            "per_kernel_tflops": {k: kern_flops[k] / (per[k] / 1e3) / 1e12 for k in kern_flops},
            "rowdot_GBps": hbm_rowdot, "rowdot_frac_of_hbm": hbm_rowdot / peaks["hbm"],
            "issued_over_algorithmic_fwd": fm["fwd_issued"] / fm["fwd"],
        }
        xs = {k: (v.cpu() if torch.is_tensor(v) else v) for k, v in x.items()}
        secs, sflops, cores, text = oracle_sample(w, xs, n_seg=1 if w.L // w.S < 4 else 2)
        cpu = {"value": sflops / secs / 1e12, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": text,
               "seconds": secs}
        prefill = None
        if not args.no_prefill:
            prefill = measure_prefill(sa, peaks)
        retrieval = None if args.no_prefill else measure_retrieval(sa, peaks)
        others = None
        if not args.no_others and world == 1 and w.name == "cfg2_gqa16k":
            del Q, K, V, dO, O, LSE, x
            torch.cuda.empty_cache()
            others = measure_other_workloads(sa, peaks, iters=3)
        t_step = ms_total / args.steps / 1e3
        value = aggregate_value(flops_step, world, t_step)
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
            "ms_per_step": ms_total / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": config_of(w, mask, fm["pairs_visible"], fm["pairs_diff"], world),
            "frac_of_bf16_peak": value / world / peaks["bf16"],
            "frac_of_bf16_sustained": value / world / peaks["bf16_sustained"],
            "roofline": roofline, "cpu_baseline": cpu,
            "e2e": {"value": aggregate_value(flops_step, world, e2e_s / e2e_steps), "unit": UNIT, "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h, "steps": e2e_steps},
            "gpu_launches": launches, "clocks": clocks, "prefill": prefill, "retrieval": retrieval, "configs": others,
        }
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    if line is not None:
        print(json.dumps(line), flush=True)


def run_table(args):
    """One JSON line per workload (configurations 1-3 and the 24 points of sweep 5): per-kernel CUDA-event
    times with inputs resident in HBM, and the throughput over unmasked work they give.  The source of
    the repository's table of measured results; not the benchmark line."""
    import paper_2605_11744_b200 as sa
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the product path has no CPU fallback")
    torch.cuda.set_device(0)
    peaks = load_peaks()
    for w in list(workloads.CONFIGS[:3]) + workloads.sweep():
        x = workloads.make_inputs(w, device="cuda")
        fm = flop_model(w, x["mask"], sa.count_pairs)
        per = sa.profile_kernels(x["Q"], x["K"], x["V"], x["dO"], w.S, w.T, x["mask"], w.sm_scale, iters=max(3, min(args.steps, 10)))
        sa.poll_status()
        bwd_ms = per["rowdot"] + per["dq"] + per["dkv"]
        tot_ms = per["fwd"] + bwd_ms
        tf = lambda flops, ms: flops / (ms / 1e3) / 1e12
        print(json.dumps({
            "workload": w.name, "B": w.B, "L": w.L, "Hq": w.Hq, "Hkv": w.Hkv, "d": w.d, "S": w.S, "T": w.T,
            "past_frac": w.past_frac, "pairs_visible": fm["pairs_visible"], "pairs_diff": fm["pairs_diff"],
            "tflop_fwd": fm["fwd"] / 1e12, "tflop_bwd": fm["bwd"] / 1e12,
            "ms": {k: round(per[k], 4) for k in ("fwd", "rowdot", "dq", "dkv")},
            "tflops_fwd": tf(fm["fwd"], per["fwd"]), "tflops_bwd": tf(fm["bwd"], bwd_ms),
            "tflops_total": tf(fm["fwd"] + fm["bwd"], tot_ms),
            "frac_of_bf16_peak": tf(fm["fwd"] + fm["bwd"], tot_ms) / peaks["bf16"],
            "frac_of_bf16_sustained": tf(fm["fwd"] + fm["bwd"], tot_ms) / peaks["bf16_sustained"],
            "issued_over_algorithmic_fwd": fm["fwd_issued"] / fm["fwd"]}), flush=True)
        del x
        torch.cuda.empty_cache()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=2, help="benchmark configuration number (1-5); default 2")
    ap.add_argument("--no-prefill", action="store_true", help="skip the configuration-4 streamed prefill measurement")
    ap.add_argument("--no-others", action="store_true",
                    help="skip the per-kernel timings of configuration 3 and three sweep points (the `configs` key)")
    ap.add_argument("--table", action="store_true",
                    help="per-kernel timings of configurations 1-3 and the sweep, one JSON line each (not the benchmark line)")
    args = ap.parse_args()
    if args.table:
        run_table(args)
        return
    w = workloads.CONFIGS[args.config - 1]
    if args.impl == "reference":
        run_reference(args, w)
    else:
        run_ours(args, w)


if __name__ == "__main__":
    main()

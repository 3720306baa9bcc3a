#!/usr/bin/env python
"""Benchmark of the mHC-lite mixing hot path (forward + backward) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload cfg2]

One "step" is one pass of the whole path over one batch of synthetic tokens: mappings + stream
pre-mix, post/residual merge, the merge's backward, and the fused backward tail (the sublayer's
output y and its backward's du are inputs).  Rank r of an N-GPU run processes its own shard of
tokens (weak scaling, no data-path collective).  Prints one JSON line on rank 0.

--impl reference times the fp64 CPU oracle on the host cores (rank 0 only) on a bounded sample.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "mhclite_mixing_fwd_bwd_tokens_per_sec"
UNIT = "tokens/s"


def algorithmic_bytes_per_token(n: int, C: int) -> dict:
    """bf16 bytes each stage must move per token when x_l is read once per pass."""
    return {
        "pre_fwd": (2 * n + 2) * C,          # read x_l, write u
        "post_fwd": (4 * n + 2) * C,         # read x_l, y; write x_next
        "post_bwd": (4 * n + 4) * C,         # read g, x_l, y; write dy
        "tail_bwd": (6 * n + 2) * C,         # read du, x_l, g; write dx
    }


def kernel_bytes_per_token(n: int, C: int) -> dict:
    """Algorithmic bf16 bytes per token of each main kernel of the fused call sequence."""
    return {
        "proj_fwd": 2 * n * C,               # read x_l
        "act_premix": (2 * n + 2) * C,       # read x_l, write u
        "postres_fwd": (4 * n + 2) * C,      # read x_l, y; write x_next
        "postres_bwd": (4 * n + 4) * C,      # read g, x_l, y; write dy
        "tail_pre": (2 * n + 2) * C,         # read x_l, du
        "tail_mma": (6 * n + 2) * C,         # read du, x_l, g; write dx
    }


def ncu_traffic(kernel: str, workload: str, T: int):
    """DRAM bytes per launch of `kernel` from the committed ncu capture of this workload, or None when
    there is none or the kernel's source has changed since (profiles/dram_traffic_<workload>.txt:
    lines `kernel  tokens  dram_bytes  source_file  sha256_of_source`)."""
    import hashlib
    path = os.path.join(ROOT, "profiles", f"dram_traffic_{workload}.txt")
    if not os.path.exists(path):
        return None
    for line in open(path):
        f = line.split()
        if len(f) == 5 and f[0] == kernel:
            src = os.path.join(ROOT, "paper_2601_05732_b200", "csrc", f[3])
            if os.path.exists(src) and hashlib.sha256(open(src, "rb").read()).hexdigest() == f[4]:
                return float(f[2]) * T / float(f[1])
    return None


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        return float(json.load(open(p))["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


# ----------------------------------------------------------------------------------------------
class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "100",
                 "-i", str(gpu_index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.strip().splitlines():
            f = [s.strip() for s in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); smax.append(float(f[2]))
            except ValueError:
                continue
            for nm, v in zip(names, f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(smax) if smax else None, "reasons": sorted(reasons), "samples": len(sm)}


# ----------------------------------------------------------------------------------------------
def oracle_sample_tokens_per_sec(wl, sample_tokens: int, repeats: int = 1):
    """Times the fp64 oracle (as it stands) on `sample_tokens` tokens of the workload, fwd+bwd."""
    from oracle import mhclite_oracle as O
    from paper_2601_05732_b200 import synth
    inp = synth.make_layer_inputs(wl.n, wl.C, sample_tokens, wl.seed, bias_std=wl.bias_std, alpha=wl.alpha, w_std=wl.w_std)
    f = synth.bf16_bits_to_f64
    x, y, g, du = f(inp["x"]), f(inp["y"]), f(inp["g"]), f(inp["du"])
    W, b, al, ga = (inp[k].astype(np.float64) for k in ("W", "b", "alpha", "gain"))
    best = float("inf")
    for _ in range(repeats):
        t0 = time.perf_counter()
        O.layer_fwd(x, y, W, b, al, ga, 1e-6)
        if wl.backward:
            O.layer_bwd(x, y, W, b, al, ga, 1e-6, g, du)
        best = min(best, time.perf_counter() - t0)
    return sample_tokens / best, best


def blas_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = [d.get("num_threads", 1) for d in threadpool_info() if d.get("user_api") == "blas"]
        return max(n) if n else 1
    except Exception:
        return os.cpu_count() or 1


def run_reference(args, wl, rank):
    """The oracle arm: each step is a bounded sample of the workload on the host cores."""
    if rank != 0:
        return
    sample = min(wl.T, 2048)
    for _ in range(args.warmup):
        oracle_sample_tokens_per_sec(wl, sample)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_sample_tokens_per_sec(wl, sample)
    dt = time.perf_counter() - t0
    value = sample * args.steps / dt
    cores = blas_threads()
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": wl.name, "n": wl.n, "C": wl.C, "T": wl.T, "note": wl.note,
                   "sample": f"{sample} tokens per step (input generation included)"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": f"{sample} tokens of {wl.name} per step, fwd+bwd, numpy fp64"},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------------------------
def run_ours(args, wl, rank, world):
    import torch
    from paper_2601_05732_b200 import dist as D
    from paper_2601_05732_b200 import synth
    from paper_2601_05732_b200 import layer as L
    from paper_2601_05732_b200.binding import MhcLite, MhcLiteError

    local = int(os.environ.get("LOCAL_RANK", 0))
    # CPU baseline first (rank 0, single-GPU run only), before the first GPU call
    cpu_baseline = None
    if world == 1 and not args.no_cpu_baseline:
        sample = min(wl.T, args.cpu_sample)
        v, secs = oracle_sample_tokens_per_sec(wl, sample)
        cpu_baseline = {"value": v, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
                        "sample": f"{sample} tokens of {wl.name}, fwd+bwd, numpy fp64, {secs:.1f} s"}

    torch.cuda.set_device(local)
    dev = f"cuda:{local}"
    D.init(world, "nccl", dev)

    n, C, T = wl.n, wl.C, wl.T
    inp = synth.make_layer_inputs(n, C, T, wl.seed, bias_std=wl.bias_std, alpha=wl.alpha, w_std=wl.w_std,
                                  shard=D.shard_of(rank))
    ctx = MhcLite(n, C, local)
    P = L.LayerParams(inp["W"], inp["b"], inp["alpha"], inp["gain"], dev)
    B = L.LayerBuffers(ctx, T, "lite")
    x, y, g, du = (L.to_device_bf16(inp[k], dev) for k in ("x", "y", "g", "du"))
    eps = 1e-6

    fused = not args.unfused

    def step():
        L.pre_fwd(ctx, P, B, x, eps, fused)
        L.post_fwd(ctx, B, x, y)
        if wl.backward:
            L.post_bwd(ctx, B, x, y, g, fused)
            L.tail_bwd(ctx, P, B, x, g, du, eps, fused)

    def barrier():
        D.barrier(world)

    for _ in range(max(args.warmup, 3)):
        step()
    barrier()

    # One step's launches (all issued by the library through the C ABI) captured once in a CUDA graph and
    # replayed: the nine kernels of a step are short enough for launch gaps to show.  Falls back to plain
    # launches when the capture is refused.
    launches_per_step = ctx.kernel_launches()
    step()
    launches_per_step = ctx.kernel_launches() - launches_per_step
    run_step, launch_mode = step, "stream"
    if not args.no_graph:
        try:
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph):
                step()
            graph.replay()
            torch.cuda.synchronize()
            run_step, launch_mode = graph.replay, "cuda_graph"
        except Exception as exc:                  # noqa: BLE001 - any capture failure means plain launches
            print(f"bench.py: CUDA graph capture refused ({exc}); timing plain launches", file=sys.stderr)
            torch.cuda.synchronize()
    for _ in range(3):
        run_step()
    barrier()

    # ---- timed region: K steps, device time, max over ranks ------------------------------------
    sampler = ClockSampler(local) if rank == 0 else None
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record()
    for _ in range(args.steps):
        run_step()
    e1.record()
    barrier()
    ms = e0.elapsed_time(e1)
    launches = launches_per_step * args.steps
    # keep the GPU busy a little longer so that the sampler sees the loaded clocks even for short runs
    t_end = time.time() + 0.6
    while rank == 0 and time.time() < t_end:
        run_step()
    torch.cuda.synchronize()
    clocks = sampler.stop() if sampler else None
    ms = D.max_over_ranks(ms, world, dev)

    # ---- per-kernel device time (same launch configuration): CUDA events recorded by the library
    #      around each of its main kernels, on the launching stream
    ctx.set_kernel_timing(True)
    ksum = {k: 0.0 for k in ctx.KERNELS}
    stage_ev = []
    for _ in range(args.steps):
        evs = [torch.cuda.Event(enable_timing=True) for _ in range(5)]
        evs[0].record(); L.pre_fwd(ctx, P, B, x, eps, fused)
        evs[1].record(); L.post_fwd(ctx, B, x, y)
        evs[2].record()
        if wl.backward:
            L.post_bwd(ctx, B, x, y, g, fused)
            evs[3].record(); L.tail_bwd(ctx, P, B, x, g, du, eps, fused)
            evs[4].record()
        torch.cuda.synchronize()
        stage_ev.append(evs)
        for i, k in enumerate(ctx.KERNELS):
            if fused and (wl.backward or i < 3):
                try:
                    ksum[k] += ctx.kernel_time_ms(i)
                except MhcLiteError:            # kernel not on this configuration's path (e.g. n = 5 fallbacks)
                    pass
    ctx.set_kernel_timing(False)
    kernel_ms = {k: v / args.steps for k, v in ksum.items() if v > 0}
    names = ["pre_fwd", "post_fwd", "post_bwd", "tail_bwd"][: 4 if wl.backward else 2]
    stage_ms = {nm: sum(e[i].elapsed_time(e[i + 1]) for e in stage_ev) / len(stage_ev) for i, nm in enumerate(names)}

    # ---- end to end through the C ABI with host buffers ----------------------------------------
    e2e = None
    if not args.no_e2e:
        pin = lambda t: t.cpu().pin_memory()
        hx, hy, hg, hdu = pin(x), pin(y), pin(g), pin(du)
        hu, hxn, hdy, hdx = (torch.empty_like(t, device="cpu").pin_memory() for t in (B.u, B.x_next, B.dy, B.dx))
        run = lambda: ctx.step_host(hx, hy, hg, hdu, P.W, P.b, P.alpha, P.gain, eps, hu, hxn, hdy, hdx,
                                    B.dW, B.db, B.dalpha, B.dgain)
        k_e2e = max(3, min(args.steps, 10))
        for _ in range(2):
            run()
        barrier()
        a, b_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(k_e2e):
            run()
        b_.record()
        barrier()
        ms_e2e = a.elapsed_time(b_)
        ms_e2e = D.max_over_ranks(ms_e2e, world, dev)
        h2d = sum(t.numel() * 2 for t in (hx, hy, hg, hdu))
        d2h = sum(t.numel() * 2 for t in (hu, hxn, hdy, hdx))
        e2e = {"value": D.job_tokens_per_s(T, world, k_e2e, ms_e2e), "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "ms_per_step": ms_e2e / k_e2e}

    # ---- the mHC (20 Sinkhorn-Knopp iterations) path on the same shapes, for comparison --------
    sk20 = None
    if not args.no_sk and wl.backward and rank == 0:
        ski = synth.make_layer_inputs(n, C, T, wl.seed, bias_std=wl.bias_std, alpha=wl.alpha, w_std=wl.w_std,
                                      kind="sk", shard=D.shard_of(rank))
        Ps = L.LayerParams(ski["W"], ski["b"], ski["alpha"], ski["gain"], dev)
        Bs = L.LayerBuffers(ctx, T, "sk")

        def sk_step():
            L.pre_fwd(ctx, Ps, Bs, x, eps, True)
            L.post_fwd(ctx, Bs, x, y)
            L.post_bwd(ctx, Bs, x, y, g, True)
            L.tail_bwd(ctx, Ps, Bs, x, g, du, eps, True)

        for _ in range(3):
            sk_step()
        torch.cuda.synchronize()
        a, b_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(args.steps):
            sk_step()
        b_.record()
        torch.cuda.synchronize()
        ms_sk = a.elapsed_time(b_) / args.steps
        gap = torch.empty(T, device=dev); gap_l = torch.empty(T, device=dev)
        ctx.ds_gap(Bs.H_res, gap, None); ctx.ds_gap(B.H_res, gap_l, None)
        torch.cuda.synchronize()
        sk20 = {"tokens_per_s": T / (ms_sk * 1e-3), "ms_per_step": ms_sk, "iters": 20,
                "lite_over_sk20": ms_sk / (ms / args.steps) if world == 1 else None,
                "l1_gap_max_sk20": float(gap.max()), "l1_gap_max_lite": float(gap_l.max())}

    if rank == 0:
        peak, peak_kind = load_peaks()
        bpt = algorithmic_bytes_per_token(n, C)
        total_bytes = sum(bpt[k] for k in stage_ms) * T
        kb = kernel_bytes_per_token(n, C)
        if kernel_ms:
            dom = max(kernel_ms, key=kernel_ms.get)
            achieved = kb[dom] * T / (kernel_ms[dom] * 1e-3) / 1e9
        else:                                   # un-fused sequence: report the slowest call
            dom = max(stage_ms, key=stage_ms.get)
            achieved = bpt[dom] * T / (stage_ms[dom] * 1e-3) / 1e9
        roofline = {"bound": "hbm", "kernel": dom, "achieved": achieved, "peak": peak, "peak_kind": peak_kind,
                    "unit": "GB/s", "frac": achieved / peak, "traffic": ncu_traffic(dom, wl.name, T),
                    "whole_step_gbs": total_bytes / (ms / args.steps * 1e-3) / 1e9,
                    "whole_step_frac_of_8TBs": total_bytes / (ms / args.steps * 1e-3) / 8e12,
                    "whole_step_frac_of_measured": total_bytes / (ms / args.steps * 1e-3) / 1e9 / peak,
                    "kernel_ms": kernel_ms,
                    "kernel_gbs": {k: kb[k] * T / (v * 1e-3) / 1e9 for k, v in kernel_ms.items()},
                    "stage_ms": stage_ms,
                    "stage_gbs": {k: bpt[k] * T / (v * 1e-3) / 1e9 for k, v in stage_ms.items()}}
        line = {
            "metric": METRIC, "value": D.job_tokens_per_s(T, world, args.steps, ms), "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16 in/out, f32 accumulate",
            "data": "synthetic",
            "config": {"workload": wl.name, "n": n, "C": C, "T_per_gpu": T, "passes": "fwd+bwd" if wl.backward else "fwd", "calls": "fused" if fused else "unfused", "launch": launch_mode,
                       "note": wl.note, "l2": "inputs larger than L2 (working set %.0f MB)" % (total_bytes / 1e6)},
            "clocks": clocks, "e2e": e2e, "gpu_launches": launches, "roofline": roofline,
            "cpu_baseline": cpu_baseline, "sk20_comparison": sk20,
        }
        print(json.dumps(line), flush=True)
    D.shutdown()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg2")
    ap.add_argument("--T", type=int, default=0, help="override the token count of the workload")
    ap.add_argument("--cpu-sample", type=int, default=16384, help="tokens of the oracle's timed sample")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-sk", action="store_true", help="skip the SK-20 comparison path")
    ap.add_argument("--unfused", action="store_true", help="time the un-fused call sequence (six entry points)")
    ap.add_argument("--no-graph", action="store_true", help="time plain stream launches instead of a CUDA graph of one step")
    args = ap.parse_args()

    from paper_2601_05732_b200 import synth
    import dataclasses
    wl = synth.WORKLOADS[args.workload]
    if args.T:
        wl = dataclasses.replace(wl, T=args.T)
    rank = int(os.environ.get("RANK", 0))
    world = int(os.environ.get("WORLD_SIZE", 1))
    if args.impl == "reference":
        run_reference(args, wl, rank)
        return
    if world != args.gpus:
        if args.gpus != 1 or world != 1:
            print(f"bench.py: --gpus {args.gpus} needs torchrun with {args.gpus} ranks (WORLD_SIZE={world})", file=sys.stderr)
            sys.exit(2)
    run_ours(args, wl, rank, world)


if __name__ == "__main__":
    main()

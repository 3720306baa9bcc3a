#!/usr/bin/env python
"""Benchmark of the mHC-lite mixing hot path (forward + backward) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload cfg5] [--T tokens]

One "step" is one pass of the whole path over one batch of synthetic tokens: mappings + stream
pre-mix, post/residual merge, the merge's backward, and the fused backward tail (the sublayer's
output y and its backward's du are inputs).  Rank r of an N-GPU run processes its own shard of
tokens (weak scaling, no data-path collective).  Prints one JSON line on rank 0.

The default workload is the largest single-GPU one (cfg5: n = 4, C = 4096, T = 131072).  On one GPU the
line also carries a `workloads` table: cfg1 (forward only), cfg2, the 24-layer stack cfg3, cfg4a, cfg4b, the subset variant of the
paper's Section 5 on the cfg4b shape (24 sampled permutations of 120) and the cfg5 token sweep, each with the
mHC-lite step and (full tables) the in-library SK-20 step timed the same way (CUDA-graph replay).

--impl reference times the fp64 CPU oracle on the host cores (rank 0 only) on a bounded sample.
With --gpus N > 1 and no torchrun environment the script starts its own N ranks.
"""
from __future__ import annotations

import argparse
import dataclasses
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
NOMINAL_HBM_GBS = 8000.0
# CUDA symbol behind each timing slot of the library, by path (for reading the ncu launch list)
KERNEL_SYMBOL = {"proj_fwd": "proj_fwd_tc_k", "act_premix": "lite_act_premix_t_k / lite_act_premix_k<5>",
                 "postres_fwd": "postres_fwd_k", "postres_bwd": "postres_bwd_k",
                 "tail_pre": "lite_tailpre_w_k / lite_tailpre_k<5>", "tail_dx": "tail_ftc_k (n<=4) / tail_dx_tc_k (n=5)"}


def algorithmic_bytes_per_token(n: int, C: int, backward: bool = True) -> dict:
    """bf16 bytes each stage must move per token when x_l is read once per pass."""
    b = {
        "pre_fwd": (2 * n + 2) * C,          # read x_l, write u
        "post_fwd": (4 * n + 2) * C,         # read x_l, y; write x_next
    }
    if backward:
        b["post_bwd"] = (4 * n + 4) * C      # read g, x_l, y; write dy
        b["tail_bwd"] = (6 * n + 2) * C      # read du, x_l, g; write dx
    return b


def kernel_bytes_per_token(n: int, C: int) -> dict:
    """Algorithmic bf16 bytes per token of each main kernel of the fused call sequence."""
    return {
        "proj_fwd": 2 * n * C,               # read x_l
        "act_premix": (2 * n + 2) * C,       # read x_l, write u
        "postres_fwd": (4 * n + 2) * C,      # read x_l, y; write x_next
        "postres_bwd": (4 * n + 4) * C,      # read g, x_l, y; write dy
        "tail_pre": (2 * n + 2) * C,         # read x_l, du
        "tail_dx": (6 * n + 2) * C,          # read du, x_l, g; write dx
    }


def ncu_traffic(kernel: str, workload: str, T: int):
    """DRAM bytes per launch of `kernel` from the committed ncu capture of this workload, scaled to T tokens
    by the tokens processed, or None when there is none or the kernel's source has changed since
    (profiles/dram_traffic_<workload>.txt: lines `kernel  tokens  dram_bytes  source_file  sha256_of_source`)."""
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


_TRAFFIC_KERNELS = {"proj_fwd": ("proj_fwd_tc_k", "proj_tc.cu"), "act_premix": ("lite_act_premix_t_k", "act_kernels.cu"),
                    "postres_fwd": ("postres_fwd_k", "stream_kernels.cu"), "postres_bwd": ("postres_bwd_k", "stream_kernels.cu"),
                    "tail_pre": ("lite_tailpre_w_k", "act_kernels.cu"), "tail_dx": ("tail_ftc_k", "tail_ftc.cu")}


def write_ncu_traffic(workload: str, T: int, csv_path: str) -> None:
    """Writes profiles/dram_traffic_<workload>.txt from an `ncu --csv` log of one step of this workload at T tokens that
    holds dram__bytes_read.sum and dram__bytes_write.sum (the first launch of each kernel counts), with the hash of
    each kernel's source so that a later edit voids the figure.  Needs no GPU."""
    import csv
    import hashlib
    rows = list(csv.reader(open(csv_path)))
    head = next(r for r in rows if "Kernel Name" in r and "Metric Name" in r)
    k_i, m_i, v_i = head.index("Kernel Name"), head.index("Metric Name"), head.index("Metric Value")
    seen = {}
    for r in rows:
        if len(r) <= v_i or not r[0].isdigit():
            continue
        name = r[k_i].replace("void ", "").replace("mhcl::", "").split("<")[0].split("(")[0]
        seen.setdefault(name, {}).setdefault(r[m_i], float(r[v_i].replace(",", "")))
    lines = []
    for key, (kname, src) in _TRAFFIC_KERNELS.items():
        if kname not in seen:
            continue
        b = int(seen[kname]["dram__bytes_read.sum"] + seen[kname]["dram__bytes_write.sum"])
        h = hashlib.sha256(open(os.path.join(ROOT, "paper_2601_05732_b200", "csrc", src), "rb").read()).hexdigest()
        lines.append(f"{key} {T} {b} {src} {h}")
    out = os.path.join(ROOT, "profiles", f"dram_traffic_{workload}.txt")
    open(out, "w").write("\n".join(lines) + "\n")
    print("\n".join(lines))


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
def oracle_sample_tokens_per_sec(wl, sample_tokens: int, threads: int | None = None):
    """Times the fp64 oracle (as it stands) on `sample_tokens` tokens of the workload, fwd+bwd; with
    `threads` the numerical library underneath numpy is held to that many threads."""
    from oracle import mhclite_oracle as O
    from paper_2601_05732_b200 import synth
    inp = synth.make_layer_inputs(wl.n, wl.C, sample_tokens, wl.seed, bias_std=wl.bias_std, alpha=wl.alpha, w_std=wl.w_std)
    f = synth.bf16_bits_to_f64
    x, y, g, du = f(inp["x"]), f(inp["y"]), f(inp["g"]), f(inp["du"])
    W, b, al, ga = (inp[k].astype(np.float64) for k in ("W", "b", "alpha", "gain"))

    def run(k=None):
        t0 = time.perf_counter()
        O.layer_fwd(x[:k], y[:k], W, b, al, ga, 1e-6)
        if wl.backward:
            O.layer_bwd(x[:k], y[:k], W, b, al, ga, 1e-6, g[:k], du[:k])
        return time.perf_counter() - t0

    run(min(64, sample_tokens))          # untimed: first-call costs of the numerical library (thread pool, page faults)

    if threads is None:
        secs = run()
    else:
        from threadpoolctl import threadpool_limits
        with threadpool_limits(limits=threads):
            secs = run()
    return sample_tokens / secs, secs


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
    sample = min(wl.T, 2048 if wl.n * wl.C <= 8192 else 1024)
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
class Timer:
    """K steps per repeat, device time from CUDA events on the launching stream, barrier and synchronize on
    both sides of every repeat, the slowest rank's time; repeats until `min_total_ms` of timed work."""

    def __init__(self, torch, D, world, dev):
        self.torch, self.D, self.world, self.dev = torch, D, world, dev

    def repeat(self, run_step, steps):
        t = self.torch
        e0, e1 = t.cuda.Event(enable_timing=True), t.cuda.Event(enable_timing=True)
        self.D.barrier(self.world)
        e0.record()
        for _ in range(steps):
            run_step()
        e1.record()
        self.D.barrier(self.world)
        return self.D.max_over_ranks(e0.elapsed_time(e1), self.world, self.dev)

    def measure(self, run_step, steps, min_total_ms=500.0, max_repeats=25):
        first = self.repeat(run_step, steps)
        reps = int(min(max_repeats, max(3, math.ceil(min_total_ms / max(first, 1e-3)))))
        ms = [first] + [self.repeat(run_step, steps) for _ in range(reps - 1)]
        per = [m / steps for m in ms]
        return {"ms_per_step": statistics.median(per), "ms_min": min(per), "ms_max": max(per), "repeats": len(per),
                "timed_ms_total": sum(ms)}


def capture(torch, step, use_graph=True):
    """One step's launches (all issued by the library through the C ABI) captured once in a CUDA graph and
    replayed; plain launches when the capture is refused."""
    if use_graph:
        try:
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph):
                step()
            graph.replay()
            torch.cuda.synchronize()
            return graph.replay, "cuda_graph", graph
        except Exception as exc:                  # noqa: BLE001 - any capture failure means plain launches
            print(f"bench.py: CUDA graph capture refused ({exc}); timing plain launches", file=sys.stderr)
            torch.cuda.synchronize()
    return step, "stream", None


class Pool:
    """Device-resident synthetic activations.  The headline workload's tensors are drawn exactly as the
    parity tests draw them (synth.make_layer_inputs); the other rows of the table view the leading
    elements of the same buffers in their own shapes (iid N(0,1) bf16 either way)."""

    def __init__(self, torch, L, inp, dev, repeat=1):
        self.torch = torch
        rep = lambda t: t if repeat == 1 else t.repeat(repeat, *([1] * (t.dim() - 1)))
        self.x, self.y, self.g, self.du = (rep(L.to_device_bf16(inp[k], dev)) for k in ("x", "y", "g", "du"))

    def views(self, T, n, C):
        need_big, need_small = T * n * C, T * C
        if need_big > self.x.numel() or need_small > self.y.numel():
            raise ValueError("pool too small for this shape")
        v = lambda t, k, shape: t.reshape(-1)[:k].view(*shape)
        return (v(self.x, need_big, (T, n, C)), v(self.y, need_small, (T, C)), v(self.g, need_big, (T, n, C)),
                v(self.du, need_small, (T, C)))


def time_layer_case(mods, timer, ctx, wl, T, kind, acts, dev, steps, min_total_ms, use_graph=True, fused=True,
                    n_res=None):
    """Times one single-layer workload (kind 'lite' or 'sk') on the given activations; n_res = K when the context
    holds a subset of K permutations."""
    torch, L, synth = mods["torch"], mods["L"], mods["synth"]
    p = synth.make_layer_params(wl.n, wl.C, wl.seed, bias_std=wl.bias_std, alpha=wl.alpha, w_std=wl.w_std, kind=kind,
                                n_res=n_res)
    P = L.LayerParams(p["W"], p["b"], p["alpha"], p["gain"], dev)
    B = L.LayerBuffers(ctx, T, kind)
    x, y, g, du = acts

    def step():
        L.pre_fwd(ctx, P, B, x, 1e-6, fused)
        L.post_fwd(ctx, B, x, y)
        if wl.backward:
            L.post_bwd(ctx, B, x, y, g, fused)
            L.tail_bwd(ctx, P, B, x, g, du, 1e-6, fused)

    for _ in range(3):
        step()
    torch.cuda.synchronize()
    l0 = ctx.kernel_launches()
    step()
    launches = ctx.kernel_launches() - l0
    run_step, mode, graph = capture(torch, step, use_graph)
    for _ in range(3):
        run_step()
    res = timer.measure(run_step, steps, min_total_ms)
    res.update(launch=mode, launches_per_step=launches)
    return res, P, B, step, graph


def time_stack_case(mods, timer, ctx, wl, acts, dev, steps, min_total_ms, use_graph=True):
    """The 24-layer stack (cfg3): library calls of all layers forward, then all layers backward.  The
    sublayer's y_l and du_l are inputs (the stand-in sublayer of the parity test is harness work, not timed)."""
    torch, L, synth = mods["torch"], mods["L"], mods["synth"]
    x0, y, g_top, du = acts
    T, Ld = x0.shape[0], wl.layers
    Ps, Bs = [], []
    for l in range(Ld):
        p = synth.make_layer_params(wl.n, wl.C, wl.seed, layer=l, bias_std=wl.bias_std, alpha=wl.alpha, w_std=wl.w_std)
        Ps.append(L.LayerParams(p["W"], p["b"], p["alpha"], p["gain"], dev))
        Bs.append(L.LayerBuffers(ctx, T, "lite"))

    def step():
        L.stack_fwd(ctx, Ps, Bs, x0, lambda l, u: y, 1e-6)
        L.stack_bwd(ctx, Ps, Bs, g_top, lambda l, u, dy: du, 1e-6)

    for _ in range(2):
        step()
    torch.cuda.synchronize()
    l0 = ctx.kernel_launches()
    step()
    launches = ctx.kernel_launches() - l0
    run_step, mode, graph = capture(torch, step, use_graph)
    for _ in range(2):
        run_step()
    res = timer.measure(run_step, steps, min_total_ms)
    res.update(launch=mode, launches_per_step=launches, layers=Ld)
    return res


def rates(n, C, T, ms, peak, layers=1, backward=True):
    bpt = sum(algorithmic_bytes_per_token(n, C, backward).values())
    gbs = bpt * T * layers / (ms * 1e-3) / 1e9
    out = {"tokens_per_s": T / (ms * 1e-3), "algorithmic_gbs": gbs, "frac_of_measured_peak": gbs / peak,
           "frac_of_8TBs": gbs / NOMINAL_HBM_GBS}
    if layers > 1:
        out["token_layers_per_s"] = T * layers / (ms * 1e-3)
    return out


# ----------------------------------------------------------------------------------------------
def run_ours(args, wl, rank, world):
    import torch
    from paper_2601_05732_b200 import dist as D
    from paper_2601_05732_b200 import synth
    from paper_2601_05732_b200 import layer as L
    from paper_2601_05732_b200.binding import MhcLite, MhcLiteError
    mods = {"torch": torch, "L": L, "synth": synth}

    local = int(os.environ.get("LOCAL_RANK", 0))
    # CPU baseline first (rank 0, single-GPU run only), before the first GPU call
    cpu_baseline = None
    if world == 1 and not args.no_cpu_baseline:
        heavy = wl.n * wl.C > 8192
        sample = min(wl.T, args.cpu_sample or (8192 if heavy else 16384))
        v, secs = oracle_sample_tokens_per_sec(wl, sample)
        s1 = min(wl.T, 1024 if heavy else 2048)
        v1, secs1 = oracle_sample_tokens_per_sec(wl, s1, threads=1)
        cpu_baseline = {"value": v, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
                        "sample": f"{sample} tokens of {wl.name}, fwd+bwd, numpy fp64, {secs:.1f} s",
                        "one_core": {"value": v1, "unit": UNIT, "cores": 1,
                                     "sample": f"{s1} tokens of {wl.name}, fwd+bwd, numpy fp64, {secs1:.1f} s"}}

    torch.cuda.set_device(local)
    dev = f"cuda:{local}"
    D.init(world, "nccl", dev)
    if world > 1:
        print(f"bench.py: rank {rank}/{world} on {dev} ({torch.cuda.get_device_name(local)}), NCCL "
              f"{'.'.join(str(v) for v in torch.cuda.nccl.version())}, communicator over {world} ranks", file=sys.stderr, flush=True)

    n, C, T = wl.n, wl.C, wl.T
    peak, peak_kind = load_peaks()
    # One rank draws its T tokens exactly as the parity tests do.  Several ranks share the host's cores, so each draws
    # a block of its own shard's stream and repeats it to T tokens (the values do not enter the timing).
    T_draw = T if world == 1 else min(T, 16384)
    inp = synth.make_layer_inputs(n, C, T_draw, wl.seed, bias_std=wl.bias_std, alpha=wl.alpha, w_std=wl.w_std,
                                  shard=D.shard_of(rank))
    pool = Pool(torch, L, inp, dev, repeat=(T + T_draw - 1) // T_draw)
    ctxs = {}

    def ctx_for(n_, C_, K_=None, seed_=0):
        """One context per shape; K_: a context that holds a sampled subset of K_ permutations (paper Section 5)."""
        if (n_, C_, K_) not in ctxs:
            c_ = MhcLite(n_, C_, local)
            if K_:
                c_.set_perm_subset(torch.from_numpy(synth.sample_perm_table(n_, K_, seed_)).to(dev))
            ctxs[(n_, C_, K_)] = c_
        return ctxs[(n_, C_, K_)]

    ctx = ctx_for(n, C, args.permutations or None, wl.seed)
    timer = Timer(torch, D, world, dev)
    fused = not args.unfused
    steps = args.steps
    warm = max(args.warmup, 3)
    acts = pool.views(T, n, C)
    x, y, g, du = acts

    if wl.layers > 1:
        # a stack of layers as the headline (--workload cfg3): the library calls of all layers, nothing else
        sampler = ClockSampler(local) if rank == 0 else None
        r = time_stack_case(mods, timer, ctx, wl, acts, dev, max(2, steps // 4), args.min_ms, not args.no_graph)
        clocks = sampler.stop() if sampler else None
        ctx.device_status()
        if rank == 0:
            rt = rates(n, C, T, r["ms_per_step"], peak, layers=wl.layers)
            print(json.dumps({
                "metric": METRIC, "value": D.job_tokens_per_s(T, world, 1, r["ms_per_step"]), "unit": UNIT, "n_gpus": world,
                "steps": max(2, steps // 4), "warmup": warm, "ms_per_step": r["ms_per_step"], "repeats": r["repeats"],
                "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16 in/out, f32 accumulate",
                "data": "synthetic",
                "config": {"workload": wl.name, "n": n, "C": C, "T_per_gpu": T, "layers": wl.layers, "passes": "fwd+bwd",
                           "launch": r["launch"], "note": wl.note + "; library calls only, y_l and du_l are inputs"},
                "clocks": clocks, "e2e": None, "gpu_launches": r["launches_per_step"] * max(2, steps // 4) * r["repeats"],
                "roofline": {"bound": "hbm", "kernel": "whole stack", "achieved": rt["algorithmic_gbs"], "peak": peak,
                             "peak_kind": peak_kind, "unit": "GB/s", "frac": rt["frac_of_measured_peak"], "traffic": None},
                "token_layers_per_s": rt["token_layers_per_s"], "cpu_baseline": cpu_baseline}), flush=True)
        D.shutdown()
        return

    # ---- headline: K steps per repeat, device time, max over ranks -----------------------------
    sampler = ClockSampler(local) if rank == 0 else None
    # (the warm-up steps run inside time_layer_case: three plain, one counted, the capture, three replays)
    head, P, B, step, graph = time_layer_case(mods, timer, ctx, wl, T, "lite", acts, dev, steps, args.min_ms,
                                              use_graph=not args.no_graph, fused=fused, n_res=args.permutations or None)
    clocks = sampler.stop() if sampler else None
    ms = head["ms_per_step"]
    launch_mode = head["launch"]

    # ---- per-kernel device time (plain launches): CUDA events recorded by the library around each of its
    #      main kernels, on the launching stream
    ctx.set_kernel_timing(True)
    ksum = {k: 0.0 for k in ctx.KERNELS}
    stage_ev = []
    ksteps = min(steps, 10)
    for _ in range(ksteps):
        evs = [torch.cuda.Event(enable_timing=True) for _ in range(5)]
        evs[0].record(); L.pre_fwd(ctx, P, B, x, 1e-6, fused)
        evs[1].record(); L.post_fwd(ctx, B, x, y)
        evs[2].record()
        if wl.backward:
            L.post_bwd(ctx, B, x, y, g, fused)
            evs[3].record(); L.tail_bwd(ctx, P, B, x, g, du, 1e-6, fused)
            evs[4].record()
        torch.cuda.synchronize()
        stage_ev.append(evs)
        for i, k in enumerate(ctx.KERNELS):
            if fused and (wl.backward or i < 3):
                try:
                    ksum[k] += ctx.kernel_time_ms(i)
                except MhcLiteError:            # kernel not on this configuration's path
                    pass
    ctx.set_kernel_timing(False)
    kernel_ms = {k: v / ksteps for k, v in ksum.items() if v > 0}
    names = ["pre_fwd", "post_fwd", "post_bwd", "tail_bwd"][: 4 if wl.backward else 2]
    stage_ms = {nm: sum(e[i].elapsed_time(e[i + 1]) for e in stage_ev) / len(stage_ev) for i, nm in enumerate(names)}
    ctx.device_status()

    # ---- the mHC (20 Sinkhorn-Knopp iterations) path on the same shapes, timed the same way ----
    def sk_compare(ctx_, wl_, T_, acts_, ms_lite, B_lite=None):
        if args.no_sk or not wl_.backward:
            return None
        r, _, Bs, _, gr = time_layer_case(mods, timer, ctx_, wl_, T_, "sk", acts_, dev, steps, args.min_ms_table,
                                          use_graph=not args.no_graph)
        out = {"tokens_per_s": T_ / (r["ms_per_step"] * 1e-3), "ms_per_step": r["ms_per_step"], "iters": 20,
               "launch": r["launch"], "launches_per_step": r["launches_per_step"],
               "lite_over_sk20": r["ms_per_step"] / ms_lite}
        gap = torch.empty(T_, device=dev)
        ctx_.ds_gap(Bs.H_res, gap, None)
        out["l1_gap_max_sk20"], out["l1_gap_mean_sk20"] = float(gap.max()), float(gap.mean())
        if B_lite is not None:
            ctx_.ds_gap(B_lite.H_res, gap, None)
            out["l1_gap_max_lite"], out["l1_gap_mean_lite"] = float(gap.max()), float(gap.mean())
        del gr
        return out

    sk20 = sk_compare(ctx, wl, T, acts, ms, B) if world == 1 else None

    # ---- end to end through the C ABI with host buffers ----------------------------------------
    e2e = None
    if not args.no_e2e:
        def e2e_at(Te):
            pin = lambda a: torch.from_numpy(np.ascontiguousarray(a[:Te]).view(np.int16)).view(torch.bfloat16).pin_memory()
            hx, hy, hg, hdu = pin(inp["x"]), pin(inp["y"]), pin(inp["g"]), pin(inp["du"])
            hu, hxn, hdy, hdx = (torch.empty(s, dtype=torch.bfloat16).pin_memory()
                                 for s in ((Te, C), (Te, n, C), (Te, C), (Te, n, C)))
            run = lambda: ctx.step_host(hx, hy, hg, hdu, P.W, P.b, P.alpha, P.gain, 1e-6, hu, hxn, hdy, hdx,
                                        B.dW, B.db, B.dalpha, B.dgain)
            k = 3
            run()
            r = timer.measure(run, k, min_total_ms=0.0, max_repeats=3)
            h2d = sum(t.numel() * 2 for t in (hx, hy, hg, hdu))
            d2h = sum(t.numel() * 2 for t in (hu, hxn, hdy, hdx))
            return {"value": D.job_tokens_per_s(Te, world, 1, r["ms_per_step"]), "unit": UNIT, "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h, "ms_per_step": r["ms_per_step"], "tokens_per_step_per_gpu": Te,
                    "api": "mhclite_step_host (pinned host buffers in and out)"}
        try:
            e2e = e2e_at(T_draw)          # (several ranks: a block of tokens per rank; the ranks share the host's memory and PCIe)
        except (RuntimeError, MemoryError) as exc:     # host memory for 2 x 10 GB of pinned buffers refused
            print(f"bench.py: end-to-end run at T={T_draw} refused ({exc}); using T={T_draw // 4}", file=sys.stderr)
            e2e = e2e_at(T_draw // 4)
    del inp

    # ---- the other workloads (one GPU only): lite and SK-20 steps, same timing method ----------
    table = None
    if world == 1 and not args.no_table:
        table = []
        del B, graph
        torch.cuda.empty_cache()
        # (workload, T override, K): K = a sampled subset of K of the n! permutations (paper Section 5) on that shape
        rows = [("cfg1", None, None), ("cfg2", None, None), ("cfg3", None, None), ("cfg4a", None, None), ("cfg4b", None, None),
                ("cfg4b", None, 24)] + [("cfg5", t, None) for t in (4096, 8192, 16384, 32768, 65536, 131072)]
        for name, Tt, K in rows:
            w = synth.WORKLOADS[name]
            Tt = Tt or w.T
            if K:
                a = pool.views(Tt, w.n, w.C)
                c = ctx_for(w.n, w.C, K, w.seed)
                r, _, Bl, _, gr = time_layer_case(mods, timer, c, w, Tt, "lite", a, dev, steps, args.min_ms_table,
                                                  not args.no_graph, n_res=K)
                table.append({"workload": name, "n": w.n, "C": w.C, "T": Tt, "permutations": K,
                              "ms_per_step": r["ms_per_step"], "ms_min": r["ms_min"], "ms_max": r["ms_max"],
                              "repeats": r["repeats"], **rates(w.n, w.C, Tt, r["ms_per_step"], peak), "launch": r["launch"],
                              "launches_per_step": r["launches_per_step"], "sk20": None,
                              "note": "subset variant: Eq. (5) over %d sampled permutations of %d" % (K, math.factorial(w.n))})
                del Bl, gr
                c.device_status()
                torch.cuda.empty_cache()
                continue
            if name == wl.name and Tt == T:
                row = {"workload": name, "n": n, "C": C, "T": T, "ms_per_step": ms, **rates(n, C, T, ms, peak),
                       "launch": launch_mode, "sk20": sk20, "note": "the headline row"}
                table.append(row)
                continue
            try:
                a = pool.views(Tt, w.n, w.C)
            except ValueError:
                continue
            c = ctx_for(w.n, w.C)
            if w.layers > 1:
                r = time_stack_case(mods, timer, c, w, a, dev, max(2, steps // 4), args.min_ms_table, not args.no_graph)
                row = {"workload": name, "n": w.n, "C": w.C, "T": Tt, "layers": w.layers, "ms_per_step": r["ms_per_step"],
                       "ms_min": r["ms_min"], "ms_max": r["ms_max"], "repeats": r["repeats"],
                       **rates(w.n, w.C, Tt, r["ms_per_step"], peak, layers=w.layers), "launch": r["launch"],
                       "launches_per_step": r["launches_per_step"], "sk20": None,
                       "note": "library calls of 24 layers forward then backward; y_l, du_l are inputs"}
            else:
                r, _, Bl, _, gr = time_layer_case(mods, timer, c, w, Tt, "lite", a, dev, steps, args.min_ms_table,
                                                  not args.no_graph)
                row = {"workload": name, "n": w.n, "C": w.C, "T": Tt, "ms_per_step": r["ms_per_step"],
                       "ms_min": r["ms_min"], "ms_max": r["ms_max"], "repeats": r["repeats"],
                       **rates(w.n, w.C, Tt, r["ms_per_step"], peak, backward=w.backward), "launch": r["launch"],
                       "launches_per_step": r["launches_per_step"]}
                if not w.backward:
                    row["note"] = "forward only; 29 MB of tensors: fits L2, launch-bound (reported, not a roofline case)"
                row["sk20"] = sk_compare(c, w, Tt, a, r["ms_per_step"], Bl)
                del Bl, gr
            c.device_status()
            table.append(row)
            torch.cuda.empty_cache()

    if rank == 0:
        bpt = algorithmic_bytes_per_token(n, C, wl.backward)
        total_bytes = sum(bpt.values()) * T
        kb = kernel_bytes_per_token(n, C)
        if kernel_ms:
            dom = max(kernel_ms, key=kernel_ms.get)
            achieved = kb[dom] * T / (kernel_ms[dom] * 1e-3) / 1e9
        else:                                   # un-fused sequence: report the slowest call
            dom = max(stage_ms, key=stage_ms.get)
            achieved = bpt[dom] * T / (stage_ms[dom] * 1e-3) / 1e9
        step_gbs = total_bytes / (ms * 1e-3) / 1e9
        roofline = {"bound": "hbm", "kernel": dom, "kernel_symbol": KERNEL_SYMBOL.get(dom), "achieved": achieved,
                    "peak": peak, "peak_kind": peak_kind, "unit": "GB/s", "frac": achieved / peak,
                    "traffic": ncu_traffic(dom, wl.name, T),
                    "step": {"achieved": step_gbs, "frac": step_gbs / peak, "frac_of_8TBs": step_gbs / NOMINAL_HBM_GBS,
                             "note": "whole fwd+bwd step: algorithmic bytes (16n+10) C T over the timed step; "
                                     "roofline.frac above is the dominant kernel alone"},
                    "kernel_ms": kernel_ms,
                    "kernel_gbs": {k: kb[k] * T / (v * 1e-3) / 1e9 for k, v in kernel_ms.items()},
                    "stage_ms": stage_ms,
                    "stage_gbs": {k: bpt[k] * T / (v * 1e-3) / 1e9 for k, v in stage_ms.items()}}
        line = {
            "metric": METRIC, "value": D.job_tokens_per_s(T, world, 1, ms), "unit": UNIT, "n_gpus": world,
            "steps": steps, "warmup": warm, "ms_per_step": ms, "repeats": head["repeats"],
            "ms_per_step_min": head["ms_min"], "ms_per_step_max": head["ms_max"], "timed_ms_total": head["timed_ms_total"],
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16 in/out, f32 accumulate",
            "data": "synthetic" if world == 1 else f"synthetic ({T_draw} tokens drawn per rank, repeated to T)",
            "config": {"workload": wl.name, "n": n, "C": C, "T_per_gpu": T, "passes": "fwd+bwd" if wl.backward else "fwd",
                       "calls": "fused" if fused else "unfused", "launch": launch_mode, "note": wl.note,
                       **({"permutations": args.permutations} if args.permutations else {}),
                       "l2": "inputs larger than L2 (working set %.0f MB)" % (total_bytes / 1e6)},
            "clocks": clocks, "e2e": e2e, "gpu_launches": head["launches_per_step"] * steps * head["repeats"],
            "roofline": roofline, "cpu_baseline": cpu_baseline, "sk20_comparison": sk20, "workloads": table,
        }
        print(json.dumps(line), flush=True)
    D.shutdown()


def spawn_ranks(args_list, gpus):
    """Starts `gpus` ranks of this script under torch.distributed.run (one process per GPU, NCCL over
    NVLink for the barrier and the max-over-ranks time) and passes their exit code on."""
    import socket
    s = socket.socket(); s.bind(("127.0.0.1", 0)); port = s.getsockname()[1]; s.close()
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + args_list
    return subprocess.call(cmd)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg5")
    ap.add_argument("--T", type=int, default=0, help="override the token count of the workload")
    ap.add_argument("--layers", type=int, default=0, help="override the number of layers of a stack workload (cfg3)")
    ap.add_argument("--cpu-sample", type=int, default=0, help="tokens of the oracle's timed sample (0: by workload)")
    ap.add_argument("--min-ms", type=float, default=500.0, help="least timed work of the headline (repeats of K steps)")
    ap.add_argument("--min-ms-table", type=float, default=100.0, help="least timed work of each row of the table")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-sk", action="store_true", help="skip the SK-20 comparison path")
    ap.add_argument("--no-table", action="store_true", help="skip the table of the other workloads")
    ap.add_argument("--unfused", action="store_true", help="time the un-fused call sequence (six entry points)")
    ap.add_argument("--no-graph", action="store_true", help="time plain stream launches instead of a CUDA graph of one step")
    ap.add_argument("--permutations", type=int, default=0, metavar="K",
                    help="headline on the subset variant (paper Section 5): K sampled permutations instead of n!; "
                         "device-resident timing only")
    ap.add_argument("--traffic-from-ncu", default="", metavar="CSV",
                    help="no run: write profiles/dram_traffic_<workload>.txt from an ncu --csv log of one step at --T tokens")
    args = ap.parse_args()
    if args.permutations:
        args.no_e2e = args.no_cpu_baseline = args.no_sk = args.no_table = True
    if args.traffic_from_ncu:
        write_ncu_traffic(args.workload, args.T or synth.WORKLOADS[args.workload].T, args.traffic_from_ncu)
        return

    from paper_2601_05732_b200 import synth
    wl = synth.WORKLOADS[args.workload]
    if args.T:
        wl = dataclasses.replace(wl, T=args.T)
    if args.layers:
        wl = dataclasses.replace(wl, layers=args.layers)
    rank = int(os.environ.get("RANK", 0))
    world = int(os.environ.get("WORLD_SIZE", 1))
    if args.impl == "reference":
        run_reference(args, wl, rank)
        return
    if world != args.gpus:
        if world == 1 and args.gpus > 1:
            sys.exit(spawn_ranks(sys.argv[1:], args.gpus))
        print(f"bench.py: --gpus {args.gpus} does not match WORLD_SIZE={world}", file=sys.stderr)
        sys.exit(2)
    run_ours(args, wl, rank, world)


if __name__ == "__main__":
    main()

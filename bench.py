#!/usr/bin/env python
"""Benchmark of the pruned VAR scale step (FastVAR cached token pruning) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

One "step" = one pass of the whole hot path over one batch of synthetic input: the full scale
schedule of the workload (unpruned steps, the caching step, the pruned steps with select -> gather ->
sublayers -> restore around every attention / FFN layer).  The headline metric is forwarded (kept)
tokens per second over the pruned scale steps; ms per image is printed beside it.  Rank 0 prints ONE
JSON line.  With N > 1 every rank runs its own batch of images (replicas, no collective).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2503_23367_b200 import inputs as I  # noqa: E402

# `roofline.traffic` is the bytes one launch has to move to and from HBM (operands + results, counted by
# the library per launch), averaged over the launches of the dominant class; the notes say what an ncu
# capture of the same kernel measured against that count (summaries under profiles/).
NCU_TRAFFIC_NOTE = {
    "gemm": "A + W + out bytes per launch (the library's count), mean over the pruned steps' launches; ncu at the 128x128 step's shapes: "
            "QKV M3277 N6144 K2048 (CTA-pair kernel) dram read 38.7 MB = A + W (38.6 MB), out (40 MB) still in L2 at kernel end; second MLP "
            "GEMM M3277 N2048 K8192 (128x192 tiles) read 129.2 MB against A + W = 87.3 MB: its second round of tiles re-reads A",
    "attention": "Q + O + K + V^T bytes per launch; ncu on q820 kv5223 H16 hd128 B2 (whole work items): dram read 92.6 MB (K, V^T, Q = 92.3 MB), "
                 "write 3.8 of 6.7 MB; on q820 kv7245 B1 cut into 148 pieces: read 63.7 MB (62.7 MB), partial results stay in L2",
    "restore": "x read + written, y, cache; ncu on B2 64x64 C2048 k820: read 82.3 MB + write 14.2 MB of 149 MB (x written stays in L2)",
    "select": "x once + scores + indices; ncu on B2 64x64 C2048: score+top-k kernel reads 67.4 MB (x = 67.1 MB); on B1 128x128: 134.4 MB (134.2 MB)",
    "gather_ln": "kept rows in, bf16 rows out; ncu on B2 k820 C2048: read 13.5 MB (rows = 13.4 MB), output left in L2",
}

METRIC = "forwarded_tokens_per_s_over_pruned_scale_steps"
UNIT = "tokens/s"


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def kept(wl: I.Workload, i: int, pruned: bool = True) -> int:
    n = wl.tokens(i)
    if not pruned or wl.keep[i] >= 1.0:
        return n
    if wl.keep[i] == 0.0:
        return 0                      # skipped step: nothing forwarded, nothing cached
    import math
    return min(n, max(1, int(math.ceil(wl.keep[i] * n - 1e-9))))


# ------------------------------------------------------------------------------------------------ reference arm
def oracle_sample(wl: I.Workload):
    """Bounded sample of the workload for the CPU oracle: ONE transformer block of every pruned scale
    step, entered with a synthetic KV prefix and synthetic sublayer caches of the right sizes.
    Returns a callable that runs the sample and the kept tokens it forwards."""
    from oracle import fastvar_oracle as O
    wl1 = wl.with_depth(1)
    mt = I.model_tensors(wl1)
    widen = lambda lst: [I.bf16_bits_to_f32(a).astype(np.float64) for a in lst]
    w = {k: widen(getattr(mt, k)) for k in ("w_qkv", "b_qkv", "w_o", "b_o", "w_fc1", "b_fc1", "w_fc2", "b_fc2",
                                              "w_q_x", "w_kv_x", "w_o_x")}
    w["mod"] = mt.mod.astype(np.float64)
    w["text"] = None if mt.text is None else I.bf16_bits_to_f32(mt.text).astype(np.float64)
    steps = [i for i in range(len(wl.sides)) if 0.0 < wl.keep[i] < 1.0]   # skipped steps cost the oracle nothing worth timing
    n_c = wl.tokens(wl.cache_step)
    subs = ("attn", "xattn", "ffn") if wl.cross_len else ("attn", "ffn")
    xs = {i: I.step_input(wl, i) for i in steps}
    kv_before = {i: sum(kept(wl, j) for j in range(i)) for i in steps}
    kvmax = max(kv_before.values())
    kpre = [I.normal(wl.seed + 900 + b, (kvmax, wl.C)).astype(np.float64) for b in range(wl.B)]
    vpre = [I.normal(wl.seed + 950 + b, (kvmax, wl.C)).astype(np.float64) for b in range(wl.B)]
    caches = {s: I.normal(wl.seed + 990 + j, (wl.B, n_c, wl.C), 0.5).astype(np.float64) for j, s in enumerate(subs)}

    def run():
        for i in steps:
            orc = O.VarOracle(1, wl.C, wl.H, [(s, s) for s in wl.sides], cache_step=wl.cache_step, weights=w,
                              B=wl.B, cross_len=wl.cross_len)
            orc.step, orc.kv_len = i, kv_before[i]
            orc.Kc[0] = [kpre[b][:kv_before[i]] for b in range(wl.B)]
            orc.Vc[0] = [vpre[b][:kv_before[i]] for b in range(wl.B)]
            orc.cache[0] = dict(caches)
            orc.var_step(xs[i], i, wl.keep[i])

    tokens = sum(wl.B * kept(wl, i) for i in steps)
    desc = (f"one transformer block (of {wl.L}) of each pruned scale step (sides "
            f"{[wl.sides[i] for i in steps]}), synthetic KV prefix and caches; time x{wl.L} extrapolates to full depth")
    return run, tokens, desc


def blas_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        return max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        return os.cpu_count() or 1


ORACLE_MAX_REPS, ORACLE_MAX_WARMUP = 2, 1    # the one-block sample takes seconds to tens of seconds per run


def time_oracle(wl, reps: int, warmup: int):
    """Times the oracle's sample `reps` times after `warmup` untimed runs (both capped: the oracle is slow by
    design and the whole leg has to stay within minutes).  `value` extrapolates the one-block time to the
    workload's depth; `sample_seconds` is what one run of the sample really took."""
    run, tokens, desc = oracle_sample(wl)
    reps, warmup = max(1, min(reps, ORACLE_MAX_REPS)), max(0, min(warmup, ORACLE_MAX_WARMUP))
    for _ in range(warmup):
        run()
    ts = []
    for _ in range(reps):
        t0 = time.perf_counter(); run(); ts.append(time.perf_counter() - t0)
    t = statistics.mean(ts)
    return {"value": tokens / (t * wl.L), "unit": UNIT, "cores": blas_threads(), "kind": "oracle", "sample": desc,
            "sample_seconds": t, "runs": reps, "warmup_runs": warmup}


def config_of(wl: I.Workload, world: int) -> dict:
    """The `config` object of the JSON line, spelled the same way by both arms."""
    return {"workload": wl.name, "B_per_gpu": wl.B, "L": wl.L, "C": wl.C, "H": wl.H, "cross_len": wl.cross_len,
            "sides": list(wl.sides), "keep": list(wl.keep), "parallelism": f"replicas x{world} (images sharded, no collective)",
            "cache_hygiene": "inputs larger than L2 (weights + KV + token maps of one pass >> 126 MB)",
            "step": "one full scale schedule for one batch"}


def reference_arm(args, wl):
    if int(os.environ.get("RANK", "0")) != 0:
        return
    cb = time_oracle(wl, args.steps, args.warmup)
    # one "step" of this arm = one run of the bounded sample (one transformer block of every pruned scale step);
    # ms_per_step is the time such a run really took, the extrapolation to full depth is a key of its own
    line = {"impl": "reference", "metric": METRIC, "value": cb["value"], "unit": UNIT, "n_gpus": args.gpus,
            "steps": cb["runs"], "warmup": cb["warmup_runs"], "steps_requested": args.steps, "warmup_requested": args.warmup,
            "repetition_cap": f"at most {ORACLE_MAX_REPS} timed and {ORACLE_MAX_WARMUP} warm-up runs of the sample",
            "ms_per_step": cb["sample_seconds"] * 1e3, "ms_per_step_extrapolated_to_full_depth": cb["sample_seconds"] * wl.L * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": config_of(wl, args.gpus),
            "note": "CPU oracle (numpy fp64), pruned scale steps only, one block timed and extrapolated to the workload's depth",
            "cpu_baseline": {k: cb[k] for k in ("value", "unit", "cores", "kind", "sample")},
            "e2e": {"value": cb["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------------ our arm
class GpuTensors:
    """Random bf16 weights of the workload's shapes, drawn on the device (seeded)."""

    def __init__(self, wl: I.Workload, dev, seed: int):
        g = torch.Generator(device=dev); g.manual_seed(seed)
        C, F, L = wl.C, wl.C * wl.mlp_ratio, wl.L
        r = lambda *s, std=0.02: (torch.randn(*s, generator=g, device=dev, dtype=torch.float32) * std).to(torch.bfloat16)
        self.w_qkv = [r(3 * C, C) for _ in range(L)]; self.b_qkv = [r(3 * C) for _ in range(L)]
        self.w_o = [r(C, C) for _ in range(L)]; self.b_o = [r(C) for _ in range(L)]
        self.w_fc1 = [r(F, C) for _ in range(L)]; self.b_fc1 = [r(F) for _ in range(L)]
        self.w_fc2 = [r(C, F) for _ in range(L)]; self.b_fc2 = [r(C) for _ in range(L)]
        x = wl.cross_len > 0
        self.w_q_x = [r(C, C) for _ in range(L)] if x else []
        self.w_kv_x = [r(2 * C, C) for _ in range(L)] if x else []
        self.w_o_x = [r(C, C) for _ in range(L)] if x else []
        self.mod = torch.randn(L, wl.B, 6, C, generator=g, device=dev, dtype=torch.float32) * 0.3
        self.text = r(wl.B, wl.cross_len, C, std=1.0) if x else None


class ClockSampler:
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.p = None
        try:
            self.p = subprocess.Popen(["nvidia-smi", "-i", str(gpu_index), f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                       "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.p = None

    def stop(self) -> dict:
        if self.p is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.p.terminate()
        try:
            out, _ = self.p.communicate(timeout=5)
        except Exception:
            self.p.kill(); out = ""
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.strip().splitlines():
            f = [t.strip() for t in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); smax.append(float(f[2]))
            except ValueError:
                continue
            for nme, v in zip(names, f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(nme)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        busy = [s for s in sm if s > 0.5 * max(sm)] or sm
        return {"sm_mhz": statistics.median(busy), "sm_max_mhz": max(smax), "reasons": sorted(reasons), "samples": len(sm)}


def gemm_back_to_back(fv, wl, dev, steps_rows, sustained_tflops):
    """The GEMMs of one transformer block alone, at the row count of every pruned scale step: each of the block's
    projections as a chain of 16 launches (four rotating weight sets) captured in a CUDA graph and replayed, so that
    neither the host's enqueue time nor the side stream's restoration is in the figure.  bf16-store epilogues."""
    C, F = wl.C, int(round(wl.C * wl.mlp_ratio))
    shapes = [(3 * C, C, 0), (C, C, 0)] + ([(C, C, 0), (C, C, 0)] if wl.cross_len else []) + [(F, C, 1), (C, F, 0)]
    g = torch.Generator(device=dev); g.manual_seed(9)
    rn = lambda *sh, std=1.0: (torch.randn(*sh, generator=g, device=dev) * std).to(torch.bfloat16)
    skws = torch.zeros(fv.lib().fv_gemm_splitk_workspace_bytes(), dtype=torch.uint8, device=dev)
    st = torch.zeros(1, dtype=torch.int32, device=dev)
    nchain = 16
    by_rows, tot_fl, tot_us = {}, 0.0, 0.0
    for M in steps_rows:
        fl_m = us_m = 0.0
        for (N, K, epi) in shapes:
            a, b = rn(M, K), rn(N, std=0.02)
            ws = [rn(N, K, std=0.02) for _ in range(4)]
            out = torch.empty(M, N, dtype=torch.bfloat16, device=dev)
            for j in range(3):
                fv.fv_gemm_bf16(a, ws[j % 4], b, epilogue=epi, out=out, status=st, splitk_ws=skws)
            torch.cuda.synchronize()
            side = torch.cuda.Stream()
            gr = torch.cuda.CUDAGraph()
            with torch.cuda.stream(side):
                with torch.cuda.graph(gr, stream=side):
                    for j in range(nchain):
                        fv.fv_gemm_bf16(a, ws[j % 4], b, epilogue=epi, out=out, status=st, splitk_ws=skws)
            ts = []
            for _ in range(5):
                torch.cuda.synchronize()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(); gr.replay(); e1.record(); torch.cuda.synchronize()
                ts.append(e0.elapsed_time(e1) * 1e3 / nchain)
            us_m += statistics.median(ts)
            fl_m += 2.0 * M * N * K
            del gr, a, b, ws, out
        by_rows[str(M)] = fl_m / us_m * 1e-6
        tot_fl += fl_m; tot_us += us_m
    if int(st.item()) != 0:
        raise SystemExit("a GEMM reported an expired wait")
    mix = tot_fl / tot_us * 1e-6
    return {"what": "the projections of one block alone at the pruned steps' row counts: chains of 16 launches replayed from a CUDA graph, "
                    "four rotating weight sets (they stay in L2; inside a step the weights come from HBM and the unkept-row restoration runs beside the GEMMs)",
            "tflops_by_rows": by_rows, "mix_tflops": mix, "peak": sustained_tflops, "frac": mix / sustained_tflops if sustained_tflops else None}


def ours(args, wl):
    from paper_2503_23367_b200 import binding as fv
    from paper_2503_23367_b200 import build as fv_build
    from paper_2503_23367_b200 import replicas as R
    rank, world = int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the pruned VAR step has no CPU path")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    if rank == 0:
        fv_build.build()
    if world > 1:
        dist.barrier()
    fv.lib()

    S = len(wl.sides)
    pruned_steps = [i for i in range(S) if wl.keep[i] < 1.0]
    gt = GpuTensors(wl, dev, seed=wl.seed)          # replicas: the same weights on every rank
    cap = sum(kept(wl, i) for i in range(S))
    hw = [(s, s) for s in wl.sides]
    ctx = fv.FvContext(wl.L, wl.C, wl.H, hw, wl.cache_step, wl.B, cap, gt, cross_len=wl.cross_len, mlp_ratio=wl.mlp_ratio, device=dev)
    g = torch.Generator(device=dev); g.manual_seed(R.rank_seed(wl.seed + 77, rank))   # its own images
    xs = [torch.randn(wl.B, wl.tokens(i), wl.C, generator=g, device=dev, dtype=torch.float32) for i in range(S)]
    outs = [torch.empty_like(x) for x in xs]

    def schedule(c, keep, events=None):
        c.reset()
        for i in range(S):
            if events is not None:
                events[i].record()
            c.var_step(xs[i], i, keep[i], out=outs[i])
        if events is not None:
            events[S].record()

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            R.barrier()
            torch.cuda.synchronize()

    def max_over_ranks(v: float) -> float:
        return R.max_over_ranks(v, device=dev)

    for _ in range(args.warmup):
        schedule(ctx, wl.keep)
    barrier()
    # A timed region during which the GPU reported a thermal or hardware slowdown is taken once more (the power cap
    # alone is normal under load and kept).
    for attempt in range(2):
        fv.fv_profile_read()                                   # zero the launch counters
        evs = [[torch.cuda.Event(enable_timing=True) for _ in range(S + 1)] for _ in range(args.steps)]
        sampler = ClockSampler(local) if rank == 0 else None
        t_wall = time.perf_counter()
        for k in range(args.steps):
            schedule(ctx, wl.keep, evs[k])
        barrier()
        t_wall = time.perf_counter() - t_wall
        clocks = sampler.stop() if sampler else None
        slowed = 1.0 if clocks and any(r in ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown") for r in clocks["reasons"]) else 0.0
        if attempt == 1 or max_over_ranks(slowed) == 0.0:      # rank 0 samples; every rank follows its verdict
            if clocks is not None and attempt == 1:
                clocks["remeasured"] = True
            break
        barrier()
    launches = fv.fv_profile_read()
    gpu_launches = sum(v["launches"] for v in launches.values())
    if ctx.device_status() != 0:
        raise SystemExit("a kernel reported an expired wait")
    total_ms = sum(evs[k][0].elapsed_time(evs[k][S]) for k in range(args.steps))
    step_ms = [statistics.mean(evs[k][i].elapsed_time(evs[k][i + 1]) for k in range(args.steps)) for i in range(S)]
    total_ms = max_over_ranks(total_ms)
    pruned_ms = max_over_ranks(sum(step_ms[i] for i in pruned_steps))
    ms_per_step = total_ms / args.steps
    fwd_tokens = sum(wl.B * kept(wl, i) for i in pruned_steps)
    value = world * fwd_tokens / (pruned_ms * 1e-3)

    # ---- end to end through the public API with HOST buffers (pinned), copies inside the timed region
    hx = [torch.randn(x.shape, dtype=torch.float32).pin_memory() for x in xs]
    ho = [torch.empty(x.shape, dtype=torch.float32).pin_memory() for x in xs]
    e2e_steps = 0 if args.skip_e2e else max(2, min(args.steps, 5))

    def schedule_e2e(events=None):
        ctx.reset()
        for i in range(S):
            if events is not None:
                events[i].record()
            ctx.var_step_host(hx[i], i, wl.keep[i], ho[i])      # C ABI call with host buffers: H2D, step, D2H
        ctx.host_io_flush()                                     # the last results have landed before the region ends
        if events is not None:
            events[S].record()

    e2e = None
    if e2e_steps:
      schedule_e2e()
      barrier()
      ev2 = [[torch.cuda.Event(enable_timing=True) for _ in range(S + 1)] for _ in range(e2e_steps)]
      for k in range(e2e_steps):
          schedule_e2e(ev2[k])
      barrier()
      e2e_pruned_ms = max_over_ranks(sum(statistics.mean(ev2[k][i].elapsed_time(ev2[k][i + 1]) for k in range(e2e_steps))
                                       for i in pruned_steps))
      e2e_total_ms = max_over_ranks(statistics.mean(ev2[k][0].elapsed_time(ev2[k][S]) for k in range(e2e_steps)))
      bytes_io = sum(x.numel() * 4 for x in xs)
      e2e = {"value": world * fwd_tokens / (e2e_pruned_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": bytes_io,
             "d2h_bytes_per_step": bytes_io, "ms_per_step": e2e_total_ms, "ms_per_image": e2e_total_ms / wl.B}

    # ---- per-kernel-class device time: CUDA events around every launch, in passes of their own (the
    # event pairs serialise the launches a little, so the timed region above runs without them)
    peaks = measured_peaks()

    def class_table(only_pruned: bool, reps: int = 2):
        fv.fv_profile_read()                               # clear counters
        for _ in range(reps):
            ctx.reset()
            for i in range(S):
                fv.fv_profile_enable((not only_pruned) or (i in pruned_steps))
                ctx.var_step(xs[i], i, wl.keep[i], out=outs[i])
        raw = fv.fv_profile_read() if not only_pruned else None
        fv.fv_profile_enable(False)
        return raw, reps

    def summarise(raw, reps):
        table = {}
        for name, v in raw.items():
            if v["launches"] == 0 or v["ms"] <= 0:
                continue
            ms = v["ms"] / reps
            tensor = name in ("gemm", "attention")
            ach = (v["work"] / reps) / (ms * 1e-3) / (1e12 if tensor else 1e9)
            peak = peaks["bf16_tflops_sustained"] if tensor else peaks["hbm_gbs"]
            table[name] = {"ms_per_step": ms, "launches_per_step": v["launches"] // reps, "bound": "tensor" if tensor else "hbm",
                           "achieved": ach, "unit": "TFLOP/s" if tensor else "GB/s", "peak": peak, "frac": ach / peak,
                           "dram_bytes_per_launch": v["dram_bytes"] / max(1, v["launches"])}
        return table

    kernels, kernels_pruned, roofline = {}, {}, None
    if not args.skip_profile:
        kernels = summarise(*class_table(False))
        # pruned scale steps only: launches and work are counted always, time only while enabled, so
        # count work with the counters cleared around exactly those steps
        reps = 2
        acc = None
        for _ in range(reps):
            ctx.reset()
            for i in range(S):
                if i in pruned_steps:
                    fv.fv_profile_read(); fv.fv_profile_enable(True)
                ctx.var_step(xs[i], i, wl.keep[i], out=outs[i])
                if i in pruned_steps:
                    r = fv.fv_profile_read(); fv.fv_profile_enable(False)
                    if acc is None:
                        acc = r
                    else:
                        for n_, v_ in r.items():
                            for f_ in ("ms", "launches", "work", "dram_bytes"):
                                acc[n_][f_] += v_[f_]
        kernels_pruned = summarise(acc, reps)
        dom = max(kernels_pruned, key=lambda n: kernels_pruned[n]["ms_per_step"])
        d = kernels_pruned[dom]
        roofline = {"kernel": dom, "region": "pruned scale steps", "bound": d["bound"], "achieved": d["achieved"], "peak": d["peak"],
                    "unit": d["unit"], "frac": d["frac"], "traffic": d["dram_bytes_per_launch"],
                    "traffic_source": NCU_TRAFFIC_NOTE.get(dom, "operand + result bytes per launch (no ncu capture for this class)"),
                    "peak_source": f"of {peaks['source']} ({'sustained bf16 matmul' if d['bound'] == 'tensor' else 'copy bandwidth'})",
                    "avg_launch_ms": d["ms_per_step"] / max(1, d["launches_per_step"])}

    # ---- the generation loop around the step (Sec. 3.1, Eq. 2-3): head, greedy token choice, residual
    # accumulation and the next token map after every step, all K steps in one fv_generate call
    generation = None
    if not args.skip_generation:
        gen_t = I.generation_tensors(wl, V=4096, d=32)
        fgen = fv.FvGenerator(ctx, gen_t)
        start = torch.from_numpy(gen_t.start).to(dev)
        for _ in range(2):
            fgen.generate(start, wl.keep)
        barrier()
        ng = max(2, min(args.steps, 5))
        before = fv.fv_profile_read()
        evg = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(ng)]
        for a, b in evg:
            a.record(); fgen.generate(start, wl.keep); b.record()
        barrier()
        if ctx.device_status() != 0:
            raise SystemExit("a kernel reported an expired wait")
        g_ms = max_over_ranks(statistics.mean(a.elapsed_time(b) for a, b in evg))
        g_launches = sum(v["launches"] for v in fv.fv_profile_read().values()) // ng
        generation = {"what": "fv_generate: every scale step followed by head (V = 4096), greedy token choice, Eq. 2 (d = 32) and "
                              "the next token map; synthetic codebook and head",
                      "ms_per_step": g_ms, "ms_per_image": g_ms / wl.B, "ms_outside_the_scale_steps": g_ms - ms_per_step,
                      "gpu_launches": g_launches}
        del fgen
        torch.cuda.empty_cache()

    # ---- the coarser granularity beside it: one selection and one restoration around the whole stack of
    # blocks of a pruned step (not the paper's configuration, which is what `value` measures)
    variant = None
    ctx.close()
    del ctx
    torch.cuda.empty_cache()
    if not args.skip_variant:
        ctx_step = fv.FvContext(wl.L, wl.C, wl.H, hw, wl.cache_step, wl.B, cap, gt, cross_len=wl.cross_len, mlp_ratio=wl.mlp_ratio,
                                device=dev, granularity=1)
        for _ in range(3):
            schedule(ctx_step, wl.keep)
        barrier()
        nv = max(2, min(args.steps, 5))
        evv = [[torch.cuda.Event(enable_timing=True) for _ in range(S + 1)] for _ in range(nv)]
        for k in range(nv):
            schedule(ctx_step, wl.keep, evv[k])
        barrier()
        if ctx_step.device_status() != 0:
            raise SystemExit("a kernel reported an expired wait")
        v_total = max_over_ranks(statistics.mean(evv[k][0].elapsed_time(evv[k][S]) for k in range(nv)))
        v_pruned = max_over_ranks(sum(statistics.mean(evv[k][i].elapsed_time(evv[k][i + 1]) for k in range(nv)) for i in pruned_steps))
        variant = {"what": "selection and restoration once per scale step around all blocks (granularity 1), not the paper's per-layer wrapping",
                   "value": world * fwd_tokens / (v_pruned * 1e-3), "unit": UNIT, "ms_per_step": v_total, "ms_per_image": v_total / wl.B,
                   "ms_pruned_steps": v_pruned}
        ctx_step.close()
        del ctx_step
        torch.cuda.empty_cache()

    # ---- the optional backbone pieces switched on (cosine attention, rotary positions, bilinear restoration)
    extras = None
    if not args.skip_variant:
        qk_scale = torch.full((wl.L, wl.H), 10.0, device=dev)
        ctx_x = fv.FvContext(wl.L, wl.C, wl.H, hw, wl.cache_step, wl.B, cap, gt, cross_len=wl.cross_len, mlp_ratio=wl.mlp_ratio,
                             device=dev, rope_base=10000.0, interp_mode=1, qk_scale=qk_scale)
        for _ in range(3):
            schedule(ctx_x, wl.keep)
        barrier()
        nx = max(2, min(args.steps, 5))
        evx = [[torch.cuda.Event(enable_timing=True) for _ in range(S + 1)] for _ in range(nx)]
        for k in range(nx):
            schedule(ctx_x, wl.keep, evx[k])
        barrier()
        if ctx_x.device_status() != 0:
            raise SystemExit("a kernel reported an expired wait")
        x_total = max_over_ranks(statistics.mean(evx[k][0].elapsed_time(evx[k][S]) for k in range(nx)))
        x_pruned = max_over_ranks(sum(statistics.mean(evx[k][i].elapsed_time(evx[k][i + 1]) for k in range(nx)) for i in pruned_steps))
        extras = {"what": "same schedule with cosine attention + 2-D rotary positions (by original token index) in the QKV epilogue and "
                          "bilinear interpolation of the cache in the restoration",
                  "value": world * fwd_tokens / (x_pruned * 1e-3), "unit": UNIT, "ms_per_step": x_total, "ms_per_image": x_total / wl.B,
                  "ms_pruned_steps": x_pruned}
        ctx_x.close()
        del ctx_x
        torch.cuda.empty_cache()

    # ---- the residual stream (token maps) in bf16 instead of fp32 (fv_config.resid_dtype = 1): every pass over the
    # stream moves half the bytes, every update rounds it to bf16 once
    bf16_stream = None
    if not args.skip_variant:
        ctx_b = fv.FvContext(wl.L, wl.C, wl.H, hw, wl.cache_step, wl.B, cap, gt, cross_len=wl.cross_len, mlp_ratio=wl.mlp_ratio,
                             device=dev, resid_dtype=1)
        xs_b = [x.to(torch.bfloat16) for x in xs]
        outs_b = [torch.empty_like(x) for x in xs_b]

        def schedule_b(events=None):
            ctx_b.reset()
            for i in range(S):
                if events is not None:
                    events[i].record()
                ctx_b.var_step(xs_b[i], i, wl.keep[i], out=outs_b[i])
            if events is not None:
                events[S].record()

        for _ in range(3):
            schedule_b()
        barrier()
        nb = max(2, min(args.steps, 5))
        evb = [[torch.cuda.Event(enable_timing=True) for _ in range(S + 1)] for _ in range(nb)]
        for k in range(nb):
            schedule_b(evb[k])
        barrier()
        if ctx_b.device_status() != 0:
            raise SystemExit("a kernel reported an expired wait")
        b_total = max_over_ranks(statistics.mean(evb[k][0].elapsed_time(evb[k][S]) for k in range(nb)))
        b_pruned = max_over_ranks(sum(statistics.mean(evb[k][i].elapsed_time(evb[k][i + 1]) for k in range(nb)) for i in pruned_steps))
        bf16_stream = {"what": "same schedule with the residual stream (token maps in and out of every step) in bf16; arithmetic stays fp32",
                       "value": world * fwd_tokens / (b_pruned * 1e-3), "unit": UNIT, "ms_per_step": b_total, "ms_per_image": b_total / wl.B,
                       "ms_pruned_steps": b_pruned}
        ctx_b.close()
        del ctx_b, xs_b, outs_b
        torch.cuda.empty_cache()

    # ---- the unpruned GPU step beside it (same kernels, keep_ratio = 1 everywhere)
    unpruned = None
    if not args.skip_unpruned:
        cap_full = sum(wl.tokens(i) for i in range(S))
        ctx_full = fv.FvContext(wl.L, wl.C, wl.H, hw, wl.cache_step, wl.B, cap_full, gt, cross_len=wl.cross_len,
                                mlp_ratio=wl.mlp_ratio, device=dev)
        keep1 = (1.0,) * S
        schedule(ctx_full, keep1)
        barrier()
        evu = [[torch.cuda.Event(enable_timing=True) for _ in range(S + 1)] for _ in range(2)]
        for k in range(2):
            schedule(ctx_full, keep1, evu[k])
        barrier()
        u_total = statistics.mean(evu[k][0].elapsed_time(evu[k][S]) for k in range(2))
        u_pruned = sum(statistics.mean(evu[k][i].elapsed_time(evu[k][i + 1]) for k in range(2)) for i in pruned_steps)
        unpruned = {"ms_per_image": u_total / wl.B, "ms_same_scale_steps": u_pruned, "speedup_whole_schedule": u_total / ms_per_step,
                    "speedup_pruned_steps": u_pruned / pruned_ms}
        ctx_full.close()

    # ---- the 1024-pixel configuration beside it (13 scales up to 64x64, batch 2, keep 0.6 / 0.4 / 0.2): the same
    # device-resident timing, no other legs
    other = None
    if not args.skip_other and wl.name == "infinity_2b_2k":
        wl2 = I.WORKLOADS["infinity_2b_1k"]
        if args.blocks > 0:
            wl2 = wl2.with_depth(args.blocks)
        del gt
        torch.cuda.empty_cache()
        gt2 = GpuTensors(wl2, dev, seed=wl2.seed)
        S2 = len(wl2.sides)
        pruned2 = [i for i in range(S2) if wl2.keep[i] < 1.0]
        ctx2 = fv.FvContext(wl2.L, wl2.C, wl2.H, [(s_, s_) for s_ in wl2.sides], wl2.cache_step, wl2.B, sum(kept(wl2, i) for i in range(S2)),
                            gt2, cross_len=wl2.cross_len, mlp_ratio=wl2.mlp_ratio, device=dev)
        g2 = torch.Generator(device=dev); g2.manual_seed(R.rank_seed(wl2.seed + 77, rank))
        xs2 = [torch.randn(wl2.B, wl2.tokens(i), wl2.C, generator=g2, device=dev, dtype=torch.float32) for i in range(S2)]
        outs2 = [torch.empty_like(x) for x in xs2]

        def schedule2(events=None):
            ctx2.reset()
            for i in range(S2):
                if events is not None:
                    events[i].record()
                ctx2.var_step(xs2[i], i, wl2.keep[i], out=outs2[i])
            if events is not None:
                events[S2].record()

        for _ in range(3):
            schedule2()
        barrier()
        n2 = max(2, min(args.steps, 5))
        ev2b = [[torch.cuda.Event(enable_timing=True) for _ in range(S2 + 1)] for _ in range(n2)]
        for k in range(n2):
            schedule2(ev2b[k])
        barrier()
        if ctx2.device_status() != 0:
            raise SystemExit("a kernel reported an expired wait")
        o_total = max_over_ranks(statistics.mean(ev2b[k][0].elapsed_time(ev2b[k][S2]) for k in range(n2)))
        o_pruned = max_over_ranks(sum(statistics.mean(ev2b[k][i].elapsed_time(ev2b[k][i + 1]) for k in range(n2)) for i in pruned2))
        fwd2 = sum(wl2.B * kept(wl2, i) for i in pruned2)
        other = {"infinity_2b_1k": {"what": "the 1024-pixel configuration: 13 scales up to 64x64, batch 2, keep 0.6 / 0.4 / 0.2 on the last three",
                                    "value": world * fwd2 / (o_pruned * 1e-3), "unit": UNIT, "ms_per_step": o_total,
                                    "ms_per_image": o_total / wl2.B, "ms_pruned_steps": o_pruned, "config": config_of(wl2, world)}}
        ctx2.close()
        del ctx2, gt2, xs2, outs2
        torch.cuda.empty_cache()

    b2b = None
    if rank == 0 and not args.skip_b2b:
        b2b = gemm_back_to_back(fv, wl, dev, [wl.B * kept(wl, i) for i in pruned_steps], peaks.get("bf16_tflops_sustained"))

    cpu_baseline = None
    if rank == 0 and world == 1 and not args.skip_cpu:
        cb = time_oracle(wl, reps=1, warmup=0)
        cpu_baseline = {k: cb[k] for k in ("value", "unit", "cores", "kind", "sample")}

    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    if rank != 0:
        return
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
            "data": "synthetic",
            "config": config_of(wl, world),
            "ms_per_image": ms_per_step / wl.B, "ms_per_image_pruned_steps": pruned_ms / wl.B,
            "scale_step_ms": [round(t, 4) for t in step_ms], "wall_ms_per_step": t_wall * 1e3 / args.steps,
            "roofline": roofline, "kernels": kernels, "kernels_pruned_steps": kernels_pruned, "cpu_baseline": cpu_baseline, "e2e": e2e, "gpu_launches": gpu_launches,
            "clocks": clocks, "unpruned_gpu": unpruned, "per_step_granularity": variant, "backbone_options": extras, "bf16_residual_stream": bf16_stream, "generation_loop": generation, "other_workloads": other,
            "gemm_back_to_back": b2b, "peaks": peaks}
    print(json.dumps(line))


def sweep(args, wl):
    """Pruning-ratio and caching-step curves (the efficiency side of the paper's ablations on the pruning
    ratio and on the number of pruned steps, with synthetic weights): one JSON line, `--sweep`."""
    from dataclasses import replace
    from paper_2503_23367_b200 import binding as fv
    from paper_2503_23367_b200 import build as fv_build
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the pruned VAR step has no CPU path")
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    fv_build.build()
    fv.lib()
    S = len(wl.sides)
    gt = GpuTensors(wl, dev, seed=wl.seed)
    g = torch.Generator(device=dev); g.manual_seed(wl.seed + 77)
    xs = [torch.randn(wl.B, wl.tokens(i), wl.C, generator=g, device=dev, dtype=torch.float32) for i in range(S)]
    outs = [torch.empty_like(x) for x in xs]
    hw = [(s_, s_) for s_ in wl.sides]

    def run(keep, cache_step=None):
        w2 = replace(wl, keep=tuple(keep))
        pruned = [i for i in range(S) if keep[i] < 1.0]
        cap = sum(kept(w2, i) for i in range(S))
        ctx = fv.FvContext(wl.L, wl.C, wl.H, hw, w2.cache_step if cache_step is None else cache_step, wl.B, cap, gt,
                           cross_len=wl.cross_len, mlp_ratio=wl.mlp_ratio, device=dev)
        ev = [[torch.cuda.Event(enable_timing=True) for _ in range(S + 1)] for _ in range(3)]
        for rep in range(5):
            ctx.reset()
            for i in range(S):
                if rep >= 2:
                    ev[rep - 2][i].record()
                ctx.var_step(xs[i], i, keep[i], out=outs[i])
            if rep >= 2:
                ev[rep - 2][S].record()
        torch.cuda.synchronize()
        if ctx.device_status() != 0:
            raise SystemExit("a kernel reported an expired wait")
        total = statistics.mean(e[0].elapsed_time(e[S]) for e in ev)
        step = [statistics.mean(e[i].elapsed_time(e[i + 1]) for e in ev) for i in range(S)]
        ctx.close()
        del ctx
        torch.cuda.empty_cache()
        return total, step, pruned, w2

    base_total, base_step, _, _ = run((1.0,) * S)
    default_pruned = [i for i in range(S) if wl.keep[i] < 1.0]
    rows = []
    for ratio in (0.25, 0.4, 0.5, 0.6, 0.75, 0.9):
        keep = [1.0] * S
        for i in default_pruned:
            keep[i] = 1.0 - ratio
        total, step, pruned, w2 = run(keep)
        p_ms = sum(step[i] for i in pruned)
        rows.append({"sweep": "pruning ratio on the workload's pruned steps", "pruning_ratio": ratio, "pruned_steps": len(pruned),
                     "ms_per_image": total / wl.B, "speedup_whole_schedule": base_total / total,
                     "speedup_pruned_steps": sum(base_step[i] for i in pruned) / p_ms,
                     "forwarded_tokens_per_s": sum(wl.B * kept(w2, i) for i in pruned) / (p_ms * 1e-3)})
    for n_pruned in (1, 2, 3, 4):
        keep = [1.0] * S
        for i in range(S - n_pruned, S):
            keep[i] = 0.5
        total, step, pruned, w2 = run(keep)
        p_ms = sum(step[i] for i in pruned)
        rows.append({"sweep": "number of pruned steps N at pruning ratio 0.5 (caching step K-N)", "pruned_steps": n_pruned,
                     "cache_step": S - n_pruned - 1, "pruning_ratio": 0.5, "ms_per_image": total / wl.B,
                     "speedup_whole_schedule": base_total / total, "speedup_pruned_steps": sum(base_step[i] for i in pruned) / p_ms,
                     "forwarded_tokens_per_s": sum(wl.B * kept(w2, i) for i in pruned) / (p_ms * 1e-3)})
    # the caching step of the paper's ablation: the workload's pruned steps stay as they are, the step whose layer
    # outputs are cached moves back from K-N (the last unpruned step) to K-N-3 (smaller cached maps, upsampled further)
    first_pruned = default_pruned[0]
    for back in (0, 1, 2, 3):
        cs = first_pruned - 1 - back
        if cs < 0:
            continue
        total, step, pruned, w2 = run(list(wl.keep), cache_step=cs)
        p_ms = sum(step[i] for i in pruned)
        rows.append({"sweep": "caching step K-N-j with the workload's pruned steps fixed", "cache_step": cs, "steps_before_the_first_pruned": back + 1,
                     "cached_side": wl.sides[cs], "ms_per_image": total / wl.B, "speedup_whole_schedule": base_total / total,
                     "speedup_pruned_steps": sum(base_step[i] for i in pruned) / p_ms,
                     "forwarded_tokens_per_s": sum(wl.B * kept(w2, i) for i in pruned) / (p_ms * 1e-3)})
    print(json.dumps({"sweep": rows, "workload": wl.name, "B": wl.B, "unpruned_ms_per_image": base_total / wl.B, "data": "synthetic"}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="infinity_2b_2k", choices=sorted(I.WORKLOADS))
    ap.add_argument("--skip-cpu", action="store_true", help="omit the CPU-oracle leg")
    ap.add_argument("--skip-e2e", action="store_true", help="omit the host-buffer end-to-end leg")
    ap.add_argument("--skip-profile", action="store_true", help="omit the per-kernel-class timing passes")
    ap.add_argument("--skip-unpruned", action="store_true", help="omit the unpruned GPU comparison")
    ap.add_argument("--skip-generation", action="store_true", help="omit the generation-loop (fv_generate) timing")
    ap.add_argument("--sweep", action="store_true", help="print pruning-ratio and caching-step curves instead of the bench line")
    ap.add_argument("--skip-variant", action="store_true", help="omit the per-step-granularity comparison")
    ap.add_argument("--skip-other", action="store_true", help="omit the timing of the 1024-pixel configuration beside the default one")
    ap.add_argument("--skip-b2b", action="store_true", help="omit the back-to-back timing of a block's GEMMs")
    ap.add_argument("--blocks", type=int, default=0,
                    help="profiling only: run this many transformer blocks instead of the workload's depth (the line says so; not a bench number)")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.impl == "ours" and not args.sweep:
        # started plainly with --gpus N: become the launcher of N ranks, one per GPU (replicas; the process group
        # only carries the measurement), and pass their output through
        import socket
        with socket.socket() as sock:
            sock.bind(("127.0.0.1", 0))
            port = sock.getsockname()[1]
        cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}", "--master-addr", "127.0.0.1",
               "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
        raise SystemExit(subprocess.call(cmd))
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    wl = I.WORKLOADS[args.workload]
    if args.blocks > 0:
        wl = wl.with_depth(args.blocks)
    if args.impl == "reference":
        reference_arm(args, wl)
    elif args.sweep:
        sweep(args, wl)
    else:
        ours(args, wl)


if __name__ == "__main__":
    main()

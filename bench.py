#!/usr/bin/env python
"""Benchmark of the STILL hybrid attention layer forward on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c3] [--impl ours|reference]

One "step" is one still_hybrid_attn_fwd call (score -> top-k select -> NP-Map + linear scan ->
sparse softmax attention -> merge) over one synthetic batch of the workload; for the decode
workload (c5) a step is one still_hybrid_attn_step call.  The metric is tokens/s/layer
(B * N / time).  With N GPUs every rank runs its own batch (the (batch, head) units are
independent: no collective on the data path) and the value is the sum over ranks divided by the
slowest rank's time.

The JSON line carries, besides the contract keys:
  roofline      the softmax-attention kernel (>98% of the FLOPs): algorithmic FLOPs per launch
                divided by its CUDA-event time measured inside the timed region, against the
                measured bf16 peak of this machine (MEASURED_PEAKS.json, sustained figure)
  cpu_baseline  the CPU oracle timed on a bounded sample of the same workload on this machine
  e2e           the same metric through still_hybrid_attn_fwd_host with pinned HOST buffers
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "hybrid-attn prefill tokens/s/layer at Llama-3-8B shape"
UNIT = "tokens/s"


def algorithmic_work(w, lam=None, max_salient=0):
    """FLOPs and bytes the method itself needs for one prefill call (causal-exact pair count).  With a
    salient-cache budget a query of chunk t sees min((t-2) lam, max_salient) cached tokens."""
    lam = w.k if lam is None else lam
    C, d, N = w.C, w.d, w.N
    T = -(-N // C)
    BH, BHkv = w.B * w.H, w.B * w.Hkv
    es = 4 if w.dtype == "fp32" else 2
    if max_salient > 0:
        p_sel = C * sum(min(max(t - 2, 0) * lam, max_salient) for t in range(1, T + 1))
    else:
        p_sel = C * lam * max(T - 1, 0) * max(T - 2, 0) // 2
    p_loc = max(T - 1, 0) * C * C + T * C * (C + 1) // 2
    f_sa = 4 * d * (p_sel + p_loc) * BH
    dp = 2 * w.d_f
    la = lam < C or max_salient > 0
    f_map = 2 * d * w.d_f * N * (BH + BHkv) if la else 0
    f_la = (2 * (C - lam) + 2 * C) * dp * (d + 1) * max(T - 2, 0) * BH if la else 0
    f_score = 2 * d * (2 * C) * C * T * BH  # s_in and s_prev tiles
    by = w.B * N * d * es * (2 * w.H + 2 * w.Hkv) + 4 * BH * N + 4 * BH * T * lam
    return {"flops": f_sa + f_map + f_la + f_score, "flops_sa": f_sa, "bytes": by}


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""

    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index=0):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                 "-lms", "25"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            if len(r) < 7:
                continue
            try:
                sm.append(float(r[0]))
                mx.append(float(r[1]))
            except ValueError:
                continue
            for n, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"bf16_tflops": p["bf16_tflops"], "bf16_tflops_sustained": p["bf16_tflops_sustained"],
                "hbm_gbs": p["hbm_gbs"], "source": "measured"}
    return {"bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "hbm_gbs": 6650.0, "source": "fallback"}


def ncu_traffic(kernel_key):
    """DRAM bytes per launch of the dominant kernel from the committed ncu summary, if any."""
    path = os.path.join(ROOT, "profiles", "traffic.json")
    if os.path.exists(path):
        return json.load(open(path)).get(kernel_key)
    return None


def oracle_sample(w, lam, n_heads, n_rows, seed=0):
    """Times the CPU oracle on a bounded sample: n_heads heads in parallel, all O(N) steps in full,
    the softmax/merge step on n_rows evenly spread query rows; returns the extrapolated time of
    the whole workload, the threads used and a description of the sample."""
    import numpy as np
    import torch

    from oracle import still_oracle as oracle
    from paper_2602_02180_b200 import synth

    ws = w.with_(B=1, H=n_heads, Hkv=n_heads, k=lam)
    Q, K, V = synth.make_qkv(ws, "cpu")
    Wq, Wk = synth.make_npmap_weights(ws, "cpu")
    f64 = lambda t: t.float().numpy().astype(np.float64)  # noqa: E731
    Q, K, V, Wq, Wk = map(f64, (Q, K, V, Wq, Wk))
    hp = oracle.HeadParams(w.C, lam, w.sm_scale)
    rows = np.unique(np.linspace(0, w.N - 1, n_rows).astype(np.int64))
    t0 = time.perf_counter()
    out = oracle.layer(Q, K, V, Wq, Wk, hp, rows=rows[-1:])
    t_fixed = time.perf_counter() - t0
    t0 = time.perf_counter()
    out = oracle.layer(Q, K, V, Wq, Wk, hp, rows=rows)
    t_rows = time.perf_counter() - t0
    threads = out["threads"]
    per_row = max(t_rows - t_fixed, 1e-9) / max(len(rows) - 1, 1)
    per_head_batch = t_fixed + per_row * w.N  # n_heads heads processed side by side
    total = per_head_batch * (w.B * w.H) / n_heads
    sample = (f"{n_heads} of {w.B * w.H} heads on {threads} threads; score/select/state steps in full, "
              f"softmax+merge on {len(rows)} of {w.N} query rows, scaled by row and head count")
    return total, threads, sample, t_fixed + t_rows


def oracle_decode_sample(w, lam, n_rows=257):
    """CPU oracle for the decode workload: the per-token cost of the softmax/merge step at the end of the
    prefix (difference between n_rows and 1 answered rows, all prefix work excluded), one head per thread,
    scaled to B * H heads per step."""
    import multiprocessing

    import numpy as np

    from oracle import still_oracle as oracle
    from paper_2602_02180_b200 import synth

    n_heads = max(1, min(multiprocessing.cpu_count(), w.B * w.H))
    ws = w.with_(B=1, H=n_heads, Hkv=n_heads, k=lam, N=w.N + n_rows)
    Q, K, V = synth.make_qkv(ws, "cpu")
    Wq, Wk = synth.make_npmap_weights(ws, "cpu")
    f64 = lambda t: t.float().numpy().astype(np.float64)  # noqa: E731
    Q, K, V, Wq, Wk = map(f64, (Q, K, V, Wq, Wk))
    hp = oracle.HeadParams(w.C, lam, w.sm_scale)
    rows = np.arange(w.N, w.N + n_rows, dtype=np.int64)
    t0 = time.perf_counter()
    out = oracle.layer(Q, K, V, Wq, Wk, hp, rows=rows[:1])
    t_one = time.perf_counter() - t0
    t0 = time.perf_counter()
    out = oracle.layer(Q, K, V, Wq, Wk, hp, rows=rows)
    t_all = time.perf_counter() - t0
    per_step_heads = max(t_all - t_one, 1e-9) / (n_rows - 1)      # n_heads heads, one token each
    step_s = per_step_heads * (w.B * w.H) / n_heads
    return {"value": w.B / step_s, "unit": UNIT, "cores": out["threads"], "kind": "oracle",
            "sample": f"{n_heads} of {w.B * w.H} heads on {out['threads']} threads; softmax+merge of {n_rows} tokens after "
                      f"the {w.N}-token prefix (prefix work excluded), scaled by head count"}


def local_global_overlap(w, n_tokens=4096, n_heads=4):
    """Sec. 3.1's local-global consistency on the synthetic inputs (CPU oracle): how much of each chunk's top-C/4 by
    the windowed Self-Saliency Score is also in its top-C/4 by the full-context score.  Bounded: the first n_tokens
    tokens of n_heads heads (the full-context score costs O(N^2 d) per head)."""
    import numpy as np

    from oracle import still_oracle as oracle
    from paper_2602_02180_b200 import synth

    n = min(n_tokens, w.N)
    ws = w.with_(B=1, H=n_heads, Hkv=n_heads, N=n)
    Q, K, _ = synth.make_qkv(ws, "cpu")
    lam = max(w.C // 4, 1)
    hits = []
    for h in range(n_heads):
        q, k = (t[0, h].float().numpy().astype(np.float64) for t in (Q, K))
        loc = oracle.select(oracle.score_chunkwise(q, k, w.C, w.sm_scale), w.C, lam)
        glo = oracle.select(oracle.score_global(q, k, w.sm_scale), w.C, lam)
        for a, b in zip(loc, glo):
            sa, sb = set(a[a >= 0].tolist()), set(b[b >= 0].tolist())
            if sa:
                hits.append(len(sa & sb) / len(sa))
    return {"workload": w.name, "tokens": n, "heads": n_heads, "chunk": w.C, "topk": lam,
            "mean_overlap": float(np.mean(hits)), "min_overlap": float(np.min(hits))}


def run_reference(args, w, lam, rank, world):
    """--impl reference: the CPU oracle as it stands, on this machine's host cores."""
    if rank != 0:
        return
    import multiprocessing

    cores = multiprocessing.cpu_count()
    n_heads = max(1, min(cores, w.B * w.H))
    n_rows = 160 if w.N > 8192 else 256
    times = []
    for i in range(args.warmup + args.steps):
        total, threads, sample, spent = oracle_sample(w, lam, n_heads, n_rows)
        if i >= args.warmup:
            times.append(total)
    t = statistics.mean(times)
    value = w.B * w.N / t
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": t * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "B": w.B, "H": w.H, "Hkv": w.Hkv, "d": w.d, "N": w.N, "chunk": w.C,
                   "topk": lam, "timing": "host wall clock, extrapolated from a bounded sample"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c3", choices=["c1", "c2", "c3", "c4", "c5"])
    ap.add_argument("--topk", type=int, default=None, help="override lambda (e.g. the C/4 companion)")
    ap.add_argument("--max-salient", type=int, default=0, help="salient-cache budget per head (a multiple of topk; 0: none)")
    ap.add_argument("--B", type=int, default=None, help="override the batch (profiling of a smaller case)")
    ap.add_argument("--H", type=int, default=None, help="override the query heads (KV heads scale along)")
    ap.add_argument("--N", type=int, default=None, help="override the sequence length")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-companions", dest="companions", action="store_false",
                    help="skip the other workloads that the default single-GPU run measures after the headline")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 0)

    from paper_2602_02180_b200 import synth

    w = synth.WORKLOADS[args.workload]
    if args.B or args.H or args.N:
        H = args.H or w.H
        w = w.with_(B=args.B or w.B, H=H, Hkv=max(1, H * w.Hkv // w.H), N=args.N or w.N)
    lam = w.k if args.topk is None else args.topk
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        run_reference(args, w, lam, rank, world)
        return

    import torch

    import paper_2602_02180_b200 as still

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the CUDA library has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist

        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    dev = torch.device("cuda", local_rank)

    if w.name == "c5":
        line = bench_decode(args, w, lam, still, synth, torch, dist, dev, rank, world)
    else:
        line = bench_prefill(args, w, lam, still, synth, torch, dist, dev, rank, world)
    if rank == 0:
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def _barrier(torch, dist):
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()


def _max_over_ranks(torch, dist, x, dev):
    if dist is None:
        return x
    t = torch.tensor([x], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def roofline_times(work, peaks):
    """Roofline time of a prefill call: the slower of tensor time and HBM time, with the nominal peaks
    (2.25 PFLOP/s dense bf16, 8 TB/s) and with this pool's measured ones (burst cuBLAS bf16, copy bandwidth)."""
    nominal = max(work["flops"] / 2.25e15, work["bytes"] / 8e12)
    measured = max(work["flops"] / (peaks["bf16_tflops"] * 1e12), work["bytes"] / (peaks["hbm_gbs"] * 1e9))
    return nominal, measured


def time_prefill(w, lam, steps, warmup, still, synth, torch, dist, dev, rank, sample_clocks=True, max_salient=0):
    """Runs warmup + steps prefill calls of workload w with topk lam on resident inputs.  Every timed step
    has its own CUDA-event pair; the K steps are also bracketed as a whole.  Returns the measurements and
    the tensors (for the end-to-end leg)."""
    wl = w.with_(k=lam, seed=w.seed + 100 * rank)
    Q, K, V = synth.make_qkv(wl, dev)
    Wq, Wk = synth.make_npmap_weights(wl, dev)
    p = still.StillParams(w.B, w.H, w.Hkv, w.d, w.C, lam, w.torch_dtype, max_salient=max_salient)
    Y = torch.empty_like(Q)
    T = -(-w.N // w.C)
    scores = torch.empty(w.B, w.H, w.N, dtype=torch.float32, device=dev)
    sel = torch.empty(w.B, w.H, T, max(lam, 1), dtype=torch.int32, device=dev)
    ws_bytes = still.workspace_bytes(p, w.N)
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device=dev)
    call = lambda: still.hybrid_attn_fwd(p, Q, K, V, Wq, Wk, Y=Y, scores=scores, sel_idx=sel, workspace=ws)  # noqa: E731

    for _ in range(warmup):
        call()
    launches_per_step = still.last_launch_count()
    _barrier(torch, dist)
    sampler = ClockSampler(dev.index or 0)
    if rank == 0 and sample_clocks:
        sampler.start()
    still.profile_enable(steps)
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
    ev[0].record()
    for i in range(steps):
        call()
        ev[i + 1].record()
    _barrier(torch, dist)
    ms_total = ev[0].elapsed_time(ev[-1])
    per_step = [ev[i].elapsed_time(ev[i + 1]) for i in range(steps)]
    kernel_ms = still.profile_collect()
    clocks = sampler.stop() if rank == 0 and sample_clocks else None
    assert still.device_status(ws) == (0, 0), "a device-side wait timed out"
    return {"ms_total": ms_total, "per_step": per_step, "kernel_ms": kernel_ms, "clocks": clocks,
            "launches_per_step": launches_per_step, "workspace_bytes": ws_bytes,
            "tensors": (p, Q, K, V, Wq, Wk)}


def prefill_companion(name, w, lam, steps, still, synth, torch, dev, max_salient=0):
    """One more workload in the same run (single GPU): ms per step (median of per-step event pairs), tokens/s
    and the whole-step fraction of the roofline time, with its own clock sample."""
    m = time_prefill(w, lam, steps, 3, still, synth, torch, None, dev, 0, max_salient=max_salient)
    del m["tensors"]
    torch.cuda.empty_cache()
    work = algorithmic_work(w, lam, max_salient)
    peaks = measured_peaks()
    nominal, measured = roofline_times(work, peaks)
    ms = statistics.median(m["per_step"])
    k_ms = statistics.median(m["kernel_ms"]) if m["kernel_ms"] else None
    out = {"workload": name, "max_salient": max_salient, "B": w.B, "H": w.H, "Hkv": w.Hkv, "d": w.d, "N": w.N, "chunk": w.C, "topk": lam,
           "steps": steps, "ms_per_step": ms, "tokens_per_s": w.B * w.N / (ms * 1e-3),
           "roofline_frac_nominal": nominal / (ms * 1e-3), "roofline_frac_measured": measured / (ms * 1e-3),
           "workspace_bytes": m["workspace_bytes"], "gpu_launches_per_step": m["launches_per_step"],
           "clocks": m["clocks"]}
    if k_ms:
        ach = work["flops_sa"] / (k_ms * 1e-3) / 1e12
        out["sa_kernel"] = {"ms": k_ms, "tflops": ach, "frac_of_burst_peak": ach / peaks["bf16_tflops"],
                            "frac_of_nominal_2250": ach / 2250.0}
    return out


def bench_prefill(args, w, lam, still, synth, torch, dist, dev, rank, world):
    warmup = max(args.warmup, 10)
    m = time_prefill(w, lam, args.steps, warmup, still, synth, torch, dist, dev, rank, max_salient=args.max_salient)
    p, Q, K, V, Wq, Wk = m.pop("tensors")
    ms_total = _max_over_ranks(torch, dist, m["ms_total"], dev)
    kernel_ms, clocks, launches_per_step = m["kernel_ms"], m["clocks"], m["launches_per_step"]
    ms_step = ms_total / args.steps
    value = world * w.B * w.N / (ms_step * 1e-3)

    work = algorithmic_work(w, lam, args.max_salient)
    peaks = measured_peaks()
    nominal, measured = roofline_times(work, peaks)
    k_ms = statistics.mean(kernel_ms) if kernel_ms else None
    fp32 = w.dtype == "fp32"
    roof = None
    if k_ms:
        ach = work["flops_sa"] / (k_ms * 1e-3) / 1e12
        peak = peaks["bf16_tflops"]
        roof = {"bound": "tensor", "kernel": "softmax-attention + merge", "achieved": ach, "peak": peak,
                "unit": "TFLOP/s", "frac": ach / peak, "peak_source": peaks["source"] + " (burst cuBLAS bf16)",
                "frac_of_sustained_peak": ach / peaks["bf16_tflops_sustained"], "frac_of_nominal_2250": ach / 2250.0,
                "kernel_ms": k_ms, "kernel_ms_median": statistics.median(kernel_ms),
                "kernel_share_of_step": k_ms / ms_step,
                "traffic": ncu_traffic(f"sa_{w.name}_k{lam}"),
                "whole_step_frac_of_nominal_roofline": nominal / (ms_step * 1e-3),
                "whole_step_frac_of_measured_roofline": measured / (ms_step * 1e-3)}
        if clocks and clocks.get("sm_mhz"):
            roof["kernel_mcycles_at_sampled_clock"] = k_ms * clocks["sm_mhz"] / 1e3
        if fp32:
            roof["bound"] = "alu"
            roof["note"] = "fp32 inputs run on FMA pipes; peak shown is the bf16 tensor peak for context"

    e2e = None
    if not args.no_e2e:
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        hQ, hK, hV = (t.cpu().pin_memory() for t in (Q, K, V))
        hWq, hWk = Wq.cpu().pin_memory(), Wk.cpu().pin_memory()
        hY = torch.empty_like(hQ).pin_memory()
        arena = torch.empty(still.host_arena_bytes(p, w.N), dtype=torch.uint8, device=dev)
        n_e2e = max(2, min(args.steps, 5))
        still.hybrid_attn_fwd_host(p, hQ, hK, hV, hWq, hWk, hY=hY, arena=arena)
        _barrier(torch, dist)
        t0 = time.perf_counter()
        e0.record()
        for _ in range(n_e2e):
            still.hybrid_attn_fwd_host(p, hQ, hK, hV, hWq, hWk, hY=hY, arena=arena)
        e1.record()
        _barrier(torch, dist)
        ms_e2e = max(e0.elapsed_time(e1), (time.perf_counter() - t0) * 1e3) / n_e2e
        ms_e2e = _max_over_ranks(torch, dist, ms_e2e, dev)
        h2d = sum(t.numel() * t.element_size() for t in (hQ, hK, hV, hWq, hWk))
        d2h = hY.numel() * hY.element_size()
        e2e = {"value": world * w.B * w.N / (ms_e2e * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "ms_per_step": ms_e2e, "steps": n_e2e}
        del arena, hQ, hK, hV, hY
    del Q, K, V
    torch.cuda.empty_cache()

    # The other workloads, in the same run (single GPU only): every shape once as written and once with a
    # quarter of each chunk selected, so that selection, NP-Map, state scan and merge run at scale.
    companions = None
    if world == 1 and args.companions and args.workload == "c3" and not (args.B or args.H or args.N or args.topk is not None):
        W = synth.WORKLOADS
        companions = [
            prefill_companion("c3 topk=C/4", W["c3"], 16, 5, still, synth, torch, dev),
            prefill_companion("c2", W["c2"], 64, 10, still, synth, torch, dev),
            prefill_companion("c2 topk=C/4", W["c2"], 16, 10, still, synth, torch, dev),
            prefill_companion("c4", W["c4"], 128, 2, still, synth, torch, dev),
            prefill_companion("c4 topk=C/4", W["c4"], 32, 2, still, synth, torch, dev),
            # a capped salient cache (local window 128 + at most 896 cached tokens per head, Sec. 4.3's setting): the
            # cost per token no longer grows with the sequence -- a quarter of the length takes a quarter of the time
            prefill_companion("c4 topk=C/4 max_salient=896", W["c4"], 32, 3, still, synth, torch, dev, max_salient=896),
            prefill_companion("c4 topk=C/4 max_salient=896 N=32768", W["c4"].with_(N=32768), 32, 5, still, synth, torch, dev,
                              max_salient=896),
            decode_companion("c5", W["c5"], 64, 48, still, synth, torch, dev),
            decode_companion("c5 topk=C/4", W["c5"], 16, 48, still, synth, torch, dev),
            decode_companion("c5 topk=C/4 max_salient=448", W["c5"], 16, 48, still, synth, torch, dev, max_salient=448),
        ]

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        import multiprocessing

        n_heads = max(1, min(multiprocessing.cpu_count(), w.B * w.H))
        total, threads, sample, _ = oracle_sample(w, lam, n_heads, 160 if w.N > 8192 else 256)
        cpu = {"value": w.B * w.N / total, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample}
        if companions is not None:
            cpu["local_vs_global_selection"] = [local_global_overlap(synth.WORKLOADS[n]) for n in ("c2", "c3", "c4")]

    return {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": warmup, "ms_per_step": ms_step, "ms_per_step_median": statistics.median(m["per_step"]),
        "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16" if not fp32 else "f32", "data": "synthetic",
        "config": {"workload": w.name, "B": w.B, "H": w.H, "Hkv": w.Hkv, "d": w.d, "N": w.N, "chunk": w.C,
                   "topk": lam, "max_salient": args.max_salient, "l2": "inputs larger than L2 (no flush)", "per_gpu_batch": w.B,
                   "timing": "K steps bracketed by one CUDA-event pair (ms_per_step, value); every step also has its own "
                             "pair (ms_per_step_median)"},
        "clocks": clocks, "e2e": e2e, "gpu_launches": launches_per_step * args.steps,
        "roofline": roof, "cpu_baseline": cpu,
        "algorithmic": {"flops_per_step": work["flops"], "bytes_per_step": work["bytes"]},
        "workspace_bytes": m["workspace_bytes"], "companions": companions,
    }


def decode_bytes(w, lam, t, max_salient=0):
    """Bytes a decode step at position t has to move: K and V rows of the routed history that at least one
    query head of the KV group selected (expected size of the union of the group's selections:
    1 - (1 - lam/C)^group of the rows; all rows when lam = C), read once per KV head, plus the two-chunk local
    region and, when the linear branch is in use, its state."""
    rep = w.H // w.Hkv
    union = 1.0 - (1.0 - lam / w.C) ** rep if lam > 0 else 0.0
    n_chunks = max(t // w.C - 1, 0)
    if max_salient > 0 and lam > 0:   # only the last max_salient / lam routed chunks are still cached
        n_chunks = min(n_chunks, max_salient // lam)
    n_hist = n_chunks * w.C * union
    return (w.B * w.Hkv * (n_hist + 2 * w.C) * w.d * 2 * 2 +
            (w.B * w.H * 2 * w.d_f * (w.d + 1) * 4 if (lam < w.C or max_salient > 0) else 0))


def time_decode(w, lam, n_steps, warmup, still, synth, torch, dist, dev, rank, reserve=0, max_salient=0):
    """Summarises the prefix into a decode state with the prefill, then times n_steps decode steps (one event
    pair per step and one around all of them)."""
    p = still.StillParams(w.B, w.H, w.Hkv, w.d, w.C, lam, w.torch_dtype, max_salient=max_salient)
    cap = w.N + n_steps + warmup + reserve + 8
    state_bytes = still.state_bytes(p, cap)
    state = torch.zeros(state_bytes, dtype=torch.uint8, device=dev)
    Wq, Wk = synth.make_npmap_weights(w, dev)
    wl = w.with_(seed=w.seed + 100 * rank)
    Q, K, V = synth.make_qkv(wl, dev)
    ws = torch.empty(still.workspace_bytes(p, w.N), dtype=torch.uint8, device=dev)
    still.hybrid_attn_fwd(p, Q, K, V, Wq, Wk, state=state, state_max_tokens=cap, workspace=ws, want_y=False)
    torch.cuda.synchronize()
    del Q, K, V, ws
    torch.cuda.empty_cache()
    t = w.N
    ins = [synth.make_decode_inputs(wl, i, dev) for i in range(8)]
    y = torch.empty(w.B, w.H, w.d, dtype=w.torch_dtype, device=dev)
    for i in range(warmup):
        q, k, v = ins[i % 8]
        still.hybrid_attn_step(p, state, cap, t, q, k, v, Wq, Wk, y=y)
        t += 1
    launches = still.last_launch_count()
    _barrier(torch, dist)
    sampler = ClockSampler(dev.index or 0)
    if rank == 0:
        sampler.start()
    still.profile_enable(n_steps)
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(n_steps + 1)]
    ev[0].record()
    for i in range(n_steps):
        q, k, v = ins[i % 8]
        still.hybrid_attn_step(p, state, cap, t, q, k, v, Wq, Wk, y=y)
        ev[i + 1].record()
        t += 1
    _barrier(torch, dist)
    ms_total = ev[0].elapsed_time(ev[-1])
    per_step = [ev[i].elapsed_time(ev[i + 1]) for i in range(n_steps)]
    kernel_ms = still.profile_collect()
    clocks = sampler.stop() if rank == 0 else None
    assert still.device_status(state)[0] == 0
    return {"ms_total": ms_total, "per_step": per_step, "kernel_ms": kernel_ms, "clocks": clocks, "launches": launches,
            "state_bytes": state_bytes, "t": t, "ctx": (p, state, cap, ins, y, Wq, Wk, wl)}


def decode_companion(name, w, lam, n_steps, still, synth, torch, dev, max_salient=0):
    m = time_decode(w, lam, n_steps, 3, still, synth, torch, None, dev, 0, max_salient=max_salient)
    del m["ctx"]
    torch.cuda.empty_cache()
    peaks = measured_peaks()
    ms = statistics.median(m["per_step"])
    by = decode_bytes(w, lam, m["t"], max_salient)
    return {"workload": name, "max_salient": max_salient, "B": w.B, "H": w.H, "Hkv": w.Hkv, "d": w.d, "prefix": w.N, "chunk": w.C, "topk": lam,
            "steps": n_steps, "ms_per_step": ms, "ms_per_step_max": max(m["per_step"]),
            "tokens_per_s": w.B / (ms * 1e-3), "algorithmic_bytes_per_step": by,
            "roofline_frac_nominal": (by / 8e12) / (ms * 1e-3),
            "roofline_frac_measured": (by / (peaks["hbm_gbs"] * 1e9)) / (ms * 1e-3),
            "state_bytes": m["state_bytes"], "gpu_launches_per_step": m["launches"], "clocks": m["clocks"]}


def bench_decode(args, w, lam, still, synth, torch, dist, dev, rank, world):
    """c5: the prefix is summarised into a decode state by the prefill, then `steps` decode steps
    are timed.  HBM-bound: the salient K/V history is read once per KV head per step."""
    n_steps = args.steps
    warmup = max(args.warmup, 3)
    m = time_decode(w, lam, n_steps, warmup, still, synth, torch, dist, dev, rank, reserve=64 + w.steps,
                    max_salient=args.max_salient)
    p, state, cap, ins, y, Wq, Wk, wl = m.pop("ctx")
    t, launches, clocks, kernel_ms = m["t"], m["launches"], m["clocks"], m["kernel_ms"]
    ms_total = _max_over_ranks(torch, dist, m["ms_total"], dev)
    ms_step = ms_total / n_steps
    peaks = measured_peaks()
    by = decode_bytes(w, lam, t, args.max_salient)
    k_ms = statistics.mean(kernel_ms) if kernel_ms else ms_step
    ach = by / (k_ms * 1e-3) / 1e9
    roof = {"bound": "hbm", "kernel": "split-KV attend", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s",
            "frac": ach / peaks["hbm_gbs"], "peak_source": peaks["source"], "kernel_ms": k_ms,
            "traffic": ncu_traffic(f"attend_{w.name}_k{lam}")}
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    # end to end: every step copies that step's q, k, v from pinned host memory and reads y back
    e2e = None
    if not args.no_e2e:
        hins = [tuple(x.cpu().pin_memory() for x in ins[i]) for i in range(8)]
        dq, dk, dv = (torch.empty_like(x) for x in ins[0])
        hy = torch.empty(w.B, w.H, w.d, dtype=w.torch_dtype).pin_memory()
        n_e2e = min(n_steps, 64)
        _barrier(torch, dist)
        t0 = time.perf_counter()
        e0.record()
        for i in range(n_e2e):
            hq, hk, hv = hins[i % 8]
            dq.copy_(hq, non_blocking=True)
            dk.copy_(hk, non_blocking=True)
            dv.copy_(hv, non_blocking=True)
            still.hybrid_attn_step(p, state, cap, t, dq, dk, dv, Wq, Wk, y=y)
            hy.copy_(y, non_blocking=True)
            torch.cuda.current_stream().synchronize()
            t += 1
        e1.record()
        _barrier(torch, dist)
        ms_e2e = max(e0.elapsed_time(e1), (time.perf_counter() - t0) * 1e3) / n_e2e
        ms_e2e = _max_over_ranks(torch, dist, ms_e2e, dev)
        e2e = {"value": world * w.B / (ms_e2e * 1e-3), "unit": UNIT,
               "h2d_bytes_per_step": sum(x.numel() * x.element_size() for x in hins[0]),
               "d2h_bytes_per_step": hy.numel() * hy.element_size(), "ms_per_step": ms_e2e, "steps": n_e2e}

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu = oracle_decode_sample(w, lam)

    return {
        "metric": "hybrid-attn decode tokens/s/layer at Llama-3-8B shape", "value": world * w.B / (ms_step * 1e-3),
        "unit": UNIT, "n_gpus": world, "steps": n_steps, "warmup": warmup, "ms_per_step": ms_step,
        "ms_per_step_median": statistics.median(m["per_step"]),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": w.name, "B": w.B, "H": w.H, "Hkv": w.Hkv, "d": w.d, "prefix": w.N, "chunk": w.C,
                   "topk": lam, "max_salient": args.max_salient, "l2": "K/V history larger than L2 (no flush)"},
        "clocks": clocks, "e2e": e2e, "gpu_launches": launches * n_steps, "roofline": roof, "cpu_baseline": cpu,
    }


if __name__ == "__main__":
    main()

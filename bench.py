#!/usr/bin/env python
"""Benchmark of the Token Filtering layer step (filter + pruned attention) on B200.

One step = one pass of the whole hot path (similarity scan, fusion, selection, attention for
retained tokens) over one layer's Q/K/V of a synthetic, seeded workload.  Prints ONE JSON line.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c5|c4|c3|c2|c1]
                    [--prune 0.5] [--impl ours|reference] [--sweep]

The default workload is configuration 5, the largest that fits one GPU (Mistral-7B shape, batch 8 x
16384 tokens, window 4096).  --sweep prints one line per configuration and pruning ratio and the
1K-32K sequence sweep of configuration 5.

value   : tokens/s per layer, inputs resident in HBM, timed with CUDA events on the launch stream.
e2e     : same metric through tf_layer_filter_host (pinned host buffers; copies inside the timing).
roofline: the dominant kernel against the measured peak of the resource that bounds it.
cpu_baseline / --impl reference: the fp64 oracle, as it stands, on this machine's host cores.
N > 1   : one process per GPU (under torchrun, or started from here when no launcher set WORLD_SIZE);
          sequences are independent, so every rank runs its own replica of the workload with no
          data-path collective ("weak" scaling).
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

import numpy as np
import torch

METRIC = "filtered-attention prefill tokens/s per layer at 50% prune"
UNIT = "tokens/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            d = json.load(open(p))
            return {k: float(d[k]) for k in FALLBACK_PEAKS}, "measured"
        except Exception:
            pass
    return dict(FALLBACK_PEAKS), "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU with nvidia-smi while the timed region runs."""

    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-i", str(self.index), "-lms", "100"], stdout=subprocess.PIPE, text=True)
            self.t = threading.Thread(target=lambda: [self.lines.append(l) for l in self.proc.stdout], daemon=True)
            self.t.start()
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for l in self.lines:
            f = [x.strip() for x in l.split(",")]
            if len(f) < 6:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except ValueError:
                continue
            for n, v in zip(names, f[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def attention_flops(kept_idx: np.ndarray, n_kept: np.ndarray, Hq: int, d: int, window: int, retained_only: bool = False) -> float:
    """4*d*Hq * sum over retained tokens of the number of visible keys (the work actually needed).
    retained_only: a retained query sees retained tokens only (TF_KV_RETAINED)."""
    tot = 0.0
    for b in range(kept_idx.shape[0]):
        t = kept_idx[b, : n_kept[b]].astype(np.int64)
        if retained_only:
            first = np.searchsorted(t, t - window + 1) if window > 0 else np.zeros_like(t)
            vis = np.arange(t.size) - first + 1
        else:
            vis = t + 1
            if window > 0:
                vis = np.minimum(vis, window)
        tot += float(vis.sum())
    return 4.0 * d * Hq * tot


# --------------------------------------------------------------------------------------------------
def make_ring(wl, device, min_bytes, max_layers=8):
    """Distinct layers' (Q,K,V) of the workload until their total size exceeds min_bytes (> L2)."""
    ring, total = [], 0
    layers = list(range(max_layers)) if wl.stack is not None else [0]
    for l, q, k, v in wl.layer_qkv(layers, device):
        ring.append((q, k, v))
        total += sum(t.numel() * t.element_size() for t in (q, k, v)) * 4 // 3   # + O
        if total >= min_bytes and len(ring) >= 2:
            break
    if wl.stack is None:      # config 1 has a single layer: rotate seeds instead
        from paper_2512_07090_b200 import workloads as W
        for i in range(1, 4):
            ring.append(tuple(t.to(device) for t in W.duplicate_qkv(wl.batch, wl.seq, 32, 32, 128, 0.25, 0.05,
                                                                    wl.seed + 100 * i, wl.dtype)))
    return ring


def oracle_sample(wl, ring_cpu, prune, budget_s=12.0):
    """Time the fp64 oracle on a bounded sample of the workload: similarities, fusion and selection
    in full for one layer; attention on a seeded subset of retained rows, scaled by exact flops."""
    import oracle
    q, k, v = ring_cpu
    B, S, Hq, d = q.shape
    t0 = time.perf_counter()
    r = oracle.layer_filter(q, k, v, prune_ratio=prune, warmup_tokens=4, window=wl.window, attention=False)
    t_filter = time.perf_counter() - t0
    full_flops = attention_flops(r["kept_idx"], r["n_kept"], Hq, d, wl.window)
    rng = np.random.default_rng(0)
    rows = []
    for b in range(B):
        kept = r["kept_idx"][b, : r["n_kept"][b]]
        for t in kept:
            rows.append((b, int(t)))
    rows = np.array(rows, np.int32)
    rng.shuffle(rows)
    # grow the sample until it costs a few seconds, then one timed run sized to the budget
    n, t_attn, done_flops = min(len(rows), 64), 0.0, 0.0
    while True:
        sub = rows[:n]
        trip = np.array([(b, t, h) for b, t in sub for h in range(Hq)], np.int32)
        t0 = time.perf_counter()
        oracle.attention_rows(q, k, v, r["keep_mask"], trip, window=wl.window)
        t_attn = time.perf_counter() - t0
        vis = sub[:, 1].astype(np.int64) + 1
        if wl.window > 0:
            vis = np.minimum(vis, wl.window)
        done_flops = 4.0 * d * Hq * float(vis.sum())
        if t_attn > budget_s / 3 or n >= len(rows):
            break
        n = min(len(rows), max(n * 2, int(n * (budget_s * 0.8) / max(t_attn, 1e-3))))
    est = t_filter + t_attn * (full_flops / max(done_flops, 1.0))
    passes = 1
    if n >= len(rows) and est < budget_s / 2:
        # the whole layer costs well under the budget: time it several times over, about budget_s of CPU work in all
        passes = int(min(40, max(2, budget_s * 0.8 // est)))
        t0 = time.perf_counter()
        for _ in range(passes):
            rr = oracle.layer_filter(q, k, v, prune_ratio=prune, warmup_tokens=4, window=wl.window, attention=False)
            oracle.attention_rows(q, k, v, rr["keep_mask"], trip, window=wl.window)
        est = (time.perf_counter() - t0) / passes
    return {"value": B * S / est, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
            "sample": f"one layer: similarity+fusion+selection in full ({t_filter:.2f} s), attention on {n} of "
                      f"{len(rows)} retained rows x {Hq} heads ({t_attn:.2f} s) scaled by exact flops "
                      f"({done_flops / full_flops:.4f} of the layer)"
                      + (f"; mean of {passes} passes over the whole layer ({est * passes:.1f} s)" if passes > 1 else "")}


def run_reference(args, wl):
    """--impl reference: the oracle as it stands, on host cores; each step a bounded sample."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    layers = [0]
    _, q, k, v = next(wl.layer_qkv(layers, "cpu"))
    ring_cpu = (q.float().numpy(), k.float().numpy(), v.float().numpy())
    budget = max(2.0, min(12.0, 90.0 / max(1, args.steps + args.warmup)))
    vals = []
    for i in range(args.warmup + args.steps):
        r = oracle_sample(wl, ring_cpu, args.prune, budget_s=budget)
        if i >= args.warmup:
            vals.append(r)
    v = statistics.mean(x["value"] for x in vals)
    cb = dict(vals[-1]); cb["value"] = v
    out = {"impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
           "warmup": args.warmup, "ms_per_step": 1e3 * wl.batch * wl.seq / v, "higher_is_better": True,
           "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
           "config": workload_config(wl, args), "cpu_baseline": cb,
           "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(out))


def run_decode(args, wl, tfb, dev, local):
    """Online decode step (Algorithm 1 per token + threshold feedback + single-query attention): B sequences,
    a cache of seq tokens of the workload's layer-0 K/V, the new token at the last position.  Not the headline
    metric; one JSON line of its own."""
    _, q, k, v = next(wl.layer_qkv([0], dev))
    B, S, Hq, d = q.shape
    Hkv = k.shape[2]
    ctx = tfb.Context(local)
    params = tfb.default_params(prune_ratio=args.prune, warmup_tokens=4)
    st = tfb.DecodeState(B, Hkv, dev, tau0=10.0)      # a threshold no score reaches: every step pays the attention
    shape = tfb.make_shape(None, k, v, window=wl.window, n_q_heads=Hq)
    O = torch.empty(B, Hq, d, dtype=q.dtype, device=dev)
    shape.q_stride[:] = [q.stride(0), 0, q.stride(2)]
    shape.o_stride[:] = [O.stride(0), 0, O.stride(1)]
    ctx.ensure_workspace(shape, params)               # the decode step keeps its split-key partial results there
    pos = torch.full((B,), S - 1, dtype=torch.int32, device=dev)
    score = torch.empty(B, device=dev); skip = torch.empty(B, dtype=torch.uint8, device=dev)
    for _ in range(max(3, args.warmup)):
        ctx.tf_decode_step(shape, params, 0.0, q[:, S - 1], k, v, pos, st, O, score, skip)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    launches0 = ctx.launches
    e0.record()
    for _ in range(args.steps):
        ctx.tf_decode_step(shape, params, 0.0, q[:, S - 1], k, v, pos, st, O, score, skip)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / args.steps
    pk, pk_kind = peaks()
    vis = min(S, wl.window) if wl.window > 0 else S
    cache_bytes = 2.0 * B * Hkv * vis * d * q.element_size()          # K and V rows one query group reads once
    print(json.dumps({"metric": "online decode steps/s per layer (no skip, cache = seq tokens)", "value": B / (ms * 1e-3),
                      "unit": "tokens/s", "n_gpus": 1, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms,
                      "higher_is_better": True, "dtype": "bf16" if q.dtype == torch.bfloat16 else "f32", "data": "synthetic",
                      "config": workload_config(wl, args), "gpu_launches": int(ctx.launches - launches0),
                      "roofline": {"kernel": "decode_attention", "bound": "hbm", "achieved": cache_bytes / (ms * 1e-3) / 1e9,
                                   "peak": pk["hbm_gbs"], "unit": "GB/s", "frac": cache_bytes / (ms * 1e-3) / 1e9 / pk["hbm_gbs"],
                                   "traffic": ncu_traffic(wl.name, "decode_step", 0.0),
                                   "peak_kind": pk_kind, "algorithmic_per_launch": cache_bytes}}))
    ctx.close()


def rank_seed(seed: int, rank: int) -> int:
    """Every rank of an N-GPU run works on its own replica of the workload (sequences are independent)."""
    return seed + 7919 * rank


def max_over_ranks(ms: float, dist, device) -> float:
    """A multi-rank run is as slow as its slowest rank."""
    if dist is None:
        return ms
    t = torch.tensor([ms], device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def workload_config(wl, args):
    return {"workload": f"{wl.name}: {wl.stack.name if wl.stack else 'llama2-7b head shape'} one layer, batch {wl.batch}, "
                        f"seq {wl.seq}, {wl.n_q_heads} q heads / {wl.n_kv_heads} kv heads, head_dim 128, "
                        f"{'bf16' if wl.dtype == torch.bfloat16 else 'fp32'}, window {wl.window}, prune {args.prune}"
                        + (", retained keys only" if getattr(args, "kv_visibility", "all") == "retained" else ""),
            "global_batch": wl.batch * args.gpus, "seq_len": wl.seq, "prune_ratio": args.prune,
            "parallelism": f"replicas x{args.gpus} (independent sequences, no collective)",
            "l2": "inputs rotate over distinct layers whose total size exceeds the 126 MB L2"}


def ncu_traffic(workload: str, kernel: str, prune: float):
    """DRAM bytes per launch (read + write) of a kernel from the ncu summaries: profiles/dram_traffic.txt holds one
    line per capture, `workload kernel prune read_bytes write_bytes`; None where no capture was taken."""
    path = os.path.join(ROOT, "profiles", "dram_traffic.txt")
    if not os.path.exists(path):
        return None
    for line in open(path):
        f = line.split()
        if len(f) >= 5 and not line.startswith("#") and f[0] == workload and f[1] == kernel and abs(float(f[2]) - prune) < 1e-9:
            return int(f[3]) + int(f[4])
    return None


NOMINAL = {"hbm_gbs": 8000.0, "bf16_tflops": 2250.0}   # the figures the targets are stated against


def timed_repeats(fn, steps, sync_all, dist, dev, min_total_ms=300.0, max_repeats=200):
    """Times `steps` calls of fn(i) between two CUDA events, several times over (each repeat bracketed by a
    synchronise, and a barrier when there are ranks), until the timed work adds up to min_total_ms, so that the
    clock sampler sees the GPU under this load; returns (median ms of one repeat, all repeats, slowest rank each)."""
    times = []
    repeats = 3
    i0 = 0
    while len(times) < repeats:
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        sync_all()
        e0.record()
        for i in range(steps):
            fn(i0 + i)
        e1.record()
        sync_all()
        i0 += steps
        times.append(max_over_ranks(e0.elapsed_time(e1), dist, dev))
        if len(times) == 1:   # the same count on every rank: it comes from the slowest rank's first repeat
            repeats = int(min(max_repeats, max(3, -(-min_total_ms // max(times[0], 1e-3)))))
    return statistics.median(times), times


def measure(wl, args, tfb, dev, local, dist, world, rank, headline=True):
    """One workload at one pruning ratio: the whole layer step, each stage alone, and (headline only) the host-buffer
    entry point and the oracle on host cores.  Returns the JSON object of the line (rank 0) or None."""
    ring = make_ring(wl, dev, min_bytes=300 << 20)
    B, S, Hq, d = ring[0][0].shape
    Hkv = ring[0][1].shape[2]
    es = ring[0][0].element_size()
    ctx = tfb.Context(local)
    O = torch.empty_like(ring[0][0])
    shape = tfb.make_shape(ring[0][0], ring[0][1], ring[0][2], O, window=wl.window)
    params = tfb.default_params(prune_ratio=args.prune, warmup_tokens=4,
                                kv_visibility=tfb.TF_KV_RETAINED if args.kv_visibility == "retained" else tfb.TF_KV_ALL)
    ctx.ensure_workspace(shape, params)
    sim_k = torch.empty(B, S, Hkv, device=dev); sim_v = torch.empty_like(sim_k)
    score = torch.empty(B, S, device=dev)
    keep = torch.empty(B, S, dtype=torch.uint8, device=dev)
    idx = torch.empty(B, S, dtype=torch.int32, device=dev)
    nk = torch.empty(B, dtype=torch.int32, device=dev)

    def step(i):
        q, k, v = ring[i % len(ring)]
        ctx.tf_layer_filter(shape, params, q, k, v, O, score, keep, idx, nk)

    def sync_all():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    for i in range(args.warmup):
        step(i)
    sync_all()
    code, det = ctx.tf_get_status()
    if code != tfb.TF_OK:
        raise RuntimeError(f"device status {code}: {det}")
    scan_kernel, attn_kernel = ctx.tf_last_kernels()

    # ---- timed region: K whole steps, repeated; the median repeat is the figure -----------------------
    sampler = ClockSampler(local)
    sampler.start()
    l0 = ctx.launches
    ms, reps = timed_repeats(step, args.steps, sync_all, dist, dev)
    launches = (ctx.launches - l0) // len(reps)
    busy_ms = sum(reps)

    # ---- per-kernel durations: each stage entry point alone, K launches back to back ---------------
    # (events around the whole loop, so launch latency is not charged to the kernel; every ring entry
    #  first gets its own similarities / scores / kept list from one pass through the stages)
    names = ("kv_stats", "score_fuse", "select", "score_select", "pruned_attention")
    per = {n: 0.0 for n in names}
    per_first = {n: 0.0 for n in names}
    flops = 0.0
    state = []
    for q, k, v in ring:
        sk, sv = torch.empty_like(sim_k), torch.empty_like(sim_v)
        sc, ix, n_ = torch.empty_like(score), torch.empty_like(idx), torch.empty_like(nk)
        ctx.tf_kv_stats(shape, params, k, v, sk, sv)
        ctx.tf_score_fuse(shape, params, sk, sv, sc)
        ctx.tf_select(shape, params, sc, keep, ix, n_)
        torch.cuda.synchronize()
        flops += attention_flops(ix.cpu().numpy(), n_.cpu().numpy(), Hq, d, wl.window,
                                 args.kv_visibility == "retained") / len(ring)
        state.append((sk, sv, sc, ix, n_))

    def stage(name, i):
        q, k, v = ring[i % len(ring)]
        sk, sv, sc, ix, n_ = state[i % len(ring)]
        if name == "kv_stats": ctx.tf_kv_stats(shape, params, k, v, sim_k, sim_v)
        elif name == "score_fuse": ctx.tf_score_fuse(shape, params, sk, sv, score)
        elif name == "select": ctx.tf_select(shape, params, sc, keep, idx, nk)
        elif name == "score_select": ctx.tf_score_select(shape, params, sk, sv, score, keep, idx, nk)   # a3 + a4 as the layer step runs them
        else: ctx.tf_pruned_attention(shape, params, q, k, v, ix, n_, O)

    # Each stage's K launches are captured into a CUDA graph (the ring position advances inside it) and the graph is
    # replayed, so that the host's call path (about 10 us per call) is not what gets timed for the small kernels;
    # if capture is not possible the plain loop is timed and "host_bound" says so.
    host_bound = {}
    for n in names:
        for i in range(3):
            stage(n, i)
        torch.cuda.synchronize()
        graph = None
        try:
            side = torch.cuda.Stream()
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                for i in range(3):
                    stage(n, i)
                g_ = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g_, stream=side):
                    for i in range(args.steps):
                        stage(n, i)
            torch.cuda.current_stream().wait_stream(side)
            torch.cuda.synchronize()
            graph = g_
        except Exception as ex:                       # noqa: BLE001  (the reason goes into the line)
            host_bound[n] = f"graph capture failed ({type(ex).__name__}); plain loop timed"
            torch.cuda.synchronize()
        if graph is not None:
            graph.replay()
            torch.cuda.synchronize()

            def replay(i, graph=graph):
                if i % args.steps == 0:
                    graph.replay()
            t, ts = timed_repeats(replay, args.steps, sync_all, None, dev, min_total_ms=100.0)
        else:
            t, ts = timed_repeats(lambda i, n=n: stage(n, i), args.steps, sync_all, None, dev, min_total_ms=100.0)
        per[n] = t / args.steps
        per_first[n] = statistics.median(ts[:3]) / args.steps     # before the load has lasted tens of milliseconds
    clocks = sampler.stop()

    tokens_per_step = B * S * world
    value = tokens_per_step * args.steps / (ms * 1e-3)

    # ---- end to end through the host entry point ----------------------------------------------------
    e2e = None
    if headline:
        qh, kh, vh = (t.cpu().pin_memory() for t in ring[0])
        oh = torch.empty_like(qh).pin_memory()
        nh = torch.empty(B, dtype=torch.int32).pin_memory()
        hshape = tfb.make_shape(qh, kh, vh, oh, window=wl.window)
        e2e_steps = max(3, min(args.steps, 10))
        for _ in range(2):
            ctx.tf_layer_filter_host(hshape, params, qh, kh, vh, oh, None, None, None, nh)
        sync_all()
        f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        f0.record()
        for _ in range(e2e_steps):
            ctx.tf_layer_filter_host(hshape, params, qh, kh, vh, oh, None, None, None, nh)
        f1.record()
        sync_all()
        e2e_ms = max_over_ranks(f0.elapsed_time(f1), dist, dev)
        e2e = {"value": tokens_per_step * e2e_steps / (e2e_ms * 1e-3), "unit": UNIT,
               "h2d_bytes_per_step": int((qh.numel() + kh.numel() + vh.numel()) * es),
               "d2h_bytes_per_step": int(oh.numel() * es + nh.numel() * 4), "steps": e2e_steps}
        del qh, kh, vh, oh

    out = None
    if rank == 0:
        pk, pk_kind = peaks()
        kv_bytes = 2.0 * B * S * Hkv * d * es + 8.0 * B * S * Hkv
        sel_bytes = (4.0 * Hkv * 2 + 4.0) * B * S + 9.0 * B * S          # fusion: sims in, score out; selection: score in, mask + index out
        # us: median launch time over >= 100 ms of back-to-back launches (sustained); us_first: over the first three
        # repeats (what a peak measured as a short burst compares with)
        kern = {n: {"us": per[n] * 1e3, "us_first": per_first[n] * 1e3} for n in names}
        kv = kern["kv_stats"]
        kv.update(bound="hbm", achieved=kv_bytes / (per["kv_stats"] * 1e-3) / 1e9, unit="GB/s", peak=pk["hbm_gbs"])
        kv["frac"] = kv["achieved"] / pk["hbm_gbs"]
        kv["frac_of_nominal"] = kv["achieved"] / NOMINAL["hbm_gbs"]
        kv["frac_first"] = kv_bytes / (per_first["kv_stats"] * 1e-3) / 1e9 / pk["hbm_gbs"]
        # scoring + selection together (steps a1-a4): their bytes over the sum of their times (a3 + a4 through the entry
        # point that runs them the way the layer step does: one launch where a cluster takes the sequence, else two)
        t_filter = per["kv_stats"] + per["score_select"]
        ach_f = (kv_bytes + sel_bytes) / (t_filter * 1e-3) / 1e9
        kern["scoring_and_selection"] = {"us": t_filter * 1e3, "bound": "hbm", "achieved": ach_f, "unit": "GB/s",
                                         "peak": pk["hbm_gbs"], "frac": ach_f / pk["hbm_gbs"],
                                         "frac_of_nominal": ach_f / NOMINAL["hbm_gbs"]}
        long_run = busy_ms > 2000.0
        tpeak = pk["bf16_tflops_sustained"] if long_run else pk["bf16_tflops"]
        ach = flops / (per["pruned_attention"] * 1e-3) / 1e12
        pa = kern["pruned_attention"]
        if wl.dtype == torch.bfloat16:
            pa.update(bound="tensor", achieved=ach, unit="TFLOP/s", peak=tpeak, frac=ach / tpeak,
                      frac_of_burst=ach / pk["bf16_tflops"], frac_of_sustained=ach / pk["bf16_tflops_sustained"],
                      frac_of_nominal=ach / NOMINAL["bf16_tflops"],
                      frac_first=flops / (per_first["pruned_attention"] * 1e-3) / 1e12 / pk["bf16_tflops"])
        else:   # fp32 on the CUDA cores: 148 SMs x 128 lanes x 2 flop x max clock
            alu = 148 * 128 * 2 * 1.965e-3
            pa.update(bound="alu", achieved=ach, unit="TFLOP/s", peak=alu, frac=ach / alu)
        dom = max(names, key=lambda n: per[n])
        traffic = ncu_traffic(wl.name, dom, args.prune) if args.kv_visibility == "all" else None
        roof = {"kernel": dom, "bound": kern[dom].get("bound", "latency"), "achieved": kern[dom].get("achieved"),
                "peak": kern[dom].get("peak"), "unit": kern[dom].get("unit"), "frac": kern[dom].get("frac"),
                "traffic": traffic, "peak_kind": f"{pk_kind} ({'sustained' if long_run else 'burst'} bf16)" if dom == "pruned_attention" else pk_kind,
                "algorithmic_per_launch": flops if dom == "pruned_attention" else kv_bytes}
        cfg = workload_config(wl, args)
        cfg["timing"] = (f"median of {len(reps)} repeats of {args.steps} steps ({busy_ms:.0f} ms timed in all); "
                         f"per-kernel: each stage alone, {args.steps} launches replayed from a CUDA graph, same scheme")
        cfg["kernels_chosen"] = {"scan": scan_kernel, "attention": attn_kernel}
        if host_bound:
            cfg["host_bound"] = host_bound
        out = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
               "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak",
               "vs_baseline": None, "dtype": "bf16" if wl.dtype == torch.bfloat16 else "f32", "data": "synthetic",
               "config": cfg, "clocks": clocks, "gpu_launches": int(launches), "roofline": roof, "kernels": kern}
        if e2e is not None:
            out["e2e"] = e2e
        if headline and not args.no_cpu_baseline and world == 1 and args.kv_visibility == "all":   # the baseline arm times the default reading
            q, k, v = ring[0]
            out["cpu_baseline"] = oracle_sample(wl, (q.float().cpu().numpy(), k.float().cpu().numpy(),
                                                     v.float().cpu().numpy()), args.prune)
            out["cpu_baseline"]["c1_whole_layer_s"] = oracle_c1_times()
    ctx.close()
    del ring, state
    torch.cuda.empty_cache()
    return out


def oracle_c1_times():
    """Configuration 1 (B1 S128, 32 heads, fp32, 50 % pruning) through the whole oracle, on one thread and on all."""
    import oracle
    from paper_2512_07090_b200 import workloads as W
    wl = W.WORKLOADS["c1"]
    _, q, k, v = next(wl.layer_qkv([0], "cpu"))
    q, k, v = q.numpy(), k.numpy(), v.numpy()
    n_all = oracle.num_threads()
    res = {}
    for label, n in (("threads_1", 1), (f"threads_{n_all}", n_all)):
        oracle.set_num_threads(n)
        oracle.layer_filter(q, k, v, prune_ratio=0.5, warmup_tokens=4)
        t0 = time.perf_counter()
        for _ in range(5):
            oracle.layer_filter(q, k, v, prune_ratio=0.5, warmup_tokens=4)
        res[label] = (time.perf_counter() - t0) / 5
    oracle.set_num_threads(n_all)
    return res


def spawn_ranks(n: int) -> int:
    """`python bench.py --gpus N` without a launcher: start the N ranks here (one process per GPU, torchrun's
    environment, rendezvous on 127.0.0.1) with the same arguments and return their exit code."""
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}", "--master-addr", "127.0.0.1",
           "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.run(cmd).returncode


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="c5",
                    help="c1..c5; the default is the largest single-GPU configuration (Mistral-7B shape, batch 8 x 16384 tokens, window 4096)")
    ap.add_argument("--prune", type=float, default=0.5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--kv-visibility", default="all", choices=["all", "retained"],
                    help="retained: kept queries attend kept keys only (a different, smaller computation)")
    ap.add_argument("--decode", action="store_true",
                    help="measure the online decode step (one new token per sequence against a cache of seq tokens) instead")
    ap.add_argument("--sweep", action="store_true",
                    help="one line per configuration and pruning ratio (c1-c5), then configuration 5 at 1K-32K tokens; "
                         "device-resident figures only")
    ap.add_argument("--batch", type=int, default=0, help="override the workload's batch (a reduced case for profiler captures; named in config.workload)")
    ap.add_argument("--seq", type=int, default=0, help="override the workload's sequence length (same purpose)")
    ap.add_argument("--backend", default="nccl", help="process-group backend of an N > 1 run (gloo: CPU-only test of the launch path)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(spawn_ranks(args.gpus))

    from paper_2512_07090_b200 import workloads as W
    wl = W.WORKLOADS[args.workload]
    if args.impl == "reference":
        run_reference(args, wl)
        return

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if args.backend == "gloo":      # launch-path check without GPUs: ranks, seeds, barrier, max over ranks, one line
        import torch.distributed as dist
        dist.init_process_group("gloo")
        seed = rank_seed(wl.seed, rank)
        slow = max_over_ranks(1.0 + rank, dist, "cpu")
        dist.barrier()
        if rank == 0:
            print(json.dumps({"launch_check": True, "n_gpus": world, "slowest_ms": slow, "seed_rank0": seed,
                              "config": workload_config(wl, args)}))
        dist.destroy_process_group()
        return

    from paper_2512_07090_b200 import binding as tfb
    torch.cuda.set_device(local)
    dev = f"cuda:{local}"
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device(dev))
    import dataclasses
    base_seed = {n: w.seed for n, w in W.WORKLOADS.items()}
    wl = dataclasses.replace(wl, seed=rank_seed(wl.seed, rank))
    if args.batch or args.seq:
        wl = dataclasses.replace(wl, batch=args.batch or wl.batch, seq=args.seq or wl.seq,
                                 name=wl.name + (f"-b{args.batch}" if args.batch else "") + (f"-s{args.seq}" if args.seq else ""))

    tfb.lib()   # fails loudly if the CUDA library is not built
    if args.decode:
        run_decode(args, wl, tfb, dev, local)
        return
    if args.sweep:
        seeded = {n: dataclasses.replace(w, seed=rank_seed(base_seed[n], rank)) for n, w in W.WORKLOADS.items()}
        cases = [(seeded[n], r) for n in ("c1", "c2", "c3", "c4", "c5") for r in seeded[n].prune_ratios]
        cases += [(dataclasses.replace(seeded["c5"], name=f"c5-s{s // 1024}k", seq=s), 0.5)
                  for s in (1024, 2048, 4096, 8192, 16384, 32768)]
        for w, r in cases:
            a = argparse.Namespace(**vars(args)); a.prune = r
            out = measure(w, a, tfb, dev, local, dist, world, rank, headline=False)
            if out is not None:
                out["sweep"] = True
                print(json.dumps(out), flush=True)
    else:
        out = measure(wl, args, tfb, dev, local, dist, world, rank, headline=True)
        if out is not None:
            print(json.dumps(out))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()

"""Run ONE stage of the layer step on random tensors of a given shape: the small, self-contained
program a profiler capture wants (a few hundred MB on the device instead of a whole workload ring).

    python -m paper_2512_07090_b200.kernel_harness --stage scan --batch 8 --seq 16384 --kv-heads 8 [--q-heads 32]
           [--window 4096] [--prune 0.5] [--anchor ema --gamma 0.9] [--launches 6] [--scan-path 0..3] [--attention-path 0..6]
           [--select-path 0..2]

Stages: scan (tf_kv_stats), fuse (tf_score_fuse), select (tf_select), score_select (tf_score_select), attention
(tf_pruned_attention), step (tf_layer_filter).  Inputs are N(0,1) bf16 tensors from a fixed seed with a quarter of the tokens near-duplicates of an
earlier token (the recipe of the reduced parity cases); the stages before the requested one run once to produce its
inputs.  Prints the mean time per launch from CUDA events.
"""
from __future__ import annotations

import argparse

import torch

from . import binding as tfb


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--stage", default="scan", choices=["scan", "fuse", "select", "score_select", "attention", "step"])
    ap.add_argument("--batch", type=int, default=8)
    ap.add_argument("--seq", type=int, default=16384)
    ap.add_argument("--kv-heads", type=int, default=8)
    ap.add_argument("--q-heads", type=int, default=0)
    ap.add_argument("--window", type=int, default=0)
    ap.add_argument("--prune", type=float, default=0.5)
    ap.add_argument("--anchor", default="mean", choices=["mean", "incl", "ema"])
    ap.add_argument("--gamma", type=float, default=0.9)
    ap.add_argument("--launches", type=int, default=6)
    ap.add_argument("--scan-path", type=int, default=0)
    ap.add_argument("--attention-path", type=int, default=1)
    ap.add_argument("--select-path", type=int, default=0)
    a = ap.parse_args()
    dev = "cuda:0"
    torch.cuda.set_device(0)
    B, S, Hkv = a.batch, a.seq, a.kv_heads
    Hq = a.q_heads or Hkv
    g = torch.Generator(device=dev).manual_seed(20251207)
    k = torch.randn(B, S, Hkv, 128, generator=g, device=dev, dtype=torch.float32)
    v = torch.randn(B, S, Hkv, 128, generator=g, device=dev, dtype=torch.float32)
    dup = torch.rand(B, S, generator=g, device=dev) < 0.25                       # near-duplicates of an earlier token
    src = (torch.rand(B, S, generator=g, device=dev) * torch.arange(S, device=dev)).long().clamp_(min=0)
    dup[:, 0] = False
    for t in (k, v):
        t.copy_(torch.where(dup[..., None, None], torch.gather(t, 1, src[..., None, None].expand_as(t)) + 0.05 * torch.randn_like(t), t))
    k, v = k.bfloat16(), v.bfloat16()
    need_q = a.stage in ("attention", "step")
    q = torch.randn(B, S, Hq, 128, generator=g, device=dev, dtype=torch.bfloat16) if need_q else None
    O = torch.empty_like(q) if need_q else None
    ctx = tfb.Context(0)
    shape = tfb.make_shape(q, k, v, O, window=a.window, n_q_heads=Hq)
    params = tfb.default_params(prune_ratio=a.prune, warmup_tokens=4, gamma=a.gamma,
                                anchor_mode={"mean": tfb.TF_ANCHOR_PAST_MEAN, "incl": tfb.TF_ANCHOR_INCL_MEAN,
                                             "ema": tfb.TF_ANCHOR_EMA}[a.anchor])
    ctx.ensure_workspace(shape, params)
    ctx.tf_set_scan_path(a.scan_path)
    ctx.tf_set_attention_path(a.attention_path)
    ctx.tf_set_select_path(a.select_path)
    sim_k = torch.empty(B, S, Hkv, device=dev); sim_v = torch.empty_like(sim_k)
    score = torch.empty(B, S, device=dev)
    keep = torch.empty(B, S, dtype=torch.uint8, device=dev)
    idx = torch.empty(B, S, dtype=torch.int32, device=dev)
    nk = torch.empty(B, dtype=torch.int32, device=dev)
    ctx.tf_kv_stats(shape, params, k, v, sim_k, sim_v)
    ctx.tf_score_fuse(shape, params, sim_k, sim_v, score)
    ctx.tf_select(shape, params, score, keep, idx, nk)
    torch.cuda.synchronize()

    def run():
        if a.stage == "scan": ctx.tf_kv_stats(shape, params, k, v, sim_k, sim_v)
        elif a.stage == "fuse": ctx.tf_score_fuse(shape, params, sim_k, sim_v, score)
        elif a.stage == "select": ctx.tf_select(shape, params, score, keep, idx, nk)
        elif a.stage == "score_select": ctx.tf_score_select(shape, params, sim_k, sim_v, score, keep, idx, nk)
        elif a.stage == "attention": ctx.tf_pruned_attention(shape, params, q, k, v, idx, nk, O)
        else: ctx.tf_layer_filter(shape, params, q, k, v, O, score, keep, idx, nk)

    run()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(a.launches):
        run()
    e1.record()
    torch.cuda.synchronize()
    code, det = ctx.tf_get_status()
    print(f"{a.stage}: {e0.elapsed_time(e1) / a.launches * 1e3:.1f} us per launch over {a.launches} launches; "
          f"B{B} S{S} Hq{Hq} Hkv{Hkv} window {a.window}; status {code}; kernels {ctx.tf_last_kernels()}")
    ctx.close()


if __name__ == "__main__":
    main()

"""Parity at the full sizes of the benchmark configurations (c2-c5), in the launch configuration
bench.py times (one tf_layer_filter call, 50 % pruning, warm-up 4, the workload's window).

What the oracle can do at this size it does in full (similarities, fused scores, selection, on the
same bytes); attention is compared on a seeded sample of (sequence, retained token, query head)
rows that the oracle computes one by one; the rest is checked through properties that hold at any
size: pruned rows are exactly zero, retained rows are finite, the kept list is the ascending list of
the mask's ones padded with -1, and exactly min(E, floor(ratio*S)) tokens are pruned."""
import dataclasses

import numpy as np
import pytest
import torch

import oracle
from paper_2512_07090_b200 import binding as tfb, workloads as W
from parity import ATTN_TOL, SCORE_ATOL, mask_disagreements

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.mark.parametrize("name,layer", [("c2", 0), ("c2", 31), ("c3", 20), ("c4", 16), ("c5", 31)])
def test_layer_filter_full_size(name, layer):
    _check_layer(W.WORKLOADS[name], layer)


def test_layer_filter_sequence_of_32768_tokens():
    """Configuration 5's shape at twice its length (two sequences): the selection no longer holds the scores in
    registers, the scan chains 256 chunks per head, the windowed attention has 128 row blocks per head."""
    _check_layer(dataclasses.replace(W.WORKLOADS["c5"], name="c5-32k", batch=2, seq=32768), 3)


def _check_layer(wl, layer):
    _, q, k, v = next(wl.layer_qkv([layer], DEV))
    B, S, Hq, _ = q.shape
    Hkv = k.shape[2]
    ctx = tfb.Context(0)
    O = torch.full_like(q, float("nan"))
    shape = tfb.make_shape(q, k, v, O, window=wl.window)
    params = tfb.default_params(prune_ratio=0.5, warmup_tokens=4)
    ctx.ensure_workspace(shape, params)
    score = torch.empty(B, S, device=DEV)
    keep = torch.empty(B, S, dtype=torch.uint8, device=DEV)
    idx = torch.empty(B, S, dtype=torch.int32, device=DEV)
    nk = torch.empty(B, dtype=torch.int32, device=DEV)
    ctx.tf_layer_filter(shape, params, q, k, v, O, score, keep, idx, nk)
    torch.cuda.synchronize()
    code, det = ctx.tf_get_status()
    assert code == tfb.TF_OK, det

    # ---- filter: in full against the oracle --------------------------------------------------------
    kn, vn = k.float().cpu().numpy(), v.float().cpu().numpy()
    sim_k = oracle.anchor_similarity(kn)
    sim_v = oracle.anchor_similarity(vn)
    ref_score = oracle.score_fuse(sim_k, sim_v)
    del sim_k, sim_v
    ref = oracle.select(ref_score, 0.5, 4)
    ref["score"] = ref_score
    s_err = float(np.abs(score.cpu().numpy().astype(np.float64) - ref_score).max())
    assert s_err < SCORE_ATOL, s_err
    keep_h = keep.cpu().numpy()
    n_mis, n_out = mask_disagreements(keep_h, ref)
    assert n_out == 0, f"{n_mis} keep/prune disagreements, {n_out} outside the 1e-6 band around theta"
    idx_h, nk_h = idx.cpu().numpy(), nk.cpu().numpy()
    for b in range(B):
        assert np.array_equal(idx_h[b, :nk_h[b]], np.nonzero(keep_h[b])[0]) and np.all(idx_h[b, nk_h[b]:] == -1)
        assert nk_h[b] == S - min(S - 4, S // 2)

    # ---- attention: properties everywhere, values on a seeded sample of rows -----------------------------
    keep_d = keep.bool()
    assert bool((O[~keep_d] == 0).all()), "a pruned token's output row is not zero"
    assert bool(torch.isfinite(O[keep_d]).all())
    rng = np.random.default_rng(W.BASE_SEED + layer)
    rows = []
    for _ in range(192):
        b = int(rng.integers(B))
        t = int(idx_h[b, int(rng.integers(nk_h[b]))])
        rows.append((b, t, int(rng.integers(Hq))))
    for b in range(B):   # and the ends of every sequence: first and last retained tokens
        rows += [(b, int(idx_h[b, 0]), 0), (b, int(idx_h[b, nk_h[b] - 1]), Hq - 1)]
    rows = np.array(rows, np.int32)
    qn = q.float().cpu().numpy()
    want = oracle.attention_rows(qn, kn, vn, keep_h, rows, window=wl.window)
    got = O[rows[:, 0], rows[:, 1], rows[:, 2]].float().cpu().numpy().astype(np.float64)
    scale = np.abs(want).max(axis=-1, keepdims=True)
    rel = float((np.abs(got - want) / np.maximum(scale, 1e-30)).max())
    assert rel < ATTN_TOL[torch.bfloat16], rel
    ctx.close()

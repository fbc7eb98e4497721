"""Parity at the full sizes of the benchmark configurations (c2-c5), in the launch configuration
bench.py times (one tf_layer_filter call, warm-up 4, the workload's window), at every pruning ratio
the configuration names.

What the oracle can do at this size it does in full (similarities, fused scores, selection, on the
same bytes).  Attention: on c2 every retained row of every head against the oracle; on c3-c5 at
least 4096 seeded (sequence, retained token, query head) triples that the oracle computes one by
one (plus the first and last retained token of every sequence); the rest is checked through
properties that hold at any size: pruned rows are exactly zero, retained rows are finite, the kept
list is the ascending list of the mask's ones padded with -1, and exactly min(E, floor(ratio*S))
tokens are pruned.  The number of keep/prune disagreements inside the 1e-6 band around the
selection threshold is printed per case (run with -s to see it)."""
import dataclasses

import numpy as np
import pytest
import torch

import oracle
from paper_2512_07090_b200 import binding as tfb, workloads as W
from parity import ATTN_TOL, SCORE_ATOL, mask_disagreements

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
N_TRIPLES = 4096

_cache = {}   # (workload, layer) -> tensors and the oracle's similarities: shared by the ratios of one configuration


def _layer(wl, layer):
    key = (wl.name, layer)
    if key not in _cache:
        _cache.clear()            # one configuration's tensors at a time (c5: 2 GiB)
        _, q, k, v = next(wl.layer_qkv([layer], DEV))
        qn, kn, vn = q.float().cpu().numpy(), k.float().cpu().numpy(), v.float().cpu().numpy()
        sim_k = oracle.anchor_similarity(kn)
        sim_v = oracle.anchor_similarity(vn)
        _cache[key] = (q, k, v, qn, kn, vn, oracle.score_fuse(sim_k, sim_v))
    return _cache[key]


CASES = [("c2", 0, r) for r in W.WORKLOADS["c2"].prune_ratios] + [("c2", 31, 0.5), ("c3", 20, 0.5)] + \
        [("c4", 16, r) for r in W.WORKLOADS["c4"].prune_ratios] + [("c5", 31, 0.5)]


@pytest.mark.parametrize("name,layer,ratio", CASES)
def test_layer_filter_full_size(name, layer, ratio):
    _check_layer(W.WORKLOADS[name], layer, ratio, all_rows=(name == "c2"))


def test_layer_filter_sequence_of_32768_tokens():
    """Configuration 5's shape at twice its length (two sequences): the selection no longer holds the scores in
    registers, the scan chains 256 chunks per head, the windowed attention has 128 row blocks per head."""
    _check_layer(dataclasses.replace(W.WORKLOADS["c5"], name="c5-32k", batch=2, seq=32768), 3, 0.5)


def _check_layer(wl, layer, ratio, all_rows=False):
    q, k, v, qn, kn, vn, ref_score = _layer(wl, layer)
    B, S, Hq, _ = q.shape
    ctx = tfb.Context(0)
    O = torch.full_like(q, float("nan"))
    shape = tfb.make_shape(q, k, v, O, window=wl.window)
    params = tfb.default_params(prune_ratio=ratio, warmup_tokens=4)
    ctx.ensure_workspace(shape, params)
    score = torch.empty(B, S, device=DEV)
    keep = torch.empty(B, S, dtype=torch.uint8, device=DEV)
    idx = torch.empty(B, S, dtype=torch.int32, device=DEV)
    nk = torch.empty(B, dtype=torch.int32, device=DEV)
    ctx.tf_layer_filter(shape, params, q, k, v, O, score, keep, idx, nk)
    torch.cuda.synchronize()
    code, det = ctx.tf_get_status()
    assert code == tfb.TF_OK, det
    scan_kernel, attn_kernel = ctx.tf_last_kernels()
    assert scan_kernel in (tfb.TF_KERNEL_SCAN_GRAM_TILE, tfb.TF_KERNEL_SCAN_GRAM_PERSISTENT)
    assert attn_kernel in (tfb.TF_KERNEL_ATTN_TC_SHARED, tfb.TF_KERNEL_ATTN_TC_SPLIT, tfb.TF_KERNEL_ATTN_TC_HEAD_PAIR,
                           tfb.TF_KERNEL_ATTN_TC_HEAD_QUAD)

    # ---- filter: in full against the oracle --------------------------------------------------------
    ref = oracle.select(ref_score, ratio, 4)
    ref["score"] = ref_score
    s_err = float(np.abs(score.cpu().numpy().astype(np.float64) - ref_score).max())
    assert s_err < SCORE_ATOL, s_err
    keep_h = keep.cpu().numpy()
    n_mis, n_out = mask_disagreements(keep_h, ref)
    print(f"[{wl.name} layer {layer} ratio {ratio}] max score error {s_err:.2e}; keep/prune disagreements inside the "
          f"1e-6 band around theta: {n_mis - n_out}, outside: {n_out}")
    assert n_out == 0, f"{n_mis} keep/prune disagreements, {n_out} outside the 1e-6 band around theta"
    idx_h, nk_h = idx.cpu().numpy(), nk.cpu().numpy()
    for b in range(B):
        assert np.array_equal(idx_h[b, :nk_h[b]], np.nonzero(keep_h[b])[0]) and np.all(idx_h[b, nk_h[b]:] == -1)
        assert nk_h[b] == S - min(S - 4, int(np.floor(ratio * S)))

    # ---- attention: properties everywhere, values against the oracle ---------------------------------
    keep_d = keep.bool()
    assert bool((O[~keep_d] == 0).all()), "a pruned token's output row is not zero"
    assert bool(torch.isfinite(O[keep_d]).all())
    tol = ATTN_TOL[torch.bfloat16]
    if all_rows:
        want = oracle.pruned_attention(qn, kn, vn, keep_h, window=wl.window)
        got = O.float().cpu().numpy().astype(np.float64)
        scale = np.abs(want).max(axis=-1, keepdims=True)
        rel = float((np.abs(got - want) / np.where(scale == 0, 1.0, scale)).max())
        assert rel < tol, rel
    else:
        rng = np.random.default_rng(W.BASE_SEED + layer)
        bs = rng.integers(B, size=N_TRIPLES)
        ts = np.array([idx_h[b, rng.integers(nk_h[b])] for b in bs])
        hs = rng.integers(Hq, size=N_TRIPLES)
        rows = list(zip(bs.tolist(), ts.tolist(), hs.tolist()))
        for b in range(B):   # and the ends of every sequence: first and last retained tokens
            rows += [(b, int(idx_h[b, 0]), 0), (b, int(idx_h[b, nk_h[b] - 1]), Hq - 1)]
        rows = np.array(rows, np.int32)
        want = oracle.attention_rows(qn, kn, vn, keep_h, rows, window=wl.window)
        got = O[rows[:, 0], rows[:, 1], rows[:, 2]].float().cpu().numpy().astype(np.float64)
        scale = np.abs(want).max(axis=-1, keepdims=True)
        rel = float((np.abs(got - want) / np.maximum(scale, 1e-30)).max())
        assert rel < tol, rel
    ctx.close()

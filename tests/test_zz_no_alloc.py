"""tf_kv_stats_static: the similarity scan for callers that cannot allocate device memory.

A serving process that has handed every free byte of HBM to its KV-cache pool, or code that must
leave the device heap to a framework's allocator, cannot provide the scratch tf_kv_stats wants.
tf_kv_stats_static keeps that scratch in an array built into the library.  Here it is called
through the C-ABI twice in a row (different inputs and shapes, so the second call finds the first
call's records in the shared array) and each result is compared with tf_kv_stats on a caller-owned
workspace and with the fp64 oracle on the same bytes.  The file sorts last so that a run that stops at the first failure has already gone
through every other test.
"""
import ctypes as C

import numpy as np
import pytest
import torch

import oracle
from paper_2512_07090_b200 import binding as tfb, workloads as W
from parity import SCORE_ATOL

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _both(ctx, B, S, H, dtype, seed, check_free=True, **params):
    _, k, v = W.duplicate_qkv(B, S, H, H, 128, 0.25, 0.05, seed=seed, dtype=dtype)
    k, v = k.to(DEV), v.to(DEV)
    shape = tfb.make_shape(None, k, v)
    p = tfb.default_params(**params)
    ctx.ensure_workspace(shape, p)
    ref_k = torch.full((B, S, H), float("nan"), device=DEV); ref_v = torch.full_like(ref_k, float("nan"))
    out_k = torch.full_like(ref_k, float("nan")); out_v = torch.full_like(ref_k, float("nan"))
    ctx.tf_kv_stats(shape, p, k, v, ref_k, ref_v)
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    ctx.tf_kv_stats_static(shape, p, k, v, out_k, out_v)
    torch.cuda.synchronize()
    if check_free:   # (the very first call may make the driver load the array's module)
        assert torch.cuda.mem_get_info()[0] == free_before, "the no-allocation entry changed free device memory"
    code, det = ctx.tf_get_status()
    assert code == tfb.TF_OK, det
    assert not torch.isnan(out_k).any() and not torch.isnan(out_v).any()
    assert (out_k - ref_k).abs().max().item() < SCORE_ATOL
    assert (out_v - ref_v).abs().max().item() < SCORE_ATOL
    mode, gamma = params.get("anchor_mode", tfb.TF_ANCHOR_PAST_MEAN), params.get("gamma", 0.9)
    want_k = oracle.anchor_similarity(k.float().cpu().numpy(), mode, gamma)
    want_v = oracle.anchor_similarity(v.float().cpu().numpy(), mode, gamma)
    assert np.abs(out_k.cpu().numpy() - want_k).max() < SCORE_ATOL
    assert np.abs(out_v.cpu().numpy() - want_v).max() < SCORE_ATOL


def test_static_scratch_matches_workspace_path_twice_in_a_row():
    ctx = tfb.Context(0)
    _both(ctx, 2, 1000, 4, torch.bfloat16, seed=31, check_free=False)                 # several chunks, ragged tail
    _both(ctx, 1, 777, 3, torch.float32, seed=32)                      # other layout: region re-zeroed
    _both(ctx, 1, 777, 3, torch.float32, seed=33)                      # same layout: stale records by tag
    _both(ctx, 2, 517, 4, torch.bfloat16, seed=34, anchor_mode=tfb.TF_ANCHOR_EMA, gamma=0.9)
    ctx.close()


def test_static_scratch_works_without_a_context():
    _, k, v = W.duplicate_qkv(1, 300, 2, 2, 128, 0.25, 0.05, seed=41, dtype=torch.bfloat16)
    k, v = k.to(DEV), v.to(DEV)
    shape, p = tfb.make_shape(None, k, v), tfb.default_params()
    ctx = tfb.Context(0)
    ctx.ensure_workspace(shape, p)
    ref_k = torch.empty(1, 300, 2, device=DEV); ref_v = torch.empty_like(ref_k)
    ctx.tf_kv_stats(shape, p, k, v, ref_k, ref_v)
    out_k = torch.full_like(ref_k, float("nan")); out_v = torch.full_like(ref_k, float("nan"))
    stream = C.c_void_p(torch.cuda.current_stream().cuda_stream)
    rc = tfb.lib().tf_kv_stats_static(None, C.byref(shape), C.byref(p), C.c_void_p(k.data_ptr()),
                                      C.c_void_p(v.data_ptr()), C.c_void_p(out_k.data_ptr()),
                                      C.c_void_p(out_v.data_ptr()), None, stream)
    assert rc == tfb.TF_OK
    torch.cuda.synchronize()
    assert (out_k - ref_k).abs().max().item() < SCORE_ATOL and (out_v - ref_v).abs().max().item() < SCORE_ATOL
    ctx.close()


def test_static_scratch_rejects_shapes_beyond_its_limit():
    """Batch 4 x 4096 tokens x 40 heads needs about 22 MiB of records: refused before any launch."""
    B, S, H = 4, 4096, 40
    k = torch.zeros(B, S, H, 128, dtype=torch.bfloat16, device=DEV)
    shape, p = tfb.make_shape(None, k, k), tfb.default_params()
    out = torch.full((B, S, H), 5.0, device=DEV)
    ctx = tfb.Context(0)
    with pytest.raises(tfb.TokenFilterError) as e:
        ctx.tf_kv_stats_static(shape, p, k, k, out, out)
    assert e.value.code == tfb.TF_ERR_WORKSPACE
    torch.cuda.synchronize()
    assert (out == 5.0).all()
    ctx.close()

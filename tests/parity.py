"""Helpers shared by the GPU parity tests: run the CUDA path through the C-ABI binding, run the
oracle on the same bytes, and compare under the stated tolerances."""
import numpy as np
import torch

import oracle
from paper_2512_07090_b200 import binding as tfb

SCORE_ATOL = 1e-5          # fused scores and per-head similarities, fp32 vs fp64
BAND_REL = 1e-6            # a keep/prune disagreement is excused only this close to theta (relative)
ATTN_TOL = {torch.float32: 1e-4, torch.bfloat16: 2e-2}   # max error relative to the row's largest |value|


def to_np(t):
    return t.detach().float().cpu().numpy()


def oracle_inputs(q, k, v):
    return to_np(q), to_np(k), to_np(v)


def attn_rel_err(o_gpu, o_ref):
    """max over elements of |gpu - ref| / max_i |ref_row_i|   (rows of all zeros compare absolutely)."""
    o_gpu = np.asarray(o_gpu, dtype=np.float64)
    scale = np.abs(o_ref).max(axis=-1, keepdims=True)
    scale = np.where(scale == 0, 1.0, scale)
    return float((np.abs(o_gpu - o_ref) / scale).max()) if o_ref.size else 0.0


def mask_disagreements(gpu_mask, ref, band_rel=BAND_REL):
    """Return (n_mismatch, n_outside_band): mismatching tokens and those whose oracle score is NOT
    within band_rel*|theta| of the oracle's selection threshold theta."""
    gpu_mask = np.asarray(gpu_mask)
    mism = gpu_mask != ref["keep_mask"]
    n_out = 0
    for b in range(gpu_mask.shape[0]):
        idx = np.nonzero(mism[b])[0]
        if idx.size == 0:
            continue
        th = ref["theta"][b]
        n_out += int((np.abs(ref["score"][b, idx] - th) > band_rel * abs(th)).sum())
    return int(mism.sum()), n_out


class Gpu:
    """One context + output buffers for a given problem."""

    def __init__(self, Q, K, V, window=0, scale=0.0, **params):
        self.ctx = tfb.Context(Q.device.index or 0)
        self.Q, self.K, self.V = Q, K, V
        B, S, Hkv, _ = K.shape
        dev = K.device
        self.O = torch.full_like(Q, float("nan"))
        self.shape = tfb.make_shape(Q, K, V, self.O, window=window, softmax_scale=scale)
        self._keepalive = params
        self.params = tfb.default_params(**params)
        self.sim_k = torch.full((B, S, Hkv), float("nan"), device=dev)
        self.sim_v = torch.full((B, S, Hkv), float("nan"), device=dev)
        self.score = torch.full((B, S), float("nan"), device=dev)
        self.keep = torch.full((B, S), 7, dtype=torch.uint8, device=dev)
        self.idx = torch.full((B, S), -7, dtype=torch.int32, device=dev)
        self.nk = torch.full((B,), -7, dtype=torch.int32, device=dev)
        self.theta = torch.full((B,), float("nan"), device=dev)
        self.ctx.ensure_workspace(self.shape, self.params)

    def status_ok(self):
        code, det = self.ctx.tf_get_status()
        assert code == tfb.TF_OK, (code, det)

    def close(self):
        self.ctx.close()

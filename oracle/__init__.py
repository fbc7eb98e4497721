"""fp64 CPU oracle for the Token Filtering layer step -- TEST INFRASTRUCTURE ONLY.

Thin ctypes wrapper around ``tf_oracle.c`` (plain C, double precision, written
from the paper's Algorithm 1 and Eq. 1-3).  Nothing in the CUDA package imports
this module and this module imports nothing from the CUDA package; only the
tests, the smoke check and the benchmark's CPU-baseline / reference arm use it.

All tensors are numpy arrays, token-major ``[B, S, H, d]``.  Inputs are float32
arrays holding the exact fp32 / bf16 input values; results are float64.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "tf_oracle.c")
_LIB = os.path.join(_HERE, "libtf_oracle.so")

ANCHOR_PAST_MEAN, ANCHOR_INCL_MEAN, ANCHOR_EMA = 0, 1, 2
FUSE_INVVAR, FUSE_EQ2_LITERAL, FUSE_KEY_ONLY, FUSE_VALUE_ONLY, FUSE_MEAN = 0, 1, 2, 3, 4
SELECT_RATIO, SELECT_THRESHOLD = 0, 1
KV_ALL, KV_RETAINED = 0, 1


def build(force: bool = False) -> str:
    """Compile the C oracle into a shared library next to its source."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


_lib = None


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.tfo_num_threads.restype = C.c_int
    return _lib


def num_threads() -> int:
    return int(lib().tfo_num_threads())


def set_num_threads(n: int) -> None:
    lib().tfo_set_num_threads(C.c_int(int(n)))


def _f32(a):
    a = np.ascontiguousarray(a, dtype=np.float32)
    return a, a.ctypes.data_as(C.c_void_p)


def _ptr(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def anchor_similarity(X, anchor_mode=ANCHOR_PAST_MEAN, gamma=0.9, sum_in=None, count_in=None,
                      want_sum_out=False):
    """Cosine of every token's per-head vector to the anchor of its past.

    X ``[B,S,H,d]`` -> sim ``[B,S,H]`` float64 (and the final running sum
    ``[B,H,d]`` when ``want_sum_out``).  Algorithm 1, Section 3.2, Eq. 1.
    """
    X, xp = _f32(X)
    B, S, H, d = X.shape
    sim = np.empty((B, S, H), dtype=np.float64)
    sum_out = np.empty((B, H, d), dtype=np.float64) if want_sum_out else None
    si = ci = None
    if sum_in is not None:
        si = np.ascontiguousarray(sum_in, dtype=np.float32)
        ci = np.ascontiguousarray(count_in, dtype=np.int64)
    lib().tfo_anchor_similarity(xp, C.c_int(B), C.c_int(S), C.c_int(H), C.c_int(d),
                                C.c_int(anchor_mode), C.c_double(gamma), _ptr(si), _ptr(ci),
                                _ptr(sim), _ptr(sum_out))
    return (sim, sum_out) if want_sum_out else sim


def score_fuse(sim_k, sim_v, fuse_mode=FUSE_INVVAR, var_eps=1e-8, details=False):
    """Mean / variance over heads and the variance-aware fused score (Eq. 2-3)."""
    sim_k = np.ascontiguousarray(sim_k, dtype=np.float64)
    sim_v = np.ascontiguousarray(sim_v, dtype=np.float64)
    B, S, H = sim_k.shape
    score = np.empty((B, S), dtype=np.float64)
    extra = [np.empty((B, S), dtype=np.float64) for _ in range(5)] if details else [None] * 5
    lib().tfo_score_fuse(_ptr(sim_k), _ptr(sim_v), C.c_int(B), C.c_int(S), C.c_int(H),
                         C.c_int(fuse_mode), C.c_double(var_eps), _ptr(score),
                         *[_ptr(e) for e in extra])
    if details:
        return score, dict(zip(("s_k", "s_v", "var_k", "var_v", "alpha"), extra))
    return score


def select(score, prune_ratio=0.5, warmup_tokens=1, eligible=None, select_mode=SELECT_RATIO,
           threshold=None):
    """Keep / prune decision per token; returns a dict of mask, kept list, counts, theta."""
    score = np.ascontiguousarray(score, dtype=np.float64)
    B, S = score.shape
    keep = np.empty((B, S), dtype=np.uint8)
    kept_idx = np.empty((B, S), dtype=np.int32)
    n_kept = np.empty((B,), dtype=np.int32)
    theta = np.empty((B,), dtype=np.float64)
    n_nan = np.empty((B,), dtype=np.int32)
    el = None if eligible is None else np.ascontiguousarray(eligible, dtype=np.uint8)
    th = None
    if threshold is not None:
        th = np.ascontiguousarray(np.broadcast_to(np.asarray(threshold, dtype=np.float64), (B,)))
    lib().tfo_select(_ptr(score), C.c_int(B), C.c_int(S), C.c_double(prune_ratio),
                     C.c_int(warmup_tokens), _ptr(el), C.c_int(select_mode), _ptr(th),
                     _ptr(keep), _ptr(kept_idx), _ptr(n_kept), _ptr(theta), _ptr(n_nan))
    return dict(keep_mask=keep, kept_idx=kept_idx, n_kept=n_kept, theta=theta, n_nan=n_nan)


def _scale(scale, d):
    return float(scale) if scale else 1.0 / float(np.sqrt(d))


def pruned_attention(Q, K, V, keep_mask, window=0, scale=0.0, kv_visibility=KV_ALL):
    """Causal (windowed) attention for retained tokens; pruned rows are zero."""
    Q, qp = _f32(Q)
    K, kp = _f32(K)
    V, vp = _f32(V)
    B, S, Hq, d = Q.shape
    Hkv = K.shape[2]
    keep = np.ascontiguousarray(keep_mask, dtype=np.uint8)
    O = np.empty((B, S, Hq, d), dtype=np.float64)
    lib().tfo_pruned_attention(qp, kp, vp, C.c_int(B), C.c_int(S), C.c_int(Hq), C.c_int(Hkv),
                               C.c_int(d), C.c_int(window), C.c_double(_scale(scale, d)),
                               _ptr(keep), C.c_int(kv_visibility), _ptr(O))
    return O


def attention_rows(Q, K, V, keep_mask, rows, window=0, scale=0.0, kv_visibility=KV_ALL):
    """Selected output rows only: ``rows`` is ``[n,3]`` of (batch, token, query head)."""
    Q, qp = _f32(Q)
    K, kp = _f32(K)
    V, vp = _f32(V)
    B, S, Hq, d = Q.shape
    Hkv = K.shape[2]
    keep = np.ascontiguousarray(keep_mask, dtype=np.uint8)
    rows = np.ascontiguousarray(rows, dtype=np.int32).reshape(-1, 3)
    out = np.empty((rows.shape[0], d), dtype=np.float64)
    lib().tfo_attention_rows(qp, kp, vp, C.c_int(B), C.c_int(S), C.c_int(Hq), C.c_int(Hkv),
                             C.c_int(d), C.c_int(window), C.c_double(_scale(scale, d)),
                             _ptr(keep), C.c_int(kv_visibility), _ptr(rows),
                             C.c_int(rows.shape[0]), _ptr(out))
    return out


def layer_filter(Q, K, V, prune_ratio=0.5, warmup_tokens=1, eligible=None, window=0, scale=0.0,
                 anchor_mode=ANCHOR_PAST_MEAN, gamma=0.9, fuse_mode=FUSE_INVVAR, var_eps=1e-8,
                 select_mode=SELECT_RATIO, threshold=None, kv_visibility=KV_ALL,
                 attention=True):
    """The whole layer step in the paper's order: similarities, fused score,
    selection, attention for retained tokens.  Returns a dict of every stage."""
    sim_k = anchor_similarity(K, anchor_mode, gamma)
    sim_v = anchor_similarity(V, anchor_mode, gamma)
    score = score_fuse(sim_k, sim_v, fuse_mode, var_eps)
    sel = select(score, prune_ratio, warmup_tokens, eligible, select_mode, threshold)
    out = dict(sim_k=sim_k, sim_v=sim_v, score=score, **sel)
    if attention:
        out["O"] = pruned_attention(Q, K, V, sel["keep_mask"], window, scale, kv_visibility)
    return out


def tail_policy(p_global, tail_fraction, n_layers):
    """Section 3.3: only the last round(Y * n_layers) layers are filtered, each at P_tail = P_global / Y
    (the paper's equation for P_tail); earlier layers are not filtered.  Returns the per-layer ratios."""
    n_tail = min(n_layers, max(1, int(np.floor(tail_fraction * n_layers + 0.5))))
    return [p_global / tail_fraction if l >= n_layers - n_tail else 0.0 for l in range(n_layers)]

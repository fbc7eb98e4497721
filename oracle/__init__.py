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


# ---------------------------------------------------------------------------------------------------
# Online decode step (Algorithm 1 as a per-token procedure, with the threshold feedback of Section 3.3)
# ---------------------------------------------------------------------------------------------------
def decode_state(B, Hkv, d=128, tau0=0.0):
    """Empty per-sequence state: anchor sums, token count, threshold, decisions made, skips decided."""
    return dict(sum_k=np.zeros((B, Hkv, d)), sum_v=np.zeros((B, Hkv, d)), count=np.zeros(B, np.int64),
                tau=np.full(B, float(tau0)), steps=np.zeros(B, np.int64), skips=np.zeros(B, np.int64))


def _cos_to_anchor(x, anchor, has_past):
    """cosine of each head's vector to its anchor, each norm clamped at 1e-8; 0 where there is no past."""
    num = (x * anchor).sum(-1)
    den = np.maximum(np.sqrt((x * x).sum(-1)), 1e-8) * np.maximum(np.sqrt((anchor * anchor).sum(-1)), 1e-8)
    return np.where(has_past, num / den, 0.0)


def decode_step(state, q, K_cache, V_cache, pos, target_ratio=0.5, eta=0.05, warmup_tokens=1,
                anchor_mode=ANCHOR_PAST_MEAN, gamma=0.9, fuse_mode=FUSE_INVVAR, var_eps=1e-8,
                window=0, scale=0.0, alg1_sign=False):
    """One decoding iteration of one layer for B sequences, in the order of Algorithm 1:
    anchors -> per-head cosine of the current token's key / value -> (mean, var) over heads -> alpha ->
    s_KV -> threshold adaptation -> skip decision; then the anchor takes the current token in, and the
    attention of the current token (query q against cache positions <= pos) is computed unless skipped
    (a skipped token's attention output is zero).

    Threshold adaptation: tau += eta * (rho - target)   (Section 3.3, T_l += eta (P_current - P_tail)),
    rho = skips decided / decisions made so far (0 before the first); alg1_sign=True uses the sign
    printed in Algorithm 1, eta * (target - rho).  A token at position < warmup_tokens is never
    skipped, but its decision still counts toward rho (the thresholds keep adapting during warm-up).

    q [B,Hq,d], K_cache / V_cache [B,S,Hkv,d] with the current token already stored at pos[b].
    state is updated in place.  Returns dict(score [B], skip [B] uint8, tau [B] after the update, O [B,Hq,d])."""
    q = np.asarray(q, np.float64); K = np.asarray(K_cache, np.float64); V = np.asarray(V_cache, np.float64)
    B, S, Hkv, d = K.shape
    Hq = q.shape[1]
    pos = np.asarray(pos, np.int64)
    score = np.zeros(B); skip = np.zeros(B, np.uint8); O = np.zeros((B, Hq, d))
    for b in range(B):
        k, v = K[b, pos[b]], V[b, pos[b]]                      # [Hkv, d]
        n = int(state["count"][b])
        upd = (lambda s_, x: gamma * s_ + (1 - gamma) * x) if anchor_mode == ANCHOR_EMA else (lambda s_, x: s_ + x)
        if anchor_mode == ANCHOR_INCL_MEAN:                    # anchor takes the current token in first
            state["sum_k"][b] = upd(state["sum_k"][b], k); state["sum_v"][b] = upd(state["sum_v"][b], v)
            n += 1
        has_past = n > 0
        div = 1.0 if anchor_mode == ANCHOR_EMA else max(n, 1)
        ck = _cos_to_anchor(k, state["sum_k"][b] / div, has_past)
        cv = _cos_to_anchor(v, state["sum_v"][b] / div, has_past)
        s = float(score_fuse(ck[None, None, :], cv[None, None, :], fuse_mode, var_eps)[0, 0])
        steps, skips = int(state["steps"][b]), int(state["skips"][b])
        rho = skips / steps if steps > 0 else 0.0
        delta = eta * ((target_ratio - rho) if alg1_sign else (rho - target_ratio))
        state["tau"][b] = state["tau"][b] + delta
        decide = bool(s > state["tau"][b]) if s == s else False
        do_skip = decide and pos[b] >= warmup_tokens
        state["steps"][b] = steps + 1
        state["skips"][b] = skips + (1 if decide else 0)
        if anchor_mode != ANCHOR_INCL_MEAN:
            state["sum_k"][b] = upd(state["sum_k"][b], k); state["sum_v"][b] = upd(state["sum_v"][b], v)
            n += 1
        state["count"][b] = n
        score[b] = s; skip[b] = 1 if do_skip else 0
        if not do_skip:
            g = Hq // Hkv
            sc = scale if scale else 1.0 / np.sqrt(d)
            lo = max(0, int(pos[b]) - window + 1) if window > 0 else 0
            for h in range(Hq):
                kk = K[b, lo:pos[b] + 1, h // g]; vv = V[b, lo:pos[b] + 1, h // g]
                a = sc * (kk @ q[b, h])
                a = np.exp(a - a.max())
                O[b, h] = (a / a.sum()) @ vv
    return dict(score=score, skip=skip, tau=state["tau"].copy(), O=O)

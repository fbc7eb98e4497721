"""Pins for the fp64 oracle: closed forms, invariants, brute force and library routines.

None of these tests re-types the oracle's own formula as the expected value: each
expected value is fixed by the mathematics (a construction whose answer is known),
by an invariance the method must have, by exhaustive search on a tiny input, or
by an independent library routine (numpy mean / cumsum, torch fp64 SDPA).
"""
import itertools
import os

import numpy as np
import pytest
import torch

import oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
rng = np.random.default_rng(7)


def _rand(*shape):
    return rng.standard_normal(shape).astype(np.float32)


# ------------------------------------------------------------------ a1/a2: anchors + cosine
def test_token_equal_to_scaled_running_mean_scores_one():
    """A token that is c*(mean of its past), c>0, in every head: cosine 1 per head,
    zero variance, fused score 1 (both fuse readings)."""
    B, S, H, d = 1, 9, 4, 16
    K, V = _rand(B, S, H, d), _rand(B, S, H, d)
    t = 6
    K[0, t] = 3.5 * K[0, :t].astype(np.float64).mean(0)
    V[0, t] = 0.25 * V[0, :t].astype(np.float64).mean(0)
    sk, sv = orc.anchor_similarity(K), orc.anchor_similarity(V)
    assert np.allclose(sk[0, t], 1.0, atol=1e-6) and np.allclose(sv[0, t], 1.0, atol=1e-6)
    for mode in (orc.FUSE_INVVAR, orc.FUSE_EQ2_LITERAL):
        s, det = orc.score_fuse(sk, sv, mode, details=True)
        assert abs(s[0, t] - 1.0) < 1e-6
        assert det["var_k"][0, t] < 1e-12 and det["var_v"][0, t] < 1e-12
    # a negative multiple is anti-parallel: cosine -1
    K[0, t] = -2.0 * K[0, :t].astype(np.float64).mean(0)
    assert np.allclose(orc.anchor_similarity(K)[0, t], -1.0, atol=1e-6)


def test_all_identical_tokens_score_one_and_prune_maximally():
    B, S, H, d = 2, 12, 3, 8
    x = _rand(1, 1, H, d)
    K = np.broadcast_to(x, (B, S, H, d)).copy()
    V = np.broadcast_to(_rand(1, 1, H, d), (B, S, H, d)).copy()
    r = orc.layer_filter(K, K, V, attention=False, select_mode=orc.SELECT_THRESHOLD,
                         threshold=0.999, warmup_tokens=2)
    assert np.all(r["score"][:, 0] == 0.0)                       # no past -> 0
    assert np.allclose(r["score"][:, 1:], 1.0, atol=1e-12)
    # threshold mode: every eligible token (t >= warm-up) is pruned
    assert np.array_equal(r["keep_mask"], np.r_[[1, 1], np.zeros(S - 2)].astype(np.uint8)[None].repeat(B, 0))
    # ratio mode: all ties -> exactly the P highest-index eligible tokens go
    r = orc.layer_filter(K, K, V, attention=False, prune_ratio=0.5, warmup_tokens=1)
    exp = np.ones(S, np.uint8)
    exp[S - 6:] = 0
    assert np.array_equal(r["keep_mask"][0], exp) and r["n_kept"].tolist() == [6, 6]


def test_one_hot_tokens_are_orthogonal_to_their_past():
    d, H = 16, 2
    S = d
    K = np.zeros((1, S, H, d), np.float32)
    for t in range(S):
        K[0, t, :, t % d] = 1.0 + t
    sim = orc.anchor_similarity(K)
    assert np.all(sim == 0.0)
    r = orc.layer_filter(K, K, K, attention=False, prune_ratio=0.25, warmup_tokens=1)
    assert np.all(r["score"] == 0.0)
    assert r["kept_idx"][0, : S - 4].tolist() == list(range(S - 4))     # ties: latest pruned first
    assert r["theta"][0] == 0.0


def test_two_token_cosine_is_the_angle_between_them():
    """With one past token the anchor is that token: cos(angle) by construction."""
    d = 8
    for ang in (0.0, 0.3, np.pi / 2, 2.0, np.pi):
        a = np.zeros(d); a[0] = 2.0
        b = np.zeros(d); b[0] = 5 * np.cos(ang); b[3] = 5 * np.sin(ang)
        K = np.stack([a, b]).reshape(1, 2, 1, d).astype(np.float32)
        exp = float(np.dot(K[0, 0, 0].astype(np.float64), K[0, 1, 0]) / (2.0 * np.linalg.norm(K[0, 1, 0].astype(np.float64))))
        assert abs(orc.anchor_similarity(K)[0, 1, 0] - exp) < 1e-12
        assert abs(exp - np.cos(ang)) < 1e-6


def test_scale_and_rotation_invariance():
    B, S, H, d = 1, 20, 2, 8
    K = _rand(B, S, H, d)
    base = orc.anchor_similarity(K)
    K2 = K.copy()
    K2[0, 7] *= 4.0            # power of two: exact in fp32
    s2 = orc.anchor_similarity(K2)
    assert abs(s2[0, 7, 0] - base[0, 7, 0]) < 1e-12   # own scale does not matter
    K3 = K * 8.0                # scaling the whole past does not matter
    assert np.allclose(orc.anchor_similarity(K3), base, atol=1e-12)
    # signed permutation of coordinates = an orthogonal map that is exact in fp32
    perm = rng.permutation(d)
    sign = rng.choice([-1.0, 1.0], d).astype(np.float32)
    K4 = K[..., perm] * sign
    assert np.allclose(orc.anchor_similarity(K4), base, atol=1e-12)


def test_prefix_property_and_carry_in():
    B, S, H, d = 2, 31, 3, 8
    K = _rand(B, S, H, d)
    full = orc.anchor_similarity(K)
    K2 = K.copy(); K2[:, 20:] = _rand(B, S - 20, H, d)
    assert np.array_equal(orc.anchor_similarity(K2)[:, :20], full[:, :20])        # causal
    assert np.array_equal(orc.anchor_similarity(K[:, :13]), full[:, :13])          # truncation
    # two halves with a carry == one pass (sums of fp32 values; carry passes through fp32,
    # so build it from values exactly representable: small integers)
    Ki = rng.integers(-8, 9, (B, S, H, d)).astype(np.float32)
    one = orc.anchor_similarity(Ki)
    first, s_out = orc.anchor_similarity(Ki[:, :15], want_sum_out=True)
    second = orc.anchor_similarity(Ki[:, 15:], sum_in=s_out.astype(np.float32), count_in=np.full(B, 15))
    assert np.array_equal(np.concatenate([first, second], 1), one)


def test_final_running_sum_is_the_column_mean():
    B, S, H, d = 2, 17, 3, 8
    K = _rand(B, S, H, d)
    _, s = orc.anchor_similarity(K, want_sum_out=True)
    assert np.allclose(s / S, K.astype(np.float64).mean(axis=1), atol=1e-13)


def test_against_cumsum_formulation():
    """Independent route: exclusive cumulative sums (numpy) then a vectorised cosine."""
    B, S, H, d = 2, 40, 4, 16
    K = _rand(B, S, H, d)
    Kd = K.astype(np.float64)
    P = np.cumsum(Kd, axis=1) - Kd
    dots = (P * Kd).sum(-1)
    den = np.maximum(np.linalg.norm(P, axis=-1) / np.maximum(np.arange(S), 1)[None, :, None], 1e-8) \
        * np.maximum(np.linalg.norm(Kd, axis=-1), 1e-8) * np.maximum(np.arange(S), 1)[None, :, None]
    exp = dots / den
    exp[:, 0] = 0.0
    assert np.allclose(orc.anchor_similarity(K), exp, atol=1e-12)


def test_inclusive_mean_reading():
    """Algorithm 1 read literally (anchor already contains the current token):
    token 0 compares with itself -> exactly 1; in general cos(x_t, sum_{j<=t} x_j)."""
    B, S, H, d = 1, 10, 2, 8
    K = _rand(B, S, H, d)
    inc = orc.anchor_similarity(K, orc.ANCHOR_INCL_MEAN)
    assert np.allclose(inc[:, 0], 1.0, atol=1e-12)
    Kd = K.astype(np.float64)
    C = np.cumsum(Kd, axis=1)
    exp = (C * Kd).sum(-1) / (np.linalg.norm(C, axis=-1) * np.linalg.norm(Kd, axis=-1))
    assert np.allclose(inc, exp, atol=1e-12)


def test_ema_anchor_closed_form():
    """Eq. 1 unrolled: anchor before token t is (1-g) * sum_{j<t} g^(t-1-j) x_j."""
    B, S, H, d = 1, 12, 2, 8
    K = _rand(B, S, H, d)
    for g in (0.8, 0.9, 0.95):
        sim = orc.anchor_similarity(K, orc.ANCHOR_EMA, gamma=g)
        assert np.all(sim[:, 0] == 0)
        Kd = K.astype(np.float64)
        for t in range(1, S):
            w = (1 - g) * g ** (t - 1 - np.arange(t))
            A = (w[None, :, None, None] * Kd[:, :t]).sum(1)
            exp = (A * Kd[:, t]).sum(-1) / (np.linalg.norm(A, axis=-1) * np.linalg.norm(Kd[:, t], axis=-1))
            assert np.allclose(sim[:, t], exp, atol=1e-12)


def test_zero_vectors_give_zero_similarity_not_nan():
    K = np.zeros((1, 5, 2, 8), np.float32)
    K[0, 2] = 1.0
    s = orc.anchor_similarity(K)
    assert np.all(np.isfinite(s)) and s[0, 1, 0] == 0.0 and s[0, 3, 0] == 0.0


# ------------------------------------------------------------------ a3: fusion
def test_anchor_footprint_matches_paper():
    """Section 3.2 prints 'approximately 800 KB' for LLaMA-2-13B: one 16-bit head_dim vector
    per head per layer for K and for V."""
    with open(os.path.join(GOLDEN, "anchor_footprint.txt")) as f:
        vals = dict(l.split("=") for l in f.read().split() if "=" in l)
    n = int(vals["layers"]) * 2 * int(vals["heads"]) * int(vals["head_dim"]) * int(vals["bytes_per_elem"])
    assert n == int(vals["total_bytes"]) == 819200 and n / 1024 == 800.0


def test_fusion_hand_worked_values():
    """Two heads, numbers worked by hand.  Keys: c=(0,0.4) -> mean .2, var .04.
    Values: c=(.1,.7) -> mean .4, var .09.  Eq. 2 as printed: (1/.09)/(1/.04+1/.09) = 4/13,
    S = (4*.2 + 9*.4)/13 = 4.4/13.  Inverse-variance reading: alpha = 9/13, S = (9*.2+4*.4)/13 = 3.4/13."""
    ck = np.array([0.0, 0.4]).reshape(1, 1, 2)
    cv = np.array([0.1, 0.7]).reshape(1, 1, 2)
    lit, dl = orc.score_fuse(ck, cv, orc.FUSE_EQ2_LITERAL, var_eps=0.0, details=True)
    inv, di = orc.score_fuse(ck, cv, orc.FUSE_INVVAR, var_eps=0.0, details=True)
    assert abs(dl["var_k"][0, 0] - 0.04) < 1e-15 and abs(dl["var_v"][0, 0] - 0.09) < 1e-15
    assert abs(dl["alpha"][0, 0] - 4 / 13) < 1e-14 and abs(lit[0, 0] - 4.4 / 13) < 1e-14
    assert abs(di["alpha"][0, 0] - 9 / 13) < 1e-14 and abs(inv[0, 0] - 3.4 / 13) < 1e-14
    assert orc.score_fuse(ck, cv, orc.FUSE_KEY_ONLY)[0, 0] == pytest.approx(0.2, abs=1e-15)
    assert orc.score_fuse(ck, cv, orc.FUSE_VALUE_ONLY)[0, 0] == pytest.approx(0.4, abs=1e-15)
    assert orc.score_fuse(ck, cv, orc.FUSE_MEAN)[0, 0] == pytest.approx(0.3, abs=1e-15)


def test_fusion_bounds_symmetry_limits():
    B, S, H = 2, 50, 8
    ck, cv = rng.uniform(-1, 1, (B, S, H)), rng.uniform(-1, 1, (B, S, H))
    for mode in (orc.FUSE_INVVAR, orc.FUSE_EQ2_LITERAL):
        s, det = orc.score_fuse(ck, cv, mode, details=True)
        lo, hi = np.minimum(det["s_k"], det["s_v"]), np.maximum(det["s_k"], det["s_v"])
        assert np.all(s >= lo - 1e-15) and np.all(s <= hi + 1e-15)                # convex combination
        assert np.all((det["alpha"] >= 0) & (det["alpha"] <= 1)) and np.all(np.abs(s) <= 1)
        assert np.allclose(orc.score_fuse(cv, ck, mode), s, atol=1e-15)           # K<->V swap
        perm = rng.permutation(H)
        assert np.allclose(orc.score_fuse(ck[..., perm], cv[..., perm], mode), s, atol=1e-15)
        # replicating every head g times (GQA expansion) changes nothing
        assert np.allclose(orc.score_fuse(np.repeat(ck, 4, -1), np.repeat(cv, 4, -1), mode), s, atol=1e-14)
    # equal variances -> plain average;  zero variance on both sides (or H = 1) -> alpha = 1/2
    ck1 = np.array([0.1, 0.5]).reshape(1, 1, 2); cv1 = np.array([0.6, 0.2]).reshape(1, 1, 2)
    assert orc.score_fuse(ck1, cv1)[0, 0] == pytest.approx(0.35, abs=1e-15)
    one = orc.score_fuse(np.full((1, 1, 1), 0.8), np.full((1, 1, 1), 0.2), details=True)
    assert one[1]["alpha"][0, 0] == 0.5 and one[0][0, 0] == pytest.approx(0.5, abs=1e-15)
    # values much noisier across heads than keys: inverse-variance -> s_k, Eq. 2 literal -> s_v
    ck2 = np.array([0.300, 0.301]).reshape(1, 1, 2); cv2 = np.array([-0.9, 0.9]).reshape(1, 1, 2)
    assert abs(orc.score_fuse(ck2, cv2, orc.FUSE_INVVAR)[0, 0] - 0.3005) < 1e-6
    assert abs(orc.score_fuse(ck2, cv2, orc.FUSE_EQ2_LITERAL)[0, 0] - 0.0) < 1e-6


# ------------------------------------------------------------------ a4: selection
def _brute_force_prune_set(score, eligible, P):
    """The unique size-P subset of eligible tokens that dominates the rest in (score, index)."""
    el = [t for t in range(len(score)) if eligible[t]]
    for sub in itertools.combinations(el, P):
        rest = [t for t in el if t not in sub]
        if not sub or not rest or min((score[t], t) for t in sub) > max((score[t], t) for t in rest):
            return set(sub)
    raise AssertionError("no dominating subset")


def test_selection_matches_brute_force_on_tiny_inputs():
    for trial in range(60):
        S = int(rng.integers(1, 11))
        score = np.round(rng.uniform(-1, 1, S), 1)          # coarse grid -> many ties
        warm = int(rng.integers(0, 3))
        elig = (rng.uniform(size=S) < 0.8).astype(np.uint8)
        ratio = float(rng.choice([0.0, 0.2, 0.25, 0.5, 0.7, 0.99]))
        r = orc.select(score[None], ratio, warm, elig[None])
        ok = [(t >= warm) and bool(elig[t]) for t in range(S)]
        P = min(sum(ok), int(np.floor(ratio * S)))
        pruned = _brute_force_prune_set(score, ok, P)
        mask = r["keep_mask"][0]
        assert {t for t in range(S) if not mask[t]} == pruned
        kept = [t for t in range(S) if mask[t]]
        assert r["n_kept"][0] == S - P == len(kept)
        assert r["kept_idx"][0, : len(kept)].tolist() == kept and np.all(r["kept_idx"][0, len(kept):] == -1)
        if P:
            assert r["theta"][0] == min(score[t] for t in pruned)
        else:
            assert np.isinf(r["theta"][0])


def test_selection_edge_cases():
    s = np.array([[0.9, 0.8, np.nan, 0.7, 0.95, 0.1]])
    r = orc.select(s, 0.5, warmup_tokens=0)
    assert r["keep_mask"][0].tolist() == [0, 0, 1, 1, 0, 1] and r["n_nan"][0] == 1    # NaN never pruned
    r = orc.select(s, 0.0, warmup_tokens=0)
    assert r["keep_mask"].all() and np.isinf(r["theta"][0])                            # ratio 0
    r = orc.select(s, 0.99, warmup_tokens=4)
    assert r["keep_mask"][0].tolist() == [1, 1, 1, 1, 0, 0]                            # capped by eligibility
    r = orc.select(s, 0.5, 0, select_mode=orc.SELECT_THRESHOLD, threshold=0.8)
    assert r["keep_mask"][0].tolist() == [0, 1, 1, 1, 0, 1]                            # strict >
    r = orc.select(np.zeros((1, 0)), 0.5, 0)
    assert r["n_kept"][0] == 0


# ------------------------------------------------------------------ a5: attention
def _sdpa64(Q, K, V, window=0, key_mask=None):
    q = torch.from_numpy(Q).double().transpose(1, 2)
    g = Q.shape[2] // K.shape[2]
    k = torch.from_numpy(K).double().repeat_interleave(g, dim=2).transpose(1, 2)
    v = torch.from_numpy(V).double().repeat_interleave(g, dim=2).transpose(1, 2)
    S = Q.shape[1]
    i = torch.arange(S)[:, None]; j = torch.arange(S)[None, :]
    m = j <= i
    if window:
        m &= j > i - window
    m = m[None, None].expand(Q.shape[0], 1, S, S).clone()
    if key_mask is not None:
        m &= torch.from_numpy(key_mask.astype(bool))[:, None, None, :]
    o = torch.nn.functional.scaled_dot_product_attention(q, k, v, attn_mask=m)
    return o.transpose(1, 2).numpy()


@pytest.mark.parametrize("Hq,Hkv,window", [(4, 4, 0), (8, 2, 0), (4, 1, 5), (6, 3, 1)])
def test_zero_pruning_is_dense_causal_attention(Hq, Hkv, window):
    B, S, d = 2, 23, 16
    Q, K, V = _rand(B, S, Hq, d), _rand(B, S, Hkv, d), _rand(B, S, Hkv, d)
    O = orc.pruned_attention(Q, K, V, np.ones((B, S), np.uint8), window=window)
    assert np.allclose(O, _sdpa64(Q, K, V, window), atol=1e-12)
    # with pruning (default visibility): retained rows are unchanged, pruned rows exactly zero
    keep = (rng.uniform(size=(B, S)) < 0.5).astype(np.uint8)
    Op = orc.pruned_attention(Q, K, V, keep, window=window)
    assert np.array_equal(Op[keep.astype(bool)], O[keep.astype(bool)])
    assert np.all(Op[~keep.astype(bool)] == 0.0)
    rows = np.array([(b, t, h) for b in range(B) for t in range(0, S, 3) for h in range(Hq)], np.int32)
    R = orc.attention_rows(Q, K, V, keep, rows, window=window)
    assert np.array_equal(R, Op[rows[:, 0], rows[:, 1], rows[:, 2]])


def test_retained_only_visibility():
    B, S, Hq, Hkv, d = 1, 19, 4, 2, 8
    Q, K, V = _rand(B, S, Hq, d), _rand(B, S, Hkv, d), _rand(B, S, Hkv, d)
    keep = (rng.uniform(size=(B, S)) < 0.6).astype(np.uint8); keep[:, 0] = 1
    O = orc.pruned_attention(Q, K, V, keep, kv_visibility=orc.KV_RETAINED)
    ref = _sdpa64(Q, K, V, 0, key_mask=keep)
    kb = keep.astype(bool)
    assert np.allclose(O[kb], ref[kb], atol=1e-12) and np.all(O[~kb] == 0)


def test_attention_closed_forms():
    B, S, H, d = 1, 9, 2, 8
    Q, K, V = _rand(B, S, H, d), _rand(B, S, H, d), _rand(B, S, H, d)
    ones = np.ones((B, S), np.uint8)
    O = orc.pruned_attention(Q, K, V, ones)
    assert np.allclose(O[:, 0], V[:, 0], atol=1e-15)                       # one visible key
    assert np.allclose(orc.pruned_attention(Q, K, V, ones, window=1), V, atol=1e-15)
    Vc = np.broadcast_to(V[:, :1], V.shape).copy()
    assert np.allclose(orc.pruned_attention(Q, K, Vc, ones), Vc, atol=1e-14)   # convex weights
    # zero queries -> uniform weights -> running mean of V
    Oz = orc.pruned_attention(np.zeros_like(Q), K, V, ones)
    exp = np.cumsum(V.astype(np.float64), 1) / np.arange(1, S + 1)[None, :, None, None]
    assert np.allclose(Oz, exp, atol=1e-14)
    # scale: a huge scale picks the arg-max key
    Ob = orc.pruned_attention(Q, K, V, ones, scale=1e4)
    logits = np.einsum("bthd,bjhd->bhtj", Q.astype(np.float64), K.astype(np.float64))
    for t in range(S):
        for h in range(H):
            j = int(np.argmax(logits[0, h, t, : t + 1]))
            assert np.allclose(Ob[0, t, h], V[0, j, h], atol=1e-6)


def test_layer_filter_end_to_end_invariants():
    from paper_2512_07090_b200 import workloads as W
    q, k, v = (x.numpy() for x in W.duplicate_qkv(2, 64, 8, 2, 32, 0.25, 0.05, seed=3))
    r = orc.layer_filter(q, k, v, prune_ratio=0.5, warmup_tokens=4)
    for b in range(2):
        n = r["n_kept"][b]
        idx = r["kept_idx"][b, :n]
        assert n == 32 and np.all(np.diff(idx) > 0) and np.all(idx[:4] == np.arange(4))
        assert np.all(r["O"][b][r["keep_mask"][b] == 0] == 0.0)
        pruned = r["score"][b][r["keep_mask"][b] == 0]
        kept_el = r["score"][b][4:][r["keep_mask"][b][4:] == 1]
        assert pruned.min() >= kept_el.max() and r["theta"][b] == pruned.min()
    # GQA: statistics over KV heads == statistics over the g-fold expanded heads
    r2 = orc.layer_filter(q, np.repeat(k, 4, 2), np.repeat(v, 4, 2), prune_ratio=0.5, warmup_tokens=4)
    assert np.allclose(r2["score"], r["score"], atol=1e-13) and np.allclose(r2["O"], r["O"], atol=1e-12)


# ------------------------------------------------------------------------------- tail-focused policy
def test_tail_policy_paper_example_and_budget():
    """Section 3.3's worked example: global budget 25 %, last half of the layers => 50 % per tail layer;
    the mean over all layers is the global budget whenever Y * n_layers is whole."""
    r = orc.tail_policy(0.25, 0.5, 32)
    assert r[:16] == [0.0] * 16 and all(abs(x - 0.5) < 1e-15 for x in r[16:])
    for pg, y, L in [(0.25, 0.5, 32), (0.2, 0.4, 40), (0.33, 0.6, 40), (0.1, 1.0, 7)]:
        r = orc.tail_policy(pg, y, L)
        assert abs(sum(r) / L - pg) < 1e-12
        assert all(x == 0.0 for x in r[: L - round(y * L)])


# ------------------------------------------------------------------------------- online decode step
def _decode_run(K, V, Q, **kw):
    B, S, Hkv, d = K.shape
    st = orc.decode_state(B, Hkv, d, tau0=kw.pop("tau0", 0.0))
    out = []
    for t in range(S):
        out.append(orc.decode_step(st, Q[:, t], K, V, np.full(B, t), **kw))
    return st, out


def test_decode_steps_reproduce_the_prefill_scores_and_dense_attention():
    """Token by token with a threshold nothing reaches: the scores are the prefill oracle's scores at every
    position (same anchors, same order of compare and update) and the outputs are dense causal attention."""
    rng = np.random.default_rng(5)
    B, S, Hq, Hkv, d = 2, 40, 4, 2, 128
    Q = rng.standard_normal((B, S, Hq, d)).astype(np.float32)
    K = rng.standard_normal((B, S, Hkv, d)).astype(np.float32)
    V = rng.standard_normal((B, S, Hkv, d)).astype(np.float32)
    K[:, 20] = K[:, 3] * 1.5
    for mode, gamma in [(orc.ANCHOR_PAST_MEAN, 0.9), (orc.ANCHOR_INCL_MEAN, 0.9), (orc.ANCHOR_EMA, 0.8)]:
        ref = orc.layer_filter(Q, K, V, prune_ratio=0.0, window=7, anchor_mode=mode, gamma=gamma)
        st, out = _decode_run(K, V, Q, tau0=10.0, eta=0.0, window=7, anchor_mode=mode, gamma=gamma)
        sc = np.stack([o["score"] for o in out], 1)
        assert np.abs(sc - ref["score"]).max() < 1e-12
        O = np.stack([o["O"] for o in out], 1)
        assert np.abs(O - ref["O"]).max() < 1e-10
        assert all(o["skip"].sum() == 0 for o in out)
        assert np.all(st["count"] == S) and np.all(st["steps"] == S) and np.all(st["skips"] == 0)


def test_decode_threshold_feedback_signs_warmup_and_fixed_point():
    """Section 3.3: the threshold rises while the skip ratio is above target and falls while below; with
    Algorithm 1's printed sign it moves the other way.  Warm-up tokens are never skipped but are counted.
    On a long stream of scores the skip ratio settles at the target."""
    rng = np.random.default_rng(6)
    B, S, H, d = 1, 3000, 2, 16
    base = rng.standard_normal((1, 1, H, d))
    K = (base + 0.8 * rng.standard_normal((B, S, H, d))).astype(np.float32)
    V = (base + 0.8 * rng.standard_normal((B, S, H, d))).astype(np.float32)
    Q = rng.standard_normal((B, S, H, d)).astype(np.float32)
    st, out = _decode_run(K, V, Q, tau0=0.0, eta=0.1, target_ratio=0.3, warmup_tokens=8)
    taus = np.array([o["tau"][0] for o in out]); skips = np.array([o["skip"][0] for o in out])
    assert skips[:8].sum() == 0                                   # never inside the warm-up
    assert st["skips"][0] >= skips.sum()                          # but decided skips are counted there too
    rho = np.cumsum([1 if np.float32(o["score"][0]) > o["tau"][0] else 0 for o in out])
    # the update uses the ratio BEFORE the current decision
    prev_rho = np.concatenate([[0.0], rho[:-1] / np.arange(1, S)])
    d_tau = np.diff(np.concatenate([[0.0], taus]))
    assert np.all(np.sign(d_tau[1:]) == np.sign(np.float32(prev_rho[1:] - 0.3)))
    assert abs(st["skips"][0] / st["steps"][0] - 0.3) < 0.03     # settles at the target
    st2, out2 = _decode_run(K, V, Q, tau0=0.0, eta=0.1, target_ratio=0.3, warmup_tokens=8, alg1_sign=True)
    assert out2[0]["tau"][0] > 0 > out[0]["tau"][0]               # first update: rho = 0 < target
    # positive feedback runs away: everything or nothing is skipped in the end
    r2 = st2["skips"][0] / st2["steps"][0]
    assert r2 < 0.02 or r2 > 0.98

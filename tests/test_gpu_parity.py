"""GPU parity: the CUDA path, called through the C-ABI, against the fp64 oracle on the same
seeded inputs.  Integer results (masks, kept lists, counts) bit-exact; scores within 1e-5;
attention within 1e-4 (fp32) / 2e-2 (bf16) of the row scale."""
import ctypes as C

import numpy as np
import pytest
import torch

import oracle
from paper_2512_07090_b200 import binding as tfb, workloads as W
from parity import ATTN_TOL, SCORE_ATOL, Gpu, attn_rel_err, mask_disagreements, oracle_inputs, to_np

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _qkv(B, S, Hq, Hkv, dtype, seed=11, dup=0.25):
    q, k, v = W.duplicate_qkv(B, S, Hq, Hkv, 128, dup, 0.05, seed=seed, dtype=dtype)
    return q.to(DEV), k.to(DEV), v.to(DEV)


# ------------------------------------------------------------------------------- a1 + a2
@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
@pytest.mark.parametrize("B,S,Hkv", [(1, 1, 1), (1, 2, 3), (2, 63, 2), (1, 64, 4), (2, 65, 1),
                                      (3, 333, 5), (2, 1000, 8), (1, 4100, 2)])
@pytest.mark.parametrize("scan_path", [1, 2, 3])   # plain CUDA-core kernel / Gram-matrix kernel (one tile per CTA) / persistent Gram kernel
def test_kv_stats_matches_oracle(dtype, B, S, Hkv, scan_path):
    if scan_path >= 2 and dtype != torch.bfloat16:
        pytest.skip("the Gram-matrix kernel takes bf16 only")
    q, k, v = _qkv(B, S, Hkv, Hkv, dtype)
    g = Gpu(q, k, v)
    g.ctx.tf_set_scan_path(scan_path)
    g.ctx.tf_kv_stats(g.shape, g.params, k, v, g.sim_k, g.sim_v)
    g.status_ok()
    assert g.ctx.tf_last_kernels()[0] == scan_path          # the kernel asked for is the kernel that ran
    _, kn, vn = oracle_inputs(q, k, v)
    assert np.abs(to_np(g.sim_k) - oracle.anchor_similarity(kn)).max() < SCORE_ATOL
    assert np.abs(to_np(g.sim_v) - oracle.anchor_similarity(vn)).max() < SCORE_ATOL
    g.close()


@pytest.mark.parametrize("scan_path", [1, 2, 3])
def test_kv_stats_inclusive_mean_every_path(scan_path):
    """The inclusive-mean anchor (the token itself counted in) on each of the three scan kernels, on a length that
    leaves a ragged last tile."""
    q, k, v = _qkv(3, 1111, 5, 5, torch.bfloat16, seed=21)
    g = Gpu(q, k, v, anchor_mode=tfb.TF_ANCHOR_INCL_MEAN)
    g.ctx.tf_set_scan_path(scan_path)
    for _ in range(2):      # twice: the second launch finds the first one's records and tickets in the scratch
        g.ctx.tf_kv_stats(g.shape, g.params, k, v, g.sim_k, g.sim_v)
    g.status_ok()
    _, kn, vn = oracle_inputs(q, k, v)
    assert np.abs(to_np(g.sim_k) - oracle.anchor_similarity(kn, tfb.TF_ANCHOR_INCL_MEAN, 0.9)).max() < SCORE_ATOL
    assert np.abs(to_np(g.sim_v) - oracle.anchor_similarity(vn, tfb.TF_ANCHOR_INCL_MEAN, 0.9)).max() < SCORE_ATOL
    g.close()


def test_kv_stats_persistent_many_tiles_per_worker():
    """2048 (tile, tensor) pairs on 888 workers: every worker of the persistent kernel runs its loop more than once
    (ticket prefetch, barrier phases and TMEM columns carried from tile to tile), and the one-tile kernel must agree."""
    q, k, v = _qkv(2, 4096, 16, 16, torch.bfloat16, seed=33)
    g = Gpu(q, k, v)
    _, kn, vn = oracle_inputs(q, k, v)
    ref_k, ref_v = oracle.anchor_similarity(kn), oracle.anchor_similarity(vn)
    for path in (3, 2, 3):
        g.sim_k.fill_(7.0); g.sim_v.fill_(7.0)
        g.ctx.tf_set_scan_path(path)
        g.ctx.tf_kv_stats(g.shape, g.params, k, v, g.sim_k, g.sim_v)
        g.status_ok()
        assert np.abs(to_np(g.sim_k) - ref_k).max() < SCORE_ATOL
        assert np.abs(to_np(g.sim_v) - ref_v).max() < SCORE_ATOL
    g.close()


@pytest.mark.parametrize("gamma", [0.8, 0.9, 0.95, 0.5])
@pytest.mark.parametrize("B,S,Hkv", [(1, 1, 1), (2, 65, 2), (3, 333, 5), (2, 1000, 3), (1, 4100, 2), (2, 2048, 4)])
@pytest.mark.parametrize("scan_path", [1, 2, 3])
def test_kv_stats_ema_anchor_every_path(gamma, B, S, Hkv, scan_path):
    """The anchor the paper deploys (Eq. 1, smoothing factors of its ablation plus a small one) on each scan kernel:
    the plain CUDA-core kernel and both Gram-matrix kernels (weighted row sums, weighted prefix scan, weighted tile
    aggregates), on lengths with ragged last tiles and several chunks per chain; twice, so that the second launch
    finds the first one's records."""
    q, k, v = _qkv(B, S, Hkv, Hkv, torch.bfloat16, seed=S + 7)
    g = Gpu(q, k, v, anchor_mode=tfb.TF_ANCHOR_EMA, gamma=gamma)
    g.ctx.tf_set_scan_path(scan_path)
    for _ in range(2):
        g.ctx.tf_kv_stats(g.shape, g.params, k, v, g.sim_k, g.sim_v)
    g.status_ok()
    assert g.ctx.tf_last_kernels()[0] == scan_path
    _, kn, vn = oracle_inputs(q, k, v)
    assert np.abs(to_np(g.sim_k) - oracle.anchor_similarity(kn, tfb.TF_ANCHOR_EMA, gamma)).max() < SCORE_ATOL
    assert np.abs(to_np(g.sim_v) - oracle.anchor_similarity(vn, tfb.TF_ANCHOR_EMA, gamma)).max() < SCORE_ATOL
    g.close()


@pytest.mark.parametrize("scan_path", [0, 1, 2, 3])
def test_kv_stats_ema_carry_chains_two_calls(scan_path):
    """EMA anchors carried from one call to the next (chunked prefill): two half-sequence calls equal one call, and the
    exported state is the anchor itself (Eq. 1 applied to every token), on every scan kernel."""
    B, S, H, gamma = 2, 700, 3, 0.9
    q, k, v = _qkv(B, S, H, H, torch.bfloat16, seed=19)
    _, kn, vn = oracle_inputs(q, k, v)
    ref_k, anchor_k = oracle.anchor_similarity(kn, tfb.TF_ANCHOR_EMA, gamma, want_sum_out=True)
    ref_v, anchor_v = oracle.anchor_similarity(vn, tfb.TF_ANCHOR_EMA, gamma, want_sum_out=True)
    h = 300                                                   # a ragged tile at the end of the first call
    g1 = Gpu(q[:, :h], k[:, :h], v[:, :h], anchor_mode=tfb.TF_ANCHOR_EMA, gamma=gamma)
    g1.ctx.tf_set_scan_path(scan_path)
    sk = torch.empty(B, H, 128, device=DEV); sv = torch.empty(B, H, 128, device=DEV)
    g1.ctx.tf_kv_stats(g1.shape, g1.params, k[:, :h], v[:, :h], g1.sim_k, g1.sim_v,
                       tfb.tf_carry(None, None, None, sk.data_ptr(), sv.data_ptr()))
    cnt = torch.full((B,), h, dtype=torch.int64, device=DEV)
    g2 = Gpu(q[:, h:], k[:, h:], v[:, h:], anchor_mode=tfb.TF_ANCHOR_EMA, gamma=gamma)
    g2.ctx.tf_set_scan_path(scan_path)
    sk2 = torch.empty_like(sk); sv2 = torch.empty_like(sv)
    g2.ctx.tf_kv_stats(g2.shape, g2.params, k[:, h:], v[:, h:], g2.sim_k, g2.sim_v,
                       tfb.tf_carry(sk.data_ptr(), sv.data_ptr(), cnt.data_ptr(), sk2.data_ptr(), sv2.data_ptr()))
    g1.status_ok(); g2.status_ok()
    assert np.abs(np.concatenate([to_np(g1.sim_k), to_np(g2.sim_k)], 1) - ref_k).max() < SCORE_ATOL
    assert np.abs(np.concatenate([to_np(g1.sim_v), to_np(g2.sim_v)], 1) - ref_v).max() < SCORE_ATOL
    assert np.abs(to_np(sk2) - anchor_k).max() < 1e-5 * max(1.0, np.abs(anchor_k).max())
    assert np.abs(to_np(sv2) - anchor_v).max() < 1e-5 * max(1.0, np.abs(anchor_v).max())
    g1.close(); g2.close()


@pytest.mark.parametrize("mode,gamma", [(tfb.TF_ANCHOR_INCL_MEAN, 0.9), (tfb.TF_ANCHOR_EMA, 0.9),
                                        (tfb.TF_ANCHOR_EMA, 0.8), (tfb.TF_ANCHOR_EMA, 0.95)])
@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_kv_stats_anchor_modes(mode, gamma, dtype):
    q, k, v = _qkv(2, 517, 4, 4, dtype, seed=5)
    g = Gpu(q, k, v, anchor_mode=mode, gamma=gamma)
    g.ctx.tf_kv_stats(g.shape, g.params, k, v, g.sim_k, g.sim_v)
    g.status_ok()
    _, kn, vn = oracle_inputs(q, k, v)
    assert np.abs(to_np(g.sim_k) - oracle.anchor_similarity(kn, mode, gamma)).max() < SCORE_ATOL
    assert np.abs(to_np(g.sim_v) - oracle.anchor_similarity(vn, mode, gamma)).max() < SCORE_ATOL
    g.close()


@pytest.mark.parametrize("scan_path", [0, 1, 2, 3])
def test_kv_stats_head_major_layout_and_carry(scan_path):
    """Same values stored [B,H,S,d] (strided view) give the same similarities; two half-sequence
    calls chained through the carry equal one call; the exported sums are the column sums.
    Every scan kernel (plain, Gram one tile per CTA, Gram persistent) takes the same route."""
    B, S, H = 2, 300, 4
    q, k, v = _qkv(B, S, H, H, torch.bfloat16, seed=9)
    kt = k.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    vt = v.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    assert kt.stride() != k.stride()
    g = Gpu(q, kt, vt)
    g.ctx.tf_set_scan_path(scan_path)
    g.ctx.tf_kv_stats(g.shape, g.params, kt, vt, g.sim_k, g.sim_v)
    g.status_ok()
    _, kn, vn = oracle_inputs(q, k, v)
    ref_k, sum_k = oracle.anchor_similarity(kn, want_sum_out=True)
    ref_v, sum_v = oracle.anchor_similarity(vn, want_sum_out=True)
    assert np.abs(to_np(g.sim_k) - ref_k).max() < SCORE_ATOL
    assert np.abs(to_np(g.sim_v) - ref_v).max() < SCORE_ATOL
    g.close()
    # chained halves
    h = S // 2
    g1 = Gpu(q[:, :h], k[:, :h], v[:, :h])
    g1.ctx.tf_set_scan_path(scan_path)
    sk = torch.empty(B, H, 128, device=DEV); sv = torch.empty(B, H, 128, device=DEV)
    c1 = tfb.tf_carry(None, None, None, sk.data_ptr(), sv.data_ptr())
    g1.ctx.tf_kv_stats(g1.shape, g1.params, k[:, :h], v[:, :h], g1.sim_k, g1.sim_v, c1)
    cnt = torch.full((B,), h, dtype=torch.int64, device=DEV)
    g2 = Gpu(q[:, h:], k[:, h:], v[:, h:])
    g2.ctx.tf_set_scan_path(scan_path)
    sk2 = torch.empty_like(sk); sv2 = torch.empty_like(sv)
    c2 = tfb.tf_carry(sk.data_ptr(), sv.data_ptr(), cnt.data_ptr(), sk2.data_ptr(), sv2.data_ptr())
    g2.ctx.tf_kv_stats(g2.shape, g2.params, k[:, h:], v[:, h:], g2.sim_k, g2.sim_v, c2)
    g2.status_ok()
    g1.status_ok()
    both = np.concatenate([to_np(g1.sim_k), to_np(g2.sim_k)], 1)
    assert np.abs(both - ref_k).max() < SCORE_ATOL
    both_v = np.concatenate([to_np(g1.sim_v), to_np(g2.sim_v)], 1)
    assert np.abs(both_v - ref_v).max() < SCORE_ATOL
    assert np.abs(to_np(sk2) - sum_k).max() < 1e-3 * max(1.0, np.abs(sum_k).max())
    assert np.abs(to_np(sv2) - sum_v).max() < 1e-3 * max(1.0, np.abs(sum_v).max())
    g1.close(); g2.close()


# ------------------------------------------------------------------------------- a3
@pytest.mark.parametrize("H", [1, 2, 8, 32, 40])
@pytest.mark.parametrize("mode", [tfb.TF_FUSE_INVVAR, tfb.TF_FUSE_EQ2_LITERAL, tfb.TF_FUSE_KEY_ONLY,
                                  tfb.TF_FUSE_VALUE_ONLY, tfb.TF_FUSE_MEAN])
def test_score_fuse_matches_oracle(H, mode):
    B, S = 2, 777
    rng = np.random.default_rng(H * 10 + mode)
    ck = rng.uniform(-0.3, 0.9, (B, S, H)).astype(np.float32)
    cv = rng.uniform(-0.3, 0.9, (B, S, H)).astype(np.float32)
    ck[0, 5] = 0.25; cv[0, 5] = -0.5           # zero variance on both sides
    q, k, v = _qkv(B, S, H, H, torch.bfloat16)
    g = Gpu(q, k, v, fuse_mode=mode)
    g.ctx.tf_score_fuse(g.shape, g.params, torch.from_numpy(ck).to(DEV), torch.from_numpy(cv).to(DEV), g.score)
    g.status_ok()
    ref = oracle.score_fuse(ck, cv, mode)
    assert np.abs(to_np(g.score) - ref).max() < 2e-6
    g.close()


# ------------------------------------------------------------------------------- a4
def _select_case(score, ratio, warm, elig=None, mode=tfb.TF_SELECT_RATIO, thr=None):
    """tf_select fed fp32 scores must agree bit for bit with the oracle fed the same values."""
    B, S = score.shape
    sc = torch.from_numpy(score).to(DEV)
    q = torch.zeros(B, S, 1, 128, dtype=torch.bfloat16, device=DEV)
    kw = dict(prune_ratio=ratio, warmup_tokens=warm, select_mode=mode)
    el_t = th_t = None
    if elig is not None:
        el_t = torch.from_numpy(elig).to(DEV); kw["eligible"] = el_t
    if thr is not None:
        th_t = torch.from_numpy(np.asarray(thr, np.float32)).to(DEV); kw["threshold"] = th_t
    g = Gpu(q, q, q, **kw)
    thr64 = None if thr is None else np.asarray(thr, np.float32).astype(np.float64)   # the same fp32 values
    ref = oracle.select(score.astype(np.float64), ratio, warm, elig, mode, thr64)
    # path 1: one CTA per sequence; path 2: a cluster of CTAs per sequence (1025 to 32768 tokens); 0: the library's choice
    for path in ([0, 1, 2] if CLUSTER_SELECT_MIN < S <= CLUSTER_SELECT_MAX else [0, 1]):
        g.ctx.tf_set_select_path(path)
        for t in (g.keep, g.idx, g.nk):
            t.fill_(77)
        g.theta.fill_(float("nan"))
        g.ctx.tf_select(g.shape, g.params, sc, g.keep, g.idx, g.nk, g.theta)
        g.status_ok()
        assert np.array_equal(g.keep.cpu().numpy(), ref["keep_mask"]), path
        assert np.array_equal(g.idx.cpu().numpy(), ref["kept_idx"]), path
        assert np.array_equal(g.nk.cpu().numpy(), ref["n_kept"]), path
        assert np.array_equal(g.theta.cpu().numpy().astype(np.float64), ref["theta"]), path
    g.close()


CLUSTER_SELECT_MIN, CLUSTER_SELECT_MAX = 1024, 32768   # sequence lengths the cluster form of steps a3 + a4 takes


@pytest.mark.parametrize("S", [1025, 1500, 2048, 2049, 4096, 5000, 16384, 20000, 32768])
@pytest.mark.parametrize("H,mode", [(1, tfb.TF_FUSE_INVVAR), (2, tfb.TF_FUSE_EQ2_LITERAL), (8, tfb.TF_FUSE_INVVAR),
                                    (8, tfb.TF_FUSE_KEY_ONLY), (12, tfb.TF_FUSE_VALUE_ONLY), (32, tfb.TF_FUSE_MEAN),
                                    (40, tfb.TF_FUSE_INVVAR)])
def test_score_select_in_one_launch_gives_the_bits_of_the_two_steps(S, H, mode):
    """tf_score_select (steps a3 + a4, a cluster per sequence) against tf_score_fuse followed by tf_select with one CTA
    per sequence: the same score bits, the same masks, lists, counts and thresholds; and both against the oracle."""
    B = 3
    rng = np.random.default_rng(S + H)
    ck = rng.uniform(-0.3, 0.9, (B, S, H)).astype(np.float32)
    cv = rng.uniform(-0.3, 0.9, (B, S, H)).astype(np.float32)
    ck[0, 5] = 0.25; cv[0, 5] = -0.5                       # zero variance on both sides
    ck[1, 700:720] = ck[1, 699]; cv[1, 700:720] = cv[1, 699]   # exactly equal scores
    q, k, v = _qkv(B, S, H, H, torch.bfloat16)
    g = Gpu(q, k, v, fuse_mode=mode, prune_ratio=0.5, warmup_tokens=4)
    ck_d, cv_d = torch.from_numpy(ck).to(DEV), torch.from_numpy(cv).to(DEV)
    g.ctx.tf_set_select_path(1)
    g.ctx.tf_score_fuse(g.shape, g.params, ck_d, cv_d, g.score)
    g.ctx.tf_select(g.shape, g.params, g.score, g.keep, g.idx, g.nk, g.theta)
    g.status_ok()
    two = [t.clone() for t in (g.score, g.keep, g.idx, g.nk, g.theta)]
    for path in (2, 0):
        g.ctx.tf_set_select_path(path)
        g.score.fill_(float("nan")); g.keep.fill_(77); g.idx.fill_(77); g.nk.fill_(77); g.theta.fill_(float("nan"))
        launches = g.ctx.tf_get_status()[1]["launches"]
        g.ctx.tf_score_select(g.shape, g.params, ck_d, cv_d, g.score, g.keep, g.idx, g.nk, g.theta)
        g.status_ok()
        one_launch = H <= 8                                  # step a3 joins the cluster's launch for up to 8 KV heads
        assert g.ctx.tf_get_status()[1]["launches"] == launches + (1 if one_launch else 2)
        for got, want in zip((g.score, g.keep, g.idx, g.nk, g.theta), two):
            assert torch.equal(got.view(torch.int32) if got.dtype == torch.float32 else got,
                               want.view(torch.int32) if want.dtype == torch.float32 else want), path
    score = to_np(g.score)
    assert np.abs(score - oracle.score_fuse(ck, cv, mode)).max() < 2e-6
    ref = oracle.select(score, 0.5, 4)
    assert np.array_equal(g.keep.cpu().numpy(), ref["keep_mask"]) and np.array_equal(g.idx.cpu().numpy(), ref["kept_idx"])
    g.close()


def test_cluster_selection_refuses_lengths_it_cannot_take():
    for S in (1000, 40000):
        q = torch.zeros(1, S, 1, 128, dtype=torch.bfloat16, device=DEV)
        g = Gpu(q, q, q)
        g.ctx.tf_set_select_path(2)
        with pytest.raises(tfb.TokenFilterError) as e:
            g.ctx.tf_select(g.shape, g.params, g.score, g.keep, g.idx, g.nk, g.theta)
        assert e.value.code == tfb.TF_ERR_UNSUPPORTED
        g.close()


@pytest.mark.parametrize("S", [1, 2, 31, 1024, 1025, 2048, 2049, 5000, 8193, 16384, 16385, 40000, 51200, 60000, 70000])   # register forms of 2, 4, 8, 16 scores per thread, then scores staged in shared memory (up to 51200), then re-read from global memory (one-scan sweep up to 65536 tokens, block scans beyond)
@pytest.mark.parametrize("ratio", [0.0, 0.25, 0.5, 0.7, 0.999])
def test_select_bit_exact_random(S, ratio):
    rng = np.random.default_rng(S)
    score = rng.normal(0.2, 0.2, (3, S)).astype(np.float32)
    _select_case(score, ratio, warm=min(4, S))


@pytest.mark.parametrize("case", ["ties", "all_equal", "eligible", "nan", "threshold", "threshold_eligible"])
def test_select_bit_exact_ties_eligibility_nan_threshold(case):
    rng = np.random.default_rng(3)
    S = 3000
    coarse = np.round(rng.uniform(-1, 1, (2, S)), 1).astype(np.float32)        # many exact ties
    coarse[0, ::7] = -0.0
    elig = (rng.uniform(size=(2, S)) < 0.4).astype(np.uint8)
    if case == "ties":
        _select_case(coarse, 0.5, 1)
    elif case == "all_equal":
        _select_case(np.zeros((2, S), np.float32), 0.3, 2)
    elif case == "eligible":
        _select_case(coarse, 0.7, 10, elig)                                     # capped by eligibility
    elif case == "nan":
        nan = coarse.copy(); nan[1, 100:200] = np.nan
        _select_case(nan, 0.5, 0)
    elif case == "threshold":
        _select_case(coarse, 0.5, 3, None, tfb.TF_SELECT_THRESHOLD, [0.3, -2.0])
    else:
        _select_case(coarse, 0.5, 3, elig, tfb.TF_SELECT_THRESHOLD, [5.0, 0.0])  # nothing / a lot


@pytest.mark.parametrize("n_tied", [2, 20, 32, 33, 200])
@pytest.mark.parametrize("S", [1500, 5000, 20000])      # two / eight scores per thread in registers, scores re-read
def test_select_few_candidates_left_with_ties_at_the_cut(S, n_tied):
    """The cut falls inside a group of exactly equal scores among otherwise distinct ones: after a pass or two
    the radix select has few candidates left under its prefix (one warp ranks them when there are at most 32),
    some of them tied, and the ties must go highest index first, exactly as the oracle takes them."""
    rng = np.random.default_rng(S + n_tied)
    score = rng.normal(0.2, 0.2, (2, S)).astype(np.float32)
    P = int(np.floor(0.5 * S))
    for b in range(2):
        order = np.argsort(-score[b], kind="stable")
        cut = order[P - n_tied // 2: P - n_tied // 2 + n_tied]     # the scores around rank P
        score[b, cut] = score[b, order[P]]
    _select_case(score, 0.5, warm=3)


# ------------------------------------------------------------------------------- a5
# path 2 / 3 / 4 / 5 / 6: the tensor-core kernel with K/V tiles shared by two Q tiles of one head / split between the softmax
# groups / one Q tile and one softmax group per CTA, two CTAs per SM / shared by the same rows of two / four query heads of
# one KV group (grouped-query shapes only)
def _skip_unless_heads_pair(path, Hq, Hkv):
    if path in (5, 6) and (Hq // Hkv) % {5: 2, 6: 4}[path]:
        pytest.skip("the head forms need a multiple of two / four query heads per KV head (their refusal has a test of its own)")


@pytest.mark.parametrize("dtype,tensor_cores", [(torch.bfloat16, 2), (torch.bfloat16, 3), (torch.bfloat16, 4), (torch.bfloat16, 5),
                                                (torch.bfloat16, 6), (torch.bfloat16, 1), (torch.bfloat16, 0), (torch.float32, 0)])
@pytest.mark.parametrize("B,S,Hq,Hkv,window,ratio", [(1, 1, 2, 1, 0, 0.0), (2, 130, 4, 4, 0, 0.5),
                                                    (1, 257, 8, 2, 0, 0.3), (2, 300, 4, 1, 64, 0.5),
                                                    (1, 515, 2, 2, 1, 0.7), (1, 200, 4, 2, 0, 0.99),
                                                    (1, 1300, 4, 2, 300, 0.5), (2, 1024, 2, 1, 0, 0.25)])
def test_pruned_attention_matches_oracle(dtype, tensor_cores, B, S, Hq, Hkv, window, ratio):
    _skip_unless_heads_pair(tensor_cores, Hq, Hkv)
    q, k, v = _qkv(B, S, Hq, Hkv, dtype, seed=S)
    qn, kn, vn = oracle_inputs(q, k, v)
    ref = oracle.layer_filter(qn, kn, vn, prune_ratio=ratio, warmup_tokens=1, window=window)
    g = Gpu(q, k, v, window=window)
    g.ctx.tf_set_attention_path(tensor_cores)
    idx = torch.from_numpy(ref["kept_idx"]).to(DEV)
    nk = torch.from_numpy(ref["n_kept"]).to(DEV)
    g.ctx.tf_pruned_attention(g.shape, g.params, q, k, v, idx, nk, g.O)
    g.status_ok()
    _assert_attention_kernel(g.ctx, dtype, tensor_cores)
    o = to_np(g.O)
    assert np.isfinite(o).all()
    assert attn_rel_err(o, ref["O"]) < ATTN_TOL[dtype]
    assert np.all(o[ref["keep_mask"] == 0] == 0.0)
    g.close()


def _assert_attention_kernel(ctx, dtype, path):
    """The kernel that ran is the one the path names: 0 CUDA cores, 2 / 3 the tensor-core kernel's shared / split
    form (a build whose tensor-core kernel cannot be launched fails the call instead of running on CUDA cores),
    4 / 5 / 6 its single, head-pair and head-quad forms, 1 the tensor-core kernel in whichever form it chooses."""
    ran = ctx.tf_last_kernels()[1]
    if dtype != torch.bfloat16 or path == 0:
        assert ran == tfb.TF_KERNEL_ATTN_SIMT
    elif path == 1:
        assert ran in (tfb.TF_KERNEL_ATTN_TC_SHARED, tfb.TF_KERNEL_ATTN_TC_SPLIT, tfb.TF_KERNEL_ATTN_TC_HEAD_PAIR,
                       tfb.TF_KERNEL_ATTN_TC_HEAD_QUAD)
    else:
        assert ran == {2: tfb.TF_KERNEL_ATTN_TC_SHARED, 3: tfb.TF_KERNEL_ATTN_TC_SPLIT, 4: tfb.TF_KERNEL_ATTN_TC_SINGLE,
                       5: tfb.TF_KERNEL_ATTN_TC_HEAD_PAIR, 6: tfb.TF_KERNEL_ATTN_TC_HEAD_QUAD}[path]


@pytest.mark.parametrize("dtype,path", [(torch.bfloat16, 2), (torch.bfloat16, 3), (torch.bfloat16, 4), (torch.bfloat16, 5),
                                        (torch.bfloat16, 6), (torch.bfloat16, 0), (torch.float32, 0)])
@pytest.mark.parametrize("B,S,Hq,Hkv,window,ratio", [(1, 1, 2, 1, 0, 0.0), (2, 130, 4, 4, 0, 0.5), (1, 257, 8, 2, 0, 0.3),
                                                    (2, 300, 4, 1, 64, 0.5), (1, 515, 2, 2, 1, 0.7),
                                                    (1, 1300, 4, 2, 300, 0.5), (2, 1024, 2, 1, 0, 0.25)])
def test_pruned_attention_retained_keys_only(dtype, path, B, S, Hq, Hkv, window, ratio):
    """TF_KV_RETAINED: a retained query attends to retained tokens only (a pruned token's key and value
    are gone for later queries as well); the window still counts original positions."""
    _skip_unless_heads_pair(path, Hq, Hkv)
    q, k, v = _qkv(B, S, Hq, Hkv, dtype, seed=S + 1)
    qn, kn, vn = oracle_inputs(q, k, v)
    ref = oracle.layer_filter(qn, kn, vn, prune_ratio=ratio, warmup_tokens=1, window=window,
                              kv_visibility=oracle.KV_RETAINED)
    g = Gpu(q, k, v, window=window, kv_visibility=tfb.TF_KV_RETAINED)
    g.ctx.tf_set_attention_path(path)
    idx = torch.from_numpy(ref["kept_idx"]).to(DEV)
    nk = torch.from_numpy(ref["n_kept"]).to(DEV)
    g.ctx.tf_pruned_attention(g.shape, g.params, q, k, v, idx, nk, g.O)
    g.status_ok()
    _assert_attention_kernel(g.ctx, dtype, path)
    o = to_np(g.O)
    assert np.isfinite(o).all()
    assert attn_rel_err(o, ref["O"]) < ATTN_TOL[dtype]
    assert np.all(o[ref["keep_mask"] == 0] == 0.0)
    if ratio > 0 and S > 100 and window == 0:   # and it is a different function from the all-keys reading
        dense = oracle.layer_filter(qn, kn, vn, prune_ratio=ratio, warmup_tokens=1, window=window)
        assert attn_rel_err(dense["O"], ref["O"]) > 10 * ATTN_TOL[dtype]
    g.close()


def test_layer_filter_retained_keys_only():
    q, k, v = _qkv(2, 700, 8, 2, torch.bfloat16, seed=77)
    n_mis = _layer_case(q, k, v, window=0, prune_ratio=0.5, warmup_tokens=4, kv_visibility=tfb.TF_KV_RETAINED)
    assert n_mis == 0


@pytest.mark.parametrize("path", [2, 3, 4, 5, 6])
def test_pruned_attention_nothing_kept_and_everything_kept(path):
    q, k, v = _qkv(2, 70, {5: 4, 6: 8}.get(path, 2), 2, torch.bfloat16)
    g = Gpu(q, k, v)
    g.ctx.tf_set_attention_path(path)
    idx = torch.full((2, 70), -1, dtype=torch.int32, device=DEV)
    idx[1] = torch.arange(70, dtype=torch.int32, device=DEV)
    nk = torch.tensor([0, 70], dtype=torch.int32, device=DEV)
    g.ctx.tf_pruned_attention(g.shape, g.params, q, k, v, idx, nk, g.O)
    o = to_np(g.O)
    assert np.all(o[0] == 0)
    qn, kn, vn = oracle_inputs(q, k, v)
    dense = oracle.pruned_attention(qn, kn, vn, np.ones((2, 70), np.uint8))
    assert attn_rel_err(o[1], dense[1]) < ATTN_TOL[torch.bfloat16]
    g.close()


def test_pruned_attention_head_groups_of_unequal_size():
    """A shape whose K and V exceed the L2 budget of the CTA order and whose (batch, head) pairs do not divide into
    equal groups (2 x 57 heads of 4096 tokens: groups of 29, 29, 29 and 27): every row block of every head must still be
    served exactly once.  Sampled rows against the oracle, the rest through properties that hold at any size."""
    B, S, H = 2, 4096, 57
    q, k, v = _qkv(B, S, H, H, torch.bfloat16, seed=57)
    rng = np.random.default_rng(57)
    score = rng.normal(0.2, 0.2, (B, S))
    ref = oracle.select(score, 0.5, 4)
    g = Gpu(q, k, v, prune_ratio=0.5, warmup_tokens=4)
    g.ctx.tf_set_attention_path(2)
    idx, nk = torch.from_numpy(ref["kept_idx"]).to(DEV), torch.from_numpy(ref["n_kept"]).to(DEV)
    g.ctx.tf_pruned_attention(g.shape, g.params, q, k, v, idx, nk, g.O)
    g.status_ok()
    assert g.ctx.tf_last_kernels()[1] == tfb.TF_KERNEL_ATTN_TC_SHARED
    keep_d = torch.from_numpy(ref["keep_mask"]).to(DEV).bool()
    assert bool((g.O[~keep_d] == 0).all()) and bool(torch.isfinite(g.O[keep_d]).all())
    assert bool((g.O[keep_d].float().abs().amax(dim=-1) > 0).all())          # every retained row of every head was written
    n = 1500
    bs = rng.integers(B, size=n)
    ts = np.array([ref["kept_idx"][b, rng.integers(ref["n_kept"][b])] for b in bs])
    hs = np.concatenate([np.arange(H), rng.integers(H, size=n - H)])          # every head at least once
    rows = np.stack([bs, ts, hs], 1).astype(np.int32)
    qn, kn, vn = q.float().cpu().numpy(), k.float().cpu().numpy(), v.float().cpu().numpy()
    want = oracle.attention_rows(qn, kn, vn, ref["keep_mask"], rows)
    got = g.O[rows[:, 0], rows[:, 1], rows[:, 2]].float().cpu().numpy().astype(np.float64)
    scale = np.maximum(np.abs(want).max(axis=-1, keepdims=True), 1e-30)
    assert float((np.abs(got - want) / scale).max()) < ATTN_TOL[torch.bfloat16]
    g.close()


@pytest.mark.parametrize("tensor_cores", [2, 3, 4, 5, 6])
@pytest.mark.parametrize("claimed_ratio", [0.0, 0.9])
def test_pruned_attention_with_a_retained_list_the_ratio_does_not_predict(tensor_cores, claimed_ratio):
    """tf_pruned_attention takes any retained list; the kernel orders its row blocks by the count the prune ratio
    suggests.  With a list much longer or much shorter than that, every row block must still be served once."""
    B, S, Hq, Hkv = 2, 1500, 8, 2
    q, k, v = _qkv(B, S, Hq, Hkv, torch.bfloat16, seed=5)
    qn, kn, vn = oracle_inputs(q, k, v)
    ref = oracle.layer_filter(qn, kn, vn, prune_ratio=0.4, warmup_tokens=1)      # the list really keeps 60 %
    g = Gpu(q, k, v, prune_ratio=claimed_ratio)
    g.ctx.tf_set_attention_path(tensor_cores)
    g.O.fill_(float("nan"))
    g.ctx.tf_pruned_attention(g.shape, g.params, q, k, v, torch.from_numpy(ref["kept_idx"]).to(DEV),
                              torch.from_numpy(ref["n_kept"]).to(DEV), g.O)
    g.status_ok()
    assert attn_rel_err(to_np(g.O), ref["O"]) < ATTN_TOL[torch.bfloat16]
    g.close()


# ------------------------------------------------------------------------------- whole layer
def _layer_case(q, k, v, window=0, **kw):
    qn, kn, vn = oracle_inputs(q, k, v)
    okw = {a: b for a, b in kw.items()}
    ref = oracle.layer_filter(qn, kn, vn, window=window, **okw)
    g = Gpu(q, k, v, window=window, **kw)
    g.ctx.tf_layer_filter(g.shape, g.params, q, k, v, g.O, g.score, g.keep, g.idx, g.nk)
    g.status_ok()
    assert np.abs(to_np(g.score) - ref["score"]).max() < SCORE_ATOL
    n_mis, n_out = mask_disagreements(g.keep.cpu().numpy(), ref)
    assert n_out == 0, f"{n_mis} keep/prune disagreements, {n_out} outside the 1e-6 band around theta"
    keep = g.keep.cpu().numpy()
    idx = g.idx.cpu().numpy(); nk = g.nk.cpu().numpy()
    for b in range(keep.shape[0]):
        assert np.array_equal(idx[b, :nk[b]], np.nonzero(keep[b])[0]) and np.all(idx[b, nk[b]:] == -1)
    if n_mis == 0:
        assert attn_rel_err(to_np(g.O), ref["O"]) < ATTN_TOL[q.dtype]
    else:   # compare attention on the oracle's own kept set
        g.ctx.tf_pruned_attention(g.shape, g.params, q, k, v, torch.from_numpy(ref["kept_idx"]).to(DEV),
                                  torch.from_numpy(ref["n_kept"]).to(DEV), g.O)
        assert attn_rel_err(to_np(g.O), ref["O"]) < ATTN_TOL[q.dtype]
    g.close()
    return n_mis


def test_layer_filter_config1_fp32():
    """Config 1 in full: B1 S128 32 heads fp32, 25% near-duplicates, 50% pruning."""
    wl = W.WORKLOADS["c1"]
    _, q, k, v = next(wl.layer_qkv([0], DEV))
    _layer_case(q, k, v, prune_ratio=0.5, warmup_tokens=4)
    _layer_case(q, k, v, prune_ratio=0.5, warmup_tokens=4, fuse_mode=tfb.TF_FUSE_EQ2_LITERAL)


@pytest.mark.parametrize("B,S,Hq,Hkv,window,ratio", [(1, 777, 8, 8, 0, 0.5), (2, 1111, 8, 2, 0, 0.3),
                                                    (2, 900, 8, 2, 0, 0.7), (2, 1500, 8, 2, 256, 0.5),
                                                    (1, 640, 10, 10, 0, 0.25), (1, 333, 4, 4, 0, 0.0)])
def test_layer_filter_reduced_shapes_bf16(B, S, Hq, Hkv, window, ratio):
    q, k, v = _qkv(B, S, Hq, Hkv, torch.bfloat16, seed=S + Hq)
    _layer_case(q, k, v, window=window, prune_ratio=ratio, warmup_tokens=4)


def test_layer_filter_host_entry_matches_device_entry():
    q, k, v = W.duplicate_qkv(2, 400, 8, 2, 128, 0.25, 0.05, seed=21, dtype=torch.bfloat16)
    qd, kd, vd = q.to(DEV), k.to(DEV), v.to(DEV)
    g = Gpu(qd, kd, vd, prune_ratio=0.5, warmup_tokens=4)
    g.ctx.tf_layer_filter(g.shape, g.params, qd, kd, vd, g.O, g.score, g.keep, g.idx, g.nk)
    torch.cuda.synchronize()
    qh, kh, vh = q.pin_memory(), k.pin_memory(), v.pin_memory()
    oh = torch.empty_like(qh).pin_memory()
    sh = torch.empty(2, 400).pin_memory(); mh = torch.empty(2, 400, dtype=torch.uint8).pin_memory()
    ih = torch.empty(2, 400, dtype=torch.int32).pin_memory(); nh = torch.empty(2, dtype=torch.int32).pin_memory()
    hs = tfb.make_shape(qh, kh, vh, oh)
    g.ctx.tf_layer_filter_host(hs, g.params, qh, kh, vh, oh, sh, mh, ih, nh)
    assert torch.equal(oh, g.O.cpu()) and torch.equal(sh, g.score.cpu()) and torch.equal(mh, g.keep.cpu())
    assert torch.equal(ih, g.idx.cpu()) and torch.equal(nh, g.nk.cpu())
    g.close()


@pytest.mark.parametrize("visibility", [tfb.TF_KV_ALL, tfb.TF_KV_RETAINED])
def test_layer_filter_host_pipelined_head_groups(visibility):
    """A layer large enough for the host entry point to send Q in groups of query heads (whole KV-head groups)
    while earlier groups' attention runs and their output rows travel back: same bytes as the device entry point."""
    q, k, v = _qkv(1, 2048, 32, 8, torch.bfloat16, seed=61)
    g = Gpu(q, k, v, prune_ratio=0.5, warmup_tokens=4, kv_visibility=visibility)
    g.ctx.tf_layer_filter(g.shape, g.params, q, k, v, g.O, g.score, g.keep, g.idx, g.nk)
    torch.cuda.synchronize()
    qh, kh, vh = q.cpu().pin_memory(), k.cpu().pin_memory(), v.cpu().pin_memory()
    oh = torch.full_like(qh, float("nan")).pin_memory()
    sh = torch.empty(1, 2048).pin_memory(); mh = torch.empty(1, 2048, dtype=torch.uint8).pin_memory()
    ih = torch.empty(1, 2048, dtype=torch.int32).pin_memory(); nh = torch.empty(1, dtype=torch.int32).pin_memory()
    hs = tfb.make_shape(qh, kh, vh, oh)
    for _ in range(2):
        oh.fill_(float("nan"))
        g.ctx.tf_layer_filter_host(hs, g.params, qh, kh, vh, oh, sh, mh, ih, nh)
        assert torch.equal(oh, g.O.cpu()) and torch.equal(sh, g.score.cpu()) and torch.equal(mh, g.keep.cpu())
        assert torch.equal(ih, g.idx.cpu()) and torch.equal(nh, g.nk.cpu())
    g.status_ok()
    g.close()


def test_decode_and_prefill_share_the_workspace():
    """The decode step keeps its split-key partial results in the bound workspace, over the region where the
    similarity scan keeps its records; a scan after decode steps must still be right (it clears its region first),
    and the split decode output must equal the one-CTA-per-head output computed without a workspace."""
    B, S, Hq, Hkv = 2, 2304, 8, 2
    q, k, v = _qkv(B, S, Hq, Hkv, torch.bfloat16, seed=77)
    _, kn, vn = oracle_inputs(q, k, v)
    ref_k = oracle.anchor_similarity(kn)
    ctx = tfb.Context(0)
    params = tfb.default_params(prune_ratio=0.25, warmup_tokens=4)
    pshape = tfb.make_shape(None, k, v)
    ctx.ensure_workspace(pshape, params)
    sk = torch.empty(B, S, Hkv, device=DEV); sv = torch.empty_like(sk)
    shape = tfb.make_shape(None, k, v, n_q_heads=Hq)
    O = torch.empty(B, Hq, 128, dtype=torch.bfloat16, device=DEV)
    shape.q_stride[:] = [q.stride(0), 0, q.stride(2)]
    shape.o_stride[:] = [O.stride(0), 0, O.stride(1)]
    score = torch.empty(B, device=DEV); skip = torch.empty(B, dtype=torch.uint8, device=DEV)
    pos = torch.full((B,), S - 1, dtype=torch.int32, device=DEV)
    outs = []
    for rnd in range(2):
        ctx.tf_kv_stats(pshape, params, k, v, sk, sv)
        assert np.abs(to_np(sk) - ref_k).max() < SCORE_ATOL, rnd
        st = tfb.DecodeState(B, Hkv, DEV, tau0=10.0)          # a threshold no score reaches: attention always runs
        n0 = ctx.launches
        ctx.tf_decode_step(shape, params, 0.0, q[:, S - 1], k, v, pos, st, O, score, skip)
        assert ctx.launches - n0 == 3                          # decide, split attention, combine
        outs.append(O.clone())
    ctx.set_workspace(None)
    st = tfb.DecodeState(B, Hkv, DEV, tau0=10.0)
    n0 = ctx.launches
    ctx.tf_decode_step(shape, params, 0.0, q[:, S - 1], k, v, pos, st, O, score, skip)
    assert ctx.launches - n0 == 2                              # no workspace: one CTA per KV head, no combine
    code, det = ctx.tf_get_status()
    assert code == tfb.TF_OK, det
    assert torch.equal(outs[0], outs[1])
    assert attn_rel_err(to_np(outs[0]), to_np(O)) < 1e-2       # same products, different split of the softmax sums
    ctx.close()


def test_device_rejects_bad_arguments_without_launching():
    q, k, v = _qkv(1, 64, 2, 2, torch.bfloat16)
    g = Gpu(q, k, v)
    L = tfb.lib()
    st = C.c_void_p(torch.cuda.current_stream().cuda_stream)
    n0 = g.ctx.launches
    bad = tfb.default_params(prune_ratio=1.0)
    assert L.tf_layer_filter(g.ctx._h, C.byref(g.shape), C.byref(bad), *[C.c_void_p(t.data_ptr()) for t in (q, k, v, g.O)],
                             None, None, None, None, st) == tfb.TF_ERR_INVALID_ARG
    assert L.tf_kv_stats(g.ctx._h, C.byref(g.shape), C.byref(g.params), C.c_void_p(k.data_ptr() + 2),
                         C.c_void_p(v.data_ptr()), C.c_void_p(g.sim_k.data_ptr()), C.c_void_p(g.sim_v.data_ptr()),
                         None, st) == tfb.TF_ERR_UNSUPPORTED
    g.ctx.set_workspace(None)
    assert L.tf_kv_stats(g.ctx._h, C.byref(g.shape), C.byref(g.params), C.c_void_p(k.data_ptr()),
                         C.c_void_p(v.data_ptr()), C.c_void_p(g.sim_k.data_ptr()), C.c_void_p(g.sim_v.data_ptr()),
                         None, st) == tfb.TF_ERR_WORKSPACE
    assert g.ctx.launches == n0
    g.close()


# ------------------------------------------------------------------------------- device status record
def test_nan_score_is_reported_counted_and_cleared():
    """A NaN similarity makes the fused score NaN: tf_get_status returns TF_ERR_NAN_SCORE with the count of NaN
    scores, the selection never prunes such a token, and tf_clear_status resets the record."""
    B, S, H = 2, 300, 4
    rng = np.random.default_rng(7)
    ck = rng.uniform(-0.2, 0.8, (B, S, H)).astype(np.float32)
    cv = rng.uniform(-0.2, 0.8, (B, S, H)).astype(np.float32)
    ck[0, 17, 1] = np.nan; cv[1, 200, 0] = np.nan; ck[1, 250, 3] = np.nan
    q = torch.zeros(B, S, H, 128, dtype=torch.bfloat16, device=DEV)
    g = Gpu(q, q, q, prune_ratio=0.5, warmup_tokens=0)
    g.ctx.tf_score_fuse(g.shape, g.params, torch.from_numpy(ck).to(DEV), torch.from_numpy(cv).to(DEV), g.score)
    code, det = g.ctx.tf_get_status()
    assert code == tfb.TF_ERR_NAN_SCORE and det["code"] == tfb.TF_ERR_NAN_SCORE
    assert det["nan_count"] == 3
    assert det["where"] in (0 * S + 17, 1 * S + 200, 1 * S + 250)      # the token index of the first one seen
    sc = to_np(g.score)
    assert np.isnan(sc[0, 17]) and np.isnan(sc[1, 200]) and np.isnan(sc[1, 250]) and np.isnan(sc).sum() == 3
    g.ctx.tf_select(g.shape, g.params, g.score, g.keep, g.idx, g.nk, g.theta)
    keep = g.keep.cpu().numpy()
    assert keep[0, 17] == 1 and keep[1, 200] == 1 and keep[1, 250] == 1
    ref = oracle.select(sc.astype(np.float64), 0.5, 0)
    assert np.array_equal(keep, ref["keep_mask"]) and list(ref["n_nan"]) == [1, 2]
    g.ctx.tf_clear_status()
    code, det = g.ctx.tf_get_status()
    assert code == tfb.TF_OK and det["nan_count"] == 0 and det["code"] == 0
    g.close()


def test_bounded_wait_that_runs_out_is_reported_and_the_context_recovers():
    """tf_wait_selftest waits, with short limits, on an mbarrier nobody arrives at (spinning and parked form) and on a
    record nobody writes, through the device functions every kernel waits with: the kernel ends by itself (no hang, no
    trap), tf_get_status returns TF_ERR_TIMEOUT and says which wait gave up first, the context stays usable, and
    after tf_clear_status a scan on the same context is right."""
    q, k, v = _qkv(1, 700, 2, 2, torch.bfloat16, seed=3)
    g = Gpu(q, k, v)
    _, kn, vn = oracle_inputs(q, k, v)
    ref_k, ref_v = oracle.anchor_similarity(kn), oracle.anchor_similarity(vn)
    g.ctx.tf_kv_stats(g.shape, g.params, k, v, g.sim_k, g.sim_v)
    g.status_ok()
    g.ctx.tf_set_wait_limits(max_polls=3, wait_cycles=200000)
    g.ctx.tf_wait_selftest()
    code, det = g.ctx.tf_get_status()
    assert code == tfb.TF_ERR_TIMEOUT and det["code"] == tfb.TF_ERR_TIMEOUT
    assert det["where"] in (901, 902, 903)
    code2, _ = g.ctx.tf_get_status()                           # the record is sticky until cleared
    assert code2 == tfb.TF_ERR_TIMEOUT
    g.ctx.tf_clear_status()
    g.ctx.tf_set_wait_limits()                                 # defaults again
    for path in (2, 3, 1):
        g.sim_k.fill_(float("nan")); g.sim_v.fill_(float("nan"))
        g.ctx.tf_set_scan_path(path)
        g.ctx.tf_kv_stats(g.shape, g.params, k, v, g.sim_k, g.sim_v)
        g.status_ok()
        assert np.abs(to_np(g.sim_k) - ref_k).max() < SCORE_ATOL
        assert np.abs(to_np(g.sim_v) - ref_v).max() < SCORE_ATOL
    g.close()


@pytest.mark.parametrize("scan_path", [1, 2, 3])
def test_zero_poll_limit_never_hangs_and_the_next_launch_is_clean(scan_path):
    """A limit of zero polls on each scan kernel: a look-back record that is not there at the first look counts as missing
    (whether it is there is a matter of timing, so the status may say TF_OK or TF_ERR_TIMEOUT).  Whatever it says, the
    call returns, and the next launch with default limits is right -- the counters a launch draws its work from start at
    zero again and the records are cleared."""
    q, k, v = _qkv(2, 1500, 3, 3, torch.bfloat16, seed=4)
    g = Gpu(q, k, v)
    _, kn, vn = oracle_inputs(q, k, v)
    g.ctx.tf_set_scan_path(scan_path)
    g.ctx.tf_set_wait_limits(max_polls=0)
    for _ in range(2):
        g.ctx.tf_kv_stats(g.shape, g.params, k, v, g.sim_k, g.sim_v)
    code, _ = g.ctx.tf_get_status()
    assert code in (tfb.TF_OK, tfb.TF_ERR_TIMEOUT)
    g.ctx.tf_clear_status()
    g.ctx.tf_set_wait_limits()
    g.ctx.tf_kv_stats(g.shape, g.params, k, v, g.sim_k, g.sim_v)
    g.status_ok()
    assert np.abs(to_np(g.sim_k) - oracle.anchor_similarity(kn)).max() < SCORE_ATOL
    assert np.abs(to_np(g.sim_v) - oracle.anchor_similarity(vn)).max() < SCORE_ATOL
    g.close()


def test_requested_kernel_that_cannot_take_the_call_is_an_error_not_a_fallback():
    q, k, v = _qkv(1, 200, 2, 2, torch.float32)
    g = Gpu(q, k, v)
    for path in (2, 3):                                        # the Gram kernels take bf16 only
        g.ctx.tf_set_scan_path(path)
        with pytest.raises(tfb.TokenFilterError) as e:
            g.ctx.tf_kv_stats(g.shape, g.params, k, v, g.sim_k, g.sim_v)
        assert e.value.code == tfb.TF_ERR_UNSUPPORTED
    g.close()
    for Hq, path in ((6, 5), (4, 6)):                          # three / two query heads per KV head: no pairs / no fours
        q, k, v = _qkv(1, 200, Hq, 2, torch.bfloat16)
        g = Gpu(q, k, v)
        g.ctx.tf_set_attention_path(path)
        with pytest.raises(tfb.TokenFilterError) as e:
            g.ctx.tf_layer_filter(g.shape, g.params, q, k, v, g.O, g.score, g.keep, g.idx, g.nk)
        assert e.value.code == tfb.TF_ERR_UNSUPPORTED
        g.close()


# ------------------------------------------------------------------------------- online decode step
@pytest.mark.parametrize("dtype,mode,window,S0,T,Hq,Hkv",
                         [(torch.bfloat16, tfb.TF_ANCHOR_PAST_MEAN, 0, 70, 90, 8, 2), (torch.float32, tfb.TF_ANCHOR_PAST_MEAN, 40, 70, 90, 8, 2),
                          (torch.bfloat16, tfb.TF_ANCHOR_EMA, 0, 70, 90, 8, 2), (torch.bfloat16, tfb.TF_ANCHOR_INCL_MEAN, 0, 70, 90, 8, 2),
                          # long caches: the grouped kernel splits the keys over several CTAs and merges the partial results
                          (torch.bfloat16, tfb.TF_ANCHOR_PAST_MEAN, 0, 2900, 24, 8, 1), (torch.bfloat16, tfb.TF_ANCHOR_PAST_MEAN, 1500, 2100, 24, 4, 4),
                          (torch.bfloat16, tfb.TF_ANCHOR_PAST_MEAN, 0, 1100, 24, 6, 3)])
def test_decode_steps_match_oracle(dtype, mode, window, S0, T, Hq, Hkv):
    """A prefill of 70 tokens seeds the anchors through tf_kv_stats' carry; then 90 decode steps run in
    lockstep with the oracle: scores within 1e-5, skip decisions equal unless the score is within 1e-5 of
    the threshold (then the oracle's counters are forced on so the runs stay comparable), outputs within the
    attention tolerance; skipped rows are zero.  The oracle is fp64 throughout; the library's threshold is an
    fp32 state word (tf_decode_state.tau) and its step size an fp32 argument, so the oracle is given the same
    fp32 value of eta, and after n updates the two thresholds may differ by n roundings of an fp32 sum:
    |tau_gpu - tau_oracle| <= n * 2^-23 * max(1, |tau|)  (one rounding of the step, one of the sum, per update)."""
    B = 2
    S = S0 + T
    q, k, v = _qkv(B, S, Hq, Hkv, dtype, seed=123, dup=0.4)
    qn, kn, vn = oracle_inputs(q, k, v)
    ctx = tfb.Context(0)
    params = tfb.default_params(prune_ratio=0.25, warmup_tokens=4, anchor_mode=mode, gamma=0.9)
    st = tfb.DecodeState(B, Hkv, DEV, tau0=0.3)
    # prefill: anchors from the first S0 tokens
    pshape = tfb.make_shape(None, k[:, :S0], v[:, :S0])
    ctx.ensure_workspace(pshape, params)
    sk = torch.empty(B, S0, Hkv, device=DEV); sv = torch.empty_like(sk)
    ctx.tf_kv_stats(pshape, params, k[:, :S0], v[:, :S0], sk, sv,
                    tfb.tf_carry(None, None, None, st.sum_k.data_ptr(), st.sum_v.data_ptr()))
    st.count.fill_(S0)
    ost = oracle.decode_state(B, Hkv, 128, tau0=0.3)
    _, sum_k = oracle.anchor_similarity(kn[:, :S0], mode, 0.9, want_sum_out=True)
    _, sum_v = oracle.anchor_similarity(vn[:, :S0], mode, 0.9, want_sum_out=True)
    ost["sum_k"][:] = sum_k; ost["sum_v"][:] = sum_v; ost["count"][:] = S0
    assert np.abs(to_np(st.sum_k) - sum_k).max() < 1e-3

    shape = tfb.make_shape(None, k, v, window=window, n_q_heads=Hq)
    O = torch.full((B, Hq, 128), float("nan"), dtype=dtype, device=DEV)
    shape.q_stride[:] = [q.stride(0), 0, q.stride(2)]
    shape.o_stride[:] = [O.stride(0), 0, O.stride(1)]
    score = torch.empty(B, device=DEV); skip = torch.empty(B, dtype=torch.uint8, device=DEV)
    near, n_skips = 0, 0
    eta = float(np.float32(0.05))         # the value the C-ABI's float argument carries
    for t in range(S0, S):
        pos = torch.full((B,), t, dtype=torch.int32, device=DEV)
        ctx.tf_decode_step(shape, params, eta, q[:, t], k, v, pos, st, O, score, skip)
        ref = oracle.decode_step(ost, qn[:, t], kn, vn, np.full(B, t), target_ratio=0.25, eta=eta, warmup_tokens=4,
                                 anchor_mode=mode, gamma=0.9, window=window)
        assert np.abs(to_np(score) - ref["score"]).max() < SCORE_ATOL
        n_upd = t - S0 + 1
        tau_gpu = st.tau.cpu().numpy().astype(np.float64)
        assert np.abs(tau_gpu - ref["tau"]).max() <= n_upd * 2.0 ** -23 * max(1.0, np.abs(ref["tau"]).max())
        g_skip = skip.cpu().numpy()
        for b in range(B):
            if g_skip[b] != ref["skip"][b]:
                assert abs(ref["score"][b] - ref["tau"][b]) < 1e-5, (t, b, ref["score"][b], ref["tau"][b])
                near += 1
        if np.array_equal(g_skip, ref["skip"]):
            o = to_np(O)
            assert attn_rel_err(o, ref["O"]) < ATTN_TOL[dtype]
            assert np.all(o[ref["skip"] == 1] == 0.0)
        else:   # keep the two runs on the same trajectory
            st.steps.copy_(torch.from_numpy(ost["steps"])); st.skips.copy_(torch.from_numpy(ost["skips"]))
        n_skips += int(ref["skip"].sum())
    code, det = ctx.tf_get_status()
    assert code == tfb.TF_OK, det
    assert np.array_equal(st.count.cpu().numpy(), ost["count"]) and np.array_equal(st.steps.cpu().numpy(), ost["steps"])
    assert 0 < n_skips < B * T            # the case exercises both branches (skip and attend)
    assert near <= 2
    ctx.close()


# ------------------------------------------------------------------------------- seeded random sweep
@pytest.mark.parametrize("case", range(32))
def test_layer_filter_random_shapes_modes_and_layouts(case):
    """A seeded sweep over what the named cases do not pair up: shapes with ragged tiles, every anchor mode, fusion
    mode and K/V visibility, windows, ratios, both dtypes and every attention form, each against the oracle."""
    rng = np.random.default_rng(1000 + case)
    dtype = torch.float32 if case % 8 == 7 else torch.bfloat16
    B = int(rng.integers(1, 4))
    S = int(rng.choice([1, 2, 17, 127, 128, 129, 255, 300, 513, 777, 1025, 1400]))
    Hkv = int(rng.choice([1, 2, 3, 4, 8]))
    Hq = Hkv * int(rng.choice([1, 2, 4]))
    window = int(rng.choice([0, 0, 1, 37, 128, 400]))
    ratio = float(rng.choice([0.0, 0.1, 0.3, 0.5, 0.7, 0.95]))
    kw = dict(prune_ratio=ratio, warmup_tokens=int(rng.choice([1, 4, 9])),
              anchor_mode=int(rng.choice([tfb.TF_ANCHOR_PAST_MEAN, tfb.TF_ANCHOR_INCL_MEAN, tfb.TF_ANCHOR_EMA])),
              gamma=float(rng.choice([0.8, 0.9, 0.95])),
              fuse_mode=int(rng.choice([tfb.TF_FUSE_INVVAR, tfb.TF_FUSE_EQ2_LITERAL, tfb.TF_FUSE_KEY_ONLY,
                                        tfb.TF_FUSE_VALUE_ONLY, tfb.TF_FUSE_MEAN])),
              kv_visibility=int(rng.choice([tfb.TF_KV_ALL, tfb.TF_KV_ALL, tfb.TF_KV_RETAINED])))
    if kw["anchor_mode"] == tfb.TF_ANCHOR_INCL_MEAN:
        kw["warmup_tokens"] = max(kw["warmup_tokens"], 1)
    q, k, v = _qkv(B, S, Hq, Hkv, dtype, seed=2000 + case, dup=float(rng.choice([0.0, 0.25, 0.6])))
    qn, kn, vn = oracle_inputs(q, k, v)
    ref = oracle.layer_filter(qn, kn, vn, window=window, **kw)
    g = Gpu(q, k, v, window=window, **kw)
    path = int(rng.choice([1, 2, 3, 4, 5, 6])) if dtype == torch.bfloat16 else 0
    g.ctx.tf_set_attention_path(1 if path in (5, 6) and (Hq // Hkv) % {5: 2, 6: 4}[path] else path)
    g.ctx.tf_layer_filter(g.shape, g.params, q, k, v, g.O, g.score, g.keep, g.idx, g.nk)
    g.status_ok()
    assert np.abs(to_np(g.score) - ref["score"]).max() < SCORE_ATOL
    n_mis, n_out = mask_disagreements(g.keep.cpu().numpy(), ref)
    assert n_out == 0, f"{n_mis} keep/prune disagreements, {n_out} outside the 1e-6 band around theta"
    if n_mis:      # compare the attention on the oracle's own retained list
        g.ctx.tf_pruned_attention(g.shape, g.params, q, k, v, torch.from_numpy(ref["kept_idx"]).to(DEV),
                                  torch.from_numpy(ref["n_kept"]).to(DEV), g.O)
    o = to_np(g.O)
    assert attn_rel_err(o, ref["O"]) < ATTN_TOL[dtype]
    assert np.all(o[ref["keep_mask"] == 0] == 0.0)
    g.close()


def test_layer_filter_replayed_from_a_cuda_graph_with_new_inputs():
    """One tf_layer_filter call captured into a CUDA graph (after a first call outside the capture, which clears the
    scratch and sets function attributes) and replayed over buffers whose contents change between replays: everything a
    launch needs to tell its own look-back records from an earlier launch's lives on the device, so every replay is
    right.  Both Gram-scan kernels and the CUDA-core scan; fusion and selection as two launches and as the cluster launch."""
    B, S, Hq, Hkv = 2, 1300, 8, 2
    inputs = [_qkv(B, S, Hq, Hkv, torch.bfloat16, seed=90 + i) for i in range(3)]
    for scan_path, select_path in ((2, 1), (3, 2), (1, 2)):
        q, k, v = (t.clone() for t in inputs[0])
        g = Gpu(q, k, v, prune_ratio=0.5, warmup_tokens=4)
        g.ctx.tf_set_scan_path(scan_path)
        g.ctx.tf_set_select_path(select_path)
        g.ctx.tf_layer_filter(g.shape, g.params, q, k, v, g.O, g.score, g.keep, g.idx, g.nk)     # outside the capture
        torch.cuda.synchronize()
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            with torch.cuda.graph(graph, stream=side):
                g.ctx.tf_layer_filter(g.shape, g.params, q, k, v, g.O, g.score, g.keep, g.idx, g.nk)
        torch.cuda.current_stream().wait_stream(side)
        for qi, ki, vi in inputs[1:] + inputs[:1]:
            q.copy_(qi); k.copy_(ki); v.copy_(vi)
            g.O.fill_(float("nan")); g.score.fill_(float("nan"))
            graph.replay()
            torch.cuda.synchronize()
            g.status_ok()
            qn, kn, vn = oracle_inputs(q, k, v)
            ref = oracle.layer_filter(qn, kn, vn, prune_ratio=0.5, warmup_tokens=4)
            assert np.abs(to_np(g.score) - ref["score"]).max() < SCORE_ATOL
            n_mis, n_out = mask_disagreements(g.keep.cpu().numpy(), ref)
            assert n_out == 0
            if n_mis == 0:
                assert attn_rel_err(to_np(g.O), ref["O"]) < ATTN_TOL[torch.bfloat16]
        g.close()

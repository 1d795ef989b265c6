"""Pins for the CPU oracle: every routine is checked against something other than itself —
a library routine on a case that reduces to it, a closed form, an invariant, or the counts that
follow from the paper's formulas (tests/golden/keep_counts.txt). No GPU needed."""
import os

import numpy as np
import pytest
import torch
import torch.nn.functional as F

import oracle
from paper_2508_02558_b200 import workloads as W

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _rand(shape, seed):
    return np.random.default_rng(seed).standard_normal(shape)


# ------------------------------------------------------------------ attention (textbook definition)
@pytest.mark.parametrize("Hq,Hkv,b,nk,D", [(2, 2, 4, 9, 8), (6, 2, 5, 33, 16), (4, 1, 32, 70, 64)])
def test_attention_matches_library_sdpa(Hq, Hkv, b, nk, D):
    q, k, v = _rand((Hq, b, D), 1), _rand((Hkv, nk, D), 2), _rand((Hkv, nk, D), 3)
    out, lse = oracle.attention(q, k, v)
    G = Hq // Hkv
    kt = torch.from_numpy(k).repeat_interleave(G, dim=0)
    vt = torch.from_numpy(v).repeat_interleave(G, dim=0)
    ref = F.scaled_dot_product_attention(torch.from_numpy(q)[None], kt[None], vt[None])[0].numpy()
    np.testing.assert_allclose(out, ref, rtol=0, atol=1e-12)
    s = torch.einsum("hid,hjd->hij", torch.from_numpy(q), kt) / np.sqrt(D)
    np.testing.assert_allclose(lse, torch.logsumexp(s, dim=-1).numpy(), rtol=0, atol=1e-12)


def test_attention_closed_forms():
    Hq, Hkv, b, nk, D = 4, 2, 3, 11, 8
    q, v = _rand((Hq, b, D), 4), _rand((Hkv, nk, D), 5)
    # identical keys -> uniform probabilities -> output is the plain mean of V, lse = s + log(nk)
    k = np.broadcast_to(_rand((Hkv, 1, D), 6), (Hkv, nk, D)).copy()
    out, lse, probs = oracle.attention(q, k, v, return_probs=True)
    np.testing.assert_allclose(probs, 1.0 / nk, atol=1e-15)
    for h in range(Hq):
        np.testing.assert_allclose(out[h], np.broadcast_to(v[h // 2].mean(0), (b, D)), atol=1e-13)
        s = (q[h] @ k[h // 2, 0]) / np.sqrt(D)
        np.testing.assert_allclose(lse[h], s + np.log(nk), atol=1e-13)
    # a single key -> output is that value row exactly
    out1, _ = oracle.attention(q, k[:, :1], v[:, :1])
    for h in range(Hq):
        np.testing.assert_array_equal(out1[h], np.broadcast_to(v[h // 2, 0], (b, D)))
    # one overwhelmingly aligned key -> output tends to its value row
    k2 = _rand((Hkv, nk, D), 7) * 1e-3
    k2[:, 4] = 0.0
    qpos = np.abs(q) + 1.0
    k2[:, 4] = 50.0
    out2, _ = oracle.attention(qpos, k2, v, scale=1.0)
    for h in range(Hq):
        np.testing.assert_allclose(out2[h], np.broadcast_to(v[h // 2, 4], (b, D)), atol=1e-9)


def test_attention_invariants():
    Hq, Hkv, b, nk, D = 4, 2, 5, 17, 8
    q, k, v = _rand((Hq, b, D), 8), _rand((Hkv, nk, D), 9), _rand((Hkv, nk, D), 10)
    out, lse, probs = oracle.attention(q, k, v, return_probs=True)
    np.testing.assert_allclose(probs.sum(-1), 1.0, atol=1e-14)
    perm = np.random.default_rng(0).permutation(nk)
    out_p, lse_p = oracle.attention(q, k[:, perm], v[:, perm])
    np.testing.assert_allclose(out_p, out, atol=1e-13)
    np.testing.assert_allclose(lse_p, lse, atol=1e-13)
    # adding a constant vector along q's orthogonal complement changes nothing; scaling scale by 0 -> mean of V
    out0, _ = oracle.attention(q, k, v, scale=0.0)
    for h in range(Hq):
        np.testing.assert_allclose(out0[h], np.broadcast_to(v[h // 2].mean(0), (b, D)), atol=1e-13)


# ------------------------------------------------------------------ saliency score (Algorithm 1, mean query and score)
def test_scores_linearity_two_evaluation_orders():
    Hq, Hkv, b, L, D, o = 6, 2, 4, 29, 16, 10
    q, k = _rand((Hq, b, D), 11), _rand((Hkv, L, D), 12)
    a1 = oracle.scores_logit_mean(q, k, o)
    a2 = oracle.scores_logit_mean(q, k, o, matrix_form=True)
    assert a1.shape == (Hkv, L - b)
    np.testing.assert_allclose(a1, a2, rtol=0, atol=1e-13)


def test_scores_candidate_map_and_planted_offset_closed_form():
    Hq, Hkv, b, L, D, o = 4, 2, 4, 21, 8, 9
    q = _rand((Hq, b, D), 13)
    G = Hq // Hkv
    qbar = q.reshape(Hkv, G * b, D).mean(1)
    u = qbar / np.linalg.norm(qbar, axis=1, keepdims=True)
    # keys = position * u  ->  score_c = scale * |qbar| * pos(c): reads back the candidate position map
    k = np.arange(L)[None, :, None] * u[:, None, :]
    a = oracle.scores_logit_mean(q, k, o)
    pos = np.concatenate([np.arange(o), np.arange(o + b, L)])
    for g in range(Hkv):
        np.testing.assert_allclose(a[g], pos * np.linalg.norm(qbar[g]) / np.sqrt(D), atol=1e-12)
    np.testing.assert_array_equal(oracle.candidate_positions(L, b, o), pos)
    # planting delta*u on one key raises exactly that score by scale*delta*|qbar|, nothing else moves
    k0 = _rand((Hkv, L, D), 14)
    a0 = oracle.scores_logit_mean(q, k0, o)
    k1 = k0.copy()
    k1[:, 15] += 3.0 * u          # position 15 is candidate 15 - b = 11
    a1 = oracle.scores_logit_mean(q, k1, o)
    diff = a1 - a0
    for g in range(Hkv):
        np.testing.assert_allclose(diff[g, 11], 3.0 * np.linalg.norm(qbar[g]) / np.sqrt(D), atol=1e-12)
    diff[:, 11] = 0
    np.testing.assert_allclose(diff, 0, atol=1e-13)
    # keys orthogonal to qbar score zero; block keys never appear among the candidates
    kz = _rand((Hkv, L, D), 15)
    kz -= (kz * u[:, None, :]).sum(-1, keepdims=True) * u[:, None, :]
    np.testing.assert_allclose(oracle.scores_logit_mean(q, kz, o), 0, atol=1e-13)
    k2 = k0.copy()
    k2[:, o:o + b] += 100.0
    np.testing.assert_array_equal(oracle.scores_logit_mean(q, k2, o), a0)


def test_scores_prob_mean_mass():
    Hq, Hkv, b, L, D, o = 4, 2, 3, 14, 8, 5
    q, k, v = _rand((Hq, b, D), 16), _rand((Hkv, L, D), 17), _rand((Hkv, L, D), 18)
    _, _, probs = oracle.attention(q, k, v, return_probs=True)
    a = oracle.scores_prob_mean(probs, Hkv, o)
    G = Hq // Hkv
    block_mass = probs[:, :, o:o + b].sum(-1).reshape(Hkv, G * b).mean(1)
    np.testing.assert_allclose(a.sum(1) + block_mass, 1.0, atol=1e-14)
    # identical keys -> every candidate gets 1/L
    kc = np.broadcast_to(k[:, :1], k.shape).copy()
    _, _, pu = oracle.attention(q, kc, v, return_probs=True)
    np.testing.assert_allclose(oracle.scores_prob_mean(pu, Hkv, o), 1.0 / L, atol=1e-15)


# ------------------------------------------------------------------ pooling (Algorithm 1, MaxPool1D)
@pytest.mark.parametrize("s", [1, 3, 5, 7, 9])
def test_pool_matches_library(s):
    a = _rand((3, 41), 20 + s)
    ref = F.max_pool1d(torch.from_numpy(a)[None], kernel_size=s, stride=1, padding=s // 2)[0].numpy()
    np.testing.assert_array_equal(oracle.pool(a, s), ref)
    ref_avg = F.avg_pool1d(torch.from_numpy(a)[None], kernel_size=s, stride=1, padding=s // 2)[0].numpy()
    np.testing.assert_allclose(oracle.pool(a, s, oracle.POOL_AVG), ref_avg, atol=1e-14)
    # per-region pooling == pooling each region on its own
    seam = 17
    got = oracle.pool(a, s, seam=seam)
    for lo, hi in ((0, seam), (seam, 41)):
        part = F.max_pool1d(torch.from_numpy(a[:, lo:hi].copy())[None], s, 1, s // 2)[0].numpy()
        np.testing.assert_array_equal(got[:, lo:hi], part)


def test_pool_invariants():
    a = _rand((2, 50), 30)
    np.testing.assert_array_equal(oracle.pool(a, 1), a)
    for s in (3, 7):
        w = s // 2
        I = oracle.pool(a, s)
        assert (I >= a).all()
        t = 0.3                                   # superlevel set of I = dilation of the superlevel set of a
        hot = a >= t
        dil = np.zeros_like(hot)
        for sh in range(-w, w + 1):
            src = slice(max(0, -sh), 50 - max(0, sh)); dst = slice(max(0, sh), 50 - max(0, -sh))
            dil[:, dst] |= hot[:, src]
        np.testing.assert_array_equal(I >= t, dil)
    with pytest.raises(ValueError):
        oracle.pool(a, 4)


# ------------------------------------------------------------------ counts (Algorithm 1, n = floor(|I| r); Section 3.3.1, k = (L-b) x r)
def test_keep_counts_golden():
    rows = [l.split("#")[0].split() for l in open(os.path.join(GOLD, "keep_counts.txt")) if l.split("#")[0].strip()]
    assert len(rows) >= 8
    for L, b, o, r, mode, n_total, n_pre, n_suf in rows:
        got = oracle.keep_count(int(L), int(b), int(o), float(r), int(mode))
        assert got == (int(n_total), int(n_pre), int(n_suf)), (L, b, o, r, mode, got)


def test_keep_count_edges():
    assert oracle.keep_count(256, 32, 128, 1.0)[0] == 224
    assert oracle.keep_count(256, 32, 128, 0.0)[0] == 0
    assert oracle.keep_count(256, 32, 0, 0.5, oracle.SELECT_PER_REGION_CEIL) == (112, 0, 112)
    assert oracle.keep_count(256, 32, 224, 0.5, oracle.SELECT_PREFIX_ONLY) == (112, 112, 0)
    assert oracle.keep_count(41, 8, 10, 0.3, oracle.SELECT_PER_REGION_CEIL) == (10, 3, 7)
    with pytest.raises(ValueError):
        oracle.keep_count(256, 32, 230, 0.5)
    with pytest.raises(ValueError):
        oracle.keep_count(256, 32, 10, 1.5)


# ------------------------------------------------------------------ selection (Algorithm 1, TopKIndices)
def test_select_matches_library_stable_sort_and_tie_rule():
    rng = np.random.default_rng(40)
    for C, n in [(1, 0), (1, 1), (7, 3), (64, 64), (257, 100), (1000, 1)]:
        x = rng.standard_normal(C)
        ref = np.sort(np.argsort(-x, kind="stable")[:n])
        np.testing.assert_array_equal(oracle.select_topk(x, n), ref)
    # heavy ties: plateaus as max pooling makes them
    x = np.repeat(rng.integers(0, 4, size=40), 3).astype(np.float64)
    for n in (0, 1, 17, 59, 120):
        got = oracle.select_topk(x, n)
        ref = np.sort(np.argsort(-x, kind="stable")[:n])
        np.testing.assert_array_equal(got, ref)
        assert (np.diff(got) > 0).all()
        if 0 < n < x.size:
            evicted = np.setdiff1d(np.arange(x.size), got)
            thr = x[got].min()
            assert thr >= x[evicted].max()
            # among entries equal to the threshold, every kept one precedes every evicted one
            kept_eq, ev_eq = got[x[got] == thr], evicted[x[evicted] == thr]
            if kept_eq.size and ev_eq.size:
                assert kept_eq.max() < ev_eq.min()
    # all equal -> the first n
    np.testing.assert_array_equal(oracle.select_topk(np.zeros(9), 4), np.arange(4))


def test_select_monotone_in_retention():
    x = oracle.pool(_rand((1, 300), 41), 3)[0]
    prev = set()
    for n in (0, 30, 75, 150, 299, 300):
        cur = set(oracle.select_topk(x, n).tolist())
        assert prev <= cur and len(cur) == n
        prev = cur


# ------------------------------------------------------------------ gather (Algorithm 1, Select)
def test_gather_is_fancy_indexing_bit_exact():
    rng = np.random.default_rng(50)
    src32 = rng.standard_normal((3, 37, 8)).astype(np.float32)
    src16 = W.f32_to_bf16_bits(src32).reshape(src32.shape)
    idx = np.sort(rng.choice(37, size=(3, 11)), axis=1).astype(np.int32)
    for src in (src32, src16):
        got = oracle.gather_rows(src, idx)
        ref = np.stack([src[g, idx[g]] for g in range(3)])
        assert got.dtype == src.dtype and got.tobytes() == ref.tobytes()
    with pytest.raises(ValueError):
        oracle.gather_rows(src32, np.full((3, 2), 37, np.int32))


# ------------------------------------------------------------------ schedule (Algorithms 2 and 4)
def test_cache_state_schedule():
    assert [oracle.cache_state(i) for i in range(6)] == [0, 1, 2, 2, 2, 2]
    assert [oracle.cache_state(i, 0) for i in range(4)] == [1, 2, 2, 2]
    assert [oracle.cache_state(i, 3) for i in range(6)] == [0, 0, 0, 1, 2, 2]


# ------------------------------------------------------------------ Algorithm 1 + 3 chained
def test_refresh_keeps_planted_keys_sink_and_neighbours():
    cfg = W.CONFIGS["c1_tiny"]
    s = W.make_sequence(cfg, seed=0)
    q, k, v = s.refresh_inputs(1)
    r = oracle.refresh(q, k, v, s.block_off, cfg.retention, cfg.pool_window)
    assert r.n_keep == 112 and r.kept_idx.shape == (2, 112)
    L, b, o, w = cfg.seq_len, cfg.block_len, s.block_off, cfg.pool_window // 2
    cand_of = {int(p): c for c, p in enumerate(oracle.candidate_positions(L, b, o))}
    for g in range(cfg.n_kv_heads):
        kept = set(r.kept_idx[g].tolist())
        assert all(o > p or p >= o + b for p in kept) and max(kept) < L
        assert (np.diff(r.kept_idx[g]) > 0).all()
        must = [0] + s.planted_pos[g].tolist()
        for p in must:                          # a +3u / +6u key sits ~24 sigma above the background
            c = cand_of[p]
            for cc in range(max(0, c - w), min(L - b, c + w + 1)):
                assert int(oracle.candidate_positions(L, b, o)[cc]) in kept


def test_full_retention_reproduces_dense_attention():
    cfg = W.CONFIGS["c1_tiny"]
    s = W.make_sequence(cfg, seed=3)
    q, k, v = s.refresh_inputs(1)
    o, b = s.block_off, cfg.block_len
    r = oracle.refresh(q, k, v, o, 1.0, cfg.pool_window)
    assert r.n_keep == cfg.seq_len - b
    np.testing.assert_array_equal(r.kept_idx[0], oracle.candidate_positions(cfg.seq_len, b, o))
    k_c, v_c = oracle.gather_rows(k, r.kept_idx), oracle.gather_rows(v, r.kept_idx)
    out, lse = oracle.sparse_block_attention(q, k_c, v_c, k[:, o:o + b], v[:, o:o + b])
    np.testing.assert_allclose(out, r.out, atol=1e-13)
    np.testing.assert_allclose(lse, r.lse, atol=1e-13)


def test_dense_step_brute_force_closed_form_and_row_sampling():
    """The dense step (all L rows over all L keys, Algorithm 3) against loops written out, a closed form and the
    block rows of the refresh step."""
    rng = np.random.default_rng(11)
    Hq, Hkv, L, D = 4, 2, 7, 3
    q, k, v = rng.standard_normal((Hq, L, D)), rng.standard_normal((Hkv, L, D)), rng.standard_normal((Hkv, L, D))
    out, lse = oracle.dense_attention(q, k, v, scale=0.7)
    for h in range(Hq):
        g = h // (Hq // Hkv)                       # query heads of a group share one KV head
        for t in range(L):
            w = [np.exp(0.7 * sum(q[h, t, d] * k[g, u, d] for d in range(D))) for u in range(L)]
            z = sum(w)
            for d in range(D):
                assert abs(out[h, t, d] - sum(w[u] * v[g, u, d] for u in range(L)) / z) < 1e-12
            assert abs(lse[h, t] - np.log(z)) < 1e-12
    # no mask of any kind: with zero queries every row is the plain mean of V over the whole sequence
    out0, lse0 = oracle.dense_attention(np.zeros_like(q), k, v)
    np.testing.assert_allclose(out0, np.repeat(v.mean(axis=1), Hq // Hkv, axis=0)[:, None, :].repeat(L, axis=1), atol=1e-13)
    np.testing.assert_allclose(lse0, np.log(L), atol=1e-13)
    # a sample of rows gives those rows; the block's rows are what the refresh step computes for the block
    cfg = W.CONFIGS["c1_tiny"]
    s = W.make_sequence(cfg, seed=5)
    qf, kf, vf = s.dense_inputs(1)
    full, _ = oracle.dense_attention(qf, kf, vf)
    some, _ = oracle.dense_attention(qf, kf, vf, rows=[0, 5, cfg.seq_len - 1])
    np.testing.assert_array_equal(some, full[:, [0, 5, cfg.seq_len - 1]])
    qb, kb, vb = s.refresh_inputs(1)
    blk, _ = oracle.attention(qb, kb, vb)
    np.testing.assert_allclose(full[:, s.block_off:s.block_off + cfg.block_len], blk, atol=1e-13)


def test_sparse_attention_equals_dense_over_kept_subset():
    cfg = W.CONFIGS["c1_tiny"]
    s = W.make_sequence(cfg, seed=5)
    q, k, v = s.refresh_inputs(1)
    o, b = s.block_off, cfg.block_len
    r = oracle.refresh(q, k, v, o, 0.5, 3)
    q2, kn, vn = s.sparse_inputs(2)
    out, _ = oracle.sparse_block_attention(q2, oracle.gather_rows(k, r.kept_idx), oracle.gather_rows(v, r.kept_idx), kn, vn)
    # same thing through the library SDPA with a boolean key mask over the full sequence
    kf, vf = k.copy(), v.copy()
    kf[:, o:o + b], vf[:, o:o + b] = kn, vn
    for g in range(cfg.n_kv_heads):
        mask = np.zeros(cfg.seq_len, bool)
        mask[r.kept_idx[g]] = True
        mask[o:o + b] = True
        ref = F.scaled_dot_product_attention(torch.from_numpy(q2[g].astype(np.float64))[None],
                                             torch.from_numpy(kf[g].astype(np.float64))[None],
                                             torch.from_numpy(vf[g].astype(np.float64))[None],
                                             attn_mask=torch.from_numpy(mask)[None, None, :])[0].numpy()
        np.testing.assert_allclose(out[g], ref, atol=1e-12)


def test_refresh_policies_and_variants():
    rng = np.random.default_rng(60)
    Hq, Hkv, b, L, D, o = 4, 2, 8, 61, 16, 24
    q, k, v = rng.standard_normal((Hq, b, D)), rng.standard_normal((Hkv, L, D)), rng.standard_normal((Hkv, L, D))
    rj = oracle.refresh(q, k, v, o, 0.3, 3)
    rp = oracle.refresh(q, k, v, o, 0.3, 3, select=oracle.SELECT_PER_REGION_CEIL)
    rx = oracle.refresh(q, k, v, o, 0.3, 3, select=oracle.SELECT_PREFIX_ONLY)
    assert rj.n_keep == int(np.floor(53 * 0.3))
    n_pre, n_suf = int(np.ceil(24 * 0.3)), int(np.ceil(29 * 0.3))
    for g in range(Hkv):
        assert (rp.kept_idx[g] < o).sum() == n_pre and (rp.kept_idx[g] >= o + b).sum() == n_suf
        assert (rx.kept_idx[g] < o).sum() == int(np.floor(24 * 0.3))
        np.testing.assert_array_equal(rx.kept_idx[g][rx.kept_idx[g] >= o + b], np.arange(o + b, L))
    # the dense output does not depend on the eviction policy
    np.testing.assert_array_equal(rj.out, rp.out)
    # probability-mean scores: positive, bounded by 1, and the kept set is still valid
    rq = oracle.refresh(q, k, v, o, 0.3, 3, score=oracle.SCORE_PROB_MEAN)
    assert (rq.scores > 0).all() and (rq.scores < 1).all() and rq.kept_idx.shape == rj.kept_idx.shape


def _kept_by_library_routines(a, o, n_pre, n_suf, window, kind, per_region, joint_n=None):
    """The kept candidate set of one head rebuilt from library pieces only: torch max/avg pooling per region (or over the
    whole candidate axis) and a stable numpy sort by (score descending, index ascending)."""
    def pooled_of(x):
        t = torch.from_numpy(np.asarray(x, np.float64))[None, None]
        if kind == oracle.POOL_MAX:
            return F.max_pool1d(t, window, 1, window // 2)[0, 0].numpy()
        return F.avg_pool1d(t, window, 1, window // 2, count_include_pad=True)[0, 0].numpy()

    def top(x, n):
        order = np.argsort(-x, kind="stable")          # equal scores keep their index order: the lower index wins
        return np.sort(order[:n])
    if not per_region:
        return top(pooled_of(a), joint_n)
    pre = top(pooled_of(a[:o]), n_pre) if o > 0 else np.zeros(0, np.int64)
    if n_suf is None:                                  # prefix-sparse: the whole suffix stays
        suf = np.arange(len(a) - o)
    else:
        suf = top(pooled_of(a[o:]), n_suf) if len(a) > o else np.zeros(0, np.int64)
    return np.concatenate([pre, suf + o])


@pytest.mark.parametrize("kind", [oracle.POOL_MAX, oracle.POOL_AVG])
@pytest.mark.parametrize("window", [3, 5])
def test_refresh_variant_branches_against_library_routines(kind, window):
    """Per-region ceil, prefix-only (Algorithm 5) and the AvgPool ablation through refresh(): the kept sets must equal
    what torch's pooling and a stable sort give region by region. The inputs put a dominant score on the LAST prefix key
    and on the FIRST suffix key, so pooling across the seam, or a quota taken jointly, changes the kept sets."""
    rng = np.random.default_rng(61)
    Hq, Hkv, b, L, D, o = 4, 2, 8, 77, 16, 30
    q = rng.standard_normal((Hq, b, D))
    k, v = rng.standard_normal((Hkv, L, D)), rng.standard_normal((Hkv, L, D))
    G = Hq // Hkv
    for g in range(Hkv):
        u = q[g * G:(g + 1) * G].mean(axis=(0, 1))
        u /= np.linalg.norm(u)
        k[g, o - 1] += (9.0 if g == 0 else 0.0) * u      # head 0: the last prefix key dominates
        k[g, o + b] += (0.0 if g == 0 else 9.0) * u      # head 1: the first suffix key dominates
    r = 0.3
    C = L - b
    pos = oracle.candidate_positions(L, b, o)
    for select in (oracle.SELECT_JOINT_FLOOR, oracle.SELECT_PER_REGION_CEIL, oracle.SELECT_PREFIX_ONLY):
        res = oracle.refresh(q, k, v, o, r, window, pool_kind=kind, select=select)
        a = oracle.scores_logit_mean(q, k, o)            # pinned on its own by the linearity and planted-key tests
        per_region = select != oracle.SELECT_JOINT_FLOOR
        if select == oracle.SELECT_JOINT_FLOOR:
            n_pre = n_suf = None
            joint_n = int(np.floor(C * r))
        elif select == oracle.SELECT_PER_REGION_CEIL:
            n_pre, n_suf, joint_n = int(np.ceil(o * r)), int(np.ceil((C - o) * r)), None
        else:
            n_pre, n_suf, joint_n = int(np.floor(o * r)), None, None
        for g in range(Hkv):
            want = pos[_kept_by_library_routines(a[g], o, n_pre, n_suf, window, kind, per_region, joint_n)]
            np.testing.assert_array_equal(res.kept_idx[g], want)
    # the planted inputs bite: with max pooling the joint reading keeps the neighbour across the seam, the per-region one
    # does not reach over it
    joint = oracle.refresh(q, k, v, o, r, window, pool_kind=oracle.POOL_MAX, select=oracle.SELECT_JOINT_FLOOR)
    region = oracle.refresh(q, k, v, o, r, window, pool_kind=oracle.POOL_MAX, select=oracle.SELECT_PER_REGION_CEIL)
    assert o + b in joint.kept_idx[0] and o - 1 in joint.kept_idx[1]
    assert joint.pooled[0][o] == joint.pooled[0][o - 1] and region.pooled[0][o] < region.pooled[0][o - 1]
    assert not np.array_equal(joint.kept_idx[0], region.kept_idx[0]) or not np.array_equal(joint.kept_idx[1], region.kept_idx[1])


def test_refresh_probability_scores_against_library_softmax():
    """SCORE_PROB_MEAN through refresh(): the scores are the column means of torch.softmax over ALL keys (block included)
    taken over the group's block queries, and on the tiny config the sink and every planted key are kept."""
    cfg = W.CONFIGS["c1_tiny"]
    s = W.make_sequence(cfg, seed=0)
    q, k, v = s.refresh_inputs(1)
    o, b, L = s.block_off, cfg.block_len, cfg.seq_len
    res = oracle.refresh(q, k, v, o, cfg.retention, cfg.pool_window, score=oracle.SCORE_PROB_MEAN)
    G = cfg.n_q_heads // cfg.n_kv_heads
    scale = 1.0 / np.sqrt(cfg.head_dim)
    pos = oracle.candidate_positions(L, b, o)
    for g in range(cfg.n_kv_heads):
        logits = torch.from_numpy(q[g * G:(g + 1) * G].astype(np.float64)) @ torch.from_numpy(k[g].astype(np.float64)).T * scale
        probs = torch.softmax(logits, dim=-1).reshape(-1, L).mean(dim=0).numpy()
        np.testing.assert_allclose(res.scores[g], probs[pos], rtol=1e-12, atol=1e-15)
        kept = set(res.kept_idx[g].tolist())
        assert 0 in kept                                               # the sink
        assert set(int(x) for x in s.planted_pos[g]) <= kept           # the planted salient keys
    # and the selection on top of those scores is the library one
    a = res.scores
    for g in range(cfg.n_kv_heads):
        want = pos[_kept_by_library_routines(a[g], o, None, None, cfg.pool_window, oracle.POOL_MAX, False, res.n_keep)]
        np.testing.assert_array_equal(res.kept_idx[g], want)


# ------------------------------------------------------------------ generator sanity (shapes, rounding, determinism)
def test_workload_generator_is_deterministic_and_rounded():
    cfg = W.CONFIGS["c3_dream"]
    small = W.WorkloadConfig("t", "bf16", 14, 2, 128, 200, 64, retention=0.25, salient_frac=0.01, sink_tokens=4)
    s1, s2 = W.make_sequence(small, seed=7, layer=2, block=1), W.make_sequence(small, seed=7, layer=2, block=1)
    a, b_ = s1.refresh_inputs(1), s2.refresh_inputs(1)
    for x, y in zip(a, b_):
        assert x.tobytes() == y.tobytes()
        np.testing.assert_array_equal(W.bf16_bits_to_f32(W.f32_to_bf16_bits(x)).reshape(x.shape), x)
    assert s1.block_off == 200 + 32 and a[1].shape == (2, 264, 128) and a[0].shape == (14, 32, 128)
    q2, kn, vn = s1.sparse_inputs(2)
    assert kn.shape == (2, 32, 128) and not np.array_equal(q2, a[0])
    assert cfg.group == 7 and cfg.seq_len == 4096
    # bf16 rounding helper against torch's own conversion
    x = np.random.default_rng(1).standard_normal(1000).astype(np.float32)
    ref = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    np.testing.assert_array_equal(W.f32_to_bf16_bits(x), ref)
    bw = W.make_batch(W.CONFIGS["c5_serving"].__class__("t5", "bf16", 4, 4, 128, 64, 64), [40, 100, 64], seed=1)
    qb, kb, vb = bw.refresh_inputs()
    assert kb.shape == (3, 4, 164, 128) and list(bw.seq_len) == [104, 164, 128] and list(bw.block_off) == [40, 100, 64]
    assert np.all(kb[0, :, 104:] == 0)

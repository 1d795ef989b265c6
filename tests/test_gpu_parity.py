"""GPU parity: the CUDA path (through the C ABI) against the CPU oracle, element by element, on the same
seeded inputs. Tolerances: kept sets bit-exact outside a 1e-3 band around the threshold; compacted K/V
bit-exact; fp32 outputs within 1e-5 abs; bf16 outputs within 1e-2 + 1e-2*|ref|."""
import dataclasses

import numpy as np
import pytest
import torch

import oracle
from paper_2508_02558_b200 import binding as B
from paper_2508_02558_b200 import build as libbuild
from paper_2508_02558_b200 import workloads as W

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    libbuild.build()


def _run_sequence_case(cfg: W.WorkloadConfig, seed: int, block: int, n_sparse: int = 2, heads=None, **policy):
    import parity_util as U
    s = W.make_sequence(cfg, seed=seed, block=block)
    q, k, v = s.refresh_inputs(1)
    L, o = s.seq_len, s.block_off
    sel = policy.get("select", oracle.SELECT_JOINT_FLOOR)
    pk = policy.get("pool", oracle.POOL_MAX)
    sk = policy.get("score", oracle.SCORE_LOGIT_MEAN)
    g = U.gpu_refresh(q[None], k[None], v[None], [L], [o], cfg.dtype, cfg.retention, cfg.pool_window, **policy)
    stats = U.check_refresh_against_oracle(g, q[None], k[None], v[None], [L], [o], cfg.dtype, cfg.retention,
                                           cfg.pool_window, heads=heads, select=sel, pool_kind=pk, score=sk)
    U.check_compaction_bit_exact(g, g.k_dev, g.v_dev)
    for step in range(2, 2 + n_sparse):
        q2, kn, vn = s.sparse_inputs(step)
        out = U.gpu_sparse_step(g, q2[None], kn[None], vn[None], cfg.dtype)
        U.check_sparse_against_oracle(g, out, q2[None], kn[None], vn[None], cfg.dtype, heads=heads)
    return stats


def _small(name, dtype, Hq, Hkv, D, p, gen, **kw):
    return W.WorkloadConfig(name, dtype, Hq, Hkv, D, p, gen, **kw)


def test_c1_tiny_fp32_refresh_and_three_sparse_steps():
    stats = _run_sequence_case(W.CONFIGS["c1_tiny"], seed=0, block=0, n_sparse=3)
    assert stats["set_mismatch"] == 0


@pytest.mark.parametrize("cfg,block", [
    (_small("mha_ragged", "bf16", 4, 4, 128, 203, 130, salient_frac=0.02), 1),        # L=333: several tiles + ragged tail
    (_small("gqa7", "bf16", 14, 2, 128, 300, 96, retention=0.25, salient_frac=0.01, sink_tokens=4), 2),
    (_small("gqa4", "bf16", 8, 2, 128, 517, 64, retention=0.3, salient_frac=0.01), 0),
    (_small("d64", "bf16", 4, 2, 64, 150, 64, salient_frac=0.02), 1),
    (_small("f32_d128_gqa", "f32", 6, 2, 128, 131, 64, salient_frac=0.02), 0),
    (_small("f32_d64", "f32", 3, 3, 64, 90, 96, retention=0.7, salient_frac=0.02), 2),
    (_small("blk16", "bf16", 4, 4, 128, 100, 64, block_len=16, salient_frac=0.02), 3),
    (_small("blk64", "bf16", 2, 2, 128, 100, 128, block_len=64, salient_frac=0.02), 1),
])
def test_small_cases_span_tiles_heads_and_dtypes(cfg, block):
    _run_sequence_case(cfg, seed=11, block=block)


@pytest.mark.parametrize("cfg,block", [
    (_small("kt_gqa2", "bf16", 8, 4, 128, 517, 64, retention=0.3, salient_frac=0.01), 0),       # 64 query columns: two softmax warpgroups per tile
    (_small("kt_gqa3", "bf16", 6, 2, 128, 333, 96, retention=0.5, salient_frac=0.02), 1),       # 96: three
    (_small("kt_gqa4", "bf16", 8, 2, 128, 700, 64, retention=0.4, salient_frac=0.01), 1),       # 128: four
    (_small("kt_gqa2_d64", "bf16", 4, 2, 64, 150, 64, salient_frac=0.02), 1),
    (_small("kt_gqa4_blk16", "bf16", 16, 4, 128, 212, 32, block_len=16, salient_frac=0.02), 1), # 64 columns from four heads of 16 rows
])
@pytest.mark.parametrize("plan", [dict(kernel=3), dict(kernel=3, splits=1), dict(kernel=3, splits=8)])
def test_key_row_kernel_on_grouped_heads(cfg, block, plan, tuning):
    """Up to 128 query columns per KV head on the kernel with the keys on the accumulator rows (the planner picks it
    for such heads only when there are enough (sequence, KV head) units; here it is forced)."""
    tuning(**plan)
    _run_sequence_case(cfg, seed=21, block=block, n_sparse=2)


@pytest.mark.parametrize("p,gen,block", [(0, 96, 0), (160, 32, 0), (64, 64, 1)])
def test_block_at_sequence_edges(p, gen, block):
    """Empty prefix (block first), empty suffix (block last)."""
    if p == 0:
        cfg = _small("edge0", "bf16", 4, 4, 128, 32, 64, salient_frac=0.02)
        s = W.make_sequence(cfg, seed=2, block=0)
        # move the block to position 0 by treating the first 32 tokens as the block
        import parity_util as U
        q, k, v = s.refresh_inputs(1)
        L = s.seq_len
        g = U.gpu_refresh(q[None], k[None], v[None], [L], [0], "bf16", 0.5, 3)
        U.check_refresh_against_oracle(g, q[None], k[None], v[None], [L], [0], "bf16", 0.5, 3)
        U.check_compaction_bit_exact(g, g.k_dev, g.v_dev)
    else:
        _run_sequence_case(_small("edge", "bf16", 4, 4, 128, p, gen, salient_frac=0.02), seed=3, block=block)


@pytest.mark.parametrize("r", [0.0, 1.0, 0.1])
def test_retention_extremes(r):
    import parity_util as U
    cfg = _small("rext", "f32", 2, 2, 64, 96, 64, retention=r, salient_frac=0.02)
    _run_sequence_case(cfg, seed=4, block=0)
    if r == 1.0:
        # keeping everything and replaying the same Q/K/V must reproduce the dense refresh output
        s = W.make_sequence(cfg, seed=4, block=0)
        q, k, v = s.refresh_inputs(1)
        o, b = s.block_off, cfg.block_len
        g = U.gpu_refresh(q[None], k[None], v[None], [s.seq_len], [o], "f32", 1.0, 3)
        out = U.gpu_sparse_step(g, q[None], k[None, :, o:o + b], v[None, :, o:o + b], "f32")
        np.testing.assert_allclose(out, g.out, rtol=0, atol=1e-5)


@pytest.mark.parametrize("r", [0.0, 1.0, 0.03])
def test_retention_extremes_bf16(r):
    """Nothing kept (the reuse step attends over the block alone), everything kept, and a handful kept, on the tcgen05 path."""
    cfg = _small("rext16", "bf16", 4, 2, 128, 230, 96, retention=r, salient_frac=0.02)
    stats = _run_sequence_case(cfg, seed=16, block=1)
    assert stats["set_mismatch"] == 0 or r not in (0.0, 1.0)


@pytest.mark.parametrize("cfg,block", [
    (_small("gqa8_two_full_row_tiles", "bf16", 16, 2, 128, 200, 64, retention=0.4, salient_frac=0.02), 1),   # b*G = 256
    (_small("blk128", "bf16", 2, 2, 128, 150, 256, block_len=128, salient_frac=0.02), 1),                    # b = 128
    (_small("blk48_fallback", "bf16", 2, 2, 128, 150, 96, block_len=48, salient_frac=0.02), 1),              # not a multiple of 16
    (_small("gqa2_two_replicas", "bf16", 4, 2, 128, 333, 64, salient_frac=0.02), 0),                         # b*G = 64
    (_small("one_tile", "bf16", 4, 4, 128, 40, 64, salient_frac=0.05), 0),                                   # shorter than one key tile
])
def test_more_shapes(cfg, block):
    _run_sequence_case(cfg, seed=17, block=block)


def test_batch_with_an_empty_cache_and_a_full_one():
    """Ragged batch in which one sequence is nothing but its block (no candidates at all) beside ordinary ones."""
    import parity_util as U
    cfg = _small("rag0", "bf16", 4, 4, 128, 64, 32, salient_frac=0.02)
    bw = W.make_batch(cfg, [0, 300, 37], seed=18, block=0)
    q, k, v = bw.refresh_inputs(1, pad_value=np.nan)
    g = U.gpu_refresh(q, k, v, bw.seq_len, bw.block_off, "bf16", 0.5, 3)
    k0, v0 = np.nan_to_num(k), np.nan_to_num(v)
    U.check_refresh_against_oracle(g, q, k0, v0, bw.seq_len, bw.block_off, "bf16", 0.5, 3)
    assert int(g.kept_cnt[0]) == 0
    q2, kn, vn = bw.sparse_inputs(2)
    out = U.gpu_sparse_step(g, q2, kn, vn, "bf16")
    U.check_sparse_against_oracle(g, out, q2, kn, vn, "bf16")


@pytest.mark.parametrize("policy", [
    dict(select=B.SELECT_PER_REGION_CEIL), dict(select=B.SELECT_PREFIX_ONLY), dict(pool=B.POOL_AVG),
])
def test_policies(policy, tuning):
    cfg = _small("pol", "bf16", 4, 2, 128, 190, 96, retention=0.3, salient_frac=0.02)
    _run_sequence_case(cfg, seed=5, block=1, **policy)
    tuning(select=2)                                     # two regions, each split over the CTAs of a cluster
    _run_sequence_case(cfg, seed=5, block=1, **policy)
    tuning(select=0, kernel=2)                           # the attention kernel with the queries on the accumulator rows
    _run_sequence_case(cfg, seed=5, block=1, **policy)


@pytest.mark.parametrize("window", [1, 5, 7, 9])
def test_pool_windows(window):
    cfg = _small("win", "f32", 2, 2, 64, 120, 64, pool_window=window, salient_frac=0.03)
    stats = _run_sequence_case(cfg, seed=6, block=0, n_sparse=1)
    assert stats["set_mismatch"] == 0


@pytest.mark.parametrize("plan", [
    dict(kernel=1),                                      # cp.async + mma.sync kernels, separate merge launch
    dict(kernel=1, splits=3),
    dict(pdl=0),                                         # no programmatic dependent launch
    # the tcgen05 kernel with the keys on the accumulator rows, forced also for the grouped heads (few units: the planner
    # would give those to the query-row kernel), where one softmax warpgroup per 32 query columns shares every tile
    dict(kernel=3),
    dict(kernel=3, splits=7), dict(kernel=3, splits=1), dict(kernel=3, splits=3),      # key-split counts (cluster sizes)
    dict(kernel=3, splits=2, stages=3), dict(kernel=3, splits=1, stages=2),            # ... and ring depths
    dict(kernel=3, dual=0), dict(kernel=3, dual=0, splits=1), dict(kernel=3, dual=0, splits=3, stages=1),   # two softmax warpgroups / one
    dict(kernel=3, dual=1, splits=1, stages=1),
    dict(kernel=3, early_loads=0),                       # no loads ahead of the grid dependency
    dict(kernel=3, pdl=0),
    dict(kernel=3, splits=1, persist=1), dict(kernel=3, splits=1, persist=2),   # streaming variant (where one column group suffices)
    dict(kernel=2),                                      # the tcgen05 kernel with the queries on the accumulator rows
    dict(kernel=2, splits=7), dict(kernel=2, splits=1),
    dict(kernel=2, splits=5, fused_tail=0),              # split merge and pooling in the second launch
    dict(kernel=2, early_loads=0),
    dict(kernel=2, cluster=0, splits=4),                 # key splits merged by the last CTA instead of a cluster
    dict(kernel=2, cluster=2, splits=4),                 # ... and by a cluster of four
    dict(kernel=2, cluster=2), dict(kernel=2, cluster=2, splits=7),
    dict(kernel=2, dual=1, splits=1),                    # small-footprint variant (two CTAs per SM)
    dict(kernel=2, dual=1, splits=3),
    dict(kernel=2, key_tile=64, splits=2),               # 64-key tiles
    dict(select=2),                                      # top-k by a cluster of CTAs per head
])
def test_alternative_launch_plans_agree_with_oracle(plan, tuning):
    """Every kernel family, tail placement, tile size and split count gives the same answers."""
    tuning(**plan)
    _run_sequence_case(_small("alt_mha", "bf16", 4, 4, 128, 403, 130, salient_frac=0.02), seed=12, block=1)
    _run_sequence_case(_small("alt_gqa", "bf16", 8, 2, 128, 300, 64, retention=0.3, salient_frac=0.02), seed=13, block=0)
    _run_sequence_case(_small("alt_gqa7", "bf16", 14, 2, 128, 260, 96, retention=0.4, salient_frac=0.02), seed=14, block=1)


@pytest.mark.parametrize("cfg,block", [
    (_small("prob_mha", "bf16", 4, 4, 128, 403, 130, salient_frac=0.02), 1),            # replicated rows, ragged tail
    (_small("prob_gqa4", "bf16", 8, 2, 128, 517, 64, retention=0.3, salient_frac=0.01), 0),   # one full 128-row tile
    (_small("prob_gqa7", "bf16", 14, 2, 128, 300, 96, retention=0.25, salient_frac=0.01, sink_tokens=4), 2),   # two row tiles
    (_small("prob_d64", "bf16", 4, 2, 64, 150, 64, salient_frac=0.02), 1),
])
@pytest.mark.parametrize("plan", [{}, dict(splits=3, fused_tail=0), dict(splits=1), dict(dual=1)])
def test_softmax_probability_saliency(cfg, block, plan, tuning):
    """The second reading of "attention scores": mean softmax probability per key (two passes over K)."""
    tuning(**plan)
    _run_sequence_case(cfg, seed=15, block=block, n_sparse=1, score=B.SCORE_PROB_MEAN)


@pytest.mark.parametrize("plan", [{}, dict(splits=3), dict(lpt=1), dict(lpt=1, dual=0, splits=1), dict(dual=0, splits=1), dict(dual=0, splits=2), dict(kernel=2), dict(kernel=2, lpt=1), dict(kernel=2, lpt=1, dual=1, splits=1),
                                  dict(select=2),
                                  # streaming variant of the key-row kernel: 16 units on one CTA each, on 3 CTAs (five or six
                                  # units per CTA, in the order of the lengths) and on a single one, also in batch order
                                  dict(splits=1, persist=1), dict(splits=1, persist=3), dict(splits=1, persist=3, lpt=0), dict(splits=1, persist=2)])
def test_ragged_batch(plan, tuning):
    import parity_util as U
    tuning(**plan)
    cfg = _small("rag", "bf16", 4, 4, 128, 64, 64, salient_frac=0.02)
    bw = W.make_batch(cfg, [40, 333, 64, 200], seed=7, block=1)
    q, k, v = bw.refresh_inputs(1, pad_value=np.nan)       # padding must never be read
    g = U.gpu_refresh(q, k, v, bw.seq_len, bw.block_off, "bf16", 0.5, 3)
    k0, v0 = np.nan_to_num(k), np.nan_to_num(v)
    U.check_refresh_against_oracle(g, q, k0, v0, bw.seq_len, bw.block_off, "bf16", 0.5, 3)
    U.check_compaction_bit_exact(g, g.k_dev, g.v_dev)
    q2, kn, vn = bw.sparse_inputs(2)
    out = U.gpu_sparse_step(g, q2, kn, vn, "bf16")
    U.check_sparse_against_oracle(g, out, q2, kn, vn, "bf16")


@pytest.mark.parametrize("plan", [dict(lpt=1), dict(lpt=1, early_loads=0), dict(lpt=0)])
def test_ragged_batch_with_equal_lengths_in_length_order(plan, tuning):
    """Sequences taken from the longest to the shortest: equal lengths must still map grid slots to sequences one to one."""
    import parity_util as U
    tuning(**plan)
    cfg = _small("rag", "bf16", 4, 4, 128, 64, 64, salient_frac=0.02)
    bw = W.make_batch(cfg, [200, 64, 200, 64, 333], seed=9, block=1)
    q, k, v = bw.refresh_inputs(1, pad_value=np.nan)
    g = U.gpu_refresh(q, k, v, bw.seq_len, bw.block_off, "bf16", 0.5, 3)
    k0, v0 = np.nan_to_num(k), np.nan_to_num(v)
    U.check_refresh_against_oracle(g, q, k0, v0, bw.seq_len, bw.block_off, "bf16", 0.5, 3)
    U.check_compaction_bit_exact(g, g.k_dev, g.v_dev)


@pytest.mark.parametrize("kernel", ["default", "cluster", "single"])
def test_select_topk_alone_heavy_ties_bit_exact(kernel, tuning):
    """Plateaus of exactly equal scores (what max pooling produces) must resolve to the lowest positions. The selection
    by one CTA per head and the one by a cluster of CTAs per head (long sequences) must both be exact."""
    tuning(select={"default": 0, "single": 1, "cluster": 2}[kernel])
    rng = np.random.default_rng(8)
    for (Bn, Hkv, L, b, o, r) in [(2, 3, 300, 32, 100, 0.5), (1, 2, 2080, 32, 2048, 0.37), (1, 1, 40000, 32, 7, 0.25), (1, 1, 50000, 32, 49000, 0.6),
                                  (1, 2, 64, 32, 0, 0.5), (1, 2, 64, 32, 32, 0.99)]:
        sc = np.round(rng.standard_normal((Bn, Hkv, L)) * 2).astype(np.float32) / 2     # few distinct values
        sc[:, :, 5::17] = -np.inf
        sc[:, :, 3::29] = 0.0
        sc[:, :, 4::29] = -0.0
        d = B.make_desc(batch=Bn, n_q_heads=Hkv, n_kv_heads=Hkv, head_dim=128, seq_len_max=L, block_len=b, dtype=B.BF16,
                        retention=r, n_keep_max=L - b)
        n = B.keep_count(d, L, o)[0]
        sd = torch.from_numpy(sc).cuda()
        bo = torch.full((Bn,), o, dtype=torch.int32, device="cuda")
        idx = torch.full((Bn, Hkv, L - b), -5, dtype=torch.int32, device="cuda")
        cnt = torch.zeros((Bn,), dtype=torch.int32, device="cuda")
        B.select_topk(d, sd, None, bo, idx, cnt)
        torch.cuda.synchronize()
        pos = oracle.candidate_positions(L, b, o)
        assert (cnt.cpu().numpy() == n).all()
        for i in range(Bn):
            for h in range(Hkv):
                want = pos[oracle.select_topk(sc[i, h][pos].astype(np.float64), n)]
                got = idx[i, h].cpu().numpy()
                np.testing.assert_array_equal(got[:n], want)
                assert (got[n:] == -1).all()


def test_compact_alone_bit_exact_with_strides():
    rng = np.random.default_rng(9)
    Bn, Hkv, L, D, n = 2, 3, 77, 128, 20
    k = torch.from_numpy(rng.standard_normal((Bn, Hkv, L, D)).astype(np.float32)).cuda().to(torch.bfloat16)
    v = torch.from_numpy(rng.standard_normal((Bn, Hkv, L, D)).astype(np.float32)).cuda().to(torch.bfloat16)
    idx = np.stack([np.stack([np.sort(rng.choice(L, n, replace=False)) for _ in range(Hkv)]) for _ in range(Bn)]).astype(np.int32)
    cnt = np.array([n, 13], np.int32)
    idx[1, :, 13:] = -1
    d = B.make_desc(batch=Bn, n_q_heads=Hkv, n_kv_heads=Hkv, head_dim=D, seq_len_max=L, block_len=32, dtype=B.BF16,
                    retention=0.5, n_keep_max=n)
    kc = torch.full((Bn, Hkv, n, D), float("nan"), dtype=torch.bfloat16, device="cuda")
    vc = torch.full_like(kc, float("nan"))
    B.compact_kv(d, k, v, torch.from_numpy(idx).cuda(), torch.from_numpy(cnt).cuda(), kc, vc)
    torch.cuda.synchronize()
    for i in range(Bn):
        for h in range(Hkv):
            ref_k = oracle.gather_rows(k[i, h:h + 1].view(torch.int16).cpu().numpy(), idx[i, h:h + 1, :cnt[i]])
            ref_v = oracle.gather_rows(v[i, h:h + 1].view(torch.int16).cpu().numpy(), idx[i, h:h + 1, :cnt[i]])
            assert kc[i, h, :cnt[i]].view(torch.int16).cpu().numpy().tobytes() == ref_k.tobytes()
            assert vc[i, h, :cnt[i]].view(torch.int16).cpu().numpy().tobytes() == ref_v.tobytes()
            assert kc[i, h, cnt[i]:].float().abs().sum().item() == 0 and vc[i, h, cnt[i]:].float().abs().sum().item() == 0


def test_scores_only_and_attention_only_calls():
    """out == NULL gives scores only; pooled_scores == NULL gives attention only; both match the full call."""
    import parity_util as U
    cfg = _small("so", "bf16", 4, 2, 128, 200, 64, salient_frac=0.02)
    s = W.make_sequence(cfg, seed=10, block=0)
    q, k, v = s.refresh_inputs(1)
    g = U.gpu_refresh(q[None], k[None], v[None], [s.seq_len], [s.block_off], "bf16", 0.5, 3)
    c = g.cache
    qd, kd, vd = U.to_dev(q[None], "bf16"), g.k_dev, g.v_dev
    bo = torch.tensor([s.block_off], dtype=torch.int32, device="cuda")
    pooled2 = torch.empty_like(c.pooled)
    B.refresh_scores(c.desc, qd, kd, vd, None, bo, None, None, pooled2, c.workspace)
    out2 = torch.empty((1, 4, 32, 128), dtype=torch.bfloat16, device="cuda")
    B.refresh_scores(c.desc, qd, kd, vd, None, bo, out2, None, None, c.workspace)
    torch.cuda.synchronize()
    assert torch.equal(pooled2, torch.from_numpy(g.pooled).cuda())
    np.testing.assert_array_equal(U.to_host_f32(out2), g.out)


# ------------------------------------------------------------------ dense step (all rows over all keys)
def _dense_case(Hq, Hkv, D, lens, seed, pad=np.nan):
    """Padded batch of full-sequence inputs: q [B,Hq,Lmax,D], k/v [B,Hkv,Lmax,D]; the padding must never matter."""
    Lmax = max(max(lens), 1)
    q = np.full((len(lens), Hq, Lmax, D), pad, np.float32)
    k = np.full((len(lens), Hkv, Lmax, D), pad, np.float32)
    v = np.full((len(lens), Hkv, Lmax, D), pad, np.float32)
    for i, L in enumerate(lens):
        if L == 0:
            continue
        cfg = _small("dense", "bf16", Hq, Hkv, D, L - 16, 16, block_len=16, salient_frac=0.02)
        s = W.make_sequence(cfg, seed=seed + i)
        q[i, :, :L], k[i, :, :L], v[i, :, :L] = s.dense_inputs(0)
    return q, k, v


@pytest.mark.parametrize("Hq,Hkv,D,lens", [
    (2, 2, 128, [333]),                 # several query blocks (an odd number) and key tiles with ragged tails
    (8, 2, 64, [200]),                  # grouped heads, D = 64
    (4, 1, 128, [128]),                 # exactly one tile each way
    (2, 1, 128, [17]),                  # shorter than a tile
    (4, 2, 128, [300, 40, 0, 257]),     # ragged batch with an empty sequence
])
def test_dense_step(Hq, Hkv, D, lens):
    import parity_util as U
    q, k, v = _dense_case(Hq, Hkv, D, lens, seed=21)
    out, lse = U.gpu_dense(q, k, v, lens)
    U.check_dense_against_oracle(out, lse, np.nan_to_num(q), np.nan_to_num(k), np.nan_to_num(v), lens)


def test_dense_step_without_lengths_and_refusals():
    import parity_util as U
    q, k, v = _dense_case(2, 2, 64, [256], seed=23)
    out, _ = U.gpu_dense(q, k, v, None, want_lse=False)
    U.check_dense_against_oracle(out, None, q, k, v, None)
    d = B.make_desc(batch=1, n_q_heads=2, n_kv_heads=2, head_dim=64, seq_len_max=256, block_len=32, dtype=B.F32, retention=0.5)
    assert B.workspace_bytes(d, B.OP_DENSE_ATTN) == 0
    t = torch.zeros((1, 2, 256, 64), device="cuda:0")
    ws = torch.zeros((4096,), dtype=torch.uint8, device="cuda:0")
    with pytest.raises(B.SdllmError) as e:
        B.dense_attn(d, t, t, t, None, t, None, ws)
    assert e.value.status == B.ERR_UNSUPPORTED


def test_dense_step_two_tile_kernel_many_key_tiles():
    """Enough key tiles for every barrier phase and ring slot to wrap several times; odd number of query blocks."""
    import parity_util as U
    q, k, v = _dense_case(8, 2, 128, [1100, 640], seed=24)
    out, lse = U.gpu_dense(q, k, v, [1100, 640])
    U.check_dense_against_oracle(out, lse, np.nan_to_num(q), np.nan_to_num(k), np.nan_to_num(v), [1100, 640],
                                 rows=[0, 127, 128, 300, 639, 640, 1023, 1024, 1099])


def test_dense_step_strided_tensors_and_argument_checks():
    """q and out as column slices of wider tensors (row stride 2D), heads-last-but-one layouts left to the strides; the
    untouched half of the output buffer must stay as it was. Then the argument checks of the entry point."""
    import parity_util as U
    Hq, Hkv, D, L = 4, 2, 64, 200
    q, k, v = _dense_case(Hq, Hkv, D, [L], seed=27, pad=0.0)
    d = B.make_desc(batch=1, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=D, seq_len_max=L, block_len=32, dtype=B.BF16, retention=0.5)
    wide_q = torch.zeros((1, Hq, L, 2 * D), dtype=torch.bfloat16, device="cuda:0")
    wide_q[..., :D] = U.to_dev(q, "bf16")
    wide_o = torch.full((1, Hq, L, 2 * D), 7.0, dtype=torch.bfloat16, device="cuda:0")
    kd, vd = U.to_dev(k, "bf16"), U.to_dev(v, "bf16")
    ws = torch.zeros((max(B.workspace_bytes(d, B.OP_DENSE_ATTN), 256),), dtype=torch.uint8, device="cuda:0")
    assert B.launch_count(d, B.OP_DENSE_ATTN) >= 1
    B.dense_attn(d, wide_q[..., :D], kd, vd, None, wide_o[..., :D], None, ws)
    torch.cuda.synchronize()
    assert B.read_status(ws) == 0
    got = U.to_host_f32(wide_o)
    assert (got[..., D:] == 7.0).all()
    U.check_dense_against_oracle(np.ascontiguousarray(got[..., :D]), None, q, k, v, None)
    # argument checks: missing tensors, a workspace that is too small, a misaligned pointer
    qd = U.to_dev(q, "bf16")
    out = torch.empty_like(qd)
    for args in [(None, kd, vd, None, out, None, ws), (qd, kd, vd, None, None, None, ws)]:
        with pytest.raises(B.SdllmError) as e:
            B.dense_attn(d, *args)
        assert e.value.status == B.ERR_INVALID_ARG
    with pytest.raises(B.SdllmError) as e:
        B.dense_attn(d, qd, kd, vd, None, out, None, ws[:128])
    assert e.value.status == B.ERR_WORKSPACE
    with pytest.raises(B.SdllmError) as e:
        B.dense_attn(d, qd, kd.view(-1)[4:].view(-1), vd, None, out, None, ws)
    assert e.value.status == B.ERR_INVALID_ARG


@pytest.mark.parametrize("plan", [
    {},                                  # key-row kernel: its splits still meet in the cluster merge while they give up
    dict(splits=1),                      # ... one CTA per head
    dict(splits=1, persist=2),           # ... streaming variant: two resident CTAs walk the heads
    dict(kernel=2, cluster=0, splits=3), # query-row kernel, partials and completion counters in the workspace
    dict(kernel=2, cluster=2),           # ... cluster tail
])
def test_a_bounded_wait_that_runs_out_is_reported_and_leaves_a_usable_library(plan, tuning):
    """With the limit of the abortable device-side waits set to zero, the first wait that is not already satisfied gives
    up. Nothing hangs and nothing faults: the call returns, the status word reports the time-out, and after the workspace
    has been zeroed again the next call (normal limit) matches the oracle. The waits that let copies and MMAs in flight
    land before a CTA retires keep their own long limit."""
    import parity_util as U
    cfg = _small("timeout", "bf16", 4, 4, 128, 330, 64, salient_frac=0.02)
    s = W.make_sequence(cfg, seed=19, block=0)
    q, k, v = s.refresh_inputs(1)
    tuning(**plan)                       # before the workspace is sized
    g = U.gpu_refresh(q[None], k[None], v[None], [s.seq_len], [s.block_off], "bf16", cfg.retention, cfg.pool_window)
    q2, kn, vn = s.sparse_inputs(2)
    want = U.gpu_sparse_step(g, q2[None], kn[None], vn[None], "bf16")          # the plan itself works
    U.check_sparse_against_oracle(g, want, q2[None], kn[None], vn[None], "bf16")
    tuning(wait_cycles=0)
    qd, knd, vnd = U.to_dev(q2[None], "bf16"), U.to_dev(kn[None], "bf16"), U.to_dev(vn[None], "bf16")
    out = torch.zeros(q2[None].shape, dtype=torch.bfloat16, device=U.DEV)
    g.cache.sparse_step(qd, knd, vnd, out)
    torch.cuda.synchronize()                                                   # the call returns
    assert B.read_status(g.cache.workspace) != 0                               # ... and says that it gave up
    with pytest.raises(B.SdllmError) as e:
        B._check(B.lib().sdllm_read_status(g.cache.workspace.data_ptr(), torch.cuda.current_stream().cuda_stream,
                                           __import__("ctypes").byref(__import__("ctypes").c_int32(0))), "sdllm_read_status")
    assert e.value.status == B.ERR_TIMEOUT
    tuning(wait_cycles=400_000_000)
    g.cache.workspace.zero_()                                                  # what the header asks for after a time-out
    again = U.gpu_sparse_step(g, q2[None], kn[None], vn[None], "bf16")
    U.check_sparse_against_oracle(g, again, q2[None], kn[None], vn[None], "bf16")
    np.testing.assert_array_equal(again, want)


@pytest.mark.parametrize("plan", [{}, dict(splits=1), dict(splits=2), dict(dual=0, splits=1), dict(dual=0, splits=2), dict(kernel=2),
                                  dict(splits=1, persist=1), dict(splits=1, persist=2)])
def test_logits_far_above_the_softmax_references(plan, tuning):
    """The key-row kernel takes its softmax references from the first key of a CTA's first tile and only checks later keys
    against them; keys whose logits lie more than 2^64 above a reference make it raise the references and rescale what it
    has accumulated. Here every query shares a strong component with a few keys planted in the first tile (not its first
    row), in later tiles and in the block's fresh rows, 50 to 100 nats above everything else: refresh and reuse step must
    still match the oracle."""
    import parity_util as U
    tuning(**plan)
    rng = np.random.default_rng(23)
    Hq = Hkv = 2
    D, b, L, o = 128, 32, 900, 700
    q = rng.standard_normal((Hq, b, D)).astype(np.float32) * 0.3
    q[:, :, 0] += 3.0
    k = rng.standard_normal((Hkv, L, D)).astype(np.float32) * 0.3
    v = rng.standard_normal((Hkv, L, D)).astype(np.float32)
    for pos, gain in [(5, 300.0), (300, 250.0), (301, 250.0), (640, 200.0), (o + 40 + b, 400.0), (o + 3, 300.0)]:
        k[:, pos, :] = 0.0
        k[:, pos, 0] = gain                      # logit = gain * 3 / sqrt(128): 53 to 106 nats (76 to 153 in log2 units) above the rest
    q, k, v = (W.round_to_dtype(x, "bf16") for x in (q, k, v))
    g = U.gpu_refresh(q[None], k[None], v[None], [L], [o], "bf16", 0.5, 3)
    U.check_refresh_against_oracle(g, q[None], k[None], v[None], [L], [o], "bf16", 0.5, 3)
    U.check_compaction_bit_exact(g, g.k_dev, g.v_dev)
    q2 = W.round_to_dtype(q + 0.01 * rng.standard_normal(q.shape).astype(np.float32), "bf16")
    kn, vn = k[:, o:o + b].copy(), v[:, o:o + b].copy()
    kn[:, 17, :] = 0.0
    kn[:, 17, 0] = 500.0                         # the largest logit of all sits in the block's fresh rows (the last tile)
    out = U.gpu_sparse_step(g, q2[None], kn[None], vn[None], "bf16")
    U.check_sparse_against_oracle(g, out, q2[None], kn[None], vn[None], "bf16")


def test_planner_picks_the_kernel_families_where_they_were_measured_to_win():
    """Which kernel runs which shape on a B200 (sdllm_plan_describe): the benchmark's headline shape the key-row kernel,
    a 16-sequence serving batch its streaming variant (more units than SMs), grouped heads with few units the query-row
    kernel, grouped heads with many units the key-row kernel again."""
    def name(op=B.OP_SPARSE_BLOCK_ATTN, **kw):
        kw = dict(dict(batch=1, n_q_heads=32, n_kv_heads=32, head_dim=128, seq_len_max=1280, block_len=32, dtype=B.BF16, retention=0.5,
                       n_keep_max=496), **kw)
        return B.plan_describe(B.make_desc(**kw), op).split()[0]
    assert name() == "attn_kt_kernel" and name(B.OP_REFRESH_SCORES) == "attn_kt_kernel"
    assert name(batch=16, seq_len_max=4352, n_keep_max=2160) == "attn_kt_stream_kernel"
    assert name(B.OP_REFRESH_SCORES, batch=16, seq_len_max=4352, n_keep_max=2160) == "attn_kt_stream_kernel"
    assert name(n_q_heads=28, n_kv_heads=4, seq_len_max=4096, n_keep_max=1024) == "attn_umma_bf16_kernel"       # 224 query rows per KV head
    assert name(n_kv_heads=8, seq_len_max=32768, n_keep_max=16368) == "attn_umma_bf16_kernel"                   # 8 units of 128 rows
    assert name(batch=8, n_q_heads=16, n_kv_heads=8, seq_len_max=4352, n_keep_max=2048) == "attn_kt_kernel"     # 64 units of 64 rows
    assert name(dtype=B.F32) == "attn_f32_kernel"
    # cluster sizes follow what the device keeps resident at once: 16 units of whole-SM CTAs get clusters of six, not eight
    plan = B.plan_describe(B.make_desc(batch=2, n_q_heads=16, n_kv_heads=8, head_dim=128, seq_len_max=2080, block_len=32, dtype=B.BF16,
                                       retention=0.5, n_keep_max=1024), B.OP_SPARSE_BLOCK_ATTN)
    assert plan.startswith("attn_kt_kernel ") and " cluster=6 " in plan, plan
    # 192 units of long walks (a six-sequence serving batch): one CTA per SM with a ring of three slots, not two small CTAs
    # per SM with one slot each; short walks keep the small footprint
    for op in (B.OP_SPARSE_BLOCK_ATTN, B.OP_REFRESH_SCORES):
        plan = B.plan_describe(B.make_desc(batch=6, n_q_heads=32, n_kv_heads=32, head_dim=128, seq_len_max=4128, block_len=32,
                                           dtype=B.BF16, retention=0.5, n_keep_max=2048), op)
        assert plan.startswith("attn_kt_kernel ") and " stages=3 " in plan and " cluster=1 " in plan, plan
    plan = B.plan_describe(B.make_desc(batch=6, n_q_heads=32, n_kv_heads=32, head_dim=128, seq_len_max=1056, block_len=32,
                                       dtype=B.BF16, retention=0.5, n_keep_max=512), B.OP_SPARSE_BLOCK_ATTN)
    assert plan.startswith("attn_kt_kernel ") and " stages=1 " in plan, plan


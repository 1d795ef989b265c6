"""GPU parity at the full workload sizes, in the launch configuration the benchmark times: whole calls run on the
device, a sample of (sequence, KV head) pairs is recomputed by the CPU oracle one by one and compared element by
element; kept sets, counts and the compaction are checked for every head against properties that hold at any size."""
import numpy as np
import pytest
import torch

import oracle
from paper_2508_02558_b200 import build as libbuild
from paper_2508_02558_b200 import workloads as W

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    libbuild.build()


def _check_all_heads_properties(g, seq_len, block_off, b):
    """Every head: count, ascending unique positions outside the block and inside the sequence, -1 tail."""
    for i in range(g.kept_idx.shape[0]):
        cnt, L, o = int(g.kept_cnt[i]), int(seq_len[i]), int(block_off[i])
        idx = g.kept_idx[i]
        got = idx[:, :cnt]
        assert (np.diff(got, axis=1) > 0).all() and (got >= 0).all() and (got < L).all()
        assert not ((got >= o) & (got < o + b)).any()
        assert (idx[:, cnt:] == -1).all()
        # min kept pooled score >= max evicted pooled score, per head
        pooled = g.pooled[i]
        for h in range(idx.shape[0]):
            kept = np.zeros(pooled.shape[1], bool)
            kept[got[h]] = True
            cand = np.isfinite(pooled[h]) | (pooled[h] > -np.inf)
            cand[o:o + b] = False
            cand[L:] = False
            if cnt and (cand & ~kept).any():
                assert pooled[h][kept].min() >= pooled[h][cand & ~kept].max()


def _run(cfg, seed, heads, retention=None, window=None, score=oracle.SCORE_LOGIT_MEAN, block=0):
    import parity_util as U
    r = cfg.retention if retention is None else retention
    s_ = cfg.pool_window if window is None else window
    s = W.make_sequence(cfg, seed=seed, layer=0, block=block)
    q, k, v = s.refresh_inputs(1)
    L, o = s.seq_len, s.block_off
    g = U.gpu_refresh(q[None], k[None], v[None], [L], [o], cfg.dtype, r, s_, score=score)
    U.check_refresh_against_oracle(g, q[None], k[None], v[None], [L], [o], cfg.dtype, r, s_, heads=heads, score=score)
    _check_all_heads_properties(g, [L], [o], cfg.block_len)
    U.check_compaction_bit_exact(g, g.k_dev, g.v_dev)
    q2, kn, vn = s.sparse_inputs(2)
    out = U.gpu_sparse_step(g, q2[None], kn[None], vn[None], cfg.dtype)
    U.check_sparse_against_oracle(g, out, q2[None], kn[None], vn[None], cfg.dtype, heads=heads)
    assert np.isfinite(out).all()


def test_c2_llada_layer_full_size():
    _run(W.CONFIGS["c2_llada"], seed=21, heads=[0, 13, 31])


def test_c3_dream_layer_full_size():
    _run(W.CONFIGS["c3_dream"], seed=22, heads=[0, 3])


@pytest.mark.parametrize("name,block,r,window", [("c6_gen512", 9, 0.3, 5), ("c7_long4k", 15, None, None)])
def test_second_workload_shapes_full_size(name, block, r, window):
    """Generation length 512 (a block in the middle: prefix and suffix both long) and the 4k-prompt shape (last block)."""
    _run(W.CONFIGS[name], seed=26, heads=[4, 29], retention=r, window=window, block=block)


@pytest.mark.parametrize("r,window", [(0.1, 7), (0.5, 3)])
def test_c4_long_context_full_size(r, window):
    _run(W.CONFIGS["c4_long"], seed=23, heads=[5], retention=r, window=window)


@pytest.mark.parametrize("name,heads,r,window", [("c3_dream", [1], None, None), ("c4_long", [2], 0.25, 1)])
def test_softmax_probability_saliency_full_size(name, heads, r, window):
    _run(W.CONFIGS[name], seed=25, heads=heads, retention=r, window=window, score=oracle.SCORE_PROB_MEAN)


@pytest.mark.parametrize("batch", [4, 16])
def test_c5_serving_ragged_batch_full_size(batch):
    import parity_util as U
    cfg = W.CONFIGS["c5_serving"]
    lens = W.serving_prompt_lengths(batch, seed=5)
    bw = W.make_batch(cfg, lens, seed=24)
    q, k, v = bw.refresh_inputs(1)
    g = U.gpu_refresh(q, k, v, bw.seq_len, bw.block_off, "bf16", cfg.retention, cfg.pool_window)
    seqs = sorted({0, batch - 1, int(np.argmax(bw.seq_len)), int(np.argmin(bw.seq_len))})
    U.check_refresh_against_oracle(g, q, k, v, bw.seq_len, bw.block_off, "bf16", cfg.retention, cfg.pool_window,
                                   heads=[7, 30], seqs=seqs)
    _check_all_heads_properties(g, bw.seq_len, bw.block_off, cfg.block_len)
    q2, kn, vn = bw.sparse_inputs(2)
    out = U.gpu_sparse_step(g, q2, kn, vn, "bf16")
    U.check_sparse_against_oracle(g, out, q2, kn, vn, "bf16", heads=[7, 30], seqs=seqs)
    assert np.isfinite(out).all()


@pytest.mark.parametrize("name,heads", [("c2_llada", [0, 17]), ("c3_dream", [3]), ("c4_long", [5])])
def test_dense_step_full_size(name, heads):
    """All L rows over all L keys at the workload's size; the oracle recomputes a sample of rows of a sample of heads."""
    import parity_util as U
    cfg = W.CONFIGS[name]
    s = W.make_sequence(cfg, seed=31)
    q, k, v = s.dense_inputs(0)
    L = s.seq_len
    out, lse = U.gpu_dense(q[None], k[None], v[None], [L])
    rows = sorted({0, 1, 127, 128, L // 2 + 3, s.block_off, s.block_off + cfg.block_len - 1, L - 129, L - 1})
    U.check_dense_against_oracle(out, lse, q[None], k[None], v[None], [L], rows=rows, heads=heads)
    assert np.isfinite(out).all() and np.isfinite(lse).all()


def test_dense_step_ragged_serving_batch_full_size():
    import parity_util as U
    cfg = W.CONFIGS["c5_serving"]
    lens = W.serving_prompt_lengths(4, seed=5)
    bw = W.make_batch(cfg, lens, seed=25)
    Lm = bw.seq_len_max
    q = np.zeros((4, cfg.n_q_heads, Lm, cfg.head_dim), np.float32)
    k, v = np.zeros((4, cfg.n_kv_heads, Lm, cfg.head_dim), np.float32), np.zeros((4, cfg.n_kv_heads, Lm, cfg.head_dim), np.float32)
    for i, s in enumerate(bw.seqs):
        q[i, :, :s.seq_len], k[i, :, :s.seq_len], v[i, :, :s.seq_len] = s.dense_inputs(0)
    out, lse = U.gpu_dense(q, k, v, bw.seq_len)
    U.check_dense_against_oracle(out, lse, q, k, v, bw.seq_len, rows=[0, 130, 700, 2049, 4000], heads=[9])

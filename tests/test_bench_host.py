"""Host-side arithmetic of the benchmark (no GPU): workload overrides, token and byte counts against hand-worked
figures for the LLaDA-shaped layer, and the seeded generator of the dense step's inputs."""
import argparse
import os
import sys

import numpy as np

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
import bench
from paper_2508_02558_b200 import workloads as W


def _args(**kw):
    base = dict(workload="c2_llada", retention=None, pool_window=None)
    base.update(kw)
    return argparse.Namespace(**base)


def test_workload_overrides():
    assert bench.workload_config(_args()) == W.CONFIGS["c2_llada"]
    c = bench.workload_config(_args(retention=0.3, pool_window=7))
    assert (c.retention, c.pool_window) == (0.3, 7)
    assert (c.n_q_heads, c.seq_len, c.n_layers) == (32, 1280, 32)       # everything else is the named workload
    assert W.CONFIGS["c2_llada"].retention == 0.5                       # the table itself is untouched
    assert (W.CONFIGS["c6_gen512"].seq_len, W.CONFIGS["c7_long4k"].seq_len) == (1024, 4608)


def test_token_and_byte_counts_of_the_llada_shaped_layer():
    cfg = W.CONFIGS["c2_llada"]
    # L = 1280, b = 32, r = 0.5: n = floor((1280 - 32) / 2) = 624 kept keys; 30 reuse steps after the refresh
    assert bench.tokens_per_step(cfg, 32, [1280], [624]) == 32 * (1280 + 30 * (624 + 32))
    assert bench.tokens_per_step(cfg, 32, [1280], [624], "refresh") == 32 * 1280
    assert bench.tokens_per_step(cfg, 32, [1280], [624], "sparse") == 32 * 30 * 656
    ab = bench.algorithmic_bytes(cfg, [1280], [624])
    # sparse step: K and V of 656 keys x 32 heads x 128 x 2 B, Q and O of 32 rows x 32 heads
    assert ab["sparse"] == 2 * 656 * 32 * 128 * 2 + 2 * 32 * 32 * 128 * 2 == 11272192
    assert ab["refresh"] == 2 * 1280 * 32 * 128 * 2 + 2 * 32 * 32 * 128 * 2 + 4 * 1248 * 32
    assert ab["compact"] == 2 * (2 * 624 * 32 * 128 * 2) + 4 * 624 * 32
    assert ab["topk"] == 4 * 1248 * 32 + 4 * 624 * 32


def test_dense_inputs_are_seeded_rounded_and_share_the_block_rows():
    cfg = W.WorkloadConfig("t", "bf16", 4, 2, 64, 100, 64, salient_frac=0.02)
    a, b = W.make_sequence(cfg, seed=3, block=1), W.make_sequence(cfg, seed=3, block=1)
    qa, ka, va = a.dense_inputs(0)
    qb, kb, vb = b.dense_inputs(0)
    assert qa.shape == (4, 164, 64) and ka.shape == (2, 164, 64)
    for x, y in ((qa, qb), (ka, kb), (va, vb)):
        np.testing.assert_array_equal(x, y)
        np.testing.assert_array_equal(x, W.round_to_dtype(x, "bf16"))    # already representable in bf16
    q_blk, k_r, _ = a.refresh_inputs(0)
    np.testing.assert_array_equal(qa[:, a.block_off:a.block_off + cfg.block_len], q_blk)
    np.testing.assert_array_equal(ka, k_r)
    assert not np.array_equal(a.dense_inputs(1)[0], qa)                   # another step, other rows

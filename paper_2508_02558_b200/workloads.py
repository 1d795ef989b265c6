"""Seeded synthetic attention workloads shaped like the Sparse-dLLM decoding loop.

This module only *draws inputs*: Gaussian Q/K/V with a few "pivotal" keys planted
along the mean block-query direction (the vertical-attention pattern of Section 3.2),
a small step-to-step drift (KV states of neighbouring denoising steps are nearly
identical, Section 3.3.2) and, for 16-bit runs, one round-to-nearest-even to bf16.
It contains no scoring, pooling, selection or attention arithmetic, and is the one
module that both the CPU oracle's tests and the CUDA path's tests may import.

Only numpy is imported here.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import Dict, List, Optional, Tuple

import numpy as np

# ----------------------------------------------------------------------------- bf16
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (round-to-nearest-even) and return the uint16 bit patterns."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32).astype(np.uint64)
    rounded = (u + 0x7FFF + ((u >> 16) & 1)) >> 16
    return rounded.astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bfloat16 bit patterns to float32."""
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    return (bits.astype(np.uint32) << 16).view(np.float32)


def round_to_dtype(x: np.ndarray, dtype: str) -> np.ndarray:
    """Return float32 values that are exactly representable in `dtype` ("f32" or "bf16")."""
    x = np.asarray(x, dtype=np.float32)
    if dtype == "f32":
        return np.ascontiguousarray(x)
    if dtype == "bf16":
        return bf16_bits_to_f32(f32_to_bf16_bits(x)).reshape(x.shape)
    raise ValueError(f"unknown dtype {dtype!r}")


# ----------------------------------------------------------------------------- configs
@dataclass(frozen=True)
class WorkloadConfig:
    """Shape and recipe of one synthetic workload (one layer of one sequence unless batched)."""
    name: str
    dtype: str                  # "f32" | "bf16"
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    prompt_len: int             # p
    gen_len: int                # L - p
    block_len: int = 32         # b
    retention: float = 0.5      # r
    pool_window: int = 3        # s
    n_layers: int = 1
    steps_per_block: int = 32
    salient_frac: float = 0.0   # fraction of non-block keys planted per head (if salient_count == 0)
    salient_count: int = 0      # exact number of planted keys per head
    salient_gain: float = 3.0
    sink_tokens: int = 0        # leading positions that get the sink offset
    sink_gain: float = 6.0
    salient_spans: int = 0      # >0: planted keys are clustered in this many spans ...
    salient_span_len: int = 64  # ... of this length
    drift_std: float = 0.05     # relative to the base std 1/sqrt(D)

    @property
    def seq_len(self) -> int:
        return self.prompt_len + self.gen_len

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def n_blocks(self) -> int:
        return self.gen_len // self.block_len


CONFIGS: Dict[str, WorkloadConfig] = {
    # tiny fp32 case the oracle finishes instantly
    "c1_tiny": WorkloadConfig("c1_tiny", "f32", 2, 2, 64, 128, 128, salient_count=4, sink_tokens=1,
                              steps_per_block=5),
    # LLaDA-8B-shaped attention stack (MHA)
    "c2_llada": WorkloadConfig("c2_llada", "bf16", 32, 32, 128, 1024, 256, n_layers=32, salient_frac=0.02),
    # Dream-7B-shaped GQA stack
    "c3_dream": WorkloadConfig("c3_dream", "bf16", 28, 4, 128, 3840, 256, n_layers=28, retention=0.25,
                               salient_frac=0.01, sink_tokens=4),
    # long-context single layer
    "c4_long": WorkloadConfig("c4_long", "bf16", 32, 8, 128, 32512, 256, salient_frac=0.005,
                              salient_spans=16, salient_span_len=64),
    # one LLaDA-shaped layer for the ragged batched sweep (prompt length overridden per sequence)
    "c5_serving": WorkloadConfig("c5_serving", "bf16", 32, 32, 128, 4096, 256, salient_frac=0.02),
    # second workload shapes (LLaDA-shaped stack): generation length 512 after a 512-token prompt, and a prompt
    # truncated to 4k tokens followed by 512 generated tokens; block length 32, one denoising step per token
    "c6_gen512": WorkloadConfig("c6_gen512", "bf16", 32, 32, 128, 512, 512, n_layers=32, salient_frac=0.02),
    "c7_long4k": WorkloadConfig("c7_long4k", "bf16", 32, 32, 128, 4096, 512, n_layers=32, salient_frac=0.02),
}


def serving_prompt_lengths(batch: int, seed: int = 0, lo: int = 512, hi: int = 4096) -> List[int]:
    """Per-sequence prompt lengths of the batched serving sweep: uniform integers in [lo, hi]."""
    rng = np.random.Generator(np.random.Philox(key=[seed, 0x5E41]))
    return [int(v) for v in rng.integers(lo, hi + 1, size=batch)]


# ----------------------------------------------------------------------------- one sequence, one layer
@dataclass
class SequenceWorkload:
    """Base tensors of one (sequence, layer, block); step inputs are derived by `refresh_inputs`/`sparse_inputs`.

    Arrays are float32 holding values exactly representable in cfg.dtype.
    q_base [Hq, b, D], k_base/v_base [Hkv, L, D], planted_pos [Hkv, n_planted] (absolute positions).
    """
    cfg: WorkloadConfig
    seed: int
    layer: int
    block: int
    block_off: int
    q_base: np.ndarray
    k_base: np.ndarray
    v_base: np.ndarray
    planted_dir: np.ndarray      # [Hkv, D] unit vectors
    planted_pos: np.ndarray      # [Hkv, n_planted] int64
    _offset: np.ndarray = field(repr=False, default=None)   # [Hkv, L, D] additive K offsets (planted + sink)

    @property
    def seq_len(self) -> int:
        return self.cfg.seq_len

    def _rng(self, step: int, what: int) -> np.random.Generator:
        return np.random.Generator(np.random.Philox(key=[_mix(self.seed, self.layer, self.block), (step << 8) | what]))

    def _drift(self, shape, step: int, what: int) -> np.ndarray:
        std = self.cfg.drift_std / np.sqrt(self.cfg.head_dim)
        return self._rng(step, what).standard_normal(shape, dtype=np.float32) * np.float32(std)

    def refresh_inputs(self, step: int = 1) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
        """(Q_b, K, V) seen by the refresh step: base + this step's drift, planted offsets re-applied."""
        c = self.cfg
        q = self.q_base + self._drift(self.q_base.shape, step, 1)
        k = self.k_base + self._drift(self.k_base.shape, step, 2) + self._offset
        v = self.v_base + self._drift(self.v_base.shape, step, 3)
        return round_to_dtype(q, c.dtype), round_to_dtype(k, c.dtype), round_to_dtype(v, c.dtype)

    def sparse_inputs(self, step: int) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
        """(Q_b', K_n, V_n): the current block's fresh query/key/value rows at a cache-reuse step."""
        c = self.cfg
        o, b = self.block_off, c.block_len
        q = self.q_base + self._drift(self.q_base.shape, step, 1)
        kb = self.k_base[:, o:o + b] + self._drift((c.n_kv_heads, b, c.head_dim), step, 4) + self._offset[:, o:o + b]
        vb = self.v_base[:, o:o + b] + self._drift((c.n_kv_heads, b, c.head_dim), step, 5)
        return round_to_dtype(q, c.dtype), round_to_dtype(kb, c.dtype), round_to_dtype(vb, c.dtype)


    def dense_inputs(self, step: int = 0) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
        """(Q, K, V) of a dense step: query rows for all L positions (the block's rows are that step's Q_b), and the
        K, V of `refresh_inputs(step)`."""
        c = self.cfg
        qb, k, v = self.refresh_inputs(step)
        inv = np.float32(1.0 / np.sqrt(c.head_dim))
        q = self._rng(step, 6).standard_normal((c.n_q_heads, c.seq_len, c.head_dim), dtype=np.float32) * inv
        q[:, self.block_off:self.block_off + c.block_len] = qb
        return round_to_dtype(q, c.dtype), k, v


def _mix(*vals: int) -> int:
    """Small integer hash so (seed, layer, block) give unrelated Philox keys."""
    h = 0x9E3779B97F4A7C15
    for v in vals:
        h ^= (int(v) + 0x9E3779B97F4A7C15 + ((h << 6) & 0xFFFFFFFFFFFFFFFF) + (h >> 2)) & 0xFFFFFFFFFFFFFFFF
        h &= 0xFFFFFFFFFFFFFFFF
    return h


def make_sequence(cfg: WorkloadConfig, seed: int = 0, layer: int = 0, block: int = 0,
                  prompt_len: Optional[int] = None) -> SequenceWorkload:
    """Draw the base tensors of one (sequence, layer, block).

    Q, K, V ~ N(0, 1)/sqrt(D). Each KV head gets a unit direction u = normalised mean of its
    group's block queries; planted keys get `+ salient_gain * u`, sink positions `+ sink_gain * u`.
    Planted positions never fall inside the current block.
    """
    if prompt_len is not None:
        cfg = replace(cfg, prompt_len=int(prompt_len))
    H, Hk, D, L, b = cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.seq_len, cfg.block_len
    if not (0 <= block < cfg.n_blocks):
        raise ValueError("block index out of range")
    o = cfg.prompt_len + block * b
    rng = np.random.Generator(np.random.Philox(key=[_mix(seed, layer, block), 0]))
    inv = np.float32(1.0 / np.sqrt(D))
    q = rng.standard_normal((H, b, D), dtype=np.float32) * inv
    k = rng.standard_normal((Hk, L, D), dtype=np.float32) * inv
    v = rng.standard_normal((Hk, L, D), dtype=np.float32) * inv

    G = cfg.group
    qbar = q.reshape(Hk, G * b, D).mean(axis=1, dtype=np.float64)
    u = (qbar / np.linalg.norm(qbar, axis=1, keepdims=True)).astype(np.float32)

    cand = np.concatenate([np.arange(cfg.sink_tokens, o), np.arange(o + b, L)])   # non-block, non-sink
    n_planted = cfg.salient_count if cfg.salient_count > 0 else int(round(cfg.salient_frac * (L - b)))
    n_planted = min(n_planted, cand.size)
    pos = np.zeros((Hk, n_planted), dtype=np.int64)
    offset = np.zeros((Hk, L, D), dtype=np.float32)
    for h in range(Hk):
        if n_planted > 0:
            if cfg.salient_spans > 0:
                starts = rng.choice(cand.size - cfg.salient_span_len, size=cfg.salient_spans, replace=False)
                pool = np.unique(np.concatenate([cand[s0:s0 + cfg.salient_span_len] for s0 in starts]))
                chosen = rng.choice(pool, size=min(n_planted, pool.size), replace=False)
                if chosen.size < n_planted:
                    chosen = np.concatenate([chosen, chosen[:n_planted - chosen.size]])
            else:
                chosen = rng.choice(cand, size=n_planted, replace=False)
            pos[h] = np.sort(chosen)
            offset[h, pos[h]] += np.float32(cfg.salient_gain) * u[h]
        if cfg.sink_tokens > 0:
            offset[h, :cfg.sink_tokens] += np.float32(cfg.sink_gain) * u[h]
    return SequenceWorkload(cfg, seed, layer, block, o, round_to_dtype(q, cfg.dtype), k, v, u, pos, offset)


# ----------------------------------------------------------------------------- batches (padded)
@dataclass
class BatchWorkload:
    """Padded batch of independent sequences (ragged serving sweep). Arrays are [B, H, Lmax|b, D] float32."""
    cfg: WorkloadConfig
    seqs: List[SequenceWorkload]
    seq_len: np.ndarray       # [B] int32
    block_off: np.ndarray     # [B] int32

    @property
    def batch(self) -> int:
        return len(self.seqs)

    @property
    def seq_len_max(self) -> int:
        return int(self.seq_len.max())

    def refresh_inputs(self, step: int = 1, pad_value: float = 0.0):
        B, c, Lm = self.batch, self.cfg, self.seq_len_max
        q = np.zeros((B, c.n_q_heads, c.block_len, c.head_dim), np.float32)
        k = np.full((B, c.n_kv_heads, Lm, c.head_dim), pad_value, np.float32)
        v = np.full((B, c.n_kv_heads, Lm, c.head_dim), pad_value, np.float32)
        for i, s in enumerate(self.seqs):
            qi, ki, vi = s.refresh_inputs(step)
            q[i], k[i, :, :s.seq_len], v[i, :, :s.seq_len] = qi, ki, vi
        return q, k, v

    def sparse_inputs(self, step: int):
        parts = [s.sparse_inputs(step) for s in self.seqs]
        return tuple(np.stack([p[j] for p in parts]) for j in range(3))


def make_batch(cfg: WorkloadConfig, prompt_lens: List[int], seed: int = 0, layer: int = 0,
               block: int = 0) -> BatchWorkload:
    seqs = [make_sequence(cfg, seed=_mix(seed, i) & 0x7FFFFFFF, layer=layer, block=block, prompt_len=p)
            for i, p in enumerate(prompt_lens)]
    return BatchWorkload(cfg, seqs, np.array([s.seq_len for s in seqs], np.int32),
                         np.array([s.block_off for s in seqs], np.int32))

"""CPU oracle for the Sparse-dLLM refresh / sparse-block-attention path (TEST INFRASTRUCTURE ONLY).

A thin ctypes layer over ``sdllm_oracle.cpp`` (plain C++, double precision) plus the few lines that
chain its routines in the order of the paper's Algorithm 1 (cache refresh), Algorithm 2/4 (cache
state of a step) and Algorithm 3 (cache reuse). Only the tests, the smoke check and the benchmark's
CPU-baseline leg may import this package; the CUDA library never does, and this package never
imports the CUDA library.

Everything here works on one sequence of one layer; arrays are numpy float64 unless stated.
Parity-unpinned readings (fixed only by this project's design notes): pre-softmax logits as the
default score, one selection per KV head under GQA, the joint-vs-per-region policies, ascending
order of the kept rows.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass
from typing import List, Optional, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "sdllm_oracle.cpp")
_LIB = os.path.join(_HERE, "liboracle.so")

SCORE_LOGIT_MEAN, SCORE_PROB_MEAN = 0, 1
POOL_MAX, POOL_AVG = 0, 1
SELECT_JOINT_FLOOR, SELECT_PER_REGION_CEIL, SELECT_PREFIX_ONLY = 0, 1, 2


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (-O2, OpenMP) if the shared object is missing or stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.run(["g++", "-O2", "-std=c++17", "-fopenmp", "-fPIC", "-shared", "-o", _LIB, _SRC], check=True)
    return _LIB


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
    return _lib


def _dp(a: np.ndarray):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def _f64(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float64)


def _check(rc: int, what: str):
    if rc != 0:
        raise ValueError(f"oracle: invalid arguments to {what}")


# --------------------------------------------------------------------------- single routines
def attention(q, k, v, scale: Optional[float] = None, return_probs: bool = False):
    """Textbook softmax attention. q [Hq,b,D], k/v [Hkv,nk,D] -> out [Hq,b,D], lse [Hq,b] (, probs [Hq,b,nk])."""
    q, k, v = _f64(q), _f64(k), _f64(v)
    Hq, b, D = q.shape
    Hkv, nk, _ = k.shape
    scale = 1.0 / np.sqrt(D) if scale is None else float(scale)
    out = np.empty((Hq, b, D)); lse = np.empty((Hq, b))
    probs = np.empty((Hq, b, nk)) if return_probs else None
    rc = lib().orc_attention(_dp(q), _dp(k), _dp(v), Hq, Hkv, b, nk, D, ctypes.c_double(scale), _dp(out), _dp(lse),
                             _dp(probs) if return_probs else None)
    _check(rc, "attention")
    return (out, lse, probs) if return_probs else (out, lse)


def scores_logit_mean(q, k, block_off: int, scale: Optional[float] = None, matrix_form: bool = False) -> np.ndarray:
    """Mean-query logit saliency over the candidates (Algorithm 1, steps "Mean(Q_b)" and "MatMul(qbar, K_f^T)"). Returns [Hkv, L-b]."""
    q, k = _f64(q), _f64(k)
    Hq, b, D = q.shape
    Hkv, L, _ = k.shape
    scale = 1.0 / np.sqrt(D) if scale is None else float(scale)
    a = np.empty((Hkv, L - b))
    fn = lib().orc_scores_logit_matrix_mean if matrix_form else lib().orc_scores_logit_mean
    _check(fn(_dp(q), _dp(k), Hq, Hkv, b, L, D, int(block_off), ctypes.c_double(scale), _dp(a)), "scores_logit_mean")
    return a


def scores_prob_mean(probs, n_kv_heads: int, block_off: int) -> np.ndarray:
    """Mean softmax probability per candidate key; probs [Hq,b,L] from attention(..., return_probs=True)."""
    probs = _f64(probs)
    Hq, b, L = probs.shape
    a = np.empty((n_kv_heads, L - b))
    _check(lib().orc_scores_prob_mean(_dp(probs), Hq, n_kv_heads, b, L, int(block_off), _dp(a)), "scores_prob_mean")
    return a


def pool(a, window: int, kind: int = POOL_MAX, seam: int = -1) -> np.ndarray:
    """Key-axis pooling with stride 1 and padding window//2 (Algorithm 1, step "MaxPool1D"). a [Hkv, C]."""
    a = _f64(a)
    out = np.empty_like(a)
    _check(lib().orc_pool(_dp(a), a.shape[0], a.shape[1], int(window), int(kind), int(seam), _dp(out)), "pool")
    return out


def keep_count(seq_len: int, block_len: int, block_off: int, retention: float,
               mode: int = SELECT_JOINT_FLOOR) -> Tuple[int, int, int]:
    """(n_total, n_prefix, n_suffix); quotas are -1 in joint mode (Algorithm 1, step "n <- floor(|I| r)")."""
    n = [ctypes.c_int(0) for _ in range(3)]
    _check(lib().orc_keep_count(int(seq_len), int(block_len), int(block_off), ctypes.c_double(retention), int(mode),
                                *[ctypes.byref(x) for x in n]), "keep_count")
    return n[0].value, n[1].value, n[2].value


def select_topk(x, n: int) -> np.ndarray:
    """Indices of the n largest entries of a 1-D score array, ties to the lowest index, ascending order."""
    x = _f64(x).ravel()
    idx = np.empty(n, dtype=np.int32)
    _check(lib().orc_select_topk(_dp(x), x.size, int(n), idx.ctypes.data_as(ctypes.POINTER(ctypes.c_int32))),
           "select_topk")
    return idx


def gather_rows(src: np.ndarray, idx: np.ndarray) -> np.ndarray:
    """Bit-exact row gather: src [Hkv, L, D] (any dtype), idx [Hkv, n] absolute positions -> [Hkv, n, D]."""
    src = np.ascontiguousarray(src)
    idx = np.ascontiguousarray(idx, dtype=np.int32)
    Hkv, L, D = src.shape
    n = idx.shape[1]
    dst = np.empty((Hkv, n, D), dtype=src.dtype)
    rc = lib().orc_gather_rows(src.ctypes.data_as(ctypes.c_void_p), idx.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)),
                               Hkv, L, n, ctypes.c_size_t(D * src.dtype.itemsize), dst.ctypes.data_as(ctypes.c_void_p))
    _check(rc, "gather_rows")
    return dst


def cache_state(i: int, delay: int = 1) -> int:
    """Cache state of step i within a block: 0 dense, 1 refresh, 2 reuse (Algorithm 2; Algorithm 4 for delay != 1)."""
    return int(lib().orc_cache_state(int(i), int(delay)))


def candidate_positions(seq_len: int, block_len: int, block_off: int) -> np.ndarray:
    """Absolute positions of the candidates K_f = Concat(K[:o], K[o+b:]), in candidate order."""
    return np.concatenate([np.arange(0, block_off), np.arange(block_off + block_len, seq_len)]).astype(np.int32)


# --------------------------------------------------------------------------- Algorithm 1
@dataclass
class RefreshResult:
    out: np.ndarray          # [Hq, b, D]   dense block attention at the refresh step
    lse: np.ndarray          # [Hq, b]
    scores: np.ndarray       # [Hkv, L-b]   saliency a (candidate order)
    pooled: np.ndarray       # [Hkv, L-b]   importance I (candidate order)
    kept_idx: np.ndarray     # [Hkv, n]     absolute positions, ascending
    n_keep: int


def refresh(q, k, v, block_off: int, retention: float, window: int, *, scale: Optional[float] = None,
            score: int = SCORE_LOGIT_MEAN, pool_kind: int = POOL_MAX, select: int = SELECT_JOINT_FLOOR) -> RefreshResult:
    """The refresh step of one layer: dense attention of the block rows over all L keys, then Algorithm 1."""
    q, k, v = _f64(q), _f64(k), _f64(v)
    Hq, b, D = q.shape
    Hkv, L, _ = k.shape
    o = int(block_off)
    C = L - b
    if score == SCORE_PROB_MEAN:
        out, lse, probs = attention(q, k, v, scale, return_probs=True)
        a = scores_prob_mean(probs, Hkv, o)
    else:
        out, lse = attention(q, k, v, scale)
        a = scores_logit_mean(q, k, o, scale)
    n_total, n_pre, n_suf = keep_count(L, b, o, retention, select)
    pos = candidate_positions(L, b, o)
    kept = np.empty((Hkv, n_total), dtype=np.int32)
    if select == SELECT_JOINT_FLOOR:
        pooled = pool(a, window, pool_kind, seam=-1)
        for g in range(Hkv):
            kept[g] = pos[select_topk(pooled[g], n_total)]
    else:
        pooled = pool(a, window, pool_kind, seam=o)
        for g in range(Hkv):
            pre = select_topk(pooled[g, :o], n_pre)
            if select == SELECT_PREFIX_ONLY:
                suf = np.arange(C - o, dtype=np.int32)
            else:
                suf = select_topk(pooled[g, o:], n_suf)
            kept[g] = pos[np.concatenate([pre, suf + o])]
    return RefreshResult(out, lse, a, pooled, kept, n_total)


def sparse_block_attention(q, k_c, v_c, k_n, v_n, scale: Optional[float] = None):
    """Cache-reuse step (Algorithm 3, cache_state 2): attention over Concat(K_c, K_n), Concat(V_c, V_n)."""
    k = np.concatenate([_f64(k_c), _f64(k_n)], axis=1)
    v = np.concatenate([_f64(v_c), _f64(v_n)], axis=1)
    return attention(q, k, v, scale)


def dense_attention(q, k, v, scale: Optional[float] = None, rows: Optional[Sequence[int]] = None):
    """Dense step (Algorithm 3, cache_state 0 and the full-sequence part of cache_state 1): every row of the sequence
    attends to all L keys, no mask. q [Hq,L,D], k/v [Hkv,L,D] -> out [Hq,L,D], lse [Hq,L]. The rows are independent,
    so `rows` (query positions) restricts the work to a sample of them: out [Hq,len(rows),D]."""
    q = _f64(q)
    if rows is not None:
        q = np.ascontiguousarray(q[:, np.asarray(list(rows), dtype=np.int64)])
    return attention(q, k, v, scale)


def positions_to_candidates(kept_idx: np.ndarray, block_len: int, block_off: int) -> np.ndarray:
    """Inverse of the candidate position map for kept absolute positions."""
    kept_idx = np.asarray(kept_idx)
    return np.where(kept_idx < block_off, kept_idx, kept_idx - block_len)

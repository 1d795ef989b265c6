"""Device-memory plumbing around the C ABI: one object per (layer, batch shape) that owns the
compacted cache, the index/score buffers and the workspace (all torch CUDA tensors) and issues the
libsdllm calls in the order of the paper's Algorithm 3. It allocates and passes pointers; every
arithmetic step runs inside libsdllm.
"""
from __future__ import annotations

from typing import Optional

import torch

from . import binding as B

_TORCH_DTYPE = {B.F32: torch.float32, B.BF16: torch.bfloat16}


class LayerCache:
    """Sparse-dLLM cache of one attention layer for one decoding block of a (padded) batch."""

    def __init__(self, *, batch: int, n_q_heads: int, n_kv_heads: int, head_dim: int, seq_len_max: int,
                 block_len: int = 32, dtype: int = B.BF16, retention: float = 0.5, pool_window: int = 3,
                 pool: int = B.POOL_MAX, score: int = B.SCORE_LOGIT_MEAN, select: int = B.SELECT_JOINT_FLOOR,
                 softmax_scale: float = 0.0, n_keep_max: Optional[int] = None, device: str = "cuda:0",
                 share_scratch_with: Optional["LayerCache"] = None, fused_select: bool = True):
        if not torch.cuda.is_available():
            raise RuntimeError("libsdllm needs a CUDA device; there is no CPU path")
        B.lib()
        self.device = torch.device(device)
        self.tdtype = _TORCH_DTYPE[dtype]
        self.fused_select = fused_select    # selection and gather through sdllm_select_compact (else the two separate calls)
        probe = B.make_desc(batch=batch, n_q_heads=n_q_heads, n_kv_heads=n_kv_heads, head_dim=head_dim,
                            seq_len_max=seq_len_max, block_len=block_len, dtype=dtype, retention=retention,
                            pool_window=pool_window, pool=pool, score=score, select=select, softmax_scale=softmax_scale)
        if n_keep_max is None:
            # the count is monotone in the sequence length; per-region rounding adds at most 2
            n_keep_max = B.keep_count(probe, seq_len_max, 0)[0] + (0 if select == B.SELECT_JOINT_FLOOR else 2)
            n_keep_max = min(n_keep_max, seq_len_max - block_len)
        self.n_keep_max = int(n_keep_max)
        self.desc = B.make_desc(batch=batch, n_q_heads=n_q_heads, n_kv_heads=n_kv_heads, head_dim=head_dim,
                                seq_len_max=seq_len_max, block_len=block_len, dtype=dtype, retention=retention,
                                pool_window=pool_window, pool=pool, score=score, select=select,
                                softmax_scale=softmax_scale, n_keep_max=self.n_keep_max)
        dev, rows = self.device, max(self.n_keep_max, 1)
        self.k_c = torch.empty((batch, n_kv_heads, rows, head_dim), dtype=self.tdtype, device=dev)
        self.v_c = torch.empty_like(self.k_c)
        self.kept_idx = torch.empty((batch, n_kv_heads, rows), dtype=torch.int32, device=dev)
        self.kept_cnt = torch.zeros((batch,), dtype=torch.int32, device=dev)
        if share_scratch_with is not None:      # per-call scratch can be shared by layers that run back to back
            self.pooled, self.workspace = share_scratch_with.pooled, share_scratch_with.workspace
        else:
            self.pooled = torch.empty((batch, n_kv_heads, seq_len_max), dtype=torch.float32, device=dev)
            ws = max(B.workspace_bytes(self.desc, op) for op in range(5))
            self.workspace = torch.zeros((max(ws, 256),), dtype=torch.uint8, device=dev)   # status word starts at 0

    # cache_state 1: dense block attention + Algorithm 1
    def refresh(self, q_blk, k, v, seq_len, block_off, out=None, lse=None, stream=None):
        """q_blk [B,Hq,b,D], k/v [B,Hkv,Lmax,D], seq_len/block_off int32 [B] (seq_len may be None)."""
        d = self.desc
        B.refresh_scores(d, q_blk, k, v, seq_len, block_off, out, lse, self.pooled, self.workspace, stream)
        if self.fused_select:
            B.select_compact(d, self.pooled, seq_len, block_off, k, v, self.kept_idx, self.kept_cnt, self.k_c, self.v_c, stream)
        else:
            B.select_topk(d, self.pooled, seq_len, block_off, self.kept_idx, self.kept_cnt, None, stream)
            B.compact_kv(d, k, v, self.kept_idx, self.kept_cnt, self.k_c, self.v_c, stream)
        return out

    # cache_state 2: attention over Concat(K_c, K_n)
    def sparse_step(self, q_blk, k_blk, v_blk, out, stream=None):
        B.sparse_block_attn(self.desc, q_blk, self.k_c, self.v_c, self.kept_cnt, k_blk, v_blk, out, self.workspace, stream)
        return out

    # cache_state 0 (and the full-sequence part of cache_state 1): every row over all keys
    def dense_step(self, q, k, v, seq_len, out, lse=None, stream=None):
        """q/out [B,Hq,Lmax,D], k/v [B,Hkv,Lmax,D]; bf16 only."""
        B.dense_attn(self.desc, q, k, v, seq_len, out, lse, self.workspace, stream)
        return out

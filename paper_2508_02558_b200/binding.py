"""ctypes binding of libsdllm.so: same names as the C ABI (include/sdllm.h), argument marshalling only.

Every step of the path runs inside the CUDA library; nothing here computes. Tensors are passed as
torch tensors (their data_ptr() is taken), raw integer addresses, or None for nullable arguments.
There is no CPU fallback: a missing library raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libsdllm.so")

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT = range(6)
F32, BF16 = 0, 1
SCORE_LOGIT_MEAN, SCORE_PROB_MEAN = 0, 1
POOL_MAX, POOL_AVG = 0, 1
SELECT_JOINT_FLOOR, SELECT_PER_REGION_CEIL, SELECT_PREFIX_ONLY = 0, 1, 2
OP_REFRESH_SCORES, OP_SELECT_TOPK, OP_COMPACT_KV, OP_SPARSE_BLOCK_ATTN, OP_DENSE_ATTN, OP_SELECT_COMPACT = range(6)

EXPORTS = ("sdllm_version", "sdllm_status_string", "sdllm_workspace_bytes", "sdllm_keep_count", "sdllm_cache_state", "sdllm_launch_count",
           "sdllm_plan_describe", "sdllm_read_status",
           "sdllm_refresh_scores", "sdllm_select_topk", "sdllm_compact_kv", "sdllm_sparse_block_attn",
           "sdllm_sparse_block_attn_static", "sdllm_dense_attn", "sdllm_select_compact", "sdllm_tuning_set", "sdllm_tuning_reset")


class Desc(ctypes.Structure):
    """Mirror of `sdllm_desc`."""
    _fields_ = [
        ("struct_size", ctypes.c_uint32), ("batch", ctypes.c_int32), ("n_q_heads", ctypes.c_int32),
        ("n_kv_heads", ctypes.c_int32), ("head_dim", ctypes.c_int32), ("seq_len_max", ctypes.c_int32),
        ("block_len", ctypes.c_int32), ("dtype", ctypes.c_int32), ("softmax_scale", ctypes.c_float),
        ("pool_window", ctypes.c_int32), ("pool", ctypes.c_int32), ("score", ctypes.c_int32),
        ("select", ctypes.c_int32), ("n_keep_max", ctypes.c_int32), ("retention", ctypes.c_double),
        ("q_stride", ctypes.c_int64 * 3), ("kv_stride", ctypes.c_int64 * 3), ("o_stride", ctypes.c_int64 * 3),
        ("c_stride", ctypes.c_int64 * 3), ("blk_stride", ctypes.c_int64 * 3),
    ]


class SdllmError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} (status {status})")


_lib = None


def lib() -> ctypes.CDLL:
    """Load libsdllm.so (built by paper_2508_02558_b200.build.build()); raises if it is missing."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2508_02558_b200.build` "
                               "(there is no fallback path)")
        L = ctypes.CDLL(LIB_PATH)
        vp, i32p, dp = ctypes.c_void_p, ctypes.c_void_p, ctypes.POINTER(Desc)
        L.sdllm_version.restype = ctypes.c_int
        L.sdllm_status_string.restype = ctypes.c_char_p
        L.sdllm_status_string.argtypes = [ctypes.c_int]
        L.sdllm_workspace_bytes.restype = ctypes.c_size_t
        L.sdllm_workspace_bytes.argtypes = [dp, ctypes.c_int]
        L.sdllm_keep_count.restype = ctypes.c_int
        L.sdllm_keep_count.argtypes = [dp, ctypes.c_int32, ctypes.c_int32] + [ctypes.POINTER(ctypes.c_int32)] * 3
        L.sdllm_launch_count.restype = ctypes.c_int32
        L.sdllm_launch_count.argtypes = [ctypes.POINTER(Desc), ctypes.c_int]
        L.sdllm_plan_describe.restype = ctypes.c_int
        L.sdllm_plan_describe.argtypes = [ctypes.POINTER(Desc), ctypes.c_int, ctypes.c_char_p, ctypes.c_size_t]
        L.sdllm_cache_state.restype = ctypes.c_int32
        L.sdllm_cache_state.argtypes = [ctypes.c_int32, ctypes.c_int32]
        L.sdllm_read_status.restype = ctypes.c_int
        L.sdllm_read_status.argtypes = [vp, vp, ctypes.POINTER(ctypes.c_int32)]
        L.sdllm_refresh_scores.restype = ctypes.c_int
        L.sdllm_refresh_scores.argtypes = [dp, vp, vp, vp, i32p, i32p, vp, vp, vp, vp, ctypes.c_size_t, vp]
        L.sdllm_sparse_block_attn_static.restype = ctypes.c_int
        L.sdllm_sparse_block_attn_static.argtypes = [dp, vp, vp, vp, i32p, vp, vp, vp, vp]
        L.sdllm_select_topk.restype = ctypes.c_int
        L.sdllm_select_topk.argtypes = [dp, vp, i32p, i32p, vp, vp, vp, ctypes.c_size_t, vp]
        L.sdllm_compact_kv.restype = ctypes.c_int
        L.sdllm_compact_kv.argtypes = [dp, vp, vp, vp, vp, vp, vp, vp]
        L.sdllm_select_compact.restype = ctypes.c_int
        L.sdllm_select_compact.argtypes = [dp, vp, i32p, i32p, vp, vp, vp, vp, vp, vp, vp]
        L.sdllm_sparse_block_attn.restype = ctypes.c_int
        L.sdllm_sparse_block_attn.argtypes = [dp, vp, vp, vp, vp, vp, vp, vp, vp, ctypes.c_size_t, vp]
        L.sdllm_dense_attn.restype = ctypes.c_int
        L.sdllm_dense_attn.argtypes = [dp, vp, ctypes.POINTER(ctypes.c_int64), vp, vp, i32p, vp, ctypes.POINTER(ctypes.c_int64), vp, vp,
                                       ctypes.c_size_t, vp]
        L.sdllm_tuning_set.restype = ctypes.c_int
        L.sdllm_tuning_set.argtypes = [ctypes.c_char_p, ctypes.c_int64]
        L.sdllm_tuning_reset.restype = None
        L.sdllm_tuning_reset.argtypes = []
        _lib = L
    return _lib


def _ptr(x) -> Optional[int]:
    if x is None:
        return None
    if isinstance(x, int):
        return x
    if isinstance(x, tuple):          # (address, bytes) pair for a workspace
        return x[0]
    return x.data_ptr()


def _nbytes(x) -> int:
    if x is None or isinstance(x, int):
        return 0
    if isinstance(x, tuple):
        return int(x[1])
    return x.numel() * x.element_size()


def _stream(stream) -> Optional[int]:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    return stream if isinstance(stream, int) else stream.cuda_stream


def _check(status: int, where: str):
    if status != OK:
        raise SdllmError(status, where)


def contiguous_strides(heads: int, rows: int, head_dim: int):
    return (heads * rows * head_dim, rows * head_dim, head_dim)


def make_desc(*, batch: int, n_q_heads: int, n_kv_heads: int, head_dim: int, seq_len_max: int, block_len: int,
              dtype: int, retention: float, pool_window: int = 3, n_keep_max: int = 0, softmax_scale: float = 0.0,
              pool: int = POOL_MAX, score: int = SCORE_LOGIT_MEAN, select: int = SELECT_JOINT_FLOOR,
              q_stride: Optional[Sequence[int]] = None, kv_stride: Optional[Sequence[int]] = None,
              o_stride: Optional[Sequence[int]] = None, c_stride: Optional[Sequence[int]] = None,
              blk_stride: Optional[Sequence[int]] = None) -> Desc:
    """Fill a description; missing strides default to dense [B, H, rows, D] layouts."""
    d = Desc()
    d.struct_size = ctypes.sizeof(Desc)
    d.batch, d.n_q_heads, d.n_kv_heads, d.head_dim = batch, n_q_heads, n_kv_heads, head_dim
    d.seq_len_max, d.block_len, d.dtype, d.softmax_scale = seq_len_max, block_len, dtype, softmax_scale
    d.pool_window, d.pool, d.score, d.select = pool_window, pool, score, select
    d.n_keep_max, d.retention = n_keep_max, retention
    d.q_stride[:] = list(q_stride or contiguous_strides(n_q_heads, block_len, head_dim))
    d.kv_stride[:] = list(kv_stride or contiguous_strides(n_kv_heads, seq_len_max, head_dim))
    d.o_stride[:] = list(o_stride or contiguous_strides(n_q_heads, block_len, head_dim))
    d.c_stride[:] = list(c_stride or contiguous_strides(n_kv_heads, max(n_keep_max, 1), head_dim))
    d.blk_stride[:] = list(blk_stride or contiguous_strides(n_kv_heads, block_len, head_dim))
    return d


# ------------------------------------------------------------------------------------------ the C ABI, one to one
def version() -> int:
    return lib().sdllm_version()


def status_string(status: int) -> str:
    return lib().sdllm_status_string(int(status)).decode()


def workspace_bytes(desc: Desc, op: int) -> int:
    return int(lib().sdllm_workspace_bytes(ctypes.byref(desc), int(op)))


def keep_count(desc: Desc, seq_len: int, block_off: int):
    """(n_total, n_prefix, n_suffix) on the host; quotas are -1 when data dependent."""
    n = [ctypes.c_int32(0) for _ in range(3)]
    _check(lib().sdllm_keep_count(ctypes.byref(desc), int(seq_len), int(block_off), *[ctypes.byref(x) for x in n]),
           "sdllm_keep_count")
    return n[0].value, n[1].value, n[2].value


def launch_count(desc: Desc, op: int) -> int:
    return int(lib().sdllm_launch_count(ctypes.byref(desc), int(op)))


def plan_describe(desc: Desc, op: int) -> str:
    buf = ctypes.create_string_buffer(256)
    _check(lib().sdllm_plan_describe(ctypes.byref(desc), int(op), buf, ctypes.c_size_t(256)), "sdllm_plan_describe")
    return buf.value.decode()


def cache_state(step_in_block: int, delay: int = 1) -> int:
    return int(lib().sdllm_cache_state(int(step_in_block), int(delay)))


def read_status(workspace, stream=None) -> int:
    """Device status word of a workspace (0 = no bounded wait ever expired). Synchronises the stream."""
    v = ctypes.c_int32(0)
    st = lib().sdllm_read_status(_ptr(workspace), _stream(stream), ctypes.byref(v))
    if st not in (OK, ERR_TIMEOUT):
        raise SdllmError(st, "sdllm_read_status")
    return v.value


def refresh_scores(desc: Desc, q_blk, k, v, seq_len, block_off, out, lse, pooled_scores, workspace, stream=None):
    _check(lib().sdllm_refresh_scores(ctypes.byref(desc), _ptr(q_blk), _ptr(k), _ptr(v), _ptr(seq_len), _ptr(block_off),
                                      _ptr(out), _ptr(lse), _ptr(pooled_scores), _ptr(workspace), _nbytes(workspace),
                                      _stream(stream)), "sdllm_refresh_scores")


def select_topk(desc: Desc, pooled_scores, seq_len, block_off, kept_idx, kept_cnt, workspace=None, stream=None):
    _check(lib().sdllm_select_topk(ctypes.byref(desc), _ptr(pooled_scores), _ptr(seq_len), _ptr(block_off), _ptr(kept_idx),
                                   _ptr(kept_cnt), _ptr(workspace), _nbytes(workspace), _stream(stream)),
           "sdllm_select_topk")


def compact_kv(desc: Desc, k, v, kept_idx, kept_cnt, k_c, v_c, stream=None):
    _check(lib().sdllm_compact_kv(ctypes.byref(desc), _ptr(k), _ptr(v), _ptr(kept_idx), _ptr(kept_cnt), _ptr(k_c),
                                  _ptr(v_c), _stream(stream)), "sdllm_compact_kv")


def select_compact(desc: Desc, pooled_scores, seq_len, block_off, k, v, kept_idx, kept_cnt, k_c, v_c, stream=None):
    """sdllm_select_topk and sdllm_compact_kv in one call (one launch while a head's candidates fit a CTA)."""
    _check(lib().sdllm_select_compact(ctypes.byref(desc), _ptr(pooled_scores), _ptr(seq_len), _ptr(block_off), _ptr(k), _ptr(v),
                                      _ptr(kept_idx), _ptr(kept_cnt), _ptr(k_c), _ptr(v_c), _stream(stream)),
           "sdllm_select_compact")


def sparse_block_attn(desc: Desc, q_blk, k_c, v_c, kept_cnt, k_blk, v_blk, out, workspace, stream=None):
    _check(lib().sdllm_sparse_block_attn(ctypes.byref(desc), _ptr(q_blk), _ptr(k_c), _ptr(v_c), _ptr(kept_cnt),
                                         _ptr(k_blk), _ptr(v_blk), _ptr(out), _ptr(workspace), _nbytes(workspace),
                                         _stream(stream)), "sdllm_sparse_block_attn")


def sparse_block_attn_static(desc: Desc, q_blk, k_c, v_c, kept_cnt, k_blk, v_blk, out, stream=None):
    """The reuse step without a caller workspace (scratch built into the library; shapes above its 8 MiB are refused)."""
    _check(lib().sdllm_sparse_block_attn_static(ctypes.byref(desc), _ptr(q_blk), _ptr(k_c), _ptr(v_c), _ptr(kept_cnt),
                                                _ptr(k_blk), _ptr(v_blk), _ptr(out), _stream(stream)),
           "sdllm_sparse_block_attn_static")


def dense_attn(desc: Desc, q, k, v, seq_len, out, lse, workspace, stream=None):
    """Full-sequence bidirectional attention; q and out are [B, Hq, seq_len_max, D] tensors whose strides are passed on."""
    qs = (ctypes.c_int64 * 3)(*(q.stride()[:3] if q is not None else (0, 0, 0)))
    os_ = (ctypes.c_int64 * 3)(*(out.stride()[:3] if out is not None else (0, 0, 0)))
    _check(lib().sdllm_dense_attn(ctypes.byref(desc), _ptr(q), qs, _ptr(k), _ptr(v), _ptr(seq_len), _ptr(out), os_, _ptr(lse),
                                  _ptr(workspace), _nbytes(workspace), _stream(stream)), "sdllm_dense_attn")


def tuning_set(name: str, value: int):
    """Override one decision of the launch planner (tuning and test aid) until tuning_reset()."""
    _check(lib().sdllm_tuning_set(name.encode(), int(value)), f"sdllm_tuning_set({name})")


def tuning_reset():
    lib().sdllm_tuning_reset()

"""Helpers of the GPU parity tests: run the CUDA path through the C ABI on host-generated inputs and
compare with the CPU oracle. The CUDA side and the oracle only meet here."""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Optional, Sequence

import numpy as np
import torch

import oracle
from paper_2508_02558_b200 import binding as B
from paper_2508_02558_b200 import workloads as W
from paper_2508_02558_b200.session import LayerCache

DEV = "cuda:0"
TOL = {"f32": (1e-5, 0.0), "bf16": (1e-2, 1e-2)}      # (abs, rel): |gpu - ref| <= abs + rel * |ref|
BAND = 1e-3                                            # kept sets may differ only inside this band around the threshold


def to_dev(x: np.ndarray, dtype: str) -> torch.Tensor:
    """float32 host array (already representable in dtype) -> device tensor of that dtype, bit-exact."""
    t = torch.from_numpy(np.ascontiguousarray(x))
    if dtype == "bf16":
        bits = W.f32_to_bf16_bits(x).reshape(x.shape)
        t = torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16)
    return t.to(DEV)


def to_host_f32(t: torch.Tensor) -> np.ndarray:
    return t.detach().float().cpu().numpy()


def raw_bytes(t: torch.Tensor) -> bytes:
    t = t.detach().contiguous().cpu()
    if t.dtype == torch.bfloat16:
        t = t.view(torch.int16)
    return t.numpy().tobytes()


def assert_close(got: np.ndarray, ref: np.ndarray, dtype: str, what: str):
    a, r = TOL[dtype]
    err = np.abs(got.astype(np.float64) - ref)
    lim = a + r * np.abs(ref)
    bad = err > lim
    assert not bad.any(), f"{what}: {bad.sum()} of {bad.size} outside tolerance, max err {err.max():.3e}"
    # The stated tolerance is loose against outputs that average many small values; what the arithmetic allows
    # (bf16 P and output rounding, fp32 accumulation) is an error of a few percent of the output's own scale.
    scale = np.sqrt(np.mean(np.square(ref))) + 1e-30
    tight = (1e-6 if dtype == "f32" else 1e-2) * np.abs(ref) + (1e-5 if dtype == "f32" else 3e-2) * scale
    worse = err > tight
    assert not worse.any(), f"{what}: {worse.sum()} of {worse.size} beyond the arithmetic's own error, max err {err.max():.3e}, scale {scale:.3e}"


@dataclass
class GpuRefresh:
    cache: LayerCache
    out: np.ndarray
    lse: np.ndarray
    pooled: np.ndarray        # [B, Hkv, Lmax]
    kept_idx: np.ndarray      # [B, Hkv, n_keep_max]
    kept_cnt: np.ndarray      # [B]
    k_dev: torch.Tensor
    v_dev: torch.Tensor


def gpu_refresh(q, k, v, seq_len: Sequence[int], block_off: Sequence[int], dtype: str, retention: float, window: int,
                **policy) -> GpuRefresh:
    """q [B,Hq,b,D], k/v [B,Hkv,Lmax,D] float32 host arrays."""
    Bn, Hq, b, D = q.shape
    Hkv, Lmax = k.shape[1], k.shape[2]
    cache = LayerCache(batch=Bn, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=D, seq_len_max=Lmax, block_len=b,
                       dtype=B.BF16 if dtype == "bf16" else B.F32, retention=retention, pool_window=window, **policy)
    qd, kd, vd = to_dev(q, dtype), to_dev(k, dtype), to_dev(v, dtype)
    sl = torch.tensor(list(seq_len), dtype=torch.int32, device=DEV)
    bo = torch.tensor(list(block_off), dtype=torch.int32, device=DEV)
    out = torch.full((Bn, Hq, b, D), float("nan"), dtype=cache.tdtype, device=DEV)
    lse = torch.full((Bn, Hq, b), float("nan"), dtype=torch.float32, device=DEV)
    cache.kept_idx.fill_(-7)
    cache.k_c.fill_(float("nan")); cache.v_c.fill_(float("nan"))
    cache.refresh(qd, kd, vd, sl, bo, out=out, lse=lse)
    torch.cuda.synchronize()
    assert B.read_status(cache.workspace) == 0, "a bounded device-side wait expired"
    return GpuRefresh(cache, to_host_f32(out), lse.cpu().numpy(), cache.pooled.cpu().numpy(),
                      cache.kept_idx.cpu().numpy(), cache.kept_cnt.cpu().numpy(), kd, vd)


def check_refresh_against_oracle(g: GpuRefresh, q, k, v, seq_len, block_off, dtype, retention, window, *,
                                 heads: Optional[List[int]] = None, select=oracle.SELECT_JOINT_FLOOR,
                                 pool_kind=oracle.POOL_MAX, score_rtol: float = 1e-4, seqs: Optional[List[int]] = None,
                                 score=oracle.SCORE_LOGIT_MEAN):
    """Element-by-element comparison of one refresh (all sequences; optionally a subset of KV heads)."""
    Bn, Hq, b, D = q.shape
    Hkv = k.shape[1]
    G = Hq // Hkv
    stats = {"band_keys": 0, "set_mismatch": 0}
    for i in (range(Bn) if seqs is None else seqs):
        L, o = int(seq_len[i]), int(block_off[i])
        hs = list(range(Hkv)) if heads is None else heads
        qh = np.concatenate([q[i, h * G:(h + 1) * G] for h in hs])
        r = oracle.refresh(qh, k[i, hs, :L], v[i, hs, :L], o, retention, window, select=select, pool_kind=pool_kind,
                           score=score)
        n = r.n_keep
        assert int(g.kept_cnt[i]) == min(n, g.cache.n_keep_max), (g.kept_cnt[i], n)
        pos = oracle.candidate_positions(L, b, o)
        for j, h in enumerate(hs):
            assert_close(g.out[i, h * G:(h + 1) * G], r.out[j * G:(j + 1) * G], dtype, f"refresh out seq {i} head {h}")
            np.testing.assert_allclose(g.lse[i, h * G:(h + 1) * G], r.lse[j * G:(j + 1) * G], rtol=0, atol=1e-4)
            # pooled scores: candidates carry the score, block and padding carry -inf
            pg = g.pooled[i, h]
            scale_ref = max(np.sqrt(np.mean(r.pooled[j] ** 2)), 1e-30)
            np.testing.assert_allclose(pg[pos], r.pooled[j], rtol=0, atol=score_rtol * scale_ref)
            assert np.isneginf(pg[o:o + b]).all() and np.isneginf(pg[L:]).all()
            # kept set: valid, ascending, and equal to the oracle's outside the tie band
            kept = g.kept_idx[i, h]
            cnt = int(g.kept_cnt[i])
            got = kept[:cnt]
            assert (kept[cnt:g.cache.n_keep_max] == -1).all()
            assert (np.diff(got) > 0).all() and (got >= 0).all() and (got < L).all()
            assert not ((got >= o) & (got < o + b)).any()
            want = r.kept_idx[j]
            if not np.array_equal(got, want):
                stats["set_mismatch"] += 1
                diff = np.setxor1d(got, want)
                cand = oracle.positions_to_candidates(diff, b, o)
                _, n_pre, n_suf = oracle.keep_count(L, b, o, retention, select)
                regions = [(0, L - b, n)] if select == oracle.SELECT_JOINT_FLOOR else [(0, o, n_pre), (o, L - b, n_suf)]
                for lo, hi, nr in regions:
                    cr = cand[(cand >= lo) & (cand < hi)]
                    if cr.size == 0:
                        continue
                    assert 0 < nr < hi - lo, "kept sets differ in a region that is kept whole or dropped whole"
                    thr = np.sort(r.pooled[j][lo:hi])[::-1][nr - 1]
                    band = BAND * max(abs(thr), scale_ref)
                    assert (np.abs(r.pooled[j][cr] - thr) <= band).all(), f"kept set differs outside the tie band, seq {i} head {h}"
                stats["band_keys"] += diff.size
    return stats


def check_compaction_bit_exact(g: GpuRefresh, k_bits_src: torch.Tensor, v_bits_src: torch.Tensor):
    """K_c/V_c rows equal the source rows named by the GPU's own kept_idx, byte for byte; the rest is zero."""
    cache = g.cache
    Bn, Hkv = cache.kept_idx.shape[:2]
    kc, vc = cache.k_c.cpu(), cache.v_c.cpu()
    ks, vs = k_bits_src.cpu(), v_bits_src.cpu()
    for i in range(Bn):
        cnt = int(g.kept_cnt[i])
        for h in range(Hkv):
            idx = torch.from_numpy(g.kept_idx[i, h, :cnt].astype(np.int64))
            assert raw_bytes(kc[i, h, :cnt]) == raw_bytes(ks[i, h].index_select(0, idx))
            assert raw_bytes(vc[i, h, :cnt]) == raw_bytes(vs[i, h].index_select(0, idx))
            if cache.n_keep_max > cnt:
                assert not kc[i, h, cnt:cache.n_keep_max].float().abs().sum().item()
                assert not vc[i, h, cnt:cache.n_keep_max].float().abs().sum().item()


def gpu_sparse_step(g: GpuRefresh, q2, kn, vn, dtype: str) -> np.ndarray:
    qd, knd, vnd = to_dev(q2, dtype), to_dev(kn, dtype), to_dev(vn, dtype)
    out = torch.full(q2.shape, float("nan"), dtype=g.cache.tdtype, device=DEV)
    g.cache.sparse_step(qd, knd, vnd, out)
    torch.cuda.synchronize()
    assert B.read_status(g.cache.workspace) == 0, "a bounded device-side wait expired"
    return to_host_f32(out)


def check_sparse_against_oracle(g: GpuRefresh, out_gpu, q2, kn, vn, dtype, heads: Optional[List[int]] = None,
                                seqs: Optional[List[int]] = None):
    """Oracle attention over [K_c ; K_n], with K_c read back from the device (it is bit-exact K[kept_idx])."""
    Bn, Hq, b, D = q2.shape
    Hkv = kn.shape[1]
    G = Hq // Hkv
    for i in (range(Bn) if seqs is None else seqs):
        cnt = int(g.kept_cnt[i])
        hs = list(range(Hkv)) if heads is None else heads
        qh = np.concatenate([q2[i, h * G:(h + 1) * G] for h in hs])
        kc, vc = to_host_f32(g.cache.k_c[i, hs, :cnt]), to_host_f32(g.cache.v_c[i, hs, :cnt])
        ref, _ = oracle.sparse_block_attention(qh, kc, vc, kn[i, hs], vn[i, hs])
        for j, h in enumerate(hs):
            assert_close(out_gpu[i, h * G:(h + 1) * G], ref[j * G:(j + 1) * G], dtype, f"sparse out seq {i} head {h}")


def gpu_dense(q, k, v, seq_len: Optional[Sequence[int]], dtype: str = "bf16", want_lse: bool = True):
    """Dense step through the C ABI. q [B,Hq,Lmax,D], k/v [B,Hkv,Lmax,D] float32 host arrays -> (out, lse) with NaN
    wherever the call did not write."""
    Bn, Hq, Lmax, D = q.shape
    Hkv = k.shape[1]
    d = B.make_desc(batch=Bn, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=D, seq_len_max=Lmax, block_len=min(32, Lmax),
                    dtype=B.BF16 if dtype == "bf16" else B.F32, retention=0.5)
    qd, kd, vd = to_dev(q, dtype), to_dev(k, dtype), to_dev(v, dtype)
    sl = None if seq_len is None else torch.tensor(list(seq_len), dtype=torch.int32, device=DEV)
    out = torch.full((Bn, Hq, Lmax, D), float("nan"), dtype=qd.dtype, device=DEV)
    lse = torch.full((Bn, Hq, Lmax), float("nan"), dtype=torch.float32, device=DEV) if want_lse else None
    ws = torch.zeros((max(B.workspace_bytes(d, B.OP_DENSE_ATTN), 256),), dtype=torch.uint8, device=DEV)
    torch.cuda.synchronize()
    for _ in range(2):               # the second call runs on the counters the first one left behind
        B.dense_attn(d, qd, kd, vd, sl, out, lse, ws)
    torch.cuda.synchronize()
    assert B.read_status(ws) == 0, "a bounded device-side wait expired"
    return to_host_f32(out), (lse.cpu().numpy() if want_lse else None)


def check_dense_against_oracle(out, lse, q, k, v, seq_len: Optional[Sequence[int]], rows=None, heads=None):
    """Element by element on the rows t < seq_len[i] (all of them, or the sample `rows`); rows past the length must
    not have been written."""
    Bn, Hq, Lmax, D = q.shape
    Hkv = k.shape[1]
    G = Hq // Hkv
    for i in range(Bn):
        L = Lmax if seq_len is None else int(seq_len[i])
        assert np.isnan(out[i, :, L:]).all(), f"dense out seq {i}: rows past the length were written"
        if L == 0:
            continue
        rs = list(range(L)) if rows is None else [t for t in rows if t < L]
        for g in (range(Hkv) if heads is None else heads):
            ref, ref_lse = oracle.dense_attention(q[i, g * G:(g + 1) * G, :L], k[i, g:g + 1, :L], v[i, g:g + 1, :L], rows=rs)
            assert_close(out[i, g * G:(g + 1) * G][:, rs], ref, "bf16", f"dense out seq {i} kv head {g}")
            if lse is not None:
                np.testing.assert_allclose(lse[i, g * G:(g + 1) * G][:, rs], ref_lse, atol=1e-4, rtol=0,
                                           err_msg=f"dense lse seq {i} kv head {g}")

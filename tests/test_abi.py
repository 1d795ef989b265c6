"""Host-side checks of the C ABI that need no GPU: the library loads, exports every symbol the header
declares, and its host-only entry points (counts, schedule, workspace sizing, argument validation) behave."""
import ctypes
import os
import re

import pytest

from paper_2508_02558_b200 import binding as B
from paper_2508_02558_b200 import build as libbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    libbuild.build()


def _desc(**kw):
    base = dict(batch=1, n_q_heads=32, n_kv_heads=32, head_dim=128, seq_len_max=1280, block_len=32, dtype=B.BF16,
                retention=0.5, pool_window=3, n_keep_max=624)
    base.update(kw)
    return B.make_desc(**base)


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "sdllm.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(sdllm_[a-z_]+)\s*\(", header))
    assert declared == set(B.EXPORTS)
    L = ctypes.CDLL(B.LIB_PATH)
    for name in declared:
        assert hasattr(L, name), name
    assert B.version() == 100
    assert ctypes.sizeof(B.Desc) == 64 + 5 * 24


def test_status_strings():
    assert B.status_string(B.OK) == "ok"
    assert len({B.status_string(s) for s in range(6)}) == 6


def test_keep_count_matches_golden_table():
    rows = [l.split("#")[0].split() for l in open(os.path.join(ROOT, "tests", "golden", "keep_counts.txt"))
            if l.split("#")[0].strip()]
    for L, b, o, r, mode, n_total, n_pre, n_suf in rows:
        d = _desc(seq_len_max=int(L), block_len=int(b), retention=float(r), select=int(mode), n_q_heads=4, n_kv_heads=4)
        assert B.keep_count(d, int(L), int(o)) == (int(n_total), int(n_pre), int(n_suf))
    with pytest.raises(B.SdllmError):
        B.keep_count(_desc(), 1280, 1260)


def test_cache_state_schedule():
    assert [B.cache_state(i) for i in range(5)] == [0, 1, 2, 2, 2]             # Algorithm 2
    assert [B.cache_state(i, 3) for i in range(6)] == [0, 0, 0, 1, 2, 2]       # Algorithm 4
    assert [B.cache_state(i, 0) for i in range(3)] == [1, 2, 2]


def test_workspace_sizes():
    d = _desc()
    ws_r, ws_s = B.workspace_bytes(d, B.OP_REFRESH_SCORES), B.workspace_bytes(d, B.OP_SPARSE_BLOCK_ATTN)
    assert ws_r >= 32 * 1280 * 4 and ws_s > 0 and ws_r % 256 == 0
    assert B.workspace_bytes(d, B.OP_SELECT_TOPK) == 0 and B.workspace_bytes(d, B.OP_COMPACT_KV) == 0
    assert B.workspace_bytes(_desc(pool_window=4), B.OP_REFRESH_SCORES) == 0      # invalid description
    big = _desc(batch=16, seq_len_max=4352, n_keep_max=2160)
    assert B.workspace_bytes(big, B.OP_REFRESH_SCORES) >= 16 * 32 * 4352 * 4


def test_plan_description_is_host_only_and_checks_its_arguments():
    """Which kernel a shape gets depends on the device (without a Blackwell GPU the planner falls back to the cp.async
    kernels); the names on a B200 are checked by the GPU tests. Here: a name comes back, and bad arguments are refused."""
    assert B.plan_describe(_desc(), B.OP_SPARSE_BLOCK_ATTN).startswith("attn_")
    assert B.plan_describe(_desc(dtype=B.F32), B.OP_REFRESH_SCORES).startswith("attn_f32_kernel ")
    with pytest.raises(B.SdllmError) as e:
        B.plan_describe(_desc(), B.OP_SELECT_TOPK)
    assert e.value.status == B.ERR_INVALID_ARG
    with pytest.raises(B.SdllmError) as e:
        B.plan_describe(_desc(pool_window=2), B.OP_REFRESH_SCORES)
    assert e.value.status == B.ERR_INVALID_ARG
    assert B.lib().sdllm_plan_describe(__import__("ctypes").byref(_desc()), B.OP_REFRESH_SCORES, None, 0) == B.ERR_INVALID_ARG


@pytest.mark.parametrize("bad,status", [
    (dict(pool_window=2), B.ERR_INVALID_ARG), (dict(retention=1.5), B.ERR_INVALID_ARG),
    (dict(n_q_heads=30), B.ERR_INVALID_ARG), (dict(dtype=7), B.ERR_INVALID_ARG),
    (dict(head_dim=96), B.ERR_UNSUPPORTED), (dict(n_kv_heads=1, block_len=32), B.ERR_UNSUPPORTED),
    (dict(kv_stride=(1, 2, 3)), B.ERR_INVALID_ARG), (dict(softmax_scale=-1.0), B.ERR_INVALID_ARG),
    (dict(score=B.SCORE_PROB_MEAN, dtype=B.F32), B.ERR_UNSUPPORTED),
])
def test_bad_descriptions_are_rejected_before_any_launch(bad, status):
    d = _desc(**bad)
    fake = 0x1000   # never dereferenced: validation fails first
    for call in (lambda: B.refresh_scores(d, fake, fake, fake, None, fake, fake, None, fake, (fake, 1 << 30), stream=0),
                 lambda: B.select_topk(d, fake, None, fake, fake, fake, None, stream=0),
                 lambda: B.compact_kv(d, fake, fake, fake, fake, fake, fake, stream=0),
                 lambda: B.sparse_block_attn(d, fake, fake, fake, fake, fake, fake, fake, (fake, 1 << 30), stream=0)):
        with pytest.raises(B.SdllmError) as e:
            call()
        assert e.value.status == status


def test_null_misaligned_and_workspace_errors():
    d = _desc()
    a = 0x1000
    with pytest.raises(B.SdllmError) as e:
        B.refresh_scores(d, None, a, a, None, a, a, None, a, (a, 1 << 30), stream=0)
    assert e.value.status == B.ERR_INVALID_ARG
    with pytest.raises(B.SdllmError) as e:
        B.refresh_scores(d, a + 8, a, a, None, a, a, None, a, (a, 1 << 30), stream=0)
    assert e.value.status == B.ERR_INVALID_ARG
    for ws in (None, (a, 16), (a + 64, 1 << 30)):      # missing, too small, not 256-byte aligned
        with pytest.raises(B.SdllmError) as e:
            B.refresh_scores(d, a, a, a, None, a, a, None, a, ws, stream=0)
        assert e.value.status == B.ERR_WORKSPACE
    with pytest.raises(B.SdllmError) as e:
        B.sparse_block_attn(d, a, a, a, a, a, a, None, (a, 1 << 30), stream=0)
    assert e.value.status == B.ERR_INVALID_ARG

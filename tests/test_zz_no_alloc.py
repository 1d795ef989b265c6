"""The reuse step without a caller workspace: `sdllm_sparse_block_attn_static` against `sdllm_sparse_block_attn`.

Some hosts of the library (a server running under a fixed memory plan, a plug-in whose host owns the allocator)
may not allocate device memory once they run, so they cannot provide the workspace the regular call needs. The
static variant keeps that scratch inside the library image. This file checks, through the C ABI and on two calls
in a row (the second one finds whatever the first left in the shared scratch), that both calls give the same
output. It is collected last on purpose: a run that stops at the first failure has then run everything else."""
import numpy as np
import pytest
import torch

from paper_2508_02558_b200 import binding as B
from paper_2508_02558_b200 import build as libbuild
from paper_2508_02558_b200 import workloads as W

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    libbuild.build()


def _bf16(x):
    return torch.from_numpy(W.f32_to_bf16_bits(x).reshape(x.shape).view(np.int16)).view(torch.bfloat16).cuda()


@pytest.mark.parametrize("Hq,Hkv,n_keep,cnt", [(8, 8, 700, 700), (8, 2, 300, 211)])
def test_static_scratch_variant_matches_the_workspace_variant_twice(Hq, Hkv, n_keep, cnt):
    rng = np.random.default_rng(31)
    b, D = 32, 128
    d = B.make_desc(batch=1, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=D, seq_len_max=n_keep + b, block_len=b,
                    dtype=B.BF16, retention=0.5, n_keep_max=n_keep)
    mk = lambda *shape: _bf16((rng.standard_normal(shape) / np.sqrt(D)).astype(np.float32))
    k_c, v_c = mk(1, Hkv, n_keep, D), mk(1, Hkv, n_keep, D)
    kept = torch.tensor([cnt], dtype=torch.int32, device="cuda")
    ws = torch.zeros((max(B.workspace_bytes(d, B.OP_SPARSE_BLOCK_ATTN), 256),), dtype=torch.uint8, device="cuda")
    for call in range(2):                      # fresh block rows each time, as in consecutive denoising steps
        q, k_n, v_n = mk(1, Hq, b, D), mk(1, Hkv, b, D), mk(1, Hkv, b, D)
        want = torch.full((1, Hq, b, D), float("nan"), dtype=torch.bfloat16, device="cuda")
        got = torch.full_like(want, float("nan"))
        B.sparse_block_attn(d, q, k_c, v_c, kept, k_n, v_n, want, ws)
        B.sparse_block_attn_static(d, q, k_c, v_c, kept, k_n, v_n, got)
        torch.cuda.synchronize()
        assert B.read_status(ws) == 0
        w, g = want.float().cpu().numpy(), got.float().cpu().numpy()
        assert np.isfinite(g).all()
        assert (np.abs(g - w) <= 1e-2 + 1e-2 * np.abs(w)).all(), f"call {call}: max diff {np.abs(g - w).max():.3e}"
        np.testing.assert_array_equal(g, w)     # same kernels, same plan: the outputs are in fact identical


def test_static_scratch_variant_refuses_shapes_beyond_its_scratch():
    # a long-context GQA layer: few KV heads, so many key splits, whose partials need more than the built-in 8 MiB
    d = B.make_desc(batch=1, n_q_heads=32, n_kv_heads=8, head_dim=128, seq_len_max=32768, block_len=32, dtype=B.BF16,
                    retention=0.5, n_keep_max=16368)
    assert B.workspace_bytes(d, B.OP_SPARSE_BLOCK_ATTN) > (8 << 20)
    a = 0x1000      # never dereferenced: the size check comes first
    with pytest.raises(B.SdllmError) as e:
        B.sparse_block_attn_static(d, a, a, a, a, a, a, a, stream=0)
    assert e.value.status == B.ERR_WORKSPACE

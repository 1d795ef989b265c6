"""The reuse step without a caller workspace: `sdllm_sparse_block_attn_static` against `sdllm_sparse_block_attn`
and against the CPU oracle.

Some hosts of the library (a server running under a fixed memory plan, a plug-in whose host owns the allocator)
may not allocate device memory once they run, so they cannot provide the workspace the regular call needs. The
static variant keeps that scratch inside the library image. This file checks, through the C ABI and on two calls
in a row (the second one finds whatever the first left in the shared scratch), that both calls give the same
output and that this output is the oracle's. One of the shapes is planned so that its key splits leave partials in
the scratch and meet through the completion counters, the part of the scratch that has to start at zero.
It is collected last on purpose: a run that stops at the first failure has then run everything else."""
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


def _bf16_host(rng, shape, D):
    """Host values already representable in bf16, so the oracle and the device see the same numbers."""
    x = (rng.standard_normal(shape) / np.sqrt(D)).astype(np.float32)
    return W.bf16_bits_to_f32(W.f32_to_bf16_bits(x)).reshape(shape)


def _dev(x):
    return torch.from_numpy(W.f32_to_bf16_bits(x).reshape(x.shape).view(np.int16)).view(torch.bfloat16).cuda()


@pytest.mark.parametrize("Hq,Hkv,n_keep,cnt,plan", [
    (8, 8, 700, 700, {}),                         # few query rows per head: the splits merge inside their cluster, scratch = status word
    (8, 2, 300, 211, dict(kernel=3)),             # grouped heads on the key-row kernel: four softmax warpgroups share every tile
    (8, 2, 1500, 1333, dict(kernel=2, cluster=0)),          # key splits leave partials in the scratch; the last CTA of a head merges them (counters)
])
def test_static_scratch_variant_matches_the_workspace_variant_and_the_oracle_twice(Hq, Hkv, n_keep, cnt, plan, tuning):
    import parity_util as U
    tuning(**plan)
    rng = np.random.default_rng(31)
    b, D, G = 32, 128, Hq // Hkv
    d = B.make_desc(batch=1, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=D, seq_len_max=n_keep + b, block_len=b,
                    dtype=B.BF16, retention=0.5, n_keep_max=n_keep)
    k_c, v_c = _bf16_host(rng, (1, Hkv, n_keep, D), D), _bf16_host(rng, (1, Hkv, n_keep, D), D)
    k_cd, v_cd = _dev(k_c), _dev(v_c)
    kept = torch.tensor([cnt], dtype=torch.int32, device="cuda")
    ws_bytes = B.workspace_bytes(d, B.OP_SPARSE_BLOCK_ATTN)
    if plan.get("kernel") == 2:
        assert ws_bytes > 4096, "this case is meant to leave split partials in the scratch"
    ws = torch.zeros((max(ws_bytes, 256),), dtype=torch.uint8, device="cuda")
    for call in range(2):                      # fresh block rows each time, as in consecutive denoising steps
        q, k_n, v_n = _bf16_host(rng, (1, Hq, b, D), D), _bf16_host(rng, (1, Hkv, b, D), D), _bf16_host(rng, (1, Hkv, b, D), D)
        qd, k_nd, v_nd = _dev(q), _dev(k_n), _dev(v_n)
        want = torch.full((1, Hq, b, D), float("nan"), dtype=torch.bfloat16, device="cuda")
        got = torch.full_like(want, float("nan"))
        B.sparse_block_attn(d, qd, k_cd, v_cd, kept, k_nd, v_nd, want, ws)
        B.sparse_block_attn_static(d, qd, k_cd, v_cd, kept, k_nd, v_nd, got)
        torch.cuda.synchronize()
        assert B.read_status(ws) == 0
        w, g = want.float().cpu().numpy(), got.float().cpu().numpy()
        assert np.isfinite(g).all()
        assert (np.abs(g - w) <= 1e-2 + 1e-2 * np.abs(w)).all(), f"call {call}: max diff {np.abs(g - w).max():.3e}"
        np.testing.assert_array_equal(g, w)     # same kernels, same plan: the outputs are in fact identical
        ref, _ = oracle.sparse_block_attention(q[0], k_c[0, :, :cnt], v_c[0, :, :cnt], k_n[0], v_n[0])
        for h in range(Hkv):
            U.assert_close(g[0, h * G:(h + 1) * G], ref[h * G:(h + 1) * G], "bf16", f"static call {call} kv head {h}")


def test_static_scratch_variant_refuses_shapes_beyond_its_scratch():
    # a long-context GQA layer: few KV heads, so many key splits, whose partials need more than the built-in 8 MiB
    d = B.make_desc(batch=1, n_q_heads=32, n_kv_heads=8, head_dim=128, seq_len_max=32768, block_len=32, dtype=B.BF16,
                    retention=0.5, n_keep_max=16368)
    assert B.workspace_bytes(d, B.OP_SPARSE_BLOCK_ATTN) > (8 << 20)
    # real device buffers of the right sizes: if the size check ever moved behind the launch, the call would compute
    # something instead of touching memory it does not own
    kc = torch.zeros((1, 8, 16368, 128), dtype=torch.bfloat16, device="cuda")
    vc = torch.zeros_like(kc)
    q = torch.zeros((1, 32, 32, 128), dtype=torch.bfloat16, device="cuda")
    kn = torch.zeros((1, 8, 32, 128), dtype=torch.bfloat16, device="cuda")
    cnt = torch.zeros((1,), dtype=torch.int32, device="cuda")
    with pytest.raises(B.SdllmError) as e:
        B.sparse_block_attn_static(d, q, kc, vc, cnt, kn, kn, torch.empty_like(q))
    assert e.value.status == B.ERR_WORKSPACE

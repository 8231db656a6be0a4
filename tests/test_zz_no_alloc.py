"""adsa_decode_attn_static: attention for hosts that cannot allocate device memory.

A serving loop with a frozen memory plan, a plugin interface that forbids the allocation calls, or a
process whose device memory belongs to a pool cannot give a context its workspace.  The entry point
tested here needs none: its split-reduction scratch is a fixed array inside the library.  The test
feeds the same rows to it and to the context-based adsa_sparse_decode_attn (budget covering the whole
cache, so every row is retained) and compares the outputs, twice in a row, because the scratch is
shared between calls and keeps what the previous call left.

This file sorts last on purpose: a run that stops at the first failure has then already run
every other test.
"""
import numpy as np
import pytest
import torch

from adsa_workloads import get_workload, layer_step_qkv, prefix_kv
from adsa_workloads.configs import Workload

pytestmark = pytest.mark.gpu

OUT_MAX_ABS = 2e-2       # the tolerances of the parity tests (bf16 output)
OUT_MEAN_ABS = 2e-3
OUT_F32_MAX_ABS = 1e-4


def _dev(bits):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).to("cuda:0").view(torch.bfloat16)


def _both_paths(w, n_rows, seed, step):
    """Outputs (bf16, f32) of the context path and of the static path on the same rows."""
    import paper_2506_18226_b200 as A
    S, d = w.streams_per_layer, w.head_dim
    stride = (d + 7) // 8 * 8
    rng = np.random.default_rng(seed)
    kb = rng.standard_normal((w.batch, w.n_heads, n_rows, d)).astype(np.float32)
    vb = rng.standard_normal((w.batch, w.n_heads, n_rows, d)).astype(np.float32)
    k, v = torch.from_numpy(kb).to("cuda:0").bfloat16(), torch.from_numpy(vb).to("cuda:0").bfloat16()
    qb, knb, vnb = layer_step_qkv(w, seed, 0, step)
    q, kn, vn = _dev(qb), _dev(knb), _dev(vnb)

    eng = A.AdsaEngine(n_layers=1, batch=w.batch, n_heads=w.n_heads, head_dim=d, n_text=n_rows, grid_h=w.grid_h,
                       grid_w=w.grid_w, max_rows_per_stream=n_rows + 1, page_rows=16)
    eng.prefill_rows(0, k, v, 0)
    ref16 = torch.zeros((S, d), dtype=torch.bfloat16, device="cuda:0")
    ref32 = torch.zeros((S, d), dtype=torch.float32, device="cuda:0")
    eng.score(0, n_rows)
    eng.select(0, n_rows, n_rows + 1)                      # budget covers everything: all rows retained
    eng.sparse_decode_attn(0, n_rows, q, kn, vn, ref16, ref32)
    assert eng.get_status()[0] == 0

    # dense rows for the static path: [streams][max_rows][row_stride], stride padded with junk that must be ignored
    max_rows = n_rows + 3
    kd = torch.full((S, max_rows, stride), 7.0, dtype=torch.bfloat16, device="cuda:0")
    vd = torch.full((S, max_rows, stride), -5.0, dtype=torch.bfloat16, device="cuda:0")
    kd[:, :n_rows, :d] = k.reshape(S, n_rows, d)
    vd[:, :n_rows, :d] = v.reshape(S, n_rows, d)
    n = torch.full((S,), n_rows, dtype=torch.int32, device="cuda:0")
    outs = []
    for _ in range(2):                                      # two calls in a row share the scratch
        o16 = torch.zeros((S, d), dtype=torch.bfloat16, device="cuda:0")
        o32 = torch.zeros((S, d), dtype=torch.float32, device="cuda:0")
        A.decode_attn_static(q.reshape(S, d), kd, vd, n, kn.reshape(S, d), vn.reshape(S, d), o16, o32, head_dim=d)
        torch.cuda.synchronize()
        outs.append((o16, o32))
    return (ref16, ref32), outs


@pytest.mark.parametrize("d,n_rows,batch,heads", [
    (64, 700, 2, 12),      # several chunks per stream
    (100, 333, 1, 5),      # padded row stride, ragged tail
    (64, 40, 1, 3),        # a single chunk: no partial states at all
])
def test_static_scratch_attention_matches_context_attention(d, n_rows, batch, heads):
    w = Workload("static", 77, 1, batch, heads, d, 0, 4, 4, 1.0, 1.0)
    (ref16, ref32), outs = _both_paths(w, n_rows, seed=3, step=1)
    for o16, o32 in outs:
        e16 = (o16.float() - ref16.float()).abs()
        e32 = (o32 - ref32).abs()
        assert e16.max().item() <= OUT_MAX_ABS and e16.mean().item() <= OUT_MEAN_ABS
        assert e32.max().item() <= OUT_F32_MAX_ABS * max(1.0, ref32.abs().max().item())
    assert torch.equal(outs[0][0], outs[1][0]) and torch.equal(outs[0][1], outs[1][1])


def test_sizes_beyond_the_built_in_scratch_are_refused():
    import paper_2506_18226_b200 as A
    d = 64
    q = torch.zeros((4097, d), dtype=torch.bfloat16, device="cuda:0")
    k = torch.zeros((4097, 1, d), dtype=torch.bfloat16, device="cuda:0")
    n = torch.zeros(4097, dtype=torch.int32, device="cuda:0")
    out = torch.zeros((4097, d), dtype=torch.bfloat16, device="cuda:0")
    with pytest.raises(A.AdsaError) as e:
        A.decode_attn_static(q, k, k, n, q, q, out)
    assert e.value.status == A.binding.ENOMEM

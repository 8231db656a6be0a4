"""adsa_decode_attn_static: attention for hosts that cannot allocate device memory.

A serving loop with a frozen memory plan, a plugin interface that forbids the allocation calls, or a
process whose device memory belongs to a pool cannot give a context its workspace.  The entry point
tested here needs none: its split-reduction scratch is a fixed array inside the library.  The tests
feed the same rows to it, to the CPU oracle's attention and to the context-based
adsa_sparse_decode_attn (budget covering the whole cache, so every row is retained) and compare the
outputs, twice in a row, because the scratch is shared between calls and keeps what the previous
call left.
"""
import numpy as np
import pytest
import torch

from adsa_workloads import bf16_bits_to_f32, f32_to_bf16_bits, layer_step_qkv
from adsa_workloads.configs import Workload

pytestmark = pytest.mark.gpu

OUT_MAX_ABS = 2e-2       # the tolerances of the parity tests (bf16 output)
OUT_MEAN_ABS = 2e-3
OUT_F32_MAX_ABS = 1e-4


def _dev(bits):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).to("cuda:0").view(torch.bfloat16)


def _rows(seed, S, n_rows, d):
    """Seeded bf16 K and V rows [S, n_rows, d] as bit patterns."""
    rng = np.random.default_rng(seed)
    return (f32_to_bf16_bits(rng.standard_normal((S, n_rows, d)).astype(np.float32)),
            f32_to_bf16_bits(rng.standard_normal((S, n_rows, d)).astype(np.float32)))


def _static_tensors(kb, vb, n_each, qb, knb, vnb, d):
    """Device tensors for the static entry point: rows padded to the row stride with junk that must be ignored."""
    S, n_rows = kb.shape[0], kb.shape[1]
    stride = (d + 7) // 8 * 8
    max_rows = n_rows + 3
    kd = torch.full((S, max_rows, stride), 7.0, dtype=torch.bfloat16, device="cuda:0")
    vd = torch.full((S, max_rows, stride), -5.0, dtype=torch.bfloat16, device="cuda:0")
    kd[:, :n_rows, :d] = _dev(kb)
    vd[:, :n_rows, :d] = _dev(vb)
    n = torch.from_numpy(np.asarray(n_each, dtype=np.int32)).to("cuda:0")
    q, kn, vn = _dev(qb).reshape(S, d), _dev(knb).reshape(S, d), _dev(vnb).reshape(S, d)
    return q, kd, vd, n, kn, vn


def _static_call(A, kb, vb, n_each, qb, knb, vnb, d, repeats=2):
    q, kd, vd, n, kn, vn = _static_tensors(kb, vb, n_each, qb, knb, vnb, d)
    S = kb.shape[0]
    outs = []
    for _ in range(repeats):                                # calls in a row share the scratch
        o16 = torch.zeros((S, d), dtype=torch.bfloat16, device="cuda:0")
        o32 = torch.zeros((S, d), dtype=torch.float32, device="cuda:0")
        A.decode_attn_static(q, kd, vd, n, kn, vn, o16, o32, head_dim=d)
        torch.cuda.synchronize()
        outs.append((o16, o32))
    return outs


def _oracle_attend(kb, vb, n_each, qb, knb, vnb, d):
    """The oracle's attention over each stream's first n rows and the new row (float64)."""
    from oracle import adsa_oracle as orc
    S = kb.shape[0]
    kf, vf = bf16_bits_to_f32(kb), bf16_bits_to_f32(vb)
    qf, knf, vnf = (bf16_bits_to_f32(x).reshape(S, d) for x in (qb, knb, vnb))
    want = np.zeros((S, d))
    for s in range(S):
        n = int(n_each[s])
        want[s], _ = orc.attend(qf[s], np.concatenate([kf[s, :n], knf[s:s + 1]]), np.concatenate([vf[s, :n], vnf[s:s + 1]]))
    return want


@pytest.mark.parametrize("d,n_rows,batch,heads", [
    (64, 700, 2, 12),      # several chunks per stream
    (100, 333, 1, 5),      # padded row stride, ragged tail
    (64, 40, 1, 3),        # a single chunk: no partial states at all
])
def test_static_scratch_attention_matches_oracle_and_context_attention(d, n_rows, batch, heads):
    import paper_2506_18226_b200 as A
    w = Workload("static", 77, 1, batch, heads, d, 0, 4, 4, 1.0, 1.0)
    S = w.streams_per_layer
    kb, vb = _rows(3, S, n_rows, d)
    qb, knb, vnb = layer_step_qkv(w, 3, 0, 1)
    n_each = np.full(S, n_rows)
    outs = _static_call(A, kb, vb, n_each, qb, knb, vnb, d)
    want = _oracle_attend(kb, vb, n_each, qb, knb, vnb, d)

    # the context path on the same rows
    eng = A.AdsaEngine(n_layers=1, batch=batch, n_heads=heads, head_dim=d, n_text=n_rows, grid_h=4, grid_w=4,
                       max_rows_per_stream=n_rows + 1, page_rows=16)
    eng.prefill_rows(0, _dev(kb).reshape(batch, heads, n_rows, d), _dev(vb).reshape(batch, heads, n_rows, d), 0)
    ref16 = torch.zeros((S, d), dtype=torch.bfloat16, device="cuda:0")
    ref32 = torch.zeros((S, d), dtype=torch.float32, device="cuda:0")
    eng.score(0, n_rows)
    eng.select(0, n_rows, n_rows + 1)                      # budget covers everything: all rows retained
    eng.sparse_decode_attn(0, n_rows, _dev(qb), _dev(knb), _dev(vnb), ref16, ref32)
    assert eng.get_status()[0] == 0

    scale = max(1.0, float(np.abs(want).max()))
    for o16, o32 in outs:
        e16 = np.abs(o16.float().cpu().numpy() - want)
        e32 = np.abs(o32.cpu().numpy().astype(np.float64) - want)
        assert e16.max() <= OUT_MAX_ABS and e16.mean() <= OUT_MEAN_ABS
        assert e32.max() <= OUT_F32_MAX_ABS * scale
        k16 = (o16.float() - ref16.float()).abs()
        assert k16.max().item() <= OUT_MAX_ABS and k16.mean().item() <= OUT_MEAN_ABS
        assert (o32 - ref32).abs().max().item() <= OUT_F32_MAX_ABS * scale
    assert torch.equal(outs[0][0], outs[1][0]) and torch.equal(outs[0][1], outs[1][1])


def test_ragged_row_counts_and_nothing_allocated():
    """Streams of different lengths, empty ones among them (attention over the new row alone returns
    v_new), against the oracle; and the device's free memory is the same before and after the calls."""
    import paper_2506_18226_b200 as A
    d, S, n_rows = 64, 9, 300
    w = Workload("static-ragged", 78, 1, 1, S, d, 0, 4, 4, 1.0, 1.0)
    kb, vb = _rows(5, S, n_rows, d)
    qb, knb, vnb = layer_step_qkv(w, 5, 0, 2)
    n_each = np.array([0, 1, 31, 32, 33, 64, 199, 300, 0])
    q, kd, vd, n, kn, vn = _static_tensors(kb, vb, n_each, qb, knb, vnb, d)
    outs = [(torch.zeros((S, d), dtype=torch.bfloat16, device="cuda:0"), torch.zeros((S, d), dtype=torch.float32, device="cuda:0"))
            for _ in range(3)]
    A.decode_attn_static(q, kd, vd, n, kn, vn, *outs[0], head_dim=d)  # first use on this device: address look-up
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    for o16, o32 in outs[1:]:                                         # every tensor exists already: the calls add nothing
        A.decode_attn_static(q, kd, vd, n, kn, vn, o16, o32, head_dim=d)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before
    want = _oracle_attend(kb, vb, n_each, qb, knb, vnb, d)
    for o16, o32 in outs:
        assert np.abs(o16.float().cpu().numpy() - want).max() <= OUT_MAX_ABS
        assert np.abs(o32.cpu().numpy() - want).max() <= OUT_F32_MAX_ABS * max(1.0, float(np.abs(want).max()))
        assert torch.equal(o32, outs[0][1]) and torch.equal(o16, outs[0][0])
    vnf = bf16_bits_to_f32(vnb).reshape(S, d)
    for s in (0, 8):
        assert np.array_equal(outs[0][1][s].cpu().numpy(), vnf[s])


def test_many_wide_streams_fall_back_to_one_chunk():
    """4096 streams of 256-element rows: the partial states of even one split per stream do not fit the
    built-in array, so each stream is served by a single chunk, which needs none."""
    import paper_2506_18226_b200 as A
    d, S, n_rows = 256, 4096, 5
    w = Workload("static-wide", 79, 1, 1, S, d, 0, 4, 4, 1.0, 1.0)
    kb, vb = _rows(6, S, n_rows, d)
    qb, knb, vnb = layer_step_qkv(w, 6, 0, 3)
    n_each = np.full(S, n_rows)
    outs = _static_call(A, kb, vb, n_each, qb, knb, vnb, d)
    sample = np.arange(0, S, 97)
    want = _oracle_attend(kb[sample], vb[sample], n_each[sample], qb.reshape(S, d)[sample], knb.reshape(S, d)[sample],
                          vnb.reshape(S, d)[sample], d)
    for o16, o32 in outs:
        assert np.abs(o32.cpu().numpy()[sample] - want).max() <= OUT_F32_MAX_ABS * max(1.0, float(np.abs(want).max()))
        assert np.abs(o16.float().cpu().numpy()[sample] - want).max() <= OUT_MAX_ABS


def test_bad_arguments_and_sizes_beyond_the_built_in_scratch_are_refused():
    import paper_2506_18226_b200 as A
    B = A.binding
    d = 64
    q = torch.zeros((4097, d), dtype=torch.bfloat16, device="cuda:0")
    k = torch.zeros((4097, 1, d), dtype=torch.bfloat16, device="cuda:0")
    n = torch.zeros(4097, dtype=torch.int32, device="cuda:0")
    out = torch.zeros((4097, d), dtype=torch.bfloat16, device="cuda:0")
    with pytest.raises(A.AdsaError) as e:
        A.decode_attn_static(q, k, k, n, q, q, out)
    assert e.value.status == B.ENOMEM
    with pytest.raises(A.AdsaError) as e:                   # no output at all
        A.decode_attn_static(q[:4], k[:4], k[:4], n[:4], q[:4], q[:4], None, None)
    assert e.value.status == B.EINVAL
    flat = torch.zeros(4 * 2 * d + 8, dtype=torch.bfloat16, device="cuda:0")
    skew = flat[4:4 + 4 * 2 * d].view(4, 2, d)              # rows that do not start on a 16-byte boundary
    with pytest.raises(A.AdsaError) as e:
        A.decode_attn_static(q[:4], skew, k[:4], n[:4], q[:4], q[:4], out[:4])
    assert e.value.status == B.EINVAL
    with pytest.raises(A.AdsaError) as e:                   # head_dim below the supported range
        A.decode_attn_static(q[:4, :4], k[:4], k[:4], n[:4], q[:4, :4], q[:4, :4], out[:4], head_dim=4)
    assert e.value.status == B.EINVAL

"""GPU parity of the condition's way into the cache: dense causal attention (adsa_prefill_attn) and the 2-D
rotary embedding (adsa_rope_2d) against the CPU oracle, through the C-ABI."""
import numpy as np
import pytest
import torch

from adsa_workloads import bf16_bits_to_f32, f32_to_bf16_bits, layer_step_qkv
from adsa_workloads.configs import Workload

pytestmark = pytest.mark.gpu


def _dev(bits):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).to("cuda:0").view(torch.bfloat16)


def _bits(rng, *shape):
    return f32_to_bf16_bits(rng.standard_normal(shape).astype(np.float32))


@pytest.mark.parametrize("d,n,batch,heads", [
    (64, 120, 2, 3),       # the LlamaGen condition: 120 rows, two 64-row chunks
    (100, 37, 1, 2),       # padded row stride, rows not 16-byte aligned, a partial chunk
    (32, 200, 1, 2),       # more than 128 query rows: two rounds, four chunks
    (128, 65, 1, 1),       # one row into the second chunk
    (8, 1, 1, 2),          # a single row attends itself
])
def test_prefill_attention_matches_causal_oracle_and_fills_the_cache(d, n, batch, heads):
    import paper_2506_18226_b200 as A
    from oracle import adsa_oracle as orc
    import harness as H
    rng = np.random.default_rng(d + n)
    S = batch * heads
    qb, kb, vb = (_bits(rng, batch, heads, n, d) for _ in range(3))
    w = Workload("prefill", 60, 1, batch, heads, d, n, 4, 4, 1.0, 1.0)
    eng = H.engine_for(w, capacity=n + 16, page_rows=16)
    o16 = torch.zeros((batch, heads, n, d), dtype=torch.bfloat16, device="cuda:0")
    o32 = torch.zeros((batch, heads, n, d), dtype=torch.float32, device="cuda:0")
    eng.prefill_attn(0, _dev(qb), _dev(kb), _dev(vb), 0, o16, o32)
    assert eng.get_status()[0] == 0
    qf, kf, vf = (bf16_bits_to_f32(x).reshape(S, n, d) for x in (qb, kb, vb))
    want = np.stack([orc.causal_attend(qf[s], kf[s], vf[s]) for s in range(S)])
    e32 = np.abs(o32.cpu().numpy().reshape(S, n, d) - want)
    e16 = np.abs(o16.float().cpu().numpy().reshape(S, n, d) - want)
    assert e32.max() <= 2e-4 * max(1.0, np.abs(want).max()), e32.max()
    assert e16.max() <= 2e-2 and e16.mean() <= 2e-3
    # the rows are in the cache, in order, bit for bit
    for s in range(S):
        pos, k, v = eng.read_stream(s)
        assert pos.tolist() == list(range(n))
        assert np.array_equal(k.numpy().view(np.uint16), kb.reshape(S, n, d)[s]) and np.array_equal(v.numpy().view(np.uint16), vb.reshape(S, n, d)[s])
    # and a decode step on top of them is the oracle's step on the same rows
    st = orc.OracleStreams(S, d, n + 16, n, 4, n)
    st.append_rows(kf, vf, 0)
    q1, k1, v1 = layer_step_qkv(w, 9, 0, 0)
    out = torch.zeros((S, d), dtype=torch.bfloat16, device="cuda:0")
    eng.layer_step(0, n, n + 16, _dev(q1), _dev(k1), _dev(v1), out)
    res = st.step(*(bf16_bits_to_f32(x).reshape(S, d) for x in (q1, k1, v1)), n, n + 16)
    assert np.abs(out.float().cpu().numpy() - res.out).max() <= 2e-2
    # a second prefill into the now filled cache is refused
    with pytest.raises(A.AdsaError) as e:
        eng.prefill_attn(0, _dev(qb), _dev(kb), _dev(vb), 0, o16, None)
    assert e.value.status == A.binding.ESTATE


@pytest.mark.parametrize("d,T0,gh,gw", [(64, 120, 32, 32), (100, 7, 5, 9), (8, 0, 3, 4)])
def test_rope_2d_matches_oracle(d, T0, gh, gw):
    from oracle import adsa_oracle as orc
    import harness as H
    rng = np.random.default_rng(d)
    w = Workload("rope", 61, 1, 1, 2, d, T0, gh, gw, 1.0, 1.0)
    eng = H.engine_for(w, capacity=32, page_rows=16)
    n = 300
    xb = _bits(rng, n, d)
    pos = rng.integers(0, T0 + gh * gw, size=n).astype(np.int32)
    pos[:3] = [0, T0, T0 + gh * gw - 1]
    x = _dev(xb).clone()
    eng.rope_2d(x, torch.from_numpy(pos).to("cuda:0"))
    torch.cuda.synchronize()
    want = orc.rope_2d(bf16_bits_to_f32(xb), pos, T0, gw)
    got = x.float().cpu().numpy()
    assert (np.abs(got - want) <= 2.0 ** -7 * np.abs(want) + 1e-6).all()
    text = pos < T0
    assert np.array_equal(x.cpu().view(torch.int16).numpy()[text], xb.view(np.int16)[text])     # text rows untouched, bit for bit

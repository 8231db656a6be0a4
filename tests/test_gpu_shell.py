"""The host model's operations around the attention (adsa_rmsnorm, adsa_swiglu, adsa_cfg_sample) against the oracle.

Outputs in bf16 are compared within one rounding of the exact value (2^-8 relative: bf16 keeps 8 significant bits).
The sampled token is an integer decided by floating-point sums, taken in fp32 on the GPU and in fp64 by the oracle;
what is unique is compared exactly (the argmax, exact ties), and otherwise the token is checked to be a valid answer:
it belongs to the kept set and the caller's uniform number falls in its share of the cumulative distribution, within
the rounding of an fp32 sum.
"""
import numpy as np
import pytest
import torch

from adsa_workloads import bf16_bits_to_f32, f32_to_bf16_bits

pytestmark = pytest.mark.gpu

BF16_RTOL = 2.0 ** -8 * 1.02
CDF_EPS = 2e-5


def _dev(bits):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).to("cuda:0").view(torch.bfloat16)


def _bf16_normal(rng, shape, scale=1.0):
    return f32_to_bf16_bits((scale * rng.standard_normal(shape)).astype(np.float32))


def _host(t):
    return t.float().cpu().numpy().astype(np.float64)


@pytest.mark.parametrize("rows,dim,eps", [(32, 1280, 1e-5), (7, 96, 1e-5), (1, 8, 0.0), (513, 1024, 1e-6), (3, 4096, 1e-5)])
def test_rmsnorm_matches_the_oracle(rows, dim, eps):
    import paper_2506_18226_b200 as A
    from oracle import adsa_oracle as orc
    rng = np.random.default_rng(rows + dim)
    xb, wb = _bf16_normal(rng, (rows, dim), 3.0), _bf16_normal(rng, (dim,))
    want = orc.rmsnorm(bf16_bits_to_f32(xb), bf16_bits_to_f32(wb), eps)
    x = _dev(xb)
    got = A.rmsnorm(x, _dev(wb), eps=eps)
    torch.cuda.synchronize()
    assert np.all(np.abs(_host(got) - want) <= BF16_RTOL * np.abs(want) + 1e-30)
    A.rmsnorm(x, _dev(wb), out=x, eps=eps)                      # in place
    torch.cuda.synchronize()
    assert torch.equal(x, got)


def test_rmsnorm_of_a_zero_row_is_zero():
    import paper_2506_18226_b200 as A
    x = torch.zeros((2, 64), dtype=torch.bfloat16, device="cuda:0")
    w = torch.ones(64, dtype=torch.bfloat16, device="cuda:0")
    assert torch.equal(A.rmsnorm(x, w, eps=1e-5), x)


@pytest.mark.parametrize("rows,hidden,fused", [(32, 3584, False), (32, 3584, True), (5, 8, False), (129, 264, True)])
def test_swiglu_matches_the_oracle(rows, hidden, fused):
    import paper_2506_18226_b200 as A
    from oracle import adsa_oracle as orc
    rng = np.random.default_rng(rows * 7 + hidden)
    both = _bf16_normal(rng, (rows, 2 * hidden), 2.5)
    gate_f, up_f = bf16_bits_to_f32(both[:, :hidden]), bf16_bits_to_f32(both[:, hidden:])
    want = orc.swiglu(np.ascontiguousarray(gate_f), np.ascontiguousarray(up_f))
    if fused:                                                    # one tensor that holds both halves side by side
        t = _dev(both)
        got = A.swiglu(t[:, :hidden], t[:, hidden:])
    else:
        got = A.swiglu(_dev(np.ascontiguousarray(both[:, :hidden])), _dev(np.ascontiguousarray(both[:, hidden:])))
    torch.cuda.synchronize()
    assert np.all(np.abs(_host(got) - want) <= BF16_RTOL * np.abs(want) + 1e-30)


def _check_tokens(logits_bits, n_images, scale, top_k, temperature, uniforms, tokens):
    """Every token is a valid answer for its image (see the module docstring)."""
    from oracle import adsa_oracle as orc
    lf = bf16_bits_to_f32(logits_bits)
    exact = 0
    for b in range(n_images):
        want, mixed, cdf = orc.cfg_sample(lf[b], lf[n_images + b], scale, top_k, temperature, float(uniforms[b]))
        t = int(tokens[b])
        exact += t == want
        kth = np.sort(mixed)[-top_k]
        assert mixed[t] >= kth - 1e-5 * max(1.0, abs(kth)), (b, t, want)              # kept (or tied with the last kept one)
        before = cdf[t - 1] if t > 0 else 0.0
        assert before - CDF_EPS <= uniforms[b] <= cdf[t] + CDF_EPS, (b, t, want, before, cdf[t], uniforms[b])
    return exact


@pytest.mark.parametrize("n_images,vocab,scale,top_k,temperature", [
    (16, 16384, 7.5, 2000, 1.0),       # the codebook and the sampling defaults of the decoder family
    (16, 16384, 1.75, 16384, 1.0),     # nothing filtered
    (3, 1000, 4.0, 50, 0.7),
    (5, 32768, 2.0, 300, 1.3),         # the largest vocabulary the kernel takes
    (2, 37, 1.0, 5, 1.0),              # fewer ids than threads
])
def test_cfg_sample_tokens_are_valid_draws(n_images, vocab, scale, top_k, temperature):
    import paper_2506_18226_b200 as A
    rng = np.random.default_rng(vocab + top_k)
    lb = _bf16_normal(rng, (2 * n_images, vocab), 2.0)
    u = rng.random(n_images).astype(np.float32)
    u[0] = 0.0                                                                        # the first kept id
    toks = A.cfg_sample(_dev(lb), scale, top_k, temperature, torch.from_numpy(u).to("cuda:0"))
    toks2 = A.cfg_sample(_dev(lb), scale, top_k, temperature, torch.from_numpy(u).to("cuda:0"))
    torch.cuda.synchronize()
    assert torch.equal(toks, toks2)                                                   # a call is reproducible
    exact = _check_tokens(lb, n_images, scale, top_k, temperature, u, toks.cpu().numpy())
    assert exact >= n_images - 1                                                      # and nearly always the oracle's own token


def test_cfg_sample_top_1_is_the_argmax_with_the_lowest_id_among_equals():
    import paper_2506_18226_b200 as A
    from oracle import adsa_oracle as orc
    rng = np.random.default_rng(3)
    n, vocab = 8, 16384
    lb = _bf16_normal(rng, (2 * n, vocab), 1.0)        # bf16 values repeat: equal maxima do occur
    lf = bf16_bits_to_f32(lb)
    lf[n:] = 0.0                                       # unconditional rows zero and scale 1: the mix is the conditional row, exactly
    lf[1, 100] = lf[1, 9000] = lf[1].max() + 1.0       # a planted tie for the maximum
    lb = f32_to_bf16_bits(lf)
    u = rng.random(n).astype(np.float32)
    toks = A.cfg_sample(_dev(lb), 1.0, 1, 1.0, torch.from_numpy(u).to("cuda:0")).cpu().numpy()
    lf = bf16_bits_to_f32(lb)
    for b in range(n):
        assert toks[b] == int(np.argmax(lf[b])) == orc.cfg_sample(lf[b], lf[n + b], 1.0, 1, 1.0, float(u[b]))[0]
    assert toks[1] == 100


def test_cfg_sample_ties_at_the_threshold_keep_the_lower_ids():
    """Logits 5 at id 7, 1 at ids 20, 300 and 9000, everything else -30: top_k = 3 keeps ids 7, 20 and 300.  The
    shares are exp(0) : exp(-4) : exp(-4); a grid of u must return exactly those ids, in the oracle's proportions,
    and never id 9000."""
    import paper_2506_18226_b200 as A
    from oracle import adsa_oracle as orc
    vocab, n = 16384, 64
    row = np.full(vocab, -30.0, np.float32)
    row[7], row[20], row[300], row[9000] = 5.0, 1.0, 1.0, 1.0
    lf = np.concatenate([np.tile(row, (n, 1)), np.zeros((n, vocab), np.float32)])
    u = ((np.arange(n) + 0.5) / n).astype(np.float32)
    toks = A.cfg_sample(_dev(f32_to_bf16_bits(lf)), 1.0, 3, 1.0, torch.from_numpy(u).to("cuda:0")).cpu().numpy()
    want = np.array([orc.cfg_sample(lf[b], lf[n + b], 1.0, 3, 1.0, float(u[b]))[0] for b in range(n)])
    assert set(toks.tolist()) <= {7, 20, 300}
    assert np.array_equal(toks, want)


def test_shell_calls_refuse_bad_arguments():
    import paper_2506_18226_b200 as A
    B = A.binding
    x = torch.zeros((4, 64), dtype=torch.bfloat16, device="cuda:0")
    w = torch.ones(64, dtype=torch.bfloat16, device="cuda:0")
    with pytest.raises(A.AdsaError) as e:
        A.rmsnorm(x[:, :60], w[:60])                   # dim not a multiple of 8 (and rows no longer contiguous)
    assert e.value.status == B.EINVAL
    flat = torch.zeros(4 * 64 + 8, dtype=torch.bfloat16, device="cuda:0")
    with pytest.raises(A.AdsaError) as e:
        A.rmsnorm(flat[4:4 + 256].view(4, 64), w)      # rows that do not start on a 16-byte boundary
    assert e.value.status == B.EINVAL
    lg = torch.zeros((4, 100), dtype=torch.bfloat16, device="cuda:0")
    un = torch.zeros(2, dtype=torch.float32, device="cuda:0")
    for bad in (dict(top_k=0), dict(top_k=101), dict(temperature=0.0)):
        kw = dict(scale=1.0, top_k=10, temperature=1.0)
        kw.update(bad)
        with pytest.raises(A.AdsaError) as e:
            A.cfg_sample(lg, kw["scale"], kw["top_k"], kw["temperature"], un)
        assert e.value.status == B.EINVAL
    big = torch.zeros((2, 40000), dtype=torch.bfloat16, device="cuda:0")
    with pytest.raises(A.AdsaError) as e:
        A.cfg_sample(big, 1.0, 10, 1.0, un[:1])        # vocabulary above 32768
    assert e.value.status == B.EINVAL


def test_model_shell_generates_an_image_worth_of_tokens():
    """The LlamaGen-shaped shell (random weights) end to end on a small shape: the condition is prefilled through
    dense causal attention, every grid cell is decoded through all layers with the cache at half the context, ids
    arrive on the host; the same seed gives the same ids, the caches end at the budget, no status bit is set."""
    from paper_2506_18226_b200.shell import LlamaGenShell, ShellConfig
    cfg = ShellConfig(n_layers=2, dim=128, n_heads=2, ffn_hidden=256, vocab=512, n_text=8, grid_h=6, grid_w=6, n_images=2,
                      top_k=50)
    runs = []
    for _ in range(2):
        sh = LlamaGenShell(cfg, seed=5)
        g = torch.Generator(device="cuda:0").manual_seed(9)
        text = torch.randn(cfg.batch, cfg.n_text, cfg.dim, generator=g, device="cuda:0").to(torch.bfloat16)
        ids = sh.generate(text).clone()
        assert ids.shape == (36, 2) and int(ids.min()) >= 0 and int(ids.max()) < cfg.vocab
        assert sh.eng.get_status()[0] == 0
        n_live = sh.eng._t["n_live"].cpu().numpy()
        assert (n_live == min(sh.budget, cfg.n_text + 35)).all()      # 35 tokens were fed in after the condition
        runs.append(ids)
    assert torch.equal(runs[0], runs[1])
    assert len(set(runs[0].flatten().tolist())) > 4                    # not a constant sequence


def test_model_shell_graphs_and_eager_steps_draw_the_same_ids():
    """The decode step replayed from CUDA graphs around the attention launches gives the ids of the eager step."""
    from paper_2506_18226_b200.shell import LlamaGenShell, ShellConfig
    cfg = ShellConfig(n_layers=3, dim=128, n_heads=2, ffn_hidden=256, vocab=512, n_text=8, grid_h=6, grid_w=6, n_images=2,
                      top_k=50)
    g = torch.Generator(device="cuda:0").manual_seed(4)
    text = torch.randn(cfg.batch, cfg.n_text, cfg.dim, generator=g, device="cuda:0").to(torch.bfloat16)
    ids = [LlamaGenShell(cfg, seed=2, use_graphs=flag).generate(text).clone() for flag in (True, False)]
    assert torch.equal(ids[0], ids[1])


def test_model_shell_logits_follow_a_float64_replica():
    """The whole data flow of the shell against a replica assembled from the oracle's functions and float64 matrix
    products, rounding to bf16 where the shell stores bf16 (so that what is compared is the wiring, not the storage
    type): the logits after the condition and after each of three decode steps.  The budget covers the whole context
    here, so the attention is dense causal attention (Sec. 4.2: identical to the baseline while the cache is not
    full) and no selection can flip.  The replica is fed the ids the shell drew."""
    from oracle import adsa_oracle as orc
    from paper_2506_18226_b200.shell import LlamaGenShell, ShellConfig
    cfg = ShellConfig(n_layers=2, dim=128, n_heads=2, ffn_hidden=256, vocab=512, n_text=6, grid_h=4, grid_w=4, n_images=2,
                      top_k=40, budget_fraction=1.0)
    sh = LlamaGenShell(cfg, seed=11, use_graphs=False)
    gen = torch.Generator(device="cuda:0").manual_seed(12)
    text = torch.randn(cfg.batch, cfg.n_text, cfg.dim, generator=gen, device="cuda:0").to(torch.bfloat16)
    Bt, T, H, d, D, L = cfg.batch, cfg.n_text, cfg.n_heads, cfg.head_dim, cfg.dim, cfg.n_layers

    def f64(t):
        return t.float().cpu().numpy().astype(np.float64)

    def r(a):                                                   # round to bf16, as every stored activation is
        return bf16_bits_to_f32(f32_to_bf16_bits(np.asarray(a, dtype=np.float32))).astype(np.float64)

    W = {n: f64(getattr(sh, n)) for n in ("tok_emb", "wq", "wk", "wv", "wo", "w13", "w2", "norm1", "norm2", "norm_f", "head")}
    Kc = [[[np.zeros((0, d)) for _ in range(H)] for _ in range(Bt)] for _ in range(L)]      # the replica's caches
    Vc = [[[np.zeros((0, d)) for _ in range(H)] for _ in range(Bt)] for _ in range(L)]

    def block(l, x, positions, causal):
        h = r(orc.rmsnorm(x, W["norm1"][l], cfg.norm_eps))
        q, k, v = (r(h @ W[n][l].T).reshape(Bt, -1, H, d) for n in ("wq", "wk", "wv"))
        n_new = q.shape[1]
        attn = np.zeros((Bt, n_new, H, d))
        for b in range(Bt):
            for hh in range(H):
                qr = r(orc.rope_2d(q[b, :, hh], positions, cfg.n_text, cfg.grid_w))
                kr = r(orc.rope_2d(k[b, :, hh], positions, cfg.n_text, cfg.grid_w))
                Kall = np.concatenate([Kc[l][b][hh], kr]); Vall = np.concatenate([Vc[l][b][hh], v[b, :, hh]])
                if causal:
                    attn[b, :, hh] = orc.causal_attend(qr, kr, v[b, :, hh])
                else:
                    attn[b, 0, hh] = orc.attend(qr[0], Kall, Vall)[0]
                Kc[l][b][hh], Vc[l][b][hh] = Kall, Vall
        attn = r(attn).reshape(Bt * n_new, D)
        x = r(x + attn @ W["wo"][l].T)
        h = r(orc.rmsnorm(x, W["norm2"][l], cfg.norm_eps))
        gu = r(h @ W["w13"][l].T)
        act = r(orc.swiglu(np.ascontiguousarray(gu[:, :cfg.ffn_hidden]), np.ascontiguousarray(gu[:, cfg.ffn_hidden:])))
        return r(x + act @ W["w2"][l].T)

    def logits_of(x_last):
        return r(r(orc.rmsnorm(x_last, W["norm_f"], cfg.norm_eps)) @ W["head"].T)

    def close(got, want):
        err = np.linalg.norm(got - want) / np.linalg.norm(want)
        cos = float((got * want).sum() / (np.linalg.norm(got) * np.linalg.norm(want)))
        assert err <= 5e-2 and cos >= 0.998, (err, cos)

    # the condition
    sh.prefill(text)
    x = f64(text).reshape(Bt * T, D)
    for l in range(L):
        x = block(l, x, np.arange(T, dtype=np.int32), causal=True)
    close(f64(sh.logits), logits_of(x.reshape(Bt, T, D)[:, -1]))
    # three decode steps, fed the ids the shell drew
    for cell in range(1, 4):
        ids = sh.tokens.cpu().numpy()
        sh.decode_step(cell)
        emb = W["tok_emb"][ids]
        x = np.concatenate([emb, emb])
        for l in range(L):
            x = block(l, x, np.array([cfg.n_text + cell - 1], dtype=np.int32), causal=False)
        close(f64(sh.logits), logits_of(x))
    assert sh.eng.get_status()[0] == 0

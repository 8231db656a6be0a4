"""GPU parity: the CUDA path through the C-ABI against the CPU oracle, element by element."""
import numpy as np
import pytest
import torch

from adsa_workloads import (get_workload, late_state, layer_step_qkv, pick_page_rows, prefix_kv,
                            structured_values)
from adsa_workloads.configs import Workload

pytestmark = pytest.mark.gpu


def _harness():
    import harness
    return harness


MODES = ["calls", "fused", "two-sweep-fused", "reselect-fused", "streaming", "cluster-calls", "cluster-fused", "cores-calls", "cores-fused"]
# calls: the four C-ABI calls one by one (attention by the persistent pipelined kernel, tensor-core
#        arithmetic where the pool rows are 64 elements wide);
# fused: adsa_layer_step, one persistent kernel per layer-step, scores carried from step to step;
# two-sweep-fused: the fused kernel always scoring in a second sweep over V (by default it scores during the
#        attention sweep whenever the carried sum of normalised rows can be updated in closed form);
# reselect-fused: the fused kernel making the full selection at every step (by default, when the cache is
#        exactly full, it evicts the row the previous step noted as the highest-scoring one);
# streaming: the four calls with the staged kernels switched off (the register-streaming attention);
# cluster-*: the same two ways of calling, with the one-cluster-per-stream kernel;
# cores-*: the same, with the persistent kernel forced onto the CUDA cores.


def _apply_mode(eng, mode):
    if mode == "streaming":
        eng.set_staged(0)
    elif mode.startswith("cluster"):
        eng.set_staged(2)
    elif mode.startswith("cores"):
        eng.set_staged(3)
    elif mode.startswith("two-sweep"):
        eng.set_single_sweep(0)
    elif mode.startswith("reselect"):
        eng.set_single_sweep(1)
    return mode.endswith("fused")


def _run_trajectory(w, layer, seed, budget_fn, *, n_layers_engine=1, page_rows=None, steps=None, n_prefix=None,
                    rows_back=1, sample=None, chunk_rows=0, score_variant=0, mode="calls", score_mode=0, score_share=0):
    H = _harness()
    cap = max(budget_fn(w.n_text + g) for g in range(w.n_cells))
    eng = H.engine_for(w, n_layers=n_layers_engine, page_rows=page_rows, capacity=cap, n_prefix=n_prefix,
                       local_rows_back=rows_back, score_mode=score_mode, score_share=score_share)
    if chunk_rows:
        eng.set_attn_chunk_rows(chunk_rows)
    lh = H.LayerHarness(eng, 0, oracle_cap=w.l_max + 1, sample=sample, score_variant=score_variant,
                        fused=_apply_mode(eng, mode))
    if w.n_text:
        k, v = prefix_kv(w, seed, layer)
        lh.prefill(k, v, 0)
    for g in range(w.n_cells if steps is None else steps):
        q, k, v = layer_step_qkv(w, seed, layer, g)
        lh.step(q, k, v, w.n_text + g, budget_fn(w.n_text + g))
    status, free_state = eng.get_status()
    assert status == 0
    return lh, eng


# ---------------------------------------------------------------------------
# small shapes: several tiles, ragged tails, odd page sizes, all head-dim paths
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("d,page_rows,T0,gh,gw,beta,chunk", [
    (64, 7, 5, 6, 5, 0.5, 0),      # pages smaller than a warp tile, ragged everywhere
    (64, 16, 0, 5, 4, 0.5, 0),     # no text condition: the first step sees an empty cache
    (32, 3, 4, 4, 6, 0.6, 32),     # 4 lanes per row
    (100, 5, 9, 5, 7, 0.5, 0),     # non-power-of-two head_dim, padded row stride 104
    (128, 11, 6, 4, 4, 0.7, 0),    # 16 lanes per row
    (128, 16, 40, 7, 6, 0.6, 0),   # 256-byte rows over several blocks, pages of exactly one 16-row stage
    (128, 13, 45, 6, 7, 0.5, 0),   # 256-byte rows, pages that cut every stage into pieces
    (122, 64, 33, 6, 6, 0.5, 0),   # head_dim just below 128: the padding of a 128-element row stays out of every sum
    (48, 9, 20, 6, 7, 0.5, 0),     # 96-byte rows in 128-byte tiles: the copies fill the rest of a tile row with zeros
    (72, 10, 30, 6, 6, 0.6, 0),    # 144-byte rows in the two-half layout (the second half holds 8 elements)
    (120, 16, 35, 7, 5, 0.5, 0),   # 240-byte rows in the two-half layout
    (256, 4, 3, 3, 5, 0.5, 0),     # 32 lanes per row
    (8, 2, 2, 7, 3, 0.4, 0),       # smallest head_dim
])
@pytest.mark.parametrize("mode", MODES)
def test_small_shapes_full_trajectory(d, page_rows, T0, gh, gw, beta, chunk, mode):
    w = Workload(f"tiny-d{d}", 90 + d % 7, 1, 2, 3, d, T0, gh, gw, beta, 1.0)
    C = max(2, w.capacity())
    lh, eng = _run_trajectory(w, 0, 1, lambda cur: C, page_rows=page_rows, chunk_rows=chunk, mode=mode)
    assert lh.stats.steps == gh * gw and lh.stats.max_score_err <= 1e-6


@pytest.mark.parametrize("d,served", [(8, True), (32, True), (48, True), (64, True), (72, True), (100, True), (120, True),
                                      (128, True), (136, False), (256, False)])
def test_which_head_dims_the_tensor_core_kernel_serves(d, served):
    """Every row stride up to 128 elements runs on the tensor-core kernel (one warp group walks a whole stream in
    32-row blocks: adsa_plan_attn reports one split of 32-row steps); wider rows fall back to the other kernels."""
    H = _harness()
    w = Workload(f"plan-d{d}", 60, 1, 1, 2, d, 8, 8, 8, 0.5, 1.0)
    eng = H.engine_for(w, capacity=w.capacity(), page_rows=8)
    splits, step_rows = eng.plan_attn(40)
    assert ((splits, step_rows) == (1, 32)) == served


@pytest.mark.parametrize("n_prefix_kind,rows_back", [("none", 1), ("text+5%", 1), ("text", 2), ("text", 0)])
@pytest.mark.parametrize("mode", ["calls", "fused", "cluster-fused"])
def test_prefix_and_window_variants(n_prefix_kind, rows_back, mode):
    w = Workload("tiny-variants", 97, 1, 1, 4, 64, 10, 8, 8, 0.5, 1.0)
    n_prefix = {"none": 0, "text": w.n_text, "text+5%": w.n_text + 4}[n_prefix_kind]
    C = w.capacity()
    lh, eng = _run_trajectory(w, 0, 2, lambda cur: C, n_prefix=n_prefix, rows_back=rows_back, page_rows=8, mode=mode)
    assert lh.stats.steps == 64


@pytest.mark.parametrize("mode", MODES)
def test_budget_covering_context_is_dense_attention(mode):
    # no eviction ever: every step must equal dense causal attention (the oracle's own pin)
    w = Workload("tiny-dense", 98, 1, 1, 4, 64, 12, 10, 10, 1.0, 1.0)
    lh, eng = _run_trajectory(w, 0, 3, lambda cur: w.l_max, page_rows=16, chunk_rows=32, mode=mode)
    assert int(eng._t["n_live"].max().item()) == w.l_max


@pytest.mark.parametrize("preset", ["window", "window+prefix"])
@pytest.mark.parametrize("mode", ["calls", "fused", "two-sweep-fused", "cores-fused"])
def test_ablation_presets_without_global_tokens(preset, mode):
    """The comparison settings of Fig. 3 are corner cases of the same calls: a budget below prefix + window
    makes K = 0 at every step, so the cache keeps the local window alone (no prefix configured) or the
    prefix and the window, and nothing of the previous region."""
    w = Workload("tiny-presets", 96, 1, 1, 4, 64, 10, 9, 7, 0.5, 1.0)
    n_prefix = 0 if preset == "window" else w.n_text
    lh, eng = _run_trajectory(w, 0, 4, lambda cur: 1, n_prefix=n_prefix, page_rows=8, mode=mode)
    assert lh.stats.steps == w.n_cells
    # after the last cell: the prefix, the grid row above, the last grid row (the new row included)
    assert int(eng._t["n_live"].min().item()) == int(eng._t["n_live"].max().item()) == n_prefix + 2 * w.grid_w


# ---------------------------------------------------------------------------
# the benchmark configurations
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("seed", [0, 1, 2])
def test_config1_full_trajectory(seed, mode):
    w = get_workload(1)
    C = w.capacity()
    lh, eng = _run_trajectory(w, 0, seed, lambda cur: C, mode=mode)
    assert lh.stats.steps == 256
    assert lh.stats.max_out_err <= 2e-2 and lh.mean_out_err() <= 2e-3
    # pool never exceeds the budget's share: capacity rows per stream, in whole pages
    pr = eng.cfg.page_rows
    assert eng.pool_bytes_peak() <= w.streams_per_layer * -(-C // pr) * pr * w.row_stride * 4


@pytest.mark.parametrize("setting,n_text,grid,budget", [
    ("class-conditional", 1, 24, 384), ("class-conditional", 1, 24, 256),          # Sec. 5: context 576 cut to 384 and 256
    ("text-conditional", 120, 32, 768), ("text-conditional", 120, 32, 640), ("text-conditional", 120, 32, 512),  # 1024 cut to 768, 640, 512
])
def test_context_budgets_of_the_experiments(setting, n_text, grid, budget):
    """Whole generations at the context budgets of Sec. 5 (a class token or 120 text tokens, then a 24 x 24
    or 32 x 32 grid), a few streams of 64-element heads, fused steps against the oracle at every step."""
    w = Workload(setting, 70 + grid, 1, 1, 4, 64, n_text, grid, grid, budget / (n_text + grid * grid), 1.0)
    lh, eng = _run_trajectory(w, 0, budget, lambda cur: budget, n_prefix=n_text, mode="fused")
    assert lh.stats.steps == grid * grid
    assert lh.stats.max_out_err <= 2e-2 and lh.mean_out_err() <= 2e-3
    assert int(eng._t["n_live"].max().item()) == budget


@pytest.mark.parametrize("mode", ["calls", "fused"])
def test_config1_budget_as_fraction_of_current_context(mode):
    # the literal "50 % of the current context" schedule: budget grows with the context
    w = get_workload(1)
    lh, eng = _run_trajectory(w, 0, 0, lambda cur: max(1, -(-(cur + 1) // 2)), mode=mode)
    assert lh.stats.steps == 256


@pytest.mark.parametrize("layer,mode", [(0, "calls"), (0, "fused"), (11, "fused")])
def test_config2_full_trajectory(layer, mode):
    w = get_workload(2)
    C = w.capacity()
    lh, eng = _run_trajectory(w, layer, 0, lambda cur: C, mode=mode)
    assert lh.stats.steps == 256


def _bench_page_rows(C):
    """The page size bench.py times: the largest divisor of the capacity up to 1024 rows (one page per
    stream for the LlamaGen shapes)."""
    return pick_page_rows(C, hi=1024)


def _full_size_harness(w, C, page_rows, mode, n_sample, seed, n_rows, cur0, extra_rows=0):
    """One layer of workload `w` at full size, loaded with a seeded late-generation state of n_rows rows
    per stream as of position cur0; the oracle follows a seeded sample of the streams."""
    H = _harness()
    rng = np.random.default_rng(seed)
    eng = H.engine_for(w, n_layers=1, capacity=C, page_rows=page_rows, extra_rows=extra_rows)
    sample = sorted(rng.choice(w.streams_per_layer, size=n_sample, replace=False).tolist())
    lh = H.LayerHarness(eng, 0, oracle_cap=C + 4, sample=sample, fused=_apply_mode(eng, mode))
    pos, k, v = late_state(w, seed=seed, n_rows=n_rows, cur_pos=cur0)
    lh.prefill(k.reshape(w.batch, w.n_heads, n_rows, w.head_dim), v.reshape(w.batch, w.n_heads, n_rows, w.head_dim), 0, pos)
    lh.check_state()
    return eng, lh


def _pages_in_use(eng):
    st, fs = eng.get_status()
    assert st == 0
    return eng.cfg.n_pages - fs[2]


@pytest.mark.parametrize("cfg,beta,n_sample,steps,pages", [
    (3, 0.5, 32, 3, "paged"), (3, 0.5, 32, 3, "bench"),
    (4, 0.5, 32, 3, "paged"), (4, 0.5, 32, 3, "bench"),
    (5, 0.25, 12, 2, "bench"),
    (5, 0.5, 8, 2, "bench"),
    (5, 0.75, 6, 2, "bench"),
])
@pytest.mark.parametrize("mode", ["calls", "fused", "two-sweep-fused", "cluster-fused"])
def test_full_size_layer_steps(cfg, beta, n_sample, steps, pages, mode):
    """One layer at the full size of configs 3-5 from a seeded late-generation state (cache one row short
    of full, then full), mid-row near the end of the grid; the oracle follows a sample of streams.
    pages = "bench": the page size the benchmark times (one page per stream where the capacity allows);
    "paged": pages of at most 128 rows, several per stream."""
    w = get_workload(cfg, beta)
    C = w.capacity()
    pr = _bench_page_rows(C) if pages == "bench" else pick_page_rows(C, hi=128)
    g0 = w.n_cells - steps - w.grid_w // 2          # mid-row, near the end of the grid
    cur0 = w.n_text + g0
    eng, lh = _full_size_harness(w, C, pr, mode, n_sample, cfg * 100 + int(beta * 100), C - 1, cur0)
    for t in range(steps):
        q, kn, vn = layer_step_qkv(w, 0, 0, g0 + t)
        lh.step(q, kn, vn, cur0 + t, C)
    assert lh.stats.max_out_err <= 2e-2 and lh.mean_out_err() <= 2e-3
    n_live = eng._t["n_live"].cpu().numpy()
    assert (n_live == C).all()
    # every page in use is accounted for, none leaked
    assert _pages_in_use(eng) == w.streams_per_layer * -(-C // pr)


@pytest.mark.parametrize("cfg,pages", [(3, "bench"), (3, "paged"), (4, "bench"), (4, "paged")])
@pytest.mark.parametrize("mode", ["calls", "fused", "two-sweep-fused"])
def test_full_size_steps_that_change_the_code_path(cfg, pages, mode):
    """Configs 3 and 4 at full size, in the launch configuration the benchmark times ("bench" pages) and
    with several pages per stream, on the steps where the kernels take another branch: the step at which
    the cache fills up, the step that ends a grid row and the one that starts the next (rows leave the
    local window: the carried sum cannot be updated in closed form and the next scores come from a second
    sweep), a step whose budget is smaller than the one before (several evictions at once: the general
    selection, survivors moving into holes, pages returned), the steady steps after it, and the last two
    cells of the grid."""
    w = get_workload(cfg)
    C, W, T0 = w.capacity(), w.grid_w, w.n_text
    pr = _bench_page_rows(C) if pages == "bench" else pick_page_rows(C, hi=128)
    S = w.streams_per_layer

    # (a) two rows short of full, three cells before the end of a grid row: grow, fill up, first eviction
    #     on the row's last cell, then the first two cells of the next row
    g0 = (w.grid_h - 3) * W + W - 3
    eng, lh = _full_size_harness(w, C, pr, mode, 32, cfg * 10 + 1, C - 2, T0 + g0)
    want_rows = [C - 1, C, C, C, C]
    for t in range(5):
        q, kn, vn = layer_step_qkv(w, 1, 0, g0 + t)
        lh.step(q, kn, vn, T0 + g0 + t, C)
        assert (eng._t["n_live"].cpu().numpy() == want_rows[t]).all()
    assert _pages_in_use(eng) == S * -(-C // pr)
    # (b) the budget drops by 37 rows (general K: many rows go at once, survivors move down), stays there
    #     for a step (one eviction), then is lifted again (the cache regrows without eviction)
    g1 = g0 + 5
    for t, budget in enumerate([C - 37, C - 37, C, C]):
        q, kn, vn = layer_step_qkv(w, 1, 0, g1 + t)
        lh.step(q, kn, vn, T0 + g1 + t, budget)
    assert (eng._t["n_live"].cpu().numpy() == C - 35).all()
    assert _pages_in_use(eng) == S * -(-(C - 35) // pr)
    assert lh.stats.max_out_err <= 2e-2 and lh.mean_out_err() <= 2e-3

    # (c) the last two cells of the grid, cache full
    g2 = w.n_cells - 2
    eng, lh = _full_size_harness(w, C, pr, mode, 32, cfg * 10 + 2, C, T0 + g2)
    for t in range(2):
        q, kn, vn = layer_step_qkv(w, 2, 0, g2 + t)
        lh.step(q, kn, vn, T0 + g2 + t, C)
    assert (eng._t["n_live"].cpu().numpy() == C).all()
    assert lh.stats.max_out_err <= 2e-2 and lh.mean_out_err() <= 2e-3
    assert _pages_in_use(eng) == S * -(-C // pr)


def _wide_workload():
    """Heads of 128 elements (the 256-byte row layout) on a 24 x 24 grid with enough streams that every SM
    serves several of them."""
    return Workload("wide-d128-24x24", 41, 3, 8, 32, 128, 120, 24, 24, 0.5, 1.0)


@pytest.mark.parametrize("pages", ["bench", "paged"])
@pytest.mark.parametrize("mode", ["calls", "fused", "two-sweep-fused", "cluster-fused"])
def test_wide_rows_many_streams(pages, mode):
    """128-element heads at a size that fills the device: the cache fills up on the last cell of a grid
    row, the next row starts, the budget drops (general selection, survivors move) and is lifted again."""
    w = _wide_workload()
    C, W, T0 = w.capacity(), w.grid_w, w.n_text
    pr = _bench_page_rows(C) if pages == "bench" else pick_page_rows(C, hi=64)
    g0 = (w.grid_h - 3) * W + W - 3
    eng, lh = _full_size_harness(w, C, pr, mode, 24, 411, C - 2, T0 + g0)
    budgets = [C, C, C, C, C, C - 21, C - 21, C, C]
    for t, budget in enumerate(budgets):
        q, kn, vn = layer_step_qkv(w, 4, 0, g0 + t)
        lh.step(q, kn, vn, T0 + g0 + t, budget)
    assert (eng._t["n_live"].cpu().numpy() == C - 19).all()
    assert lh.stats.max_out_err <= 2e-2 and lh.mean_out_err() <= 2e-3
    assert _pages_in_use(eng) == w.streams_per_layer * -(-(C - 19) // pr)


@pytest.mark.parametrize("cfg,beta,n_layers,n_sample", [(4, 0.5, 4, 6), (3, 0.5, 6, 6), (5, 0.5, 2, 3), ("wide", 0.5, 4, 6)])
def test_full_size_token_step_one_launch_for_all_layers(cfg, beta, n_layers, n_sample):
    """adsa_token_step as the benchmark runs it: ONE launch of the tensor-core kernel for all layers (the
    grouping the benchmark's launch uses: two warps per stream, as many streams per SM as fit), at the full
    per-layer size of configs 3-5 with the benchmark's page size, from a seeded late state, over steps that
    include the end of a grid row and the start of the next.  The oracle follows a sample of streams of every
    layer: outputs, cache positions and payloads; and the same steps launched layer by layer agree to rounding
    and leave the same caches."""
    H = _harness()
    from oracle import adsa_oracle as orc
    from adsa_workloads import bf16_bits_to_f32, f32_to_bf16_bits
    from dataclasses import replace
    w = replace(_wide_workload() if cfg == "wide" else get_workload(cfg, beta), n_layers=n_layers)
    cfg = 6 if cfg == "wide" else cfg
    C, T0, W, S, d = w.capacity(), w.n_text, w.grid_w, w.streams_per_layer, w.head_dim
    pr = _bench_page_rows(C)
    g0 = (w.grid_h - 2) * W + W - 3                      # three cells before a row ends: cells W-3, W-2, W-1, then 0, 1
    steps = 5
    rng = np.random.default_rng(cfg)
    sample = [sorted(rng.choice(S, size=n_sample, replace=False).tolist()) for _ in range(n_layers)]
    engs = [H.engine_for(w, n_layers=n_layers, capacity=C, page_rows=pr) for _ in range(2)]
    engs[1].set_token_launch(0)                          # the same steps, one launch per layer
    ost = orc.OracleStreams(n_layers * n_sample, d, C + 4, T0, W, T0)
    for l in range(n_layers):
        pos, k, v = late_state(w, seed=100 * cfg + l, n_rows=C, cur_pos=T0 + g0)
        for e in engs:
            e.prefill_rows(l, H.dev_bf16(k.reshape(w.batch, w.n_heads, C, d)), H.dev_bf16(v.reshape(w.batch, w.n_heads, C, d)), 0,
                           torch.from_numpy(pos.reshape(w.batch, w.n_heads, C)).to("cuda:0"))
        for i, s_ in enumerate(sample[l]):
            ost.load(l * n_sample + i, pos[s_], bf16_bits_to_f32(k[s_]), bf16_bits_to_f32(v[s_]))
    shape = (n_layers, w.batch, w.n_heads, d)
    outs = [torch.zeros(shape, dtype=torch.bfloat16, device="cuda:0") for _ in range(2)]
    alive = np.ones(n_layers * n_sample, dtype=bool)     # streams still in step with the oracle (a tolerated tie ends a stream's comparison)
    for t in range(steps):
        per = [layer_step_qkv(w, 7, l, g0 + t) for l in range(n_layers)]
        bits = [np.stack([x[i] for x in per]).reshape(shape) for i in range(3)]
        dev = [H.dev_bf16(b) for b in bits]
        before = engs[0].launch_count()
        for e, o in zip(engs, outs):
            e.token_step(T0 + g0 + t, C, dev[0], dev[1], dev[2], o)
        if t > 0:
            assert engs[0].launch_count() - before == 1          # scores are carried in: one launch for the whole stack
        # (the two ways may give a stream a different number of warps, so partial sums merge in another order)
        assert (outs[0].float() - outs[1].float()).abs().max().item() <= 4e-3, f"step {t}: one launch and per-layer launches differ"
        pick = lambda b: np.concatenate([bf16_bits_to_f32(b).reshape(n_layers, S, d)[l, sample[l]] for l in range(n_layers)])
        res = ost.step(pick(bits[0]), pick(bits[1]), pick(bits[2]), T0 + g0 + t, C)
        got = outs[0].float().cpu().numpy().reshape(n_layers, S, d)
        n_live = engs[0]._t["n_live"].cpu().numpy()
        pos_now = engs[0]._t["pos"].cpu().numpy()
        for l in range(n_layers):
            for i, s_ in enumerate(sample[l]):
                j = l * n_sample + i
                if not alive[j]:
                    continue
                sid = l * S + s_
                g_pos = set(pos_now[sid, :n_live[sid]].tolist())
                o_pos = set(ost.rows(j)[0].tolist())
                if g_pos != o_pos:                           # only a near-tie at the selection threshold may differ
                    sc = dict(zip(res.cand_pos[j].tolist(), res.cand_score[j].tolist()))
                    theta = max(sc[p_] for p_ in res.kept_pos[j].tolist() if p_ in sc)
                    assert len(g_pos) == len(o_pos) and all(abs(sc[p_] - theta) <= 1e-6 for p_ in g_pos ^ o_pos), (t, l, s_)
                    alive[j] = False
                    continue
                assert np.abs(got[l, s_] - res.out[j]).max() <= 2e-2, (t, l, s_)
    assert alive.sum() >= alive.size - 2
    for e in engs:
        assert e.get_status()[0] == 0
        assert (e._t["n_live"].cpu().numpy() == C).all()
    same = np.sort(engs[0]._t["pos"].cpu().numpy(), axis=1) == np.sort(engs[1]._t["pos"].cpu().numpy(), axis=1)
    assert same.all(axis=1).mean() >= 0.999              # (a near-tie may fall the other way with another summation order)
    # payloads of the sampled streams, bit for bit
    for l in range(n_layers):
        for i, s_ in enumerate(sample[l]):
            j = l * n_sample + i
            if not alive[j]:
                continue
            pos, k, v = engs[0].read_stream(l * S + s_)
            opos, ok, ov = ost.rows(j)
            og, oo = np.argsort(pos.numpy()), np.argsort(opos)
            assert np.array_equal(pos.numpy()[og], opos[oo])
            assert np.array_equal(k.numpy().view(np.uint16)[og], f32_to_bf16_bits(ok)[oo])
            assert np.array_equal(v.numpy().view(np.uint16)[og], f32_to_bf16_bits(ov)[oo])


# ---------------------------------------------------------------------------
# selection under structure: clusters, exact ties, equal and zero rows, any K
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("kind", ["clusters", "duplicates", "equal", "zeros", "iid"])
@pytest.mark.parametrize("mode", ["calls", "fused", "cluster-fused"])
def test_selection_on_structured_values(kind, mode):
    H = _harness()
    T0, gh, gw, d = 4, 20, 16, 64
    w = Workload("struct", 99, 1, 1, 6, d, T0, gh, gw, 0.5, 1.0)
    n_rows = T0 + 250
    cur = T0 + 18 * gw + 5                      # local window = 21 rows, the rest are candidates
    for budget in (n_rows + 1, n_rows, n_rows - 1, 200, 120, T0 + 21 + 2, T0 + 21 + 1, 3):
        eng = H.engine_for(w, capacity=n_rows + 1, page_rows=32)
        lh = H.LayerHarness(eng, 0, oracle_cap=n_rows + 2, fused=_apply_mode(eng, mode))
        rng = np.random.default_rng(5)
        pos = np.stack([rng.permutation(np.concatenate([np.arange(T0), T0 + np.sort(rng.choice(cur - T0, n_rows - T0, replace=False))]))
                        for _ in range(6)]).astype(np.int32)
        v = np.stack([structured_values(kind, n_rows, d, seed=10 + s) for s in range(6)]).reshape(1, 6, n_rows, d)
        k = np.stack([structured_values("iid", n_rows, d, seed=20 + s) for s in range(6)]).reshape(1, 6, n_rows, d)
        lh.prefill(k, v, 0, pos)
        q, kn, vn = layer_step_qkv(w, 0, 0, cur - T0)
        lh.step(q, kn, vn, cur, budget)


@pytest.mark.parametrize("kind", ["duplicates", "equal"])
@pytest.mark.parametrize("mode", ["fused", "two-sweep-fused", "calls"])
def test_exact_ties_over_many_steps_follow_the_position_rule(kind, mode):
    """A full cache whose V rows come in identical pairs (or are all identical), stepped many times with new rows
    that repeat cached ones: at every step several candidates share the highest score exactly, so the row that
    goes is decided by position (Eq. 3 with the tie rule), also on the steps where the fused kernel would
    otherwise take the evictee the previous step noted.  Not one selection may differ from the oracle's."""
    H = _harness()
    T0, gh, gw, d = 4, 20, 16, 64
    w = Workload("ties", 93, 1, 1, 6, d, T0, gh, gw, 0.5, 1.0)
    n_rows = T0 + 250
    g0 = 17 * gw + 3
    cur0 = T0 + g0
    eng = H.engine_for(w, capacity=n_rows, page_rows=32)
    lh = H.LayerHarness(eng, 0, oracle_cap=n_rows + 2, fused=_apply_mode(eng, mode))
    rng = np.random.default_rng(7)
    recent = np.arange(cur0 - 2 * gw, cur0)                 # the cells of the local window and the row above are cached
    older = np.arange(T0, cur0 - 2 * gw)
    pos = np.stack([rng.permutation(np.concatenate([np.arange(T0), recent, np.sort(rng.choice(older, n_rows - T0 - recent.size, replace=False))]))
                    for _ in range(6)]).astype(np.int32)
    vals = np.stack([structured_values(kind, n_rows, d, seed=30 + s) for s in range(6)])
    k = np.stack([structured_values("iid", n_rows, d, seed=40 + s) for s in range(6)]).reshape(1, 6, n_rows, d)
    lh.prefill(k, vals.reshape(1, 6, n_rows, d), 0, pos)
    for t in range(2 * gw + 5):                             # across two grid-row boundaries
        q, kn, vn = layer_step_qkv(w, 3, 0, g0 + t)
        vn = vn.copy().reshape(6, d)
        if t % 3 != 2:                                      # two steps in three: the new row repeats a cached one
            for s_ in range(6):
                vn[s_] = vals[s_, (7 * t + s_) % n_rows]
        lh.step(q, kn, vn.reshape(1, 6, d), cur0 + t, n_rows)
    assert lh.stats.tolerated_divergences == 0
    assert lh.stats.steps == 2 * gw + 5


@pytest.mark.parametrize("mode", ["calls", "fused"])
def test_repeat_runs_are_bit_identical(mode):
    outs = []
    for _ in range(3):
        w = get_workload(1)
        lh, eng = _run_trajectory(w, 0, 0, lambda cur: w.capacity(), steps=160, mode=mode)
        outs.append((lh.out_f32.cpu().numpy().copy(), np.sort(eng._t["pos"][:, :w.capacity()].cpu().numpy(), axis=1)))
    for o in outs[1:]:
        assert np.array_equal(o[0], outs[0][0]) and np.array_equal(o[1], outs[0][1])


@pytest.mark.parametrize("warps,depth,ahead", [(1, 2, -1), (2, 2, -1), (3, 3, -1), (4, 2, -1), (1, 8, -1), (2, 0, -1),
                                               (2, 2, 0), (2, 2, 3), (1, 2, 5)])
def test_tensor_core_kernel_group_sizes_and_ring_depths(warps, depth, ahead):
    """The warp-group kernel with 1-4 warps per stream, several ring depths and several L2 look-ahead
    distances: a trajectory that grows, fills up and evicts, on a grid whose rows are not a multiple of
    the 32-row tile."""
    H = _harness()
    w = Workload("groups", 96, 1, 2, 3, 64, 40, 12, 11, 0.55, 1.0)
    C = w.capacity()
    for fused in (True, False):
        eng = H.engine_for(w, capacity=C, page_rows=13)
        eng.set_staged(4)
        eng.set_stream_warps(warps)
        eng.set_ring_stages(depth)
        eng.set_l2_lookahead(ahead)
        lh = H.LayerHarness(eng, 0, oracle_cap=w.l_max + 1, fused=fused)
        k, v = prefix_kv(w, 4, 0)
        lh.prefill(k, v, 0)
        for g in range(w.n_cells):
            q, kn, vn = layer_step_qkv(w, 4, 0, g)
            lh.step(q, kn, vn, w.n_text + g, C)
        assert eng.get_status()[0] == 0 and lh.stats.steps == w.n_cells


# ---------------------------------------------------------------------------
# the comparison method of Section 3.4: attention-mass pruning (score_mode 1)
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("mode", ["calls", "fused"])
@pytest.mark.parametrize("seed", [0, 1])
def test_attention_mass_mode_config1_full_trajectory(seed, mode):
    """Config 1 (its eight keys scaled x4 are made for this rule) under attention-mass pruning: masses, kept
    and evicted sets, outputs and cache contents against the oracle at every step."""
    w = get_workload(1)
    C = w.capacity()
    lh, eng = _run_trajectory(w, 0, seed, lambda cur: C, mode=mode, score_mode=1)
    assert lh.stats.steps == 256
    assert lh.stats.max_out_err <= 2e-2 and lh.mean_out_err() <= 2e-3


@pytest.mark.parametrize("d,page_rows,T0,gh,gw,beta,n_prefix", [
    (64, 7, 5, 6, 5, 0.5, None),
    (100, 5, 9, 5, 7, 0.5, None),
    (32, 3, 4, 6, 6, 0.4, 0),        # no prefix: the text rows compete too, with zero mass at first
])
def test_attention_mass_mode_small_shapes(d, page_rows, T0, gh, gw, beta, n_prefix):
    w = Workload(f"mass-d{d}", 80 + d % 7, 1, 2, 3, d, T0, gh, gw, beta, 1.0)
    C = max(2, w.capacity())
    lh, eng = _run_trajectory(w, 0, 3, lambda cur: C, page_rows=page_rows, n_prefix=n_prefix, score_mode=1)
    assert lh.stats.steps == gh * gw
    # a budget that moves: several rows go at once, survivors (and their masses) move
    lh, eng = _run_trajectory(w, 0, 4, lambda cur: C - (3 if (cur // 4) % 2 else 0), page_rows=page_rows, n_prefix=n_prefix, score_mode=1)
    assert lh.stats.steps == gh * gw


def test_attention_mass_mode_update_needs_the_attention_first():
    import paper_2506_18226_b200 as A
    H = _harness()
    w = get_workload(1)
    eng = H.engine_for(w, capacity=w.capacity(), score_mode=1)
    k, v = prefix_kv(w, 0, 0)
    eng.prefill_rows(0, H.dev_bf16(k), H.dev_bf16(v), 0)
    q, kn, vn = (H.dev_bf16(x) for x in layer_step_qkv(w, 0, 0, 0))
    eng.score(0, 120)
    eng.select(0, 120, w.capacity())
    with pytest.raises(A.AdsaError) as e:
        eng.kv_update(0, 120, kn, vn)
    assert e.value.status == A.binding.ESTATE


# ---------------------------------------------------------------------------
# granularity variant: one score per token over all heads of a layer (score_share 1)
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("d,heads,page_rows,T0,gh,gw,beta", [
    (64, 4, 16, 6, 7, 6, 0.5),
    (100, 3, 5, 9, 5, 7, 0.5),
    (32, 12, 8, 4, 6, 6, 0.4),
])
@pytest.mark.parametrize("mode", ["calls", "fused"])
def test_head_shared_selection_full_trajectory(d, heads, page_rows, T0, gh, gw, beta, mode):
    """Eq. 1-2 on a token's V over all heads: scores, kept and evicted sets (the same for every head of a
    batch row), outputs and caches against the oracle; then a budget that moves (several rows at once)."""
    w = Workload(f"shared-d{d}", 70 + d % 7, 1, 2, heads, d, T0, gh, gw, beta, 1.0)
    C = max(2, w.capacity())
    lh, eng = _run_trajectory(w, 0, 5, lambda cur: C, page_rows=page_rows, mode=mode, score_share=1)
    assert lh.stats.steps == gh * gw and lh.stats.max_score_err <= 1e-6
    pos = np.sort(eng._t["pos"][:, :C].cpu().numpy(), axis=1).reshape(w.batch, heads, C)
    assert (pos == pos[:, :1]).all()                     # every head of a batch row holds the same tokens
    lh, eng = _run_trajectory(w, 0, 6, lambda cur: C - (3 if (cur // 4) % 2 else 0), page_rows=page_rows, mode=mode, score_share=1)
    assert lh.stats.steps == gh * gw


# ---------------------------------------------------------------------------
# the one-call and host-buffer entry points agree with the four separate calls
# ---------------------------------------------------------------------------
def test_layer_step_and_host_variant_match_separate_calls():
    """adsa_layer_step (fused kernel) and its host-buffer variant are bit-identical to each other; against
    the four separate calls (different kernels, same arithmetic up to summation order) the outputs agree
    to bf16 rounding and the caches hold the same positions."""
    H = _harness()
    w = get_workload(1)
    C = w.capacity()
    engs = [H.engine_for(w, capacity=C) for _ in range(3)]
    k, v = prefix_kv(w, 0, 0)
    for e in engs:
        e.prefill_rows(0, H.dev_bf16(k), H.dev_bf16(v), 0)
    outs = [torch.zeros((w.streams_per_layer, w.head_dim), dtype=torch.bfloat16, device="cuda:0") for _ in range(2)]
    out_h = torch.zeros((w.streams_per_layer, w.head_dim), dtype=torch.bfloat16).pin_memory()
    for g in range(100):
        qb, kb, vb = layer_step_qkv(w, 0, 0, g)
        q, kn, vn = H.dev_bf16(qb), H.dev_bf16(kb), H.dev_bf16(vb)
        cur = w.n_text + g
        engs[0].score(0, cur)
        engs[0].select(0, cur, C)
        engs[0].sparse_decode_attn(0, cur, q, kn, vn, outs[0])
        engs[0].kv_update(0, cur, kn, vn)
        engs[1].layer_step(0, cur, C, q, kn, vn, outs[1])
        hq, hk, hv = (torch.from_numpy(x.view(np.int16)).view(torch.bfloat16).pin_memory() for x in (qb, kb, vb))
        engs[2].layer_step_host(0, cur, C, hq, hk, hv, out_h)
        assert torch.equal(outs[1].cpu(), out_h)
        assert (outs[0].float() - outs[1].float()).abs().max().item() <= 2e-2
    pos = [np.sort(e._t["pos"][:, :C].cpu().numpy(), axis=1) for e in engs]
    assert np.array_equal(pos[0], pos[1]) and np.array_equal(pos[1], pos[2])
    # four kernels per step against one (plus one scoring launch on the first step, nothing carried in yet)
    assert engs[0].launch_count() - 2 == 4 * 100 and engs[1].launch_count() - 2 == 100 + 1


def test_back_to_back_layers_match_serialised_launches():
    """Launches of consecutive layers overlap (the next kernel's set-up, and, when the kernel ahead serves
    another layer, its reading and selection of the cache run under the previous kernel's tail).  The
    results must be bit-identical to the same steps with the device synchronised after every launch, for
    the fused step and for the four separate calls with the layers interleaved (score and select for every
    layer, then every layer's attention back to back, then every update: what each call leaves for the next
    is stored per layer), over a trajectory that fills up and evicts.  A third way of issuing the fused
    steps alternates two streams ordered by events.  The free-running fused and four-call runs are also
    compared with the oracle following every stream of every layer."""
    H = _harness()
    from oracle import adsa_oracle as orc
    from adsa_workloads import bf16_bits_to_f32
    w = Workload("layers", 95, 3, 2, 3, 64, 24, 10, 9, 0.5, 1.0)
    C, L, S, T, d = w.capacity(), w.n_layers, w.streams_per_layer, w.n_cells, w.head_dim
    bits, qs, ks, vs = [], [], [], []
    for g in range(T):
        per = [layer_step_qkv(w, 5, l, g) for l in range(L)]
        bits.append([np.stack([x[i] for x in per]).reshape(L * S, d) for i in range(3)])
        qs.append(torch.stack([H.dev_bf16(x[0]) for x in per]))
        ks.append(torch.stack([H.dev_bf16(x[1]) for x in per]))
        vs.append(torch.stack([H.dev_bf16(x[2]) for x in per]))
    # the oracle: all L * S streams side by side (stream index = layer * S + stream within the layer)
    ost = orc.OracleStreams(L * S, d, w.l_max + 1, w.n_text, w.grid_w, w.n_text)
    pk = np.concatenate([bf16_bits_to_f32(prefix_kv(w, 5, l)[0]).reshape(S, w.n_text, d) for l in range(L)])
    pv = np.concatenate([bf16_bits_to_f32(prefix_kv(w, 5, l)[1]).reshape(S, w.n_text, d) for l in range(L)])
    ost.append_rows(pk, pv, 0)
    want = np.zeros((T, L * S, d))
    for g in range(T):
        res = ost.step(*(bf16_bits_to_f32(b) for b in bits[g]), w.n_text + g, C)
        want[g] = res.out
    want_pos = np.sort(ost.pos[:, :C], axis=1)

    side = torch.cuda.Stream()
    results = {}
    for variant in ("fused-free", "fused-synced", "fused-two-streams", "calls-free", "calls-synced"):
        eng = H.engine_for(w, capacity=C, page_rows=16)
        for l in range(L):
            k, v = prefix_kv(w, 5, l)
            eng.prefill_rows(l, H.dev_bf16(k), H.dev_bf16(v), 0)
        outs = torch.zeros((T, L, S, w.head_dim), dtype=torch.bfloat16, device="cuda:0")
        synced = variant.endswith("synced")
        main = torch.cuda.current_stream()
        for g in range(T):
            cur = w.n_text + g
            if variant == "fused-two-streams":
                for l in range(L):                  # odd layers on the side stream, each launch ordered after the one before
                    st = side if l & 1 else main
                    other = main if l & 1 else side
                    st.wait_stream(other)
                    with torch.cuda.stream(st):
                        eng.layer_step(l, cur, C, qs[g][l], ks[g][l], vs[g][l], outs[g, l])
                main.wait_stream(side)
            elif variant.startswith("fused"):
                if synced:
                    for l in range(L):
                        eng.layer_step(l, cur, C, qs[g][l], ks[g][l], vs[g][l], outs[g, l])
                        torch.cuda.synchronize()
                else:
                    eng.token_step(cur, C, qs[g], ks[g], vs[g], outs[g].view(L, w.batch, w.n_heads, w.head_dim))
            else:
                for l in range(L):
                    eng.score(l, cur)
                    eng.select(l, cur, C)
                for l in range(L):      # attention launches of consecutive layers back to back
                    eng.sparse_decode_attn(l, cur, qs[g][l], ks[g][l], vs[g][l], outs[g, l])
                    if synced:
                        torch.cuda.synchronize()
                for l in range(L):
                    eng.kv_update(l, cur, ks[g][l], vs[g][l])
        torch.cuda.synchronize()
        assert eng.get_status()[0] == 0
        n_live = eng._t["n_live"].cpu().numpy()
        pos = np.sort(eng._t["pos"][:, :C].cpu().numpy(), axis=1)
        results[variant] = (outs.cpu(), n_live, pos)
    for a, b in (("fused-free", "fused-synced"), ("fused-free", "fused-two-streams"), ("calls-free", "calls-synced")):
        assert torch.equal(results[a][0], results[b][0]), (a, b)
        assert np.array_equal(results[a][1], results[b][1]) and np.array_equal(results[a][2], results[b][2]), (a, b)
    for a in ("fused-free", "calls-free"):
        got = results[a][0].float().numpy().reshape(T, L * S, d)
        err = np.abs(got - want)
        assert err.max() <= 2e-2 and err.mean() <= 2e-3, (a, err.max(), err.mean())
        assert (results[a][1] == C).all() and np.array_equal(results[a][2], want_pos), a


def test_interleaved_layers_keep_their_own_selection():
    """score/select of two layers, then both attentions, then both updates: each layer attends and evicts by
    its own keep mask.  The layers get different budgets, so a mix-up changes the row counts."""
    H = _harness()
    w = Workload("layers2", 93, 2, 1, 4, 64, 12, 6, 6, 0.5, 1.0)
    S, d = w.streams_per_layer, w.head_dim
    eng = H.engine_for(w, capacity=w.l_max, page_rows=16)
    for l in range(2):
        k, v = prefix_kv(w, 7, l)
        eng.prefill_rows(l, H.dev_bf16(k), H.dev_bf16(v), 0)
    out = torch.zeros((2, S, d), dtype=torch.bfloat16, device="cuda:0")
    for g in range(20):                                  # grow both layers without eviction
        for l in range(2):
            q, kn, vn = (H.dev_bf16(x) for x in layer_step_qkv(w, 7, l, g))
            eng.layer_step(l, w.n_text + g, w.l_max, q, kn, vn, out[l])
    cur = w.n_text + 20
    budgets = (32, 25)                                   # 32 live rows each; layer 0 evicts 1, layer 1 evicts 8
    counts = torch.zeros((2, S, 4), dtype=torch.int32, device="cuda:0")
    qkv = [[H.dev_bf16(x) for x in layer_step_qkv(w, 7, l, 20)] for l in range(2)]
    for l in range(2):
        eng.score(l, cur)
        eng.select(l, cur, budgets[l], counts=counts[l])
    for l in range(2):
        eng.sparse_decode_attn(l, cur, *qkv[l], out[l])
    for l in range(2):
        eng.kv_update(l, cur, qkv[l][1], qkv[l][2])
    assert eng.get_status()[0] == 0
    n_live = eng._t["n_live"].cpu().numpy().reshape(2, S)
    assert (n_live[0] == 32).all() and (n_live[1] == 25).all()
    c = counts.cpu().numpy()
    assert (c[0, :, 1] == 1).all() and (c[1, :, 1] == 8).all()
    # and each layer's output is what the same layer gives when stepped on its own
    ref = H.engine_for(w, capacity=w.l_max, page_rows=16)
    for l in range(2):
        k, v = prefix_kv(w, 7, l)
        ref.prefill_rows(l, H.dev_bf16(k), H.dev_bf16(v), 0)
    o2 = torch.zeros((2, S, d), dtype=torch.bfloat16, device="cuda:0")
    for g in range(20):
        for l in range(2):
            q, kn, vn = (H.dev_bf16(x) for x in layer_step_qkv(w, 7, l, g))
            ref.layer_step(l, w.n_text + g, w.l_max, q, kn, vn, o2[l])
    for l in range(2):
        ref.score(l, cur)
        ref.select(l, cur, budgets[l])
        ref.sparse_decode_attn(l, cur, *qkv[l], o2[l])
        ref.kv_update(l, cur, qkv[l][1], qkv[l][2])
    assert torch.equal(out.cpu(), o2.cpu())
    assert np.array_equal(np.sort(eng._t["pos"].cpu().numpy(), axis=1), np.sort(ref._t["pos"].cpu().numpy(), axis=1))


@pytest.mark.parametrize("n_layers,pinned_out,chunks", [(1, True, 0), (4, True, 0), (8, False, 0), (13, True, 0), (13, False, 3)])
def test_token_step_host_matches_device_call(n_layers, pinned_out, chunks):
    """adsa_token_step_host (inputs in pinned host memory, moved in chunks of layers while other layers compute;
    the output either in pinned memory, which the kernels write themselves, or in pageable memory, which is
    filled by copies) gives bit for bit what adsa_token_step gives on device tensors, and leaves the same cache."""
    H = _harness()
    w = Workload("host", 94, n_layers, 2, 2, 64, 16, 8, 7, 0.5, 1.0)
    C, L, T = w.capacity(), w.n_layers, w.n_cells
    engs = [H.engine_for(w, capacity=C, page_rows=16) for _ in range(2)]
    for e in engs:
        for l in range(L):
            k, v = prefix_kv(w, 6, l)
            e.prefill_rows(l, H.dev_bf16(k), H.dev_bf16(v), 0)
    shape = (L, w.batch, w.n_heads, w.head_dim)
    out_d = torch.zeros(shape, dtype=torch.bfloat16, device="cuda:0")
    out_h = torch.zeros(shape, dtype=torch.bfloat16)
    if pinned_out:
        out_h = out_h.pin_memory()
    engs[1].set_host_chunks(chunks)
    for g in range(T):
        per = [layer_step_qkv(w, 6, l, g) for l in range(L)]
        bits = [np.stack([x[i] for x in per]).reshape(shape) for i in range(3)]
        dev = [H.dev_bf16(b) for b in bits]
        host = [torch.from_numpy(b.view(np.int16)).view(torch.bfloat16).pin_memory() for b in bits]
        cur = w.n_text + g
        engs[0].token_step(cur, C, dev[0], dev[1], dev[2], out_d)
        engs[1].token_step_host(cur, C, host[0], host[1], host[2], out_h)
        assert torch.equal(out_d.cpu(), out_h), f"cell {g}"
    for e in engs:
        assert e.get_status()[0] == 0
    assert torch.equal(engs[0]._t["n_live"].cpu(), engs[1]._t["n_live"].cpu())
    pos = [np.sort(e._t["pos"][:, :C].cpu().numpy(), axis=1) for e in engs]
    assert np.array_equal(pos[0], pos[1])


def test_token_step_host_full_size_waits_for_its_inputs():
    """At the per-layer size of config 4 with 12 layers, the inputs of the later layers are still crossing the bus
    when the one launch that serves the whole stack is already running: it must wait for each layer's inputs.
    Every step has new inputs and the staging buffers still hold the previous step's, so a layer read too early
    shows up as a difference from the call on device tensors."""
    H = _harness()
    from dataclasses import replace
    w = replace(get_workload(4), n_layers=12)
    C, L, T0, d = w.capacity(), 12, w.n_text, w.head_dim
    pr = _bench_page_rows(C)
    g0 = w.n_cells - 6
    engs = [H.engine_for(w, n_layers=L, capacity=C, page_rows=pr) for _ in range(2)]
    for l in range(L):
        pos, k, v = late_state(w, seed=300 + l, n_rows=C, cur_pos=T0 + g0)
        for e in engs:
            e.prefill_rows(l, H.dev_bf16(k.reshape(w.batch, w.n_heads, C, d)), H.dev_bf16(v.reshape(w.batch, w.n_heads, C, d)), 0,
                           torch.from_numpy(pos.reshape(w.batch, w.n_heads, C)).to("cuda:0"))
    shape = (L, w.batch, w.n_heads, d)
    out_d = torch.zeros(shape, dtype=torch.bfloat16, device="cuda:0")
    out_h = torch.zeros(shape, dtype=torch.bfloat16).pin_memory()
    for t in range(6):
        per = [layer_step_qkv(w, 8, l, g0 + t) for l in range(L)]
        bits = [np.stack([x[i] for x in per]).reshape(shape) for i in range(3)]
        dev = [H.dev_bf16(b) for b in bits]
        host = [torch.from_numpy(b.view(np.int16)).view(torch.bfloat16).pin_memory() for b in bits]
        engs[0].token_step(T0 + g0 + t, C, dev[0], dev[1], dev[2], out_d)
        before = engs[1].launch_count()
        engs[1].token_step_host(T0 + g0 + t, C, host[0], host[1], host[2], out_h)
        if t > 0:
            assert engs[1].launch_count() - before == 1
        assert torch.equal(out_d.cpu(), out_h), f"step {t}"
    for e in engs:
        assert e.get_status()[0] == 0


def test_gated_token_step_waits_for_its_words_and_gives_up_after_a_bounded_time():
    """adsa_token_step_gated reads a layer's inputs only after the layer's word says they have landed.  With the
    words set it equals adsa_token_step bit for bit.  With words that nothing ever sets the kernel does not hang:
    every wait runs out after a bounded time, the device status reports ADSA_DEV_COPY_TIMEOUT, the call returns,
    and after a reset the context works as before."""
    import time
    import paper_2506_18226_b200 as A
    H = _harness()
    w = Workload("gated", 95, 3, 2, 4, 64, 12, 8, 8, 0.5, 1.0)
    C, L = w.capacity(), w.n_layers
    shape = (L, w.batch, w.n_heads, w.head_dim)

    def fresh():
        e = H.engine_for(w, capacity=C, page_rows=16)
        for l in range(L):
            k, v = prefix_kv(w, 6, l)
            e.prefill_rows(l, H.dev_bf16(k), H.dev_bf16(v), 0)
        return e

    def inputs(g):
        per = [layer_step_qkv(w, 6, l, g) for l in range(L)]
        return [H.dev_bf16(np.stack([x[i] for x in per]).reshape(shape)) for i in range(3)]

    ref, eng = fresh(), fresh()
    ready = torch.zeros(L, dtype=torch.int32, device="cuda:0")
    out_r, out_g = (torch.zeros(shape, dtype=torch.bfloat16, device="cuda:0") for _ in range(2))
    for g in range(6):                                        # words written before the call: no waiting at all
        q, k, v = inputs(g)
        ready.fill_(g + 1)
        ref.token_step(w.n_text + g, C, q, k, v, out_r)
        eng.token_step_gated(w.n_text + g, C, q, k, v, out_g, ready, g + 1)
        assert torch.equal(out_r, out_g)
    assert eng.get_status()[0] == 0
    # words that stay behind: the step ends by itself and says so
    q, k, v = inputs(6)
    t0 = time.perf_counter()
    eng.token_step_gated(w.n_text + 6, C, q, k, v, out_g, ready, 1000)
    torch.cuda.synchronize()
    waited = time.perf_counter() - t0
    assert eng.get_status()[0] & A.binding.DEV_COPY_TIMEOUT
    assert 0.05 < waited < 20.0
    # the context is usable again after a reset
    eng.reset()
    for l in range(L):
        kk, vv = prefix_kv(w, 6, l)
        eng.prefill_rows(l, H.dev_bf16(kk), H.dev_bf16(vv), 0)
    ref2 = fresh()
    q, k, v = inputs(0)
    ready.fill_(5)
    ref2.token_step(w.n_text, C, q, k, v, out_r)
    eng.token_step_gated(w.n_text, C, q, k, v, out_g, ready, 5)
    assert torch.equal(out_r, out_g) and eng.get_status()[0] == 0


def test_error_paths_return_status_and_launch_nothing():
    import paper_2506_18226_b200 as A
    H = _harness()
    w = get_workload(1)
    eng = H.engine_for(w, capacity=w.capacity())
    before = eng.launch_count()
    with pytest.raises(A.AdsaError) as e:
        eng.select(0, 120, 50)                  # select before score
    assert e.value.status == A.binding.ESTATE
    eng.score(0, 120)
    with pytest.raises(A.AdsaError) as e:
        eng.select(0, 121, 50)                  # cur_pos changed inside a layer-step
    assert e.value.status == A.binding.ESTATE
    with pytest.raises(A.AdsaError) as e:
        eng.score(7, 120)                       # no such layer
    assert e.value.status == A.binding.EINVAL
    assert eng.launch_count() == before + 1
    # a pool that cannot hold the text condition is refused on the host
    small = A.AdsaEngine(n_layers=1, batch=1, n_heads=12, head_dim=64, n_text=120, grid_h=16, grid_w=16,
                         max_rows_per_stream=188, page_rows=47, n_pages=12 * 2)
    k, v = prefix_kv(w, 0, 0)
    with pytest.raises(A.AdsaError) as e:
        small.prefill_rows(0, H.dev_bf16(k), H.dev_bf16(v), 0)
    assert e.value.status == A.binding.ENOMEM
    assert small.get_status()[0] == 0

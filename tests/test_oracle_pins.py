"""Pins of the CPU oracle against what the paper and the mathematics fix.

None of these tests retypes the oracle's formulas: each compares the oracle with
a closed form, a hand-computable case, an invariant, a library routine
(torch SDPA, scikit-learn's cosine similarity), exhaustive search on tiny
inputs, or a value the paper prints (Tables 1-2).
"""
import itertools
import os

import numpy as np
import pytest
import torch

from adsa_workloads import bf16_bits_to_f32, f32_to_bf16_bits, structured_values
from oracle import adsa_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "tables_1_2_cache_rows.txt")


def _bf16(x):
    return bf16_bits_to_f32(f32_to_bf16_bits(np.asarray(x, dtype=np.float32)))


def _randn(rng, *shape):
    return _bf16(rng.standard_normal(shape))


# --------------------------------------------------------------------------
# Section 4.1 partition: local window against brute-force grid enumeration
# --------------------------------------------------------------------------
@pytest.mark.parametrize("H,W", [(1, 1), (1, 5), (5, 1), (3, 4), (4, 4), (16, 16)])
@pytest.mark.parametrize("R", [1, 2])
def test_local_window_matches_grid_neighbour_enumeration(H, W, R):
    T0 = 7
    for r in range(H):
        for c in range(W):
            cur = T0 + r * W + c
            # brute force over every cell (r2, c2): earlier in raster order, at most R rows up
            want = set()
            for r2 in range(H):
                for c2 in range(W):
                    earlier = (r2 < r) or (r2 == r and c2 < c)
                    if earlier and (r - r2) <= R:
                        want.add(T0 + r2 * W + c2)
            got = {p for p in range(cur) if orc.region(p, cur, T0, W, T0, R) == orc.REGION_LOCAL}
            assert got == want
            assert len(got) == min(r, R) * W + c
            # the two attention peaks of Fig. 2: previous token and same column one row up
            if c > 0 or r > 0:
                assert (cur - 1) in got or cur - 1 < T0
            if r > 0:
                assert (cur - W) in got
            # text rows are never local; with n_prefix = T0 they are all prefix
            assert all(orc.region(p, cur, T0, W, T0, R) == orc.REGION_PREFIX for p in range(T0))


def test_partition_is_exhaustive_and_prefix_threshold_moves():
    T0, W = 5, 4
    cur = T0 + 11
    for n_prefix in (0, 3, T0, T0 + 2):
        regions = [orc.region(p, cur, T0, W, n_prefix, 1) for p in range(cur)]
        assert all(r in (0, 1, 2) for r in regions)
        assert [r == orc.REGION_PREFIX for r in regions] == [p < n_prefix for p in range(cur)]
    # rows at or beyond the current position cannot be cached
    assert orc.region(cur, cur, T0, W, T0, 1) == orc.REGION_INVALID
    assert orc.region(-1, cur, T0, W, T0, 1) == orc.REGION_INVALID
    # while decoding the text condition itself nothing is local
    assert orc.region(2, 4, T0, W, 0, 1) == orc.REGION_PREVIOUS


# --------------------------------------------------------------------------
# Eq. 1-2: hand cases, closed forms, invariants, library routine
# --------------------------------------------------------------------------
def test_score_identical_rows_is_one_and_orthogonal_rows_is_zero():
    v = np.tile(_bf16([[0.5, -2.0, 3.0, 1.0]]), (6, 1))
    np.testing.assert_allclose(orc.score_definition(v), 1.0, atol=1e-6)
    np.testing.assert_allclose(orc.score_definition(np.eye(5, 8, dtype=np.float32) * 3.0), 0.0, atol=1e-7)


def test_score_two_orthogonal_clusters_closed_form():
    a, b = 3, 5
    e0, e1 = np.zeros(6, np.float32), np.zeros(6, np.float32)
    e0[1], e1[4] = 2.0, 0.25
    v = np.stack([e0] * a + [e1] * b)
    s = orc.score_definition(v)
    p = a + b
    np.testing.assert_allclose(s[:a], (a - 1) / (p - 1), atol=1e-6)
    np.testing.assert_allclose(s[a:], (b - 1) / (p - 1), atol=1e-6)


def test_score_antipodal_pair_and_known_angle():
    # rows: x, -x, y with y orthogonal to x  ->  S = (-1+0)/2, (-1+0)/2, 0
    v = np.array([[1, 0, 0], [-4, 0, 0], [0, 2, 0]], dtype=np.float32)
    np.testing.assert_allclose(orc.score_definition(v), [-0.5, -0.5, 0.0], atol=1e-7)
    # 60 degrees apart: cos = 1/2, p = 2 so S_i = S_ij
    v = np.array([[1, 0], [0.5, np.sqrt(3) / 2]], dtype=np.float32)
    np.testing.assert_allclose(orc.score_definition(v), [0.5, 0.5], atol=1e-6)


def test_score_zero_row_and_degenerate_sizes():
    v = np.array([[0, 0, 0], [1, 1, 0], [1, 1, 0]], dtype=np.float32)
    np.testing.assert_allclose(orc.score_definition(v), [0.0, 0.5, 0.5], atol=1e-6)
    assert orc.score_definition(np.ones((1, 4), np.float32)).tolist() == [0.0]
    assert orc.score_definition(np.zeros((0, 4), np.float32)).shape == (0,)


def test_score_matches_sklearn_cosine_similarity_offdiagonal_mean():
    from sklearn.metrics.pairwise import cosine_similarity
    rng = np.random.default_rng(3)
    for p, d in [(2, 4), (17, 64), (50, 100)]:
        v = _randn(rng, p, d)
        c = cosine_similarity(v.astype(np.float64))
        want = (c.sum(axis=1) - np.diag(c)) / (p - 1)
        np.testing.assert_allclose(orc.score_definition(v), want, atol=2e-7)


def test_score_scale_invariance_permutation_equivariance():
    rng = np.random.default_rng(4)
    v = _randn(rng, 23, 16)
    s = orc.score_definition(v)
    scales = (2.0 ** rng.integers(-3, 4, size=(23, 1))).astype(np.float32)  # exact in bf16
    np.testing.assert_allclose(orc.score_definition(v * scales), s, atol=1e-7)
    perm = rng.permutation(23)
    np.testing.assert_allclose(orc.score_definition(v[perm]), s[perm], atol=1e-7)
    # sum over i of (p-1) S_i counts every unordered pair twice
    from sklearn.metrics.pairwise import cosine_similarity
    c = cosine_similarity(v.astype(np.float64))
    np.testing.assert_allclose(s.astype(np.float64).sum() * 22, c.sum() - np.trace(c), rtol=1e-5)


@pytest.mark.parametrize("kind", ["iid", "clusters", "duplicates", "equal", "zeros"])
def test_rowsum_variant_agrees_with_definition(kind):
    v = bf16_bits_to_f32(structured_values(kind, 97, 64, seed=11))
    np.testing.assert_allclose(orc.score_rowsum(v), orc.score_definition(v), atol=1e-6)


# --------------------------------------------------------------------------
# Eq. 3: exhaustive subset search, ties, the eviction special case
# --------------------------------------------------------------------------
def _brute_force_subset(score, pos, K):
    best = None
    for sub in itertools.combinations(range(len(score)), K):
        key = (sum(float(score[i]) for i in sub), tuple(sorted(int(pos[i]) for i in sub)))
        if best is None or key < best[0]:
            best = (key, sub)
    return set(best[1]) if best else set()


def test_select_equals_argmin_over_all_subsets():
    rng = np.random.default_rng(5)
    for trial in range(30):
        p = int(rng.integers(1, 11))
        # dyadic scores: subset sums are exact, ties are frequent
        score = (rng.integers(-4, 5, size=p) / 8.0).astype(np.float32)
        pos = rng.permutation(40)[:p].astype(np.int32)
        for K in range(p + 1):
            keep = orc.select_lowest(score, pos, K)
            assert set(np.flatnonzero(keep).tolist()) == _brute_force_subset(score, pos, K)


def test_select_all_equal_scores_keeps_lowest_positions_and_clamps():
    pos = np.array([9, 2, 7, 4, 30, 1], dtype=np.int32)
    score = np.full(6, 0.25, dtype=np.float32)
    keep = orc.select_lowest(score, pos, 3)
    assert sorted(pos[keep == 1].tolist()) == [1, 2, 4]
    assert orc.select_lowest(score, pos, 0).sum() == 0
    assert orc.select_lowest(score, pos, 99).sum() == 6


def test_select_k_equals_p_minus_one_evicts_the_most_similar_token():
    # Section 4.2: when the cache is full the token most similar to the others goes
    v = np.eye(12, 16, dtype=np.float32) * 2.0   # mutually orthogonal rows: S = 0
    v[7] = v[3]                                  # rows 3 and 7 are duplicates: S = 1/(p-1) for both
    s = orc.score_definition(v)
    pos = np.arange(100, 112, dtype=np.int32)
    keep = orc.select_lowest(s, pos, 11)
    evicted = int(np.flatnonzero(keep == 0)[0])
    assert s[evicted] == s.max()
    assert evicted == 7  # equal scores: the lower position (row 3) is kept


# --------------------------------------------------------------------------
# Attention: closed forms, invariants, library routine
# --------------------------------------------------------------------------
def test_attention_closed_forms():
    d = 4
    v = np.array([[1, 2, 3, 4], [5, 6, 7, 8], [-1, 0, 1, 0]], dtype=np.float32)
    # equal keys -> uniform weights -> mean of V
    out, w = orc.attend(np.ones(d, np.float32), np.ones((3, d), np.float32), v)
    np.testing.assert_allclose(w, 1 / 3, atol=1e-12)
    np.testing.assert_allclose(out, v.mean(axis=0), atol=1e-12)
    # q = 0 -> the same
    out, _ = orc.attend(np.zeros(d, np.float32), np.arange(12, dtype=np.float32).reshape(3, d), v)
    np.testing.assert_allclose(out, v.mean(axis=0), atol=1e-12)
    # two keys whose logits differ by ln 3 -> weights 3/4 and 1/4 (scale given explicitly)
    q = np.array([1, 0, 0, 0], np.float32)
    k = np.array([[2, 9, 9, 9], [1, -5, 0, 3]], np.float32)
    out, w = orc.attend(q, k, v[:2], scale=np.log(3.0))
    np.testing.assert_allclose(w, [0.75, 0.25], atol=1e-12)
    np.testing.assert_allclose(out, 0.75 * v[0] + 0.25 * v[1], atol=1e-12)
    # default scale is 1/sqrt(d): d = 4 halves the logits, so a gap of 2 ln 3 gives 3:1 again
    k2 = np.array([[2 * np.log(3.0), 0, 0, 0], [0, 0, 0, 0]], np.float32)
    _, w = orc.attend(q, k2, v[:2])
    np.testing.assert_allclose(w, [0.75, 0.25], atol=1e-6)
    # one dominant key -> its value row
    out, _ = orc.attend(q * 100, np.array([[5, 0, 0, 0], [0, 0, 0, 0], [-5, 0, 0, 0]], np.float32), v)
    np.testing.assert_allclose(out, v[0], atol=1e-9)


def test_attention_invariants_and_sdpa():
    rng = np.random.default_rng(7)
    for n, d in [(1, 8), (37, 64), (200, 100)]:
        q, k, v = _randn(rng, d), _randn(rng, n, d), _randn(rng, n, d)
        out, w = orc.attend(q, k, v)
        assert abs(w.sum() - 1.0) < 1e-12 and (w >= 0).all()
        assert (out <= v.max(axis=0) + 1e-9).all() and (out >= v.min(axis=0) - 1e-9).all()
        # shifting every key by the same vector moves all logits equally
        out2, _ = orc.attend(q, k + _bf16(np.ones(d)), v)
        np.testing.assert_allclose(out2, out, atol=1e-9)
        ref = torch.nn.functional.scaled_dot_product_attention(
            torch.from_numpy(q.astype(np.float64))[None, None, None, :],
            torch.from_numpy(k.astype(np.float64))[None, None],
            torch.from_numpy(v.astype(np.float64))[None, None])[0, 0, 0].numpy()
        np.testing.assert_allclose(out, ref, atol=1e-10)


# --------------------------------------------------------------------------
# The layer-step: dense equivalence, set invariants, Tables 1-2
# --------------------------------------------------------------------------
def _run_steps(T0, H, W, d, budget_fn, n_prefix, seed, score_variant=0, n_streams=2):
    rng = np.random.default_rng(seed)
    L = T0 + H * W
    st = orc.OracleStreams(n_streams, d, L, T0, W, n_prefix, score_variant=score_variant)
    hist_k = np.zeros((n_streams, L, d), np.float32)
    hist_v = np.zeros((n_streams, L, d), np.float32)
    if T0:
        hist_k[:, :T0], hist_v[:, :T0] = _randn(rng, n_streams, T0, d), _randn(rng, n_streams, T0, d)
        st.append_rows(hist_k[:, :T0], hist_v[:, :T0], 0)
    log = []
    for g in range(H * W):
        cur = T0 + g
        q, kn, vn = _randn(rng, n_streams, d), _randn(rng, n_streams, d), _randn(rng, n_streams, d)
        hist_k[:, cur], hist_v[:, cur] = kn, vn
        before = [set(st.rows(s)[0].tolist()) for s in range(n_streams)]
        res = st.step(q, kn, vn, cur, budget_fn(cur))
        log.append((cur, q, before, res, st.n_live.copy()))
    return st, hist_k, hist_v, log


def test_budget_covering_the_context_is_dense_attention():
    # Section 4.2: as long as the cache has room nothing is evicted, so the method is plain dense attention
    T0, H, W, d = 6, 4, 5, 16
    st, hk, hv, log = _run_steps(T0, H, W, d, lambda cur: 10_000, T0, seed=8)
    for cur, q, before, res, n_live in log:
        assert (n_live == cur + 1).all()
        for s in range(2):
            assert len(res.evict_pos[s]) == 0
            ref = torch.nn.functional.scaled_dot_product_attention(
                torch.from_numpy(q[s].astype(np.float64))[None, None, None, :],
                torch.from_numpy(hk[s, :cur + 1].astype(np.float64))[None, None],
                torch.from_numpy(hv[s, :cur + 1].astype(np.float64))[None, None])[0, 0, 0].numpy()
            np.testing.assert_allclose(res.out[s], ref, atol=1e-10)


def test_sparse_step_attends_exactly_the_retained_rows():
    # the output must equal library attention restricted to kept_pos + the new row
    T0, H, W, d = 5, 6, 6, 8
    C = (T0 + H * W) // 2
    st, hk, hv, log = _run_steps(T0, H, W, d, lambda cur: C, T0, seed=9)
    for cur, q, before, res, n_live in log:
        for s in range(2):
            idx = np.array(sorted(res.kept_pos[s].tolist()) + [cur])
            ref = torch.nn.functional.scaled_dot_product_attention(
                torch.from_numpy(q[s].astype(np.float64))[None, None, None, :],
                torch.from_numpy(hk[s, idx].astype(np.float64))[None, None],
                torch.from_numpy(hv[s, idx].astype(np.float64))[None, None])[0, 0, 0].numpy()
            np.testing.assert_allclose(res.out[s], ref, atol=1e-10)


@pytest.mark.parametrize("n_prefix_kind", ["text", "none", "text+5%"])
def test_update_invariants(n_prefix_kind):
    T0, H, W, d = 6, 6, 5, 8
    L = T0 + H * W
    C = L // 2
    n_prefix = {"text": T0, "none": 0, "text+5%": T0 + int(np.ceil(0.05 * H * W))}[n_prefix_kind]
    st, hk, hv, log = _run_steps(T0, H, W, d, lambda cur: C, n_prefix, seed=10)
    gone = [set(), set()]
    for cur, q, before, res, n_live in log:
        g = cur - T0
        r, c = divmod(g, W)
        for s in range(2):
            kept, ev = set(res.kept_pos[s].tolist()), set(res.evict_pos[s].tolist())
            assert kept | ev == before[s] and not (kept & ev)
            assert not (ev & {p for p in before[s] if p < n_prefix})            # prefix never leaves
            local = {T0 + g2 for g2 in range(g) if r - g2 // W <= 1}
            assert local <= kept or local <= kept | {p for p in local if p < n_prefix}
            assert set(res.cand_pos[s].tolist()) == before[s] - local - set(range(n_prefix))
            mandatory = len(before[s] & (local | set(range(n_prefix))))
            assert n_live[s] == max(min(len(before[s]) + 1, C), mandatory + 1)
            assert not (before[s] & gone[s])                                     # evicted rows never return
            gone[s] |= ev
            # the evicted rows are the highest-scoring candidates
            if len(ev):
                sc = dict(zip(res.cand_pos[s].tolist(), res.cand_score[s].tolist()))
                assert min(sc[p] for p in ev) >= max([sc[p] for p in kept if p in sc] or [-np.inf])
    for s in range(2):
        pos, k, v = st.rows(s)
        assert len(set(pos.tolist())) == len(pos)
        np.testing.assert_array_equal(k, hk[s, pos])                             # payload bit-identical
        np.testing.assert_array_equal(v, hv[s, pos])


def test_step_scores_the_value_rows_and_not_the_keys():
    """Section 4.1 (the sentence before Eq. 1) takes the similarity between V rows, because rotary position
    embedding sits on Q and K; Section 4.2 evicts the row most similar to the others.  A hand case the step
    must get right: eight cached rows, all in the previous region, whose V rows are mutually orthogonal
    except that the row at position 5 is a positive multiple of the row at position 2 (cosine 1); the K rows
    are unrelated, with their own duplicate pair at positions 1 and 6.  With a budget of one row less than
    cache + new row exactly one row goes: of the two V duplicates (equal scores 1/(p-1), all others 0) the
    higher position, 5.  Scoring the keys instead would evict 6."""
    d, W = 16, 4
    rng = np.random.default_rng(21)
    v = np.zeros((8, d), np.float32)
    for i in range(8):
        v[i, i] = 2.0
    v[5] = 3.0 * v[2]
    k = _randn(rng, 8, d)
    k[6] = k[1]
    cur = 5 * W + 1                      # grid row 5: the local window is rows 4-5, positions 0..7 are "previous"
    for order in (np.arange(8), rng.permutation(8)):        # the physical order of the cache must not matter
        st = orc.OracleStreams(1, d, 16, 0, W, 0)
        st.load(0, np.arange(8)[order], k[order], v[order])
        res = st.step(_randn(rng, 1, d), _randn(rng, 1, d), _randn(rng, 1, d), cur, budget=8)
        assert res.evict_pos[0].tolist() == [5]
        assert sorted(res.kept_pos[0].tolist()) == [0, 1, 2, 3, 4, 6, 7]
        sc = dict(zip(res.cand_pos[0].tolist(), res.cand_score[0].tolist()))
        assert sc[2] == sc[5] == pytest.approx(1.0 / 7.0, abs=1e-7)
        assert all(abs(sc[p_]) < 1e-7 for p_ in (0, 1, 3, 4, 6, 7))


def test_step_scores_equal_eq_1_2_on_the_cached_value_rows():
    """Over whole trajectories with independent K and V draws: the scores the step reports for its
    candidates are Eq. 1-2 of exactly those positions' V rows (taken from the full history, which the
    step never sees), and they are not what the K rows would give."""
    T0, H, W, d = 6, 6, 5, 8
    C = (T0 + H * W) // 2
    st, hk, hv, log = _run_steps(T0, H, W, d, lambda cur: C, T0, seed=22)
    differs = 0
    for cur, q, before, res, n_live in log:
        for s in range(2):
            cp = res.cand_pos[s]
            if len(cp) == 0:
                continue
            np.testing.assert_array_equal(res.cand_score[s], orc.score_definition(hv[s, cp]))
            if len(cp) >= 3 and np.abs(res.cand_score[s] - orc.score_definition(hk[s, cp])).max() > 1e-3:
                differs += 1
    assert differs >= 20


# --------------------------------------------------------------------------
# The comparison method of Section 3.4 (attention-mass pruning, score_mode 1)
# --------------------------------------------------------------------------
def test_select_highest_equals_argmax_over_all_subsets():
    rng = np.random.default_rng(31)
    for trial in range(30):
        p = int(rng.integers(1, 11))
        score = (rng.integers(0, 9, size=p) / 8.0).astype(np.float32)      # dyadic masses: exact sums, frequent ties
        pos = rng.permutation(40)[:p].astype(np.int32)
        for K in range(p + 1):
            best = None
            for sub in itertools.combinations(range(p), K):
                key = (-sum(float(score[i]) for i in sub), tuple(sorted(int(pos[i]) for i in sub)))
                if best is None or key < best[0]:
                    best = (key, sub)
            keep = orc.select_highest(score, pos, K)
            assert set(np.flatnonzero(keep).tolist()) == (set(best[1]) if best else set())


def _run_mass_steps(T0, H, W, d, budget_fn, n_prefix, seed, n_streams=2, k_scale=None):
    rng = np.random.default_rng(seed)
    L = T0 + H * W
    st = orc.OracleStreams(n_streams, d, L, T0, W, n_prefix, score_mode=1)
    hk, hv = np.zeros((n_streams, L, d), np.float32), np.zeros((n_streams, L, d), np.float32)
    hq = np.zeros((n_streams, L, d), np.float32)
    if T0:
        hk[:, :T0], hv[:, :T0] = _randn(rng, n_streams, T0, d), _randn(rng, n_streams, T0, d)
        st.append_rows(hk[:, :T0], hv[:, :T0], 0)
    log = []
    for g in range(H * W):
        cur = T0 + g
        q, kn, vn = _randn(rng, n_streams, d), _randn(rng, n_streams, d), _randn(rng, n_streams, d)
        if k_scale is not None:
            kn = kn * np.float32(k_scale(cur))
        hq[:, cur], hk[:, cur], hv[:, cur] = q, kn, vn
        res = st.step(q, kn, vn, cur, budget_fn(cur))
        log.append((cur, res, st.n_live.copy()))
    return st, hq, hk, hv, log


def test_mass_without_eviction_is_the_column_sum_of_the_attention_matrix():
    """With room for everything the method is dense attention, and a row's mass is the sum of its softmax
    weights over the steps since its insertion: the column sums of the causal attention matrix, here from
    torch's softmax in float64.  Every step hands out a total weight of 1."""
    T0, H, W, d = 5, 5, 4, 16
    st, hq, hk, hv, log = _run_mass_steps(T0, H, W, d, lambda cur: 10_000, T0, seed=32)
    L = T0 + H * W
    for s in range(2):
        pos, k, v = st.rows(s)
        want = np.zeros(L)
        for cur in range(T0, L):
            logits = torch.from_numpy(hk[s, :cur + 1].astype(np.float64)) @ torch.from_numpy(hq[s, cur].astype(np.float64)) / np.sqrt(d)
            want[:cur + 1] += torch.softmax(logits, dim=0).numpy()
        got = st.mass[s, :len(pos)]
        np.testing.assert_allclose(got, want[pos], atol=2e-6)
        assert abs(float(got.astype(np.float64).sum()) - H * W) < 1e-4


def test_mass_is_conserved_under_eviction_and_the_least_attended_row_goes():
    T0, H, W, d = 4, 7, 6, 8
    C = (T0 + H * W) // 2
    st, hq, hk, hv, log = _run_mass_steps(T0, H, W, d, lambda cur: C, T0, seed=33)
    for s in range(2):
        lost = 0.0
        for cur, res, n_live in log:
            sc = dict(zip(res.cand_pos[s].tolist(), res.cand_score[s].tolist()))
            ev = res.evict_pos[s].tolist()
            lost += sum(sc[p_] for p_ in ev)
            if len(ev) == 1:      # cache full: exactly the least attended candidate goes, the higher position on a tie
                lo = min(sc.values())
                assert sc[ev[0]] == lo and ev[0] == max(p_ for p_, m in sc.items() if m == lo)
            kept_c = [sc[p_] for p_ in res.kept_pos[s].tolist() if p_ in sc]
            assert not ev or not kept_c or max(sc[p_] for p_ in ev) <= min(kept_c)
        n = int(st.n_live[s])
        total = float(st.mass[s, :n].astype(np.float64).sum()) + lost
        assert abs(total - H * W) < 1e-3


def test_a_key_that_draws_the_attention_survives_where_similarity_pruning_would_not_care():
    """Keys of some positions scaled x4 (the benchmark's 'global' keys) draw far more attention than the rest;
    under attention-mass pruning their rows, once candidates, carry more mass than the median candidate and
    outlive it.  The V-cosine rule of the paper is blind to key scale."""
    T0, H, W, d = 6, 10, 8, 32
    big = {T0 + 3, T0 + 11, T0 + 20}
    C = (T0 + H * W) // 2
    st, hq, hk, hv, log = _run_mass_steps(T0, H, W, d, lambda cur: C, T0, seed=34, n_streams=4,
                                          k_scale=lambda cur: 4.0 if cur in big else 1.0)
    above, seen = 0, 0
    for cur, res, n_live in log:
        for s in range(4):
            sc = dict(zip(res.cand_pos[s].tolist(), res.cand_score[s].tolist()))
            if len(sc) < 8:
                continue
            med = float(np.median(list(sc.values())))
            for p_ in big & set(sc):
                seen += 1
                above += sc[p_] > med
    assert seen > 100 and above / seen > 0.9
    for s in range(4):                       # and they are still cached at the end, in every stream
        assert big <= set(st.rows(s)[0].tolist())


# --------------------------------------------------------------------------
# Granularity variant: one score per token over all heads of a layer
# --------------------------------------------------------------------------
def _run_shared_steps(T0, Hg, W, d, n_heads, budget, seed, share):
    rng = np.random.default_rng(seed)
    L = T0 + Hg * W
    st = orc.OracleStreams(n_heads, d, L, T0, W, T0, share_heads=n_heads if share else 0)
    hv = np.zeros((n_heads, L, d), np.float32)
    hk = np.zeros((n_heads, L, d), np.float32)
    hk[:, :T0], hv[:, :T0] = _randn(rng, n_heads, T0, d), _randn(rng, n_heads, T0, d)
    st.append_rows(hk[:, :T0], hv[:, :T0], 0)
    log = []
    for g in range(Hg * W):
        cur = T0 + g
        q, kn, vn = _randn(rng, n_heads, d), _randn(rng, n_heads, d), _randn(rng, n_heads, d)
        hk[:, cur], hv[:, cur] = kn, vn
        log.append((cur, q, st.step(q, kn, vn, cur, budget)))
    return st, hk, hv, log


def test_shared_selection_scores_the_concatenated_value_rows():
    """One score per token: Eq. 1-2 on the token's V rows of all heads laid end to end (taken from the full
    history, which the step never sees); every head keeps the same tokens; each head's output is library
    attention over its own rows at those tokens."""
    T0, Hg, W, d, NH = 4, 6, 5, 8, 3
    C = (T0 + Hg * W) // 2
    st, hk, hv, log = _run_shared_steps(T0, Hg, W, d, NH, C, seed=41, share=True)
    evictions = 0
    for cur, q, res in log:
        cp = res.cand_pos[0]
        if len(cp):
            cat = np.concatenate([hv[h, cp] for h in range(NH)], axis=1)
            want = orc.score_definition(cat)
            for h in range(NH):
                assert np.array_equal(res.cand_pos[h], cp)
                np.testing.assert_array_equal(res.cand_score[h], want)
        for h in range(NH):
            assert np.array_equal(res.kept_pos[h], res.kept_pos[0]) and np.array_equal(res.evict_pos[h], res.evict_pos[0])
            idx = np.array(sorted(res.kept_pos[h].tolist()) + [cur])
            ref = torch.nn.functional.scaled_dot_product_attention(
                torch.from_numpy(q[h].astype(np.float64))[None, None, None, :],
                torch.from_numpy(hk[h, idx].astype(np.float64))[None, None],
                torch.from_numpy(hv[h, idx].astype(np.float64))[None, None])[0, 0, 0].numpy()
            np.testing.assert_allclose(res.out[h], ref, atol=1e-10)
        evictions += len(res.evict_pos[0])
    assert evictions > 5


def test_shared_selection_with_one_head_is_the_per_stream_step():
    a = _run_shared_steps(5, 5, 4, 8, 1, 12, seed=42, share=True)
    b = _run_shared_steps(5, 5, 4, 8, 1, 12, seed=42, share=False)
    for (cur, q, ra), (_, _, rb) in zip(a[3], b[3]):
        assert np.array_equal(ra.kept_pos[0], rb.kept_pos[0]) and np.array_equal(ra.cand_score[0], rb.cand_score[0])
        assert np.array_equal(ra.out, rb.out)


def test_shared_selection_sees_redundancy_that_one_head_alone_misjudges():
    """Tokens 1 and 5 have the same V in head 0 but orthogonal V in head 1; tokens 2 and 6 have the same V in
    both heads.  Over both heads the pair (2, 6) is the most redundant (cosine 1 against 1/2) and, with room for
    all but one, token 6 goes; head 0 on its own sees two equally redundant pairs and, by the position rule,
    would drop token 6 as well only by luck of the order: with the pairs swapped it drops the wrong one."""
    d, W = 8, 4
    e = np.eye(16, d, dtype=np.float32)
    def build(full_pair, half_pair):
        v0 = np.stack([e[i % d] * 2 for i in range(8)])
        v1 = np.stack([e[(i + 3) % d] * 2 for i in range(8)])
        v0[:] = 0; v1[:] = 0
        for i in range(8):
            v0[i, i] = 2.0; v1[i, (i + 1) % 8] = 2.0
        a, b = full_pair
        v0[b], v1[b] = v0[a], v1[a]
        a, b = half_pair
        v0[b] = v0[a]
        return np.stack([v0, v1])
    rng = np.random.default_rng(43)
    cur = 5 * W + 1
    for full_pair, half_pair, want in (((2, 6), (1, 5), 6), ((1, 5), (2, 6), 5)):
        v = build(full_pair, half_pair)
        st = orc.OracleStreams(2, d, 16, 0, W, 0, share_heads=2)
        for h in range(2):
            st.load(h, np.arange(8), _randn(rng, 8, d), v[h])
        res = st.step(_randn(rng, 2, d), _randn(rng, 2, d), _randn(rng, 2, d), cur, budget=8)
        assert res.evict_pos[0].tolist() == [want] and res.evict_pos[1].tolist() == [want]
    # head 0 alone: both pairs score the same, the highest position (6) goes whichever pair is the full one
    v = build((1, 5), (2, 6))
    st = orc.OracleStreams(1, d, 16, 0, W, 0)
    st.load(0, np.arange(8), _randn(rng, 8, d), v[0])
    res = st.step(_randn(rng, 1, d), _randn(rng, 1, d), _randn(rng, 1, d), cur, budget=8)
    assert res.evict_pos[0].tolist() == [6]


# --------------------------------------------------------------------------
# Prefill of the condition (dense causal attention) and 2-D rotary embedding
# --------------------------------------------------------------------------
def test_causal_attend_is_library_causal_attention():
    rng = np.random.default_rng(51)
    for n, d in [(1, 8), (17, 64), (120, 100)]:
        q, k, v = _randn(rng, n, d), _randn(rng, n, d), _randn(rng, n, d)
        out = orc.causal_attend(q, k, v)
        t = lambda x: torch.from_numpy(x.astype(np.float64))[None, None]
        ref = torch.nn.functional.scaled_dot_product_attention(t(q), t(k), t(v), is_causal=True)[0, 0].numpy()
        np.testing.assert_allclose(out, ref, atol=1e-10)
        np.testing.assert_allclose(out[0], v[0], atol=1e-12)              # the first row sees only itself


def test_rope_2d_hand_values_and_invariants():
    T0, W, d = 3, 5, 8                                   # two pairs per axis: angles index * 1 and index * base^(-1/2)
    base = 10000.0
    x = np.zeros((3, d), np.float32)
    x[:, 0] = 1.0; x[:, 2] = 1.0; x[:, 4] = 1.0; x[:, 6] = 1.0     # every pair is (1, 0)
    pos = np.array([1, T0 + 0, T0 + 2 * W + 3])          # a text token, cell (0, 0), cell (row 2, column 3)
    out = orc.rope_2d(x, pos, T0, W, base)
    np.testing.assert_allclose(out[0], x[0], atol=1e-15)             # text tokens are not rotated
    np.testing.assert_allclose(out[1], x[1], atol=1e-15)             # neither is the grid's origin
    th = base ** -0.5
    want = [np.cos(2), np.sin(2), np.cos(2 * th), np.sin(2 * th), np.cos(3), np.sin(3), np.cos(3 * th), np.sin(3 * th)]
    np.testing.assert_allclose(out[2], want, atol=1e-12)
    # a rotation: pair norms are kept
    rng = np.random.default_rng(52)
    y = _randn(rng, 40, 16)
    p = rng.integers(0, T0 + 7 * W, size=40)
    r = orc.rope_2d(y, p, T0, W)
    np.testing.assert_allclose((r.reshape(40, 8, 2) ** 2).sum(-1), (y.astype(np.float64).reshape(40, 8, 2) ** 2).sum(-1), rtol=1e-12)


def test_rope_2d_makes_the_logit_depend_on_the_grid_offset_only():
    """q.k after the embedding depends on the row and column distances of the two cells, not on where they
    lie (the reason RoPE sits on Q and K): shifting both cells by the same rows and columns changes nothing."""
    T0, W, d = 4, 9, 32
    rng = np.random.default_rng(53)
    q, k = _randn(rng, 1, d), _randn(rng, 1, d)
    cell = lambda r, c: np.array([T0 + r * W + c])
    ref = (orc.rope_2d(q, cell(3, 5), T0, W) @ orc.rope_2d(k, cell(1, 2), T0, W).T).item()
    for dr, dc in [(1, 0), (0, 3), (4, 2), (-1, -2)]:
        got = (orc.rope_2d(q, cell(3 + dr, 5 + dc), T0, W) @ orc.rope_2d(k, cell(1 + dr, 2 + dc), T0, W).T).item()
        assert abs(got - ref) < 1e-9
    other = (orc.rope_2d(q, cell(3, 5), T0, W) @ orc.rope_2d(k, cell(2, 2), T0, W).T).item()
    assert abs(other - ref) > 1e-3


def _golden_rows():
    rows = []
    with open(GOLDEN) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                t, h, w, dense, cache, red = line.split()
                rows.append((int(t), int(h), int(w), int(dense), int(cache), float(red)))
    return rows


@pytest.mark.parametrize("table,H,W,dense,cache,printed", _golden_rows())
def test_cache_sizes_of_tables_1_and_2(table, H, W, dense, cache, printed):
    assert H * W == dense
    # the reduction the paper prints next to each cache size
    assert abs((1 - cache / dense) * 100 - printed) < 0.06
    # image tokens only (T0 = 0, no text condition), fixed capacity = the printed cache size
    st, hk, hv, log = _run_steps(0, H, W, 4, lambda cur: cache, 0, seed=12, n_streams=1)
    peak = 0
    for cur, q, before, res, n_live in log:
        peak = max(peak, int(n_live[0]))
        if cur + 1 <= cache:
            assert len(res.evict_pos[0]) == 0 and n_live[0] == cur + 1           # dense until full
        else:
            assert len(res.evict_pos[0]) == 1 and n_live[0] == cache             # then one eviction per step
    assert peak == cache


# ---------------------------------------------------------------------------
# the host model's operations around the attention (Section 5: the method is integrated with LlamaGen)
# ---------------------------------------------------------------------------
def test_rmsnorm_unit_mean_square_scale_invariance_and_torch():
    import torch
    rng = np.random.default_rng(11)
    x = rng.standard_normal((5, 96)).astype(np.float32)
    w = rng.standard_normal(96).astype(np.float32)
    y = orc.rmsnorm(x, np.ones(96, np.float32), eps=0.0)
    assert np.allclose((y ** 2).mean(axis=1), 1.0, atol=1e-12)                 # unit mean square without eps
    assert np.allclose(orc.rmsnorm(4.0 * x, w, eps=0.0), orc.rmsnorm(x, w, eps=0.0), atol=1e-12)   # scale-free
    want = torch.nn.functional.rms_norm(torch.from_numpy(x).double(), (96,), torch.from_numpy(w).double(), eps=1e-5)
    assert np.allclose(orc.rmsnorm(x, w, eps=1e-5), want.numpy(), atol=1e-12)
    # hand case: x = (3, 4), w = (1, 2): mean square 12.5, y = (3, 8) / sqrt(12.5)
    y = orc.rmsnorm(np.array([[3.0, 4.0]], np.float32), np.array([1.0, 2.0], np.float32), eps=0.0)
    assert np.allclose(y, np.array([[3.0, 8.0]]) / np.sqrt(12.5), atol=1e-14)
    # eps matters for a zero row: the output is zero, not NaN
    assert np.array_equal(orc.rmsnorm(np.zeros((1, 8), np.float32), np.ones(8, np.float32), eps=1e-5), np.zeros((1, 8)))


def test_swiglu_hand_values_and_torch():
    import torch
    g = np.array([0.0, 1.0, -1.0, 20.0, -20.0], np.float32)
    u = np.array([2.0, 2.0, 2.0, 0.5, 3.0], np.float32)
    got = orc.swiglu(g, u)
    assert got[0] == 0.0
    assert np.isclose(got[1], 2.0 / (1.0 + np.exp(-1.0)), atol=1e-15)
    assert np.isclose(got[1] - got[2], 2.0, atol=1e-15)                         # silu(g) - silu(-g) = g (both times up = 2)
    assert np.isclose(got[3], 10.0, atol=1e-7) and abs(got[4]) < 1e-6             # silu -> identity / zero far out
    rng = np.random.default_rng(12)
    a, b = rng.standard_normal(200).astype(np.float32), rng.standard_normal(200).astype(np.float32)
    want = torch.nn.functional.silu(torch.from_numpy(a).double()) * torch.from_numpy(b).double()
    assert np.allclose(orc.swiglu(a, b), want.numpy(), atol=1e-14)


def test_cfg_sample_mixing_top_k_and_inverse_cdf():
    lc = np.array([1.0, 2.0, 3.0, 0.0, 3.0], np.float32)
    lu = np.array([0.0, 1.0, 0.0, 4.0, 0.0], np.float32)
    # scale 1 is the conditional logits, scale 0 the unconditional ones, scale 2 extrapolates
    for scale, want in ((1.0, lc), (0.0, lu), (2.0, 2.0 * lc - lu)):
        _, mixed, _ = orc.cfg_sample(lc, lu, scale, 5, 1.0, 0.0)
        assert np.array_equal(mixed, want.astype(np.float64))
    # top_k = 1 is the argmax, whatever u; equal maxima: the lower id
    for u in (0.0, 0.3, 0.999999):
        assert orc.cfg_sample(lc, lu, 1.0, 1, 1.0, u)[0] == 2
    # top_k = 2 at scale 1 keeps ids 2 and 4 (both 3.0): each has half of the mass
    tok, _, cdf = orc.cfg_sample(lc, lu, 1.0, 2, 1.0, 0.49)
    assert tok == 2 and np.allclose(cdf, [0.0, 0.0, 0.5, 0.5, 1.0])
    assert orc.cfg_sample(lc, lu, 1.0, 2, 1.0, 0.51)[0] == 4
    # top_k = 3: the threshold value 2.0 is unique here; ids 1, 2, 4 with weights e^-1 : 1 : 1
    tok, _, cdf = orc.cfg_sample(lc, lu, 1.0, 3, 1.0, 0.0)
    z = np.exp(-1.0) + 2.0
    assert tok == 1 and np.allclose(cdf, [0.0, np.exp(-1.0) / z, (np.exp(-1.0) + 1.0) / z, (np.exp(-1.0) + 1.0) / z, 1.0])
    # a tie AT the threshold: logits (5, 1, 1, 1), top_k = 2 keeps id 0 and the lowest of the equal ids
    tie = np.array([5.0, 1.0, 1.0, 1.0], np.float32)
    _, _, cdf = orc.cfg_sample(tie, tie, 1.0, 2, 1.0, 0.0)
    assert cdf[1] == 1.0 and cdf[0] < 1.0
    # temperature: T -> 0 concentrates on the largest kept logit, a large T flattens the kept ones
    assert orc.cfg_sample(lc, lu, 1.0, 3, 1e-3, 0.9)[0] in (2, 4)
    _, _, cdf = orc.cfg_sample(lc, lu, 1.0, 3, 1e6, 0.0)
    assert np.allclose(cdf[[1, 2, 4]], [1 / 3, 2 / 3, 1.0], atol=1e-5)


def test_cfg_sample_frequencies_follow_the_softmax_of_the_kept_logits():
    """Over a grid of u the share of each token equals its softmax probability among the kept tokens
    (torch.softmax on torch.topk as the independent statement)."""
    import torch
    rng = np.random.default_rng(13)
    lc, lu = rng.standard_normal(40).astype(np.float32), rng.standard_normal(40).astype(np.float32)
    scale, k, T = 1.75, 7, 0.8
    mixed = torch.from_numpy(lu).double() + scale * (torch.from_numpy(lc).double() - torch.from_numpy(lu).double())
    top = torch.topk(mixed, k)
    want = np.zeros(40)
    want[top.indices.numpy()] = torch.softmax(top.values / T, 0).numpy()
    n = 4000
    counts = np.zeros(40)
    for i in range(n):
        counts[orc.cfg_sample(lc, lu, scale, k, T, (i + 0.5) / n)[0]] += 1
    assert np.abs(counts / n - want).max() <= 1.0 / n + 1e-12

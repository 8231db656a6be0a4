"""Teacher-forced comparison of the CUDA path with the CPU oracle (GPU tests only).

Both sides receive the same seeded bf16 inputs.  After every layer-step the
harness compares, per stream: Eq. 2 scores, the retained/evicted position sets,
the attention output and the cache contents.  Selection is destructive, so one
tolerated near-tie (scores within 1e-6 of the selection threshold) would change
every later state: when it happens the GPU stream is overwritten with the
oracle's state before the next step and the event is counted.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np
import torch

from adsa_workloads import bf16_bits_to_f32
from oracle import adsa_oracle as orc
from paper_2506_18226_b200 import AdsaEngine

SCORE_ATOL = 1e-6        # GPU fp32 row-sum identity vs definition in double
TIE_BAND = 1e-6          # selection may differ only on scores this close to the threshold
OUT_MAX_ABS = 2e-2       # bf16 output vs oracle
OUT_MEAN_ABS = 2e-3
OUT_F32_MAX_ABS = 1e-4   # fp32 output: only summation order and exp2 vs exp differ (scaled by max|out|, >= 1)
# attention-mass mode (score_mode 1): the score is a running fp32 sum of softmax weights, one rounding of the sum and
# one of the weight (exp2, division: a few 1e-7) per step attended, so the bands are per accumulated quantity
MASS_ATOL = 2e-5


def dev_bf16(bits: np.ndarray, device="cuda:0") -> torch.Tensor:
    """uint16 bf16 patterns -> device bfloat16 tensor of the same shape."""
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).to(device).view(torch.bfloat16)


@dataclass
class Stats:
    steps: int = 0
    streams_checked: int = 0
    tolerated_divergences: int = 0
    max_score_err: float = 0.0
    max_out_err: float = 0.0
    sum_out_err: float = 0.0
    n_out: int = 0
    max_out_f32_err: float = 0.0
    log: list = field(default_factory=list)


class LayerHarness:
    """One layer of an engine next to an OracleStreams of the same streams."""

    def __init__(self, eng: AdsaEngine, layer: int, oracle_cap: int, score_variant: int = 0, sample=None,
                 fused: bool = False):
        """fused=False drives the four calls one by one; fused=True drives adsa_layer_step (one fused
        kernel carrying the scores from step to step) and reads the selection off the cache contents."""
        cfg = eng.cfg
        self.eng, self.layer, self.fused = eng, layer, fused
        self.S, self.d = eng.S, cfg.head_dim
        # sample: the streams (indices within the layer) the oracle follows; None = all
        self.sample = list(range(self.S)) if sample is None else list(sample)
        assert not cfg.score_share or sample is None, "head-shared selection: the oracle follows whole batch rows"
        self.mass_mode = cfg.score_mode == 1
        self.score_atol = MASS_ATOL if self.mass_mode else SCORE_ATOL
        self.tie_band = MASS_ATOL if self.mass_mode else TIE_BAND
        self.orc = orc.OracleStreams(len(self.sample), self.d, oracle_cap, cfg.n_text, cfg.grid_w, cfg.n_prefix,
                                     cfg.local_rows_back, float(cfg.softmax_scale), score_variant, score_mode=cfg.score_mode,
                                     share_heads=cfg.n_heads if cfg.score_share else 0)
        dev = eng.device
        R = cfg.max_rows_per_stream
        self.scores = torch.zeros((self.S, R), dtype=torch.float32, device=dev)
        self.sel_slots = torch.zeros((self.S, R), dtype=torch.int32, device=dev)
        self.sel_pos = torch.zeros((self.S, R), dtype=torch.int32, device=dev)
        self.evict_pos = torch.zeros((self.S, R), dtype=torch.int32, device=dev)
        self.counts = torch.zeros((self.S, 4), dtype=torch.int32, device=dev)
        self.out_bf16 = torch.zeros((self.S, self.d), dtype=torch.bfloat16, device=dev)
        self.out_f32 = torch.zeros((self.S, self.d), dtype=torch.float32, device=dev)
        self.stats = Stats()

    # -- loading -----------------------------------------------------------
    def prefill(self, k_bits, v_bits, first_pos=0, pos=None):
        """k_bits, v_bits: uint16 [batch, heads, n, d]; pos: optional int32 [S, n]."""
        n = k_bits.shape[2]
        kd, vd = dev_bf16(k_bits, self.eng.device), dev_bf16(v_bits, self.eng.device)
        pd = None if pos is None else torch.from_numpy(np.ascontiguousarray(pos, dtype=np.int32)).to(self.eng.device)
        self.eng.prefill_rows(self.layer, kd, vd, first_pos, pd)
        kf = bf16_bits_to_f32(k_bits).reshape(self.S, n, self.d)
        vf = bf16_bits_to_f32(v_bits).reshape(self.S, n, self.d)
        for i, s in enumerate(self.sample):
            p = np.arange(first_pos, first_pos + n) if pos is None else pos[s]
            a = int(self.orc.n_live[i])
            self.orc.pos[i, a:a + n] = p
            self.orc.k[i, a:a + n] = kf[s]
            self.orc.v[i, a:a + n] = vf[s]
            self.orc.n_live[i] = a + n

    def _resync(self, i, s):
        pos, k, v = self.orc.rows(i)
        self.orc.load(i, pos, k, v)          # (attention-mass mode: a reloaded stream starts from zero mass on both sides)
        from adsa_workloads import f32_to_bf16_bits
        b, h = divmod(s, self.eng.cfg.n_heads)
        dev = self.eng.device
        self.eng.set_stream_rows(self.layer, b, h, dev_bf16(f32_to_bf16_bits(k), dev), dev_bf16(f32_to_bf16_bits(v), dev),
                                 torch.from_numpy(pos.astype(np.int32)).to(dev))

    # -- one step ----------------------------------------------------------
    def step(self, q_bits, k_bits, v_bits, cur_pos, budget, check_state=True, n_threads=0):
        eng, L, S, d = self.eng, self.layer, self.S, self.d
        dev = eng.device
        q, kn, vn = dev_bf16(q_bits, dev), dev_bf16(k_bits, dev), dev_bf16(v_bits, dev)
        self.scores.fill_(float("nan"))
        eng.score(L, cur_pos, self.scores)           # fused: the scores carried in from the previous step
        sid0 = eng.stream_index(L, 0, 0)
        pos_before = eng._t["pos"][sid0:sid0 + S].cpu().numpy()
        n_before = eng._t["n_live"][sid0:sid0 + S].cpu().numpy()
        if self.fused:
            eng.layer_step(L, cur_pos, budget, q, kn, vn, self.out_bf16)
            self.out_f32.copy_(self.out_bf16.float())
            pos_after = eng._t["pos"][sid0:sid0 + S].cpu().numpy()
            n_after = eng._t["n_live"][sid0:sid0 + S].cpu().numpy()
        else:
            eng.select(L, cur_pos, budget, self.sel_slots, self.sel_pos, self.evict_pos, self.counts)
            eng.sparse_decode_attn(L, cur_pos, q, kn, vn, self.out_bf16, self.out_f32)
            eng.kv_update(L, cur_pos, kn, vn)

        qf = bf16_bits_to_f32(q_bits).reshape(S, d)[self.sample]
        kf = bf16_bits_to_f32(k_bits).reshape(S, d)[self.sample]
        vf = bf16_bits_to_f32(v_bits).reshape(S, d)[self.sample]
        res = self.orc.step(qf, kf, vf, cur_pos, budget, n_threads=n_threads)

        scores = self.scores.cpu().numpy()
        counts = self.counts.cpu().numpy()
        sel_pos = self.sel_pos.cpu().numpy()
        evict_pos = self.evict_pos.cpu().numpy()
        out_bf16 = self.out_bf16.float().cpu().numpy()
        out_f32 = self.out_f32.cpu().numpy()
        st = self.stats
        st.steps += 1
        diverged = []
        step_err_sum, step_err_n = 0.0, 0
        for i, s in enumerate(self.sample):
            st.streams_checked += 1
            n = int(n_before[s])
            if self.fused:
                before = set(pos_before[s, :n].tolist())
                after = pos_after[s, :int(n_after[s])].tolist()
                assert len(set(after)) == len(after) and cur_pos in after, (cur_pos, s)
                g_keep = set(after) - {cur_pos}
                g_ev = before - g_keep
                assert g_keep <= before, (cur_pos, s)
                n_keep, n_ev = len(g_keep), len(g_ev)
                p = int(np.count_nonzero(~np.isnan(scores[s, :n])))
            else:
                p, n_ev, n_keep, K = (int(x) for x in counts[s])
                g_keep, g_ev = set(sel_pos[s, :n_keep].tolist()), set(evict_pos[s, :n_ev].tolist())
            assert n_keep + n_ev == n, (cur_pos, s, n_keep, n_ev, n)
            assert p == len(res.cand_pos[i]), (cur_pos, s, p, len(res.cand_pos[i]))
            # Eq. 2 scores, matched by position
            slot_of = {int(pp): j for j, pp in enumerate(pos_before[s, :n])}
            if p:
                g = np.array([scores[s, slot_of[int(pp)]] for pp in res.cand_pos[i]], dtype=np.float64)
                err = float(np.max(np.abs(g - res.cand_score[i].astype(np.float64))))
                st.max_score_err = max(st.max_score_err, err)
                assert err <= self.score_atol, f"score mismatch {err} at pos {cur_pos} stream {s}"
            # Eq. 3 + always-kept regions: retained / evicted position sets
            o_keep, o_ev = set(res.kept_pos[i].tolist()), set(res.evict_pos[i].tolist())
            assert len(g_keep) == n_keep and len(g_ev) == n_ev
            assert g_keep | g_ev == o_keep | o_ev
            if g_keep != o_keep:
                assert len(g_keep) == len(o_keep), f"retained set sizes differ at pos {cur_pos} stream {s}"
                sc = dict(zip(res.cand_pos[i].tolist(), res.cand_score[i].tolist()))
                kept_sc = [sc[pp] for pp in o_keep if pp in sc]
                theta = (min(kept_sc) if self.mass_mode else max(kept_sc)) if kept_sc else float('-inf')
                for pp in g_keep ^ o_keep:
                    assert abs(sc[pp] - theta) <= self.tie_band, \
                        f"selection differs outside the tie band at pos {cur_pos} stream {s}: {sc[pp]} vs {theta}"
                st.tolerated_divergences += 1
                st.log.append((cur_pos, s, sorted(g_keep ^ o_keep)))
                diverged.append((i, s))
                continue
            # attention output
            e16 = np.abs(out_bf16[s] - res.out[i])
            e32 = np.abs(out_f32[s] - res.out[i])
            st.max_out_err = max(st.max_out_err, float(e16.max()))
            st.max_out_f32_err = max(st.max_out_f32_err, float(e32.max()))
            st.sum_out_err += float(e16.sum())
            st.n_out += e16.size
            step_err_sum += float(e16.sum())
            step_err_n += e16.size
            assert e16.max() <= OUT_MAX_ABS, f"attention mismatch {e16.max()} at pos {cur_pos} stream {s}"
            scale = max(1.0, float(np.abs(res.out[i]).max()))
            assert self.fused or e32.max() <= OUT_F32_MAX_ABS * scale, \
                f"fp32 attention mismatch {e32.max()} at pos {cur_pos} stream {s}"
        # the mean is taken over the output tensor of the call ([batch, heads, d]), as the max is
        assert step_err_sum <= OUT_MEAN_ABS * max(1, step_err_n), \
            f"mean attention error {step_err_sum / max(1, step_err_n)} at pos {cur_pos}"
        for i, s in diverged:
            self._resync(i, s)
        if check_state:
            self.check_state(skip={s for _, s in diverged})
        return res

    def check_state(self, skip=()):
        """Cache contents as a set keyed by position, payloads bit-identical."""
        from adsa_workloads import f32_to_bf16_bits
        eng = self.eng
        for i, s in enumerate(self.sample):
            if s in skip:
                continue
            b, h = divmod(s, eng.cfg.n_heads)
            pos, k, v = eng.read_stream(eng.stream_index(self.layer, b, h))
            opos, ok, ov = self.orc.rows(i)
            order_g, order_o = np.argsort(pos.numpy()), np.argsort(opos)
            assert np.array_equal(pos.numpy()[order_g], opos[order_o]), f"cache positions differ, stream {s}"
            assert np.array_equal(k.numpy().view(np.uint16)[order_g], f32_to_bf16_bits(ok)[order_o]), f"K payload, stream {s}"
            assert np.array_equal(v.numpy().view(np.uint16)[order_g], f32_to_bf16_bits(ov)[order_o]), f"V payload, stream {s}"

    def mean_out_err(self):
        return self.stats.sum_out_err / max(1, self.stats.n_out)


def engine_for(w, n_layers=None, page_rows=None, capacity=None, extra_rows=0, **kw) -> AdsaEngine:
    """An engine shaped like workload `w` (optionally fewer layers)."""
    from adsa_workloads import pick_page_rows
    cap = w.capacity() if capacity is None else capacity
    max_rows = max(cap, w.n_text + 2 * w.grid_w) + extra_rows
    pr = pick_page_rows(cap) if page_rows is None else page_rows
    return AdsaEngine(n_layers=w.n_layers if n_layers is None else n_layers, batch=w.batch, n_heads=w.n_heads,
                      head_dim=w.head_dim, n_text=w.n_text, grid_h=w.grid_h, grid_w=w.grid_w,
                      max_rows_per_stream=max_rows, page_rows=pr, **kw)

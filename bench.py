#!/usr/bin/env python
"""Benchmark of the ADSA decode-attention hot path on B200.

A *step* is one decoded image token for the whole batch: every layer runs score ->
select -> sparse decode attention -> cache update (libadsa's adsa_token_step).  The
workload is a LlamaGen-shaped attention stack on synthetic seeded q/k/v (no dataset,
no trained weights); the default is the XL shape (36 layers, batch 32 = 16 prompts x CFG,
20 heads x 64, 120 text rows + a 32x32 grid, budget 50 %).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfgN] [--beta B]
  python bench.py --impl reference ...      # times the CPU oracle instead (a deliberately slow program)

The timed region is the LAST K grid cells of a generation (cache full: the most expensive
cells); the cells before them are decoded untimed first, which is also the warm-up.  With
the default K = H*W the whole generation is timed and a full untimed generation precedes it.
One JSON line is printed by rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402
import torch  # noqa: E402

from adsa_workloads import get_workload, late_state, pick_page_rows  # noqa: E402

METRIC, UNIT = "image_tokens_per_s", "image-tokens/s"
INPUT_RING_BYTES = 24 << 30   # q/k/v for all steps are kept in HBM up to this size, else a ring of steps is cycled

# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) from the ncu captures summarised
# under profiles/, keyed by workload; None where no capture of the current kernel exists.
STEP_DRAM_TRAFFIC_BYTES = {"cfg4": 98622720 + 3850112}    # profiles/step_kernel_cfg4_2layers.md
ATTN_DRAM_TRAFFIC_BYTES = {"cfg4": 94057600 + 3473536}     # profiles/attn_kernel_cfg4_2layers.md


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg4")
    ap.add_argument("--beta", type=float, default=None)
    ap.add_argument("--layers", type=int, default=None, help="override the layer count (small profiling cases)")
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--chunk-rows", type=int, default=0, help="override rows per attention chunk (0 = automatic)")
    ap.add_argument("--page-rows", type=int, default=0, help="rows per pool page (0 = the largest divisor of the capacity up to 128)")
    ap.add_argument("--kernel-mode", type=int, default=1,
                    help="0 streaming, 1 automatic, 2 cluster, 3 persistent on CUDA cores, 4 persistent with MMA")
    ap.add_argument("--stream-warps", type=int, default=0, help="warps per stream of the tensor-core kernel (0 = automatic)")
    ap.add_argument("--l2-ahead", type=int, default=-1, help="tiles per warp asked into L2 beyond the ring (-1 = automatic)")
    ap.add_argument("--sweep-mode", type=int, default=2, help="adsa_set_single_sweep: 0 two sweeps, 1 single sweep, 2 single sweep + carried evictee")
    ap.add_argument("--token-launch", type=int, default=1, help="adsa_set_token_launch: 1 one launch per token, 0 one launch per layer")
    ap.add_argument("--next-tiles", type=int, default=-1, help="adsa_set_next_layer_hint (-1 = the library's default)")
    ap.add_argument("--ring-stages", type=int, default=0, help="cap on the persistent kernel's ring (0 = as many as fit)")
    ap.add_argument("--profiler-range", action="store_true",
                    help="bracket the timed region with cudaProfilerStart/Stop (for `ncu --profile-from-start off`)")
    return ap.parse_args()


def _workload(args):
    from dataclasses import replace
    w = get_workload(int(args.workload.replace("cfg", "")), args.beta)
    return w if args.layers is None else replace(w, n_layers=args.layers, name=f"{w.name}-{args.layers}layers")


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


# --------------------------------------------------------------------------------------
# multi-process aggregation (replicas only: the path shards by nothing, ranks are independent)
# --------------------------------------------------------------------------------------
def aggregate(ms_local: float, units_local: float, world: int):
    """(max over ranks of the time, sum over ranks of the units).  Uses the default process group."""
    if world == 1:
        return ms_local, units_local
    import torch.distributed as dist
    dev = torch.device("cuda", torch.cuda.current_device()) if dist.get_backend() == "nccl" else torch.device("cpu")
    t = torch.tensor([ms_local], dtype=torch.float64, device=dev)
    u = torch.tensor([units_local], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


class ClockSampler:
    """nvidia-smi clock/throttle samples of one GPU while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.proc = index, None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "100", "-i", str(self.index)], stdout=subprocess.PIPE, text=True)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        out = self.proc.communicate()[0]
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except ValueError:
                continue
            for n, val in zip(names, f[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# --------------------------------------------------------------------------------------
# the CUDA path
# --------------------------------------------------------------------------------------
def make_inputs(w, n_steps, dev, seed):
    """Seeded N(0, sigma^2) bf16 q/k/v [n_steps, L, batch, heads, d] and the text-condition rows, in HBM."""
    g = torch.Generator(device=dev).manual_seed(seed)
    shape = (w.n_layers, w.batch, w.n_heads, w.head_dim)
    per_step = 3 * int(np.prod(shape)) * 2
    ring = min(n_steps, max(8, INPUT_RING_BYTES // per_step))
    qkv = [torch.empty((ring,) + shape, dtype=torch.bfloat16, device=dev) for _ in range(3)]
    for t in qkv:
        for i in range(ring):
            t[i] = (torch.randn(shape, generator=g, device=dev) * w.sigma).to(torch.bfloat16)
    pshape = (w.n_layers, w.batch, w.n_heads, w.n_text, w.head_dim)
    pk = (torch.randn(pshape, generator=g, device=dev) * w.sigma).to(torch.bfloat16)
    pv = (torch.randn(pshape, generator=g, device=dev) * w.sigma).to(torch.bfloat16)
    return qkv, (pk, pv), ring


def run_ours(args, rank, world, local_rank):
    from paper_2506_18226_b200 import AdsaEngine

    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    w = _workload(args)
    C, HW, T0, L = w.capacity(), w.n_cells, w.n_text, w.n_layers
    K = HW if args.steps is None else max(1, args.steps)
    W = max(3, args.warmup)
    # Large pages keep a stream's rows contiguous, so that one TMA box covers a whole tile; the default is
    # the largest divisor of the capacity up to 1024 rows (cfg4: one 572-row page per stream), which also
    # makes a full stream occupy whole pages: pool bytes = the budget's share of dense, exactly.
    pr = args.page_rows if args.page_rows else pick_page_rows(C, hi=1024)
    pages_per_stream = -(-C // pr)
    eng = AdsaEngine(n_layers=L, batch=w.batch, n_heads=w.n_heads, head_dim=w.head_dim, n_text=T0, grid_h=w.grid_h,
                     grid_w=w.grid_w, max_rows_per_stream=max(C, T0 + 2 * w.grid_w), page_rows=pr,
                     n_pages=L * w.streams_per_layer * max(pages_per_stream, -(-(T0 + 2 * w.grid_w) // pr)),
                     device=str(dev))
    if args.chunk_rows:
        eng.set_attn_chunk_rows(args.chunk_rows)
    eng.set_staged(args.kernel_mode)
    if args.sweep_mode != 2:
        eng.set_single_sweep(args.sweep_mode)
    eng.set_token_launch(args.token_launch)
    if args.next_tiles >= 0:
        eng.set_next_layer_hint(args.next_tiles)
    if args.ring_stages:
        eng.set_ring_stages(args.ring_stages)
    if args.l2_ahead >= 0:
        eng.set_l2_lookahead(args.l2_ahead)
    if args.stream_warps:
        eng.set_stream_warps(args.stream_warps)
    (q, k, v), (pk, pv), ring = make_inputs(w, HW, dev, args.seed + 1000 * rank)
    out = torch.zeros((2, L, w.batch, w.n_heads, w.head_dim), dtype=torch.bfloat16, device=dev)

    def start_generation():
        eng.reset()
        if T0:
            for l in range(L):
                eng.prefill_rows(l, pk[l], pv[l], 0)

    def decode(g):
        eng.token_step(T0 + g, C, q[g % ring], k[g % ring], v[g % ring], out[g & 1])

    # ---- warm-up generation; its last cells also time the attention kernel on its own ----------
    M = min(8, HW // 2)
    start_generation()
    for g in range(HW - 2 * M):
        decode(g)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    # the fused layer-step kernel on its own, cache full: L launches per cell, each a different layer's KV
    step_ms, step_launches = 0.0, 0
    for g in range(HW - 2 * M, HW - M):
        torch.cuda.synchronize(dev)
        n0 = eng.launch_count()
        e0.record()
        decode(g)
        e1.record()
        torch.cuda.synchronize(dev)
        step_ms += e0.elapsed_time(e1)
        step_launches += eng.launch_count() - n0
    rows_step = int(eng._t["n_live"].max().item())
    # (the keep mask and counts are stored per layer, so grouping the calls like this is a valid trajectory: every
    # layer attends and evicts by its own selection; the timed generation below starts from a reset all the same)
    attn_ms, attn_launches = 0.0, 0
    call_ms = {"adsa_score": [], "adsa_select": [], "adsa_sparse_decode_attn": [], "adsa_kv_update": []}
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(5)]
    for g in range(HW - M, HW):
        cur, r = T0 + g, g % ring
        ev[0].record()
        for l in range(L):
            eng.score(l, cur)
        ev[1].record()
        for l in range(L):
            eng.select(l, cur, C)
        ev[2].record()
        for l in range(L):                          # L launches back to back, each reads a different layer's KV
            eng.sparse_decode_attn(l, cur, q[r, l], k[r, l], v[r, l], out[g & 1, l])
        ev[3].record()
        for l in range(L):
            eng.kv_update(l, cur, k[r, l], v[r, l])
        ev[4].record()
        torch.cuda.synchronize(dev)
        attn_ms += ev[2].elapsed_time(ev[3])
        attn_launches += L
        if g > HW - M:      # in the first of these cells the scores were left behind by the fused step: no score kernel runs
            for i, name in enumerate(call_ms):
                call_ms[name].append(ev[i].elapsed_time(ev[i + 1]) * 1e3 / L)
    status, _ = eng.get_status()
    assert status == 0, f"device status {status} after the warm-up generation"
    n_live = eng._t["n_live"]
    rows_full = int(n_live.max().item())
    assert int(n_live.min().item()) == rows_full == min(C, T0 + HW)
    peak_pool_bytes = eng.pool_bytes_peak()

    # ---- timed: the last K cells of a generation ----------------------------------------------
    start_generation()
    first = (HW - K) % HW if K % HW else 0
    for g in range(first):
        decode(g)
    torch.cuda.synchronize(dev)
    if world > 1:
        torch.distributed.barrier()
    sampler = ClockSampler(local_rank if "CUDA_VISIBLE_DEVICES" not in os.environ else
                           os.environ["CUDA_VISIBLE_DEVICES"].split(",")[local_rank])
    sampler.start()
    launches0 = eng.launch_count()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if args.profiler_range:
        torch.cuda.profiler.start()
    t0.record()
    g = first
    cell_ev = []                                    # one event per cell: where in the generation the time goes
    for _ in range(K):
        if g == HW:                                 # K > H*W: start another generation inside the timed region
            start_generation()
            g = 0
        decode(g)
        g += 1
        if K <= 4096:
            e = torch.cuda.Event(enable_timing=True)
            e.record()
            cell_ev.append((g - 1, e))
    t1.record()
    torch.cuda.synchronize(dev)
    if args.profiler_range:
        torch.cuda.profiler.stop()
    if world > 1:
        torch.distributed.barrier()
    ms_local = t0.elapsed_time(t1)
    clocks = sampler.stop()
    launches = eng.launch_count() - launches0
    status, _ = eng.get_status()
    assert status == 0, f"device status {status} after the timed region"

    prompts = w.batch // 2 if w.batch >= 2 else w.batch
    ms, tokens = aggregate(ms_local, float(prompts * K), world)

    # ---- end to end: same cells through the host-buffer entry point -----------------------------
    e2e = None
    if not args.no_e2e:
        Ke = min(K, 256, HW)
        start_generation()
        for g in range(HW - Ke):
            decode(g)
        shape = (L, w.batch, w.n_heads, w.head_dim)
        hq, hk, hv = (torch.empty((Ke,) + shape, dtype=torch.bfloat16).pin_memory() for _ in range(3))
        for i, g in enumerate(range(HW - Ke, HW)):
            hq[i].copy_(q[g % ring]); hk[i].copy_(k[g % ring]); hv[i].copy_(v[g % ring])
        ho = torch.empty(shape, dtype=torch.bfloat16).pin_memory()
        torch.cuda.synchronize(dev)
        if world > 1:
            torch.distributed.barrier()
        tw = time.perf_counter()
        for i, g in enumerate(range(HW - Ke, HW)):
            eng.token_step_host(T0 + g, C, hq[i], hk[i], hv[i], ho)      # synchronises: the result is on the host
        e2e_ms_local = (time.perf_counter() - tw) * 1e3
        e2e_ms, e2e_tokens = aggregate(e2e_ms_local, float(prompts * Ke), world)
        per = int(np.prod(shape)) * 2
        e2e = {"value": e2e_tokens / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": 3 * per,
               "d2h_bytes_per_step": per, "steps": Ke, "ms_per_step": e2e_ms / Ke,
               "api": "adsa_token_step_host (pinned host q/k/v in, host output out, copies in chunks of layers under the "
                      "compute, one sync per token)"}

    if rank != 0:
        return
    # per call (cache full, median over cells, per layer) and per cell of the timed generation
    detail = {"per_call_us_cache_full": {n: float(np.median(v)) for n, v in call_ms.items() if v}}
    if detail["per_call_us_cache_full"]:
        detail["per_call_us_cache_full"]["four_call_sequence"] = float(sum(detail["per_call_us_cache_full"].values()))
    if len(cell_ev) >= 48 and K == HW and first == 0:
        prev, per_cell = t0, {}
        for gcell, e in cell_ev:
            per_cell[gcell] = prev.elapsed_time(e) * 1e3 / L
            prev = e
        span = lambda a: float(np.median([per_cell[i] for i in range(a, a + 16)]))
        detail["fused_layer_step_us_by_cell"] = {"start_cells_0_15": span(0), "middle": span(HW // 2 - 8),
                                                  "end_last_16": span(HW - 16),
                                                  "rows_at": {"start": T0 + 1, "middle": min(C, T0 + HW // 2), "end": min(C, T0 + HW)}}
    # ---- rooflines, steady state (cache full, one eviction per step) ----------------------------
    # The dominant kernel is the fused layer-step (one launch per layer-step: select, attend, the next
    # step's scores, update).  Algorithmic bytes per stream: retained rows x (K + V) + 16 B of metadata per
    # live row (position, carried score, inverse norm read; next score written) + q, k_new, v_new, out and
    # the new row's K and V.  The attention kernel alone (adsa_sparse_decode_attn) is reported beside it.
    peak, peak_kind = peaks()
    d2 = w.head_dim * 2
    retained = rows_full - 1 if rows_full == C else rows_full          # one eviction per step once full
    step_bytes = w.streams_per_layer * (retained * 2 * d2 + rows_step * 16 + 6 * d2)
    step_us = step_ms * 1e3 / max(1, step_launches)
    step_gbs = step_bytes / (step_us * 1e-6) / 1e9
    roofline = {"bound": "hbm", "kernel": "fused layer-step (adsa_layer_step / adsa_token_step)", "achieved": step_gbs,
                "peak": peak, "unit": "GB/s", "frac": step_gbs / peak, "peak_kind": f"of {peak_kind}",
                "frac_of_nominal_8000": step_gbs / 8000.0, "us_per_launch": step_us, "launches_timed": step_launches,
                "algorithmic_bytes_per_launch": step_bytes, "traffic": STEP_DRAM_TRAFFIC_BYTES.get(args.workload)}
    attn_bytes = w.streams_per_layer * (retained * 2 * d2 + 4 * d2)
    attn_us = attn_ms * 1e3 / attn_launches
    achieved = attn_bytes / (attn_us * 1e-6) / 1e9
    roofline_attn = {"bound": "hbm", "kernel": "attention alone (adsa_sparse_decode_attn)", "achieved": achieved,
                     "peak": peak, "unit": "GB/s", "frac": achieved / peak, "peak_kind": f"of {peak_kind}",
                     "frac_of_nominal_8000": achieved / 8000.0, "us_per_launch": attn_us,
                     "launches_timed": attn_launches, "algorithmic_bytes_per_launch": attn_bytes,
                     "traffic": ATTN_DRAM_TRAFFIC_BYTES.get(args.workload)}

    line = {
        "metric": METRIC, "value": tokens / (ms * 1e-3), "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
        "data": "synthetic", "impl": "ours",
        "config": {"workload": w.name, "layers": L, "batch": w.batch, "heads": w.n_heads, "head_dim": w.head_dim,
                   "n_text": T0, "grid": [w.grid_h, w.grid_w], "budget_fraction": w.beta, "capacity_rows": C,
                   "page_rows": pr, "storage": "bf16 KV pool, fp32 arithmetic", "parallelism": "replicas only",
                   "cells_timed": [first, first + K] if K <= HW else "whole generations",
                   "l2": "inputs larger than L2: every step sweeps the whole KV pool "
                         f"({peak_pool_bytes / 1e9:.2f} GB) against 126 MB of L2",
                   "inputs": f"q/k/v ring of {ring} steps resident in HBM"},
        "us_per_layer_step": ms * 1e3 / (K * L),
        "batch_rows_per_s": tokens / (ms * 1e-3) * (w.batch / prompts),
        "gpu_launches": launches, "clocks": clocks, "roofline": roofline, "roofline_attn": roofline_attn,
        "detail": detail,
        # peak_bytes counts whole pool rows (row_stride elements: d rounded up to a 16-byte multiple);
        # payload_bytes the d elements of each row, which is what dense_bytes counts
        "kv_pool": {"peak_bytes": peak_pool_bytes, "dense_bytes": w.dense_kv_bytes(),
                    "ratio": peak_pool_bytes / w.dense_kv_bytes(),
                    "payload_bytes": peak_pool_bytes * w.head_dim // eng.cfg.row_stride,
                    "payload_ratio": peak_pool_bytes * w.head_dim / eng.cfg.row_stride / w.dense_kv_bytes(),
                    "row_stride": eng.cfg.row_stride, "budget_fraction": w.beta},
    }
    if e2e:
        line["e2e"] = e2e
    if world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline(w, C, args.seed, budget_s=15.0)
    print(json.dumps(line), flush=True)


# --------------------------------------------------------------------------------------
# the CPU oracle as a timed baseline (the only place outside tests that runs oracle/)
# --------------------------------------------------------------------------------------
def _oracle_state(w, C, seed, n_streams):
    from adsa_workloads import bf16_bits_to_f32
    from oracle import adsa_oracle as orc
    cur = w.n_text + w.n_cells - w.grid_w // 2 - 1       # a late cell, mid-row: cache full, one eviction per step
    ids = list(range(n_streams))
    pos, k, v = late_state(w, seed, C, cur, streams=ids)
    st = orc.OracleStreams(n_streams, w.head_dim, C + 2, w.n_text, w.grid_w, w.n_text)
    rng = np.random.Generator(np.random.Philox(key=[seed, 0xBE7C]))
    qkv = [bf16_bits_to_f32(_bf16(rng.standard_normal((n_streams, w.head_dim), dtype=np.float32) * np.float32(w.sigma)))
           for _ in range(3)]
    return st, (pos, bf16_bits_to_f32(k), bf16_bits_to_f32(v)), qkv, cur


def _bf16(x):
    from adsa_workloads import f32_to_bf16_bits
    return f32_to_bf16_bits(x)


def _oracle_step_seconds(st, state, qkv, cur, C, n_threads):
    pos, k, v = state
    for s in range(st.n_streams):
        st.load(s, pos[s], k[s], v[s])
    t = time.perf_counter()
    st.step(qkv[0], qkv[1], qkv[2], cur, C, n_threads=n_threads)
    return time.perf_counter() - t


def cpu_baseline(w, C, seed, budget_s):
    """The oracle as it stands, on the host cores: one layer-step (Eq. 1-2 by definition, Eq. 3,
    attention, update) over a sample of streams at a late cell, extrapolated to all streams and layers."""
    from oracle import adsa_oracle as orc
    threads = orc.max_threads()
    n = min(w.streams_per_layer, max(threads, 8))
    st, state, qkv, cur = _oracle_state(w, C, seed, n)
    t_probe = _oracle_step_seconds(st, state, qkv, cur, C, threads)
    n2 = int(min(w.streams_per_layer, max(n, n * budget_s / max(t_probe, 1e-4))))
    if n2 > n:
        st, state, qkv, cur = _oracle_state(w, C, seed, n2)
        t_probe, n = _oracle_step_seconds(st, state, qkv, cur, C, threads), n2
    token_s = t_probe * (w.streams_per_layer / n) * w.n_layers
    prompts = w.batch // 2 if w.batch >= 2 else w.batch
    return {"value": prompts / token_s, "unit": UNIT, "cores": threads, "kind": "oracle",
            "sample": f"{n} of {w.streams_per_layer} streams of 1 of {w.n_layers} layers, one layer-step at cell "
                      f"{cur - w.n_text} (cache full, {C} rows), {t_probe:.2f} s, extrapolated to a whole token"}


def run_reference(args):
    """--impl reference: the CPU oracle, timed K steps after W warm-up steps; each step is one layer-step
    over a bounded sample of streams at a late cell (cache full), extrapolated to the whole batch and stack."""
    from oracle import adsa_oracle as orc
    w = _workload(args)
    C = w.capacity()
    K = w.n_cells if args.steps is None else max(1, args.steps)
    W = max(0, args.warmup)
    threads = orc.max_threads()
    n = min(w.streams_per_layer, threads)
    st, state, qkv, cur = _oracle_state(w, C, args.seed, n)
    t_probe = _oracle_step_seconds(st, state, qkv, cur, C, threads)
    # size the per-step sample so that K + W steps take about two minutes
    n2 = int(max(1, min(w.streams_per_layer, n * 120.0 / max(t_probe * (K + W), 1e-3))))
    if n2 != n:
        n = n2
        st, state, qkv, cur = _oracle_state(w, C, args.seed, n)
    for _ in range(W):
        _oracle_step_seconds(st, state, qkv, cur, C, threads)
    total = 0.0
    for _ in range(K):
        total += _oracle_step_seconds(st, state, qkv, cur, C, threads)
    step_s = total / K
    token_s = step_s * (w.streams_per_layer / n) * w.n_layers
    prompts = w.batch // 2 if w.batch >= 2 else w.batch
    value = prompts / token_s
    sample = (f"each step: {n} of {w.streams_per_layer} streams of 1 of {w.n_layers} layers, one layer-step at cell "
              f"{cur - w.n_text} (cache full, {C} rows); extrapolated to a whole token")
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": K, "warmup": W,
            "ms_per_step": token_s * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f64", "data": "synthetic", "impl": "reference",
            "config": {"workload": w.name, "layers": w.n_layers, "batch": w.batch, "heads": w.n_heads,
                       "head_dim": w.head_dim, "n_text": w.n_text, "grid": [w.grid_h, w.grid_w],
                       "budget_fraction": w.beta, "capacity_rows": C, "parallelism": "host cores only"},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def main():
    args = parse_args()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        if rank == 0:
            run_reference(args)
        return
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    if world > 1:
        torch.cuda.set_device(local_rank)
        torch.distributed.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    try:
        run_ours(args, rank, world, local_rank)
    finally:
        if world > 1:
            torch.distributed.destroy_process_group()


if __name__ == "__main__":
    main()

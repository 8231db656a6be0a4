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
cells).  With K below H*W the cache is loaded with a seeded late-generation state (text rows, the
two most recent grid rows, a random subset of older cells per stream), W cells are decoded untimed
and K cells timed; this is repeated until about half a second has been timed and the median
region is reported.  With the default K = H*W a whole generation is timed after a whole untimed one.
One JSON line is printed by rank 0; besides the headline workload it carries short measurements of
the other configurations (`detail.all_configs`) and a memory-against-batch table (`detail.memory_vs_batch`).
"""
from __future__ import annotations

import argparse
import json
import os
import socket
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
INPUT_RING_BYTES = 12 << 30   # q/k/v of the decoded cells are kept in HBM up to this size, else a ring of cells is cycled
TIMED_SECONDS = 0.5           # repeats of the timed region add up to about this much device time
LLAMAGEN_XL_PARAM_BYTES = 775_000_000 * 2   # bf16 weights of the 775 M-parameter XL decoder (context for the memory table)


def parse_args(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference", "selftest"])
    ap.add_argument("--workload", default="cfg4", help="cfg1 .. cfg5: the headline workload of the JSON line")
    ap.add_argument("--beta", type=float, default=None)
    ap.add_argument("--layers", type=int, default=None, help="override the layer count (small profiling cases)")
    ap.add_argument("--head-dim", type=int, default=0, help="override the head dimension (experiments with other row widths)")
    ap.add_argument("--shell", default="", choices=["", "B", "L", "XL"],
                    help="also time whole generations of the LlamaGen-shaped model shell of this size (detail.model_shell)")
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-all-configs", action="store_true", help="skip the short runs of the other configurations")
    ap.add_argument("--no-memory-sweep", action="store_true", help="skip the memory-against-batch table")
    ap.add_argument("--no-detail", action="store_true",
                    help="headline region only: no per-call, attention-alone or per-layer-launch timing")
    ap.add_argument("--chunk-rows", type=int, default=0, help="override rows per attention chunk (0 = automatic)")
    ap.add_argument("--page-rows", type=int, default=0, help="rows per pool page (0 = the largest divisor of the capacity up to 1024)")
    ap.add_argument("--kernel-mode", type=int, default=1,
                    help="0 streaming, 1 automatic, 2 cluster, 3 persistent on CUDA cores, 4 persistent with MMA")
    ap.add_argument("--stream-warps", type=int, default=0, help="warps per stream of the tensor-core kernel (0 = automatic)")
    ap.add_argument("--l2-ahead", type=int, default=-1, help="tiles per warp asked into L2 beyond the ring (-1 = automatic)")
    ap.add_argument("--sweep-mode", type=int, default=2,
                    help="adsa_set_single_sweep: 0 two sweeps, 1 single sweep, 2 single sweep + carried evictee")
    ap.add_argument("--token-launch", type=int, default=1, help="adsa_set_token_launch: 1 one launch per token, 0 one launch per layer")
    ap.add_argument("--host-chunks", type=int, default=0, help="adsa_set_host_chunks (0 = the library's default)")
    ap.add_argument("--next-tiles", type=int, default=-1, help="adsa_set_next_layer_hint (-1 = the library's default)")
    ap.add_argument("--ring-stages", type=int, default=0, help="cap on the persistent kernel's ring (0 = as many as fit)")
    ap.add_argument("--profiler-range", action="store_true",
                    help="bracket ONE timed region with cudaProfilerStart/Stop (for `ncu --profile-from-start off`); no repeats")
    ap.add_argument("--backend", default="nccl", choices=["nccl", "gloo"], help="process-group backend when several ranks run")
    return ap.parse_args(argv)


def _workload(args, name=None, beta=None):
    from dataclasses import replace
    w = get_workload(int((name or args.workload).replace("cfg", "")), beta if name else args.beta)
    if name:
        return w
    if args.head_dim:      # an experiment, not one of the benchmark configurations: the same stack with other heads
        w = replace(w, head_dim=args.head_dim, name=f"{w.name}-headdim{args.head_dim}")
    return w if args.layers is None else replace(w, n_layers=args.layers, name=f"{w.name}-{args.layers}layers")


def _traffic_key(w):
    """The workload name the ncu captures are filed under: "cfg4" ...; a head-dim experiment has none."""
    return w.name if "headdim" in w.name else w.name[:4]


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def kernel_source_digest():
    """SHA-256 over the sources of the timed kernel: counters taken from another version of them are not reported."""
    import hashlib
    h = hashlib.sha256()
    for name in ("adsa_wstep.cu", "adsa_dev.cuh", "adsa_select.cuh", "adsa_async.cuh"):
        with open(os.path.join(ROOT, "paper_2506_18226_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()


def dram_traffic(kind, workload, page_rows, launch, capacity_rows):
    """DRAM bytes (read + written) per layer-step from the ncu captures summarised under profiles/, or None
    when no capture matches the kernel configuration that was timed, or the kernel's sources have changed
    since the captures were taken."""
    path = os.path.join(ROOT, "profiles", "dram_traffic.json")
    try:
        with open(path) as f:
            rec = json.load(f)
            if rec.get("kernel_source_sha256") != kernel_source_digest():
                return None
            for e in rec["entries"]:
                if (e["kind"], e["workload"], e["page_rows"], e["launch"], e["capacity_rows"]) == (kind, workload, page_rows, launch, capacity_rows):
                    return e["dram_bytes_per_layer_step"]
    except (OSError, KeyError, ValueError):
        pass
    return None


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


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def spawn_replicas(n, argv):
    """`--gpus N` given to a plain `python bench.py`: start N ranks of this file under torch.distributed.run
    (one per GPU; rank 0 prints the line), as a multi-process launcher would, and return its exit code."""
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}", "--master-addr", "127.0.0.1",
           "--master-port", str(_free_port()), os.path.abspath(__file__), *argv]
    return subprocess.call(cmd)


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


def gpu_index(local_rank):
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    return vis.split(",")[local_rank] if vis else local_rank


# --------------------------------------------------------------------------------------
# the CUDA path: one attention stack, its inputs and the ways of decoding a grid cell
# --------------------------------------------------------------------------------------
class Stack:
    """An engine shaped like workload `w` with seeded q/k/v for `n_cells` grid cells resident in HBM."""

    def __init__(self, w, args, dev, rank, n_cells):
        from paper_2506_18226_b200 import AdsaEngine
        self.w, self.dev = w, dev
        self.C, self.T0, self.L, self.HW = w.capacity(), w.n_text, w.n_layers, w.n_cells
        # Large pages keep a stream's rows contiguous, so that one TMA box covers a whole tile; the default is
        # the largest divisor of the capacity up to 1024 rows (cfg4: one 572-row page per stream), which also
        # makes a full stream occupy whole pages: pool bytes = the budget's share of dense, exactly.
        self.page_rows = args.page_rows if args.page_rows else pick_page_rows(self.C, hi=1024)
        max_rows = max(self.C, self.T0 + 2 * w.grid_w)
        self.eng = eng = AdsaEngine(n_layers=self.L, batch=w.batch, n_heads=w.n_heads, head_dim=w.head_dim, n_text=self.T0,
                                    grid_h=w.grid_h, grid_w=w.grid_w, max_rows_per_stream=max_rows, page_rows=self.page_rows,
                                    n_pages=self.L * w.streams_per_layer * -(-max_rows // self.page_rows), device=str(dev))
        if args.chunk_rows:
            eng.set_attn_chunk_rows(args.chunk_rows)
        eng.set_staged(args.kernel_mode)
        eng.set_single_sweep(args.sweep_mode)
        eng.set_token_launch(args.token_launch)
        if args.host_chunks:
            eng.set_host_chunks(args.host_chunks)
        if args.next_tiles >= 0:
            eng.set_next_layer_hint(args.next_tiles)
        if args.ring_stages:
            eng.set_ring_stages(args.ring_stages)
        if args.l2_ahead >= 0:
            eng.set_l2_lookahead(args.l2_ahead)
        if args.stream_warps:
            eng.set_stream_warps(args.stream_warps)
        self.seed = args.seed + 1000 * rank
        g = torch.Generator(device=dev).manual_seed(self.seed)
        self.shape = (self.L, w.batch, w.n_heads, w.head_dim)
        per_cell = 3 * int(np.prod(self.shape)) * 2
        self.ring = max(1, min(n_cells, max(8, INPUT_RING_BYTES // per_cell)))
        self.qkv = [torch.empty((self.ring,) + self.shape, dtype=torch.bfloat16, device=dev) for _ in range(3)]
        for t in self.qkv:
            for i in range(self.ring):
                t[i] = (torch.randn(self.shape, generator=g, device=dev) * w.sigma).to(torch.bfloat16)
        self.out = torch.zeros((2,) + self.shape, dtype=torch.bfloat16, device=dev)

    # -- cache states ----------------------------------------------------------------
    def _rows(self, g, n):
        w = self.w
        return (torch.randn((w.batch, w.n_heads, n, w.head_dim), generator=g, device=self.dev) * w.sigma).to(torch.bfloat16)

    def start_generation(self):
        """Empty caches, then the text condition of every layer."""
        self.eng.reset()
        g = torch.Generator(device=self.dev).manual_seed(self.seed + 1)
        if self.T0:
            for l in range(self.L):
                self.eng.prefill_rows(l, self._rows(g, self.T0), self._rows(g, self.T0), 0)

    def load_late(self, cell):
        """The caches as they look when `cell` is about to be decoded, without decoding the cells before it:
        the text rows, the two most recent grid rows and, per stream, a random subset of the older cells
        (min(capacity, context) rows in all), in shuffled physical order, with seeded N(0, sigma^2) payloads."""
        w, T0 = self.w, self.T0
        if cell <= 0:
            return self.start_generation()
        cur = T0 + cell
        n = min(self.C, cur)
        lo = max(T0, cur - 2 * w.grid_w)
        text = torch.arange(0, T0, device=self.dev)
        recent = torch.arange(lo, cur, device=self.dev)
        older = torch.arange(T0, lo, device=self.dev)
        n_old = n - T0 - recent.numel()
        assert 0 <= n_old <= older.numel(), "capacity below text condition + two grid rows"
        S = w.streams_per_layer
        self.eng.reset()
        g = torch.Generator(device=self.dev).manual_seed(self.seed + 2 + cell)
        for l in range(self.L):
            parts = [text.expand(S, -1)]
            if n_old:
                pick = torch.rand((S, older.numel()), generator=g, device=self.dev).argsort(dim=1)[:, :n_old]
                parts.append(older[pick])
            parts.append(recent.expand(S, -1))
            rows = torch.cat(parts, dim=1)
            perm = torch.rand((S, n), generator=g, device=self.dev).argsort(dim=1)
            pos = rows.gather(1, perm).to(torch.int32).view(w.batch, w.n_heads, n).contiguous()
            self.eng.prefill_rows(l, self._rows(g, n), self._rows(g, n), 0, pos)

    # -- decoding one grid cell --------------------------------------------------------
    def decode(self, g):
        """One token through the whole stack (adsa_token_step)."""
        i = g % self.ring
        self.eng.token_step(self.T0 + g, self.C, self.qkv[0][i], self.qkv[1][i], self.qkv[2][i], self.out[g & 1])

    def full_cell(self):
        """First grid cell at which the cache is full before the step (one eviction per step from there on)."""
        return max(0, self.C - self.T0)

    def bytes_per_layer_step(self, rows_before):
        """Algorithmic bytes of one fused layer-step and of attention alone, for `rows_before` live rows per
        stream at a full cache: retained rows x (K + V) + 16 B of metadata per live row (position, carried score,
        inverse norm read; next score written) + q, k_new, v_new, out and the new row's K and V."""
        w = self.w
        d2 = w.head_dim * 2
        retained = rows_before - 1 if rows_before >= self.C else rows_before
        step = w.streams_per_layer * (retained * 2 * d2 + rows_before * 16 + 6 * d2)
        attn = w.streams_per_layer * (retained * 2 * d2 + 4 * d2)
        return step, attn


def timed_region(st, first, K, W, world, profiler=False):
    """Decode cells first .. first+K-1 between two CUDA events, after W untimed cells from a loaded state
    (or, for a whole generation, after an untimed generation).  Returns (ms, launches, per-cell events)."""
    HW = st.HW
    if first == 0 and K >= HW:
        st.start_generation()
        for g in range(HW):                       # the warm-up generation
            st.decode(g)
        st.start_generation()
    else:
        st.load_late(max(0, first - W))
        for g in range(max(0, first - W), first):
            st.decode(g)
    torch.cuda.synchronize(st.dev)
    if world > 1:
        torch.distributed.barrier()
    n0 = st.eng.launch_count()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    cells = []
    if profiler:
        torch.cuda.profiler.start()
    t0.record()
    g = first
    for _ in range(K):
        if g == HW:                               # K > H*W: another generation inside the timed region
            st.start_generation()
            g = 0
        st.decode(g)
        g += 1
        if first == 0 and K == HW:
            e = torch.cuda.Event(enable_timing=True)
            e.record()
            cells.append((g - 1, e))
    t1.record()
    torch.cuda.synchronize(st.dev)
    if profiler:
        torch.cuda.profiler.stop()
    if world > 1:
        torch.distributed.barrier()
    return t0.elapsed_time(t1), st.eng.launch_count() - n0, (t0, cells)


def _roofline(kind, label, bytes_per_unit, us_per_unit, units_per_launch, launches, traffic):
    peak, peak_kind = peaks()
    gbs = bytes_per_unit / (us_per_unit * 1e-6) / 1e9
    return {"bound": "hbm", "kernel": label, "achieved": gbs, "peak": peak, "unit": "GB/s", "frac": gbs / peak,
            "peak_kind": f"of {peak_kind}", "frac_of_nominal_8000": gbs / 8000.0,
            "us_per_layer_step": us_per_unit, "layer_steps_per_launch": units_per_launch,
            "us_per_launch": us_per_unit * units_per_launch, "launches_timed": launches,
            "algorithmic_bytes_per_layer_step": bytes_per_unit,
            "algorithmic_bytes_per_launch": bytes_per_unit * units_per_launch,
            "traffic": None if traffic is None else traffic * units_per_launch, "kind": kind}


def pool_record(st, peak_pool_bytes):
    """Bytes of the paged pool at its high-water mark against a dense cache, with the per-row and per-stream
    state the library keeps beside the pool (positions, inverse norms, carried scores: 12 B per row slot;
    carried sum, masks, counts, notes, page table per stream) counted as metadata."""
    w, cfg = st.w, st.eng.cfg
    n_streams = st.L * w.streams_per_layer
    mask_words = (cfg.max_rows_per_stream + 31) // 32
    max_pages = -(-cfg.max_rows_per_stream // cfg.page_rows)
    meta = n_streams * (cfg.max_rows_per_stream * 12 + 256 * 4 + 2 * mask_words * 4 + 16 + 16 + max_pages * 4 + 4)
    dense = w.dense_kv_bytes() * st.L // w.n_layers
    return {"peak_bytes": peak_pool_bytes, "dense_bytes": dense, "ratio": peak_pool_bytes / dense,
            "payload_bytes": peak_pool_bytes * w.head_dim // cfg.row_stride,
            "payload_ratio": peak_pool_bytes * w.head_dim / cfg.row_stride / dense,
            "metadata_bytes": meta, "ratio_with_metadata": (peak_pool_bytes + meta) / dense,
            "row_stride": cfg.row_stride, "page_rows": cfg.page_rows, "budget_fraction": w.beta}


def measure(w, args, dev, rank, world, local_rank, K, W, detail=True):
    """The timed region of one workload (median of repeats), its rooflines and, on request, the separate
    timings at a full cache: per-layer launches, attention alone, the four calls one by one."""
    HW = w.n_cells
    K = HW if K is None else max(1, K)
    first = (HW - K) % HW if K % HW else 0
    whole = first == 0 and K >= HW
    M = max(1, min(8, HW // 4))
    st = Stack(w, args, dev, rank, HW if whole else min(HW, K + W + M + 4))
    eng, L, C, T0 = st.eng, st.L, st.C, st.T0
    prompts = w.batch // 2 if w.batch >= 2 else w.batch

    sampler = ClockSampler(gpu_index(local_rank))
    sampler.start()
    ms0, launches, (t0, cells) = timed_region(st, first, K, W, world, profiler=args.profiler_range)
    regions = [ms0]
    if not whole and not args.profiler_range:
        worst, _ = aggregate(ms0, 0.0, world)              # every rank repeats the same number of times
        repeats = int(min(40, max(3, np.ceil(TIMED_SECONDS * 1e3 / max(worst, 1e-3)))))
        for _ in range(repeats - 1):
            regions.append(timed_region(st, first, K, W, world)[0])
    clocks = sampler.stop()
    status, _ = eng.get_status()
    assert status == 0, f"device status {status} after the timed region"
    ms_local = float(np.median(regions))
    ms, tokens = aggregate(ms_local, float(prompts * K), world)
    rows_now = int(eng._t["n_live"].max().item())
    assert int(eng._t["n_live"].min().item()) == rows_now == min(C, T0 + HW)
    peak_pool_bytes = eng.pool_bytes_peak()

    res = {"workload": w, "stack": st, "K": K, "W": W, "first": first, "ms": ms, "tokens": tokens, "launches": launches,
           "clocks": clocks, "regions": len(regions), "region_ms_min_max": [float(min(regions)), float(max(regions))],
           "kv_pool": pool_record(st, peak_pool_bytes), "prompts": prompts, "detail": {}}

    # ---- roofline of the headline path at a full cache -------------------------------------------
    step_bytes, attn_bytes = st.bytes_per_layer_step(rows_now)
    launch_kind = "token-launch" if launches == K else "layer-launch"
    if whole:
        prev, per_cell = t0, {}
        for gcell, e in cells:
            per_cell[gcell] = prev.elapsed_time(e) * 1e3 / L
            prev = e
        span = lambda a, n=16: float(np.median([per_cell[i] for i in range(a, min(HW, a + n))]))
        res["detail"]["fused_layer_step_us_by_cell"] = {
            "start_cells_0_15": span(0), "middle": span(max(0, HW // 2 - 8)), "end_last_16": span(max(0, HW - 16)),
            "rows_at": {"start": T0 + 1, "middle": min(C, T0 + HW // 2), "end": min(C, T0 + HW)}}
        us_unit, n_timed = span(max(0, HW - 16)), 16 * launches // K
    elif first >= st.full_cell():
        us_unit, n_timed = ms_local * 1e3 / (K * L), launches
    else:
        us_unit, n_timed = None, 0
    if us_unit:
        per_launch = L if launch_kind == "token-launch" else 1
        res["roofline"] = _roofline("fused", f"fused layer-step (adsa_token_step, {launch_kind}: {per_launch} layer-step(s) per launch)",
                                    step_bytes, us_unit, per_launch, n_timed,
                                    dram_traffic("fused", _traffic_key(w), st.page_rows, launch_kind, C))
    if detail and rank == 0 and T0 + HW > C:
        res["detail"].update(full_cache_detail(st, args, M, step_bytes, attn_bytes))
    return res


def full_cache_detail(st, args, M, step_bytes, attn_bytes):
    """Separate timings over the last M cells (cache full): the fused step launched layer by layer, the
    attention call alone (every layer's launch back to back, after every layer's score and select), and each
    of the four calls.  The keep masks are per layer, so the grouped calls are a valid trajectory."""
    eng, L, C, T0, HW, dev = st.eng, st.L, st.C, st.T0, st.HW, st.dev
    out = {}
    wname = _traffic_key(st.w)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    # (1) one launch per layer, as a decoder whose layers feed each other has to do
    eng.set_token_launch(0)                      # adsa_token_step now launches layer after layer, from C
    st.load_late(HW - M - 2)
    for g in range(HW - M - 2, HW - M):
        st.decode(g)
    torch.cuda.synchronize(dev)
    n0 = eng.launch_count()
    e0.record()
    for g in range(HW - M, HW):
        st.decode(g)
    e1.record()
    torch.cuda.synchronize(dev)
    launches = eng.launch_count() - n0
    out["roofline_layer_launch"] = _roofline("fused", "fused layer-step, one launch per layer (adsa_layer_step)", step_bytes,
                                             e0.elapsed_time(e1) * 1e3 / launches, 1, launches,
                                             dram_traffic("fused", wname, st.page_rows, "layer-launch", C))
    eng.set_token_launch(args.token_launch)
    # (2) the four calls
    st.load_late(HW - M)
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(5)]
    call_us = {"adsa_score": [], "adsa_select": [], "adsa_sparse_decode_attn": [], "adsa_kv_update": []}
    attn_ms = 0.0
    for g in range(HW - M, HW):
        cur, i = T0 + g, g % st.ring
        q, k, v = (t[i] for t in st.qkv)
        ev[0].record()
        for l in range(L):
            eng.score(l, cur)
        ev[1].record()
        for l in range(L):
            eng.select(l, cur, C)
        ev[2].record()
        for l in range(L):                          # L launches back to back, each reads a different layer's KV
            eng.sparse_decode_attn(l, cur, q[l], k[l], v[l], st.out[g & 1, l])
        ev[3].record()
        for l in range(L):
            eng.kv_update(l, cur, k[l], v[l])
        ev[4].record()
        torch.cuda.synchronize(dev)
        attn_ms += ev[2].elapsed_time(ev[3])
        for j, name in enumerate(call_us):
            call_us[name].append(ev[j].elapsed_time(ev[j + 1]) * 1e3 / L)
    assert eng.get_status()[0] == 0
    out["roofline_attn"] = _roofline("attn", "attention alone (adsa_sparse_decode_attn)", attn_bytes, attn_ms * 1e3 / (M * L), 1,
                                     M * L, dram_traffic("attn", wname, st.page_rows, "layer-launch", C))
    per_call = {n: float(np.median(v)) for n, v in call_us.items()}
    per_call["four_call_sequence"] = float(sum(per_call.values()))
    out["per_call_us_cache_full"] = per_call
    return out


def end_to_end(st, args, K, W, world, prompts):
    """The same cells through adsa_token_step_host: pinned host q/k/v in, host output out, every step's copies
    inside the timed region, which is bracketed by wall-clock reads after a device synchronisation."""
    HW, T0, C = st.HW, st.T0, st.C
    Ke = min(K, 64, HW)
    hq, hk, hv = (torch.empty((Ke,) + st.shape, dtype=torch.bfloat16).pin_memory() for _ in range(3))
    ho = torch.empty(st.shape, dtype=torch.bfloat16).pin_memory()
    for i, g in enumerate(range(HW - Ke, HW)):
        j = g % st.ring
        hq[i].copy_(st.qkv[0][j]); hk[i].copy_(st.qkv[1][j]); hv[i].copy_(st.qkv[2][j])
    regions = []
    for _ in range(5):
        st.load_late(max(0, HW - Ke - W))
        for g in range(max(0, HW - Ke - W), HW - Ke):
            st.decode(g)
        torch.cuda.synchronize(st.dev)
        if world > 1:
            torch.distributed.barrier()
        tw = time.perf_counter()
        for i, g in enumerate(range(HW - Ke, HW)):
            st.eng.token_step_host(T0 + g, C, hq[i], hk[i], hv[i], ho)      # synchronises: the result is on the host
        regions.append((time.perf_counter() - tw) * 1e3)
    ms, tokens = aggregate(float(np.median(regions)), float(prompts * Ke), world)
    per = int(np.prod(st.shape)) * 2
    return {"value": tokens / (ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": 3 * per, "d2h_bytes_per_step": per,
            "steps": Ke, "ms_per_step": ms / Ke, "regions": len(regions),
            "api": "adsa_token_step_host (q/k/v from pinned host memory by copy-engine copies in chunks of layers, queued beside "
                   "ONE launch for all layers that waits for each layer's inputs to land; the output rows are written "
                   "by the kernel into pinned host memory; one sync per token, wall clock around the calls)"}


def compact(res):
    """One configuration's figures for detail.all_configs."""
    w, L = res["workload"], res["workload"].n_layers
    d = res["detail"]
    out = {"workload": w.name, "budget_fraction": w.beta, "capacity_rows": w.capacity(),
           "image_tokens_per_s": res["tokens"] / (res["ms"] * 1e-3), "ms_per_token": res["ms"] / res["K"],
           "us_per_layer_step": res["ms"] * 1e3 / (res["K"] * L), "cells_timed": [res["first"], res["first"] + res["K"]],
           "regions": res["regions"], "gpu_launches": res["launches"],
           "pool_ratio": res["kv_pool"]["ratio"], "pool_payload_ratio": res["kv_pool"]["payload_ratio"],
           "pool_ratio_with_metadata": res["kv_pool"]["ratio_with_metadata"], "page_rows": res["kv_pool"]["page_rows"],
           "clocks": res["clocks"]}
    for key, r in (("fused", res.get("roofline")), ("fused_layer_launch", d.get("roofline_layer_launch")),
                   ("attn_alone", d.get("roofline_attn"))):
        if r:
            out[key] = {"us_per_layer_step": r["us_per_layer_step"], "achieved_gbs": r["achieved"], "frac": r["frac"],
                        "frac_of_nominal_8000": r["frac_of_nominal_8000"]}
    return out


def memory_vs_batch(args, dev):
    """Fig. 8-style table on the XL shape: bytes of the KV pool (+ the library's metadata) against a dense
    cache for batch 2 .. 64, with the XL decoder's bf16 weights beside them as context."""
    from dataclasses import replace
    rows = []
    base = get_workload(4)
    for batch in (2, 4, 8, 16, 32, 64):
        w = replace(base, batch=batch, name=f"cfg4-batch{batch}")
        st = Stack(w, args, dev, 0, 4)
        st.load_late(st.HW - 3)
        for g in range(st.HW - 3, st.HW):
            st.decode(g)
        assert st.eng.get_status()[0] == 0
        rec = pool_record(st, st.eng.pool_bytes_peak())
        rows.append({"batch": batch, "adsa_pool_bytes": rec["peak_bytes"], "metadata_bytes": rec["metadata_bytes"],
                     "dense_kv_bytes": rec["dense_bytes"], "kv_ratio": rec["ratio"], "kv_ratio_with_metadata": rec["ratio_with_metadata"],
                     "weights_bytes": LLAMAGEN_XL_PARAM_BYTES,
                     "total_ratio_with_weights": (rec["peak_bytes"] + rec["metadata_bytes"] + LLAMAGEN_XL_PARAM_BYTES) /
                                                 (rec["dense_bytes"] + LLAMAGEN_XL_PARAM_BYTES)})
        del st
        torch.cuda.empty_cache()
    return rows


def model_shell(args, dev):
    """Whole generations through the LlamaGen-shaped shell (random weights): the condition is prefilled, every grid
    cell is decoded through all layers (torch GEMMs around libadsa's kernels, one ADSA layer-step launch per layer,
    because every layer's q/k/v depend on the layer before), ids go to the host as they are drawn."""
    from paper_2506_18226_b200.shell import SHAPES, LlamaGenShell, ShellConfig
    grid = {"B": 16, "L": 24, "XL": 32}[args.shell]
    n_images = {"B": 1, "L": 8, "XL": 16}[args.shell]
    cfg = ShellConfig(grid_h=grid, grid_w=grid, n_images=n_images, **SHAPES[args.shell])
    sh = LlamaGenShell(cfg, seed=args.seed, device=str(dev))
    g = torch.Generator(device=dev).manual_seed(args.seed + 1)
    text = torch.randn(cfg.batch, cfg.n_text, cfg.dim, generator=g, device=dev).to(torch.bfloat16)
    sh.generate(text, n_cells=min(64, grid * grid))          # warm-up: kernels loaded, cuBLAS handles made
    times = []
    for _ in range(2):
        torch.cuda.synchronize(dev)
        t0 = time.perf_counter()
        ids = sh.generate(text)
        times.append(time.perf_counter() - t0)
    t = min(times)
    cells = grid * grid
    status = int(sh.eng.get_status()[0])
    weights = sum(x.numel() for x in (sh.wq, sh.wk, sh.wv, sh.wo, sh.w13, sh.w2, sh.head, sh.tok_emb)) * 2
    n_ids = int(ids.numel())
    # the three stateless kernels on their own, at sizes larger than L2 (CUDA events, 20 launches each)
    import paper_2506_18226_b200 as A
    hbm, _ = peaks()

    def timed(fn):
        for _ in range(3):
            fn()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(20):
            fn()
        e1.record()
        torch.cuda.synchronize(dev)
        return e0.elapsed_time(e1) / 20 * 1e3     # us

    rows = 65536
    x = torch.randn(rows, cfg.dim, device=dev).to(torch.bfloat16)
    y = torch.empty_like(x)
    us_norm = timed(lambda: A.rmsnorm(x, sh.norm_f, out=y, eps=cfg.norm_eps))
    gu = torch.randn(rows, 2 * cfg.ffn_hidden, device=dev).to(torch.bfloat16)
    act = torch.empty(rows, cfg.ffn_hidden, dtype=torch.bfloat16, device=dev)
    us_act = timed(lambda: A.swiglu(gu[:, :cfg.ffn_hidden], gu[:, cfg.ffn_hidden:], out=act))
    us_sample = timed(lambda: A.cfg_sample(sh.logits, cfg.cfg_scale, min(cfg.top_k, cfg.vocab), cfg.temperature, sh.uniforms[0],
                                           tokens=sh.tokens))
    b_norm, b_act = 2 * x.numel() * 2, 3 * act.numel() * 2
    ops = {"rmsnorm": {"rows": rows, "dim": cfg.dim, "us": us_norm, "gbs": b_norm / us_norm * 1e-3, "frac_of_measured_copy": b_norm / us_norm * 1e-3 / hbm},
           "swiglu": {"rows": rows, "hidden": cfg.ffn_hidden, "us": us_act, "gbs": b_act / us_act * 1e-3, "frac_of_measured_copy": b_act / us_act * 1e-3 / hbm},
           "cfg_sample": {"n_images": n_images, "vocab": cfg.vocab, "top_k": min(cfg.top_k, cfg.vocab), "us": us_sample}}
    del x, y, gu, act
    # Device memory the shell holds (weights, KV pool with its metadata, workspace, activations) against the number of
    # images, with the cache at the budget and with a cache for the whole context: allocated bytes, not a formula
    # (Sec. 5, "GPU Memory-efficient Image Generation", Fig. 8).
    del sh
    torch.cuda.empty_cache()
    # the same generation with a cache for the whole context (nothing is ever evicted: dense attention)
    dense = LlamaGenShell(ShellConfig(grid_h=grid, grid_w=grid, n_images=n_images, budget_fraction=1.0, **SHAPES[args.shell]),
                          seed=args.seed, device=str(dev))
    dense.generate(text, n_cells=min(64, grid * grid))
    torch.cuda.synchronize(dev)
    t0 = time.perf_counter()
    dense.generate(text)
    t_dense = time.perf_counter() - t0
    del dense
    torch.cuda.empty_cache()
    mem = []
    for n_img in (1, 2, 4, 8, 16, 32):
        row = {"n_images": n_img, "batch_rows": 2 * n_img}
        for key, frac in (("adsa_bytes", cfg.budget_fraction), ("dense_bytes", 1.0)):
            base = torch.cuda.memory_allocated(dev)
            tmp = LlamaGenShell(ShellConfig(grid_h=grid, grid_w=grid, n_images=n_img, budget_fraction=frac, **SHAPES[args.shell]),
                                seed=args.seed, device=str(dev))
            row[key] = torch.cuda.memory_allocated(dev) - base
            del tmp
            torch.cuda.empty_cache()
        row["ratio"] = row["adsa_bytes"] / row["dense_bytes"]
        mem.append(row)
    return {"shape": args.shell, "layers": cfg.n_layers, "dim": cfg.dim, "heads": cfg.n_heads, "ffn_hidden": cfg.ffn_hidden,
            "vocab": cfg.vocab, "n_images": n_images, "batch_rows": cfg.batch, "grid": [grid, grid], "capacity_rows": cfg.capacity,
            "image_tokens_per_s": n_images * cells / t, "ms_per_token": t / cells * 1e3, "seconds_per_generation": t,
            "whole_context_cache": {"ms_per_token": t_dense / cells * 1e3, "image_tokens_per_s": n_images * cells / t_dense,
                                    "time_ratio_adsa_over_dense": t / t_dense},
            "weights_bytes": weights, "ids_on_host": n_ids, "data": "random weights, random condition embeddings",
            "timing": "wall clock around prefill + every decode step + the final synchronisation, best of 2",
            "kernels_alone": ops, "memory_vs_images_allocated": mem, "status": status}


def run_ours(args, rank, world, local_rank):
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    w = _workload(args)
    W = max(3, args.warmup)
    res = measure(w, args, dev, rank, world, local_rank, args.steps, W, detail=not args.no_detail)
    st, K, L, C = res["stack"], res["K"], w.n_layers, w.capacity()
    e2e = None if args.no_e2e else end_to_end(st, args, K, W, world, res["prompts"])
    peak_pool_gb = res["kv_pool"]["peak_bytes"] / 1e9
    ring = st.ring
    res["stack"] = None
    del st
    torch.cuda.empty_cache()
    if rank != 0:
        return
    detail = res["detail"]
    if not args.no_all_configs and world == 1:      # short runs of every configuration (one GPU only: ranks are not held for it)
        import copy
        rows = []
        for name, beta in [("cfg1", None), ("cfg2", None), ("cfg3", None), ("cfg4", None), ("cfg5", 0.25), ("cfg5", 0.5), ("cfg5", 0.75)]:
            w2 = _workload(args, name, beta)
            if w2.name == w.name and w2.beta == w.beta and args.layers is None:
                rows.append(compact(res))
                continue
            a2 = copy.copy(args)
            a2.page_rows, a2.layers, a2.workload, a2.profiler_range = 0, None, name, False
            r2 = measure(w2, a2, dev, 0, 1, local_rank, min(20, w2.n_cells), 5, detail=True)
            r2["stack"] = None
            rows.append(compact(r2))
            del r2
            torch.cuda.empty_cache()
        detail["all_configs"] = rows
        # the headline workload once more with several pages per stream (the headline uses the largest divisor of the
        # capacity up to 1024 rows, i.e. one page per stream where the capacity allows)
        small = pick_page_rows(C, hi=64)
        if small != res["kv_pool"]["page_rows"] and args.page_rows == 0:
            a2 = copy.copy(args)
            a2.page_rows, a2.profiler_range = small, False
            r2 = measure(w, a2, dev, 0, 1, local_rank, min(20, w.n_cells), 5, detail=True)
            r2["stack"] = None
            detail["several_pages_per_stream"] = compact(r2)
            del r2
            torch.cuda.empty_cache()
    if not args.no_memory_sweep and world == 1:
        detail["memory_vs_batch"] = memory_vs_batch(args, dev)
    if args.shell and world == 1:
        detail["model_shell"] = model_shell(args, dev)

    ms, tokens = res["ms"], res["tokens"]
    line = {
        "metric": METRIC, "value": tokens / (ms * 1e-3), "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
        "data": "synthetic", "impl": "ours",
        "config": {"workload": w.name, "layers": L, "batch": w.batch, "heads": w.n_heads, "head_dim": w.head_dim,
                   "n_text": w.n_text, "grid": [w.grid_h, w.grid_w], "budget_fraction": w.beta, "capacity_rows": C,
                   "page_rows": res["kv_pool"]["page_rows"], "storage": "bf16 KV pool, fp32 arithmetic",
                   "parallelism": "replicas only",
                   "cells_timed": [res["first"], res["first"] + K] if K <= w.n_cells else "whole generations",
                   "timed_regions": f"median of {res['regions']} regions of {K} steps each (min {res['region_ms_min_max'][0]:.3f} ms, "
                                    f"max {res['region_ms_min_max'][1]:.3f} ms), each after a reload of the cache state and {W} untimed steps",
                   "launch": "one launch per token (all layers)" if res["launches"] == K else "one launch per layer",
                   "l2": f"inputs larger than L2: every step sweeps the whole KV pool ({peak_pool_gb:.2f} GB) against 126 MB of L2",
                   "inputs": f"q/k/v ring of {ring} steps resident in HBM"},
        "us_per_layer_step": ms * 1e3 / (K * L),
        "batch_rows_per_s": tokens / (ms * 1e-3) * (w.batch / res["prompts"]),
        "gpu_launches": res["launches"], "clocks": res["clocks"],
    }
    if "roofline" in res:
        line["roofline"] = res["roofline"]
    for key in ("roofline_layer_launch", "roofline_attn"):
        if key in detail:
            line[key] = detail.pop(key)
    line["detail"] = detail
    line["kv_pool"] = res["kv_pool"]
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
    reps = int(min(40, max(1, budget_s / max(t_probe, 1e-3))))      # small shapes: the same layer-step again, about budget_s in all
    if reps > 1:
        t_probe = sum(_oracle_step_seconds(st, state, qkv, cur, C, threads) for _ in range(reps)) / reps
    token_s = t_probe * (w.streams_per_layer / n) * w.n_layers
    prompts = w.batch // 2 if w.batch >= 2 else w.batch
    return {"value": prompts / token_s, "unit": UNIT, "cores": threads, "kind": "oracle",
            "sample": f"{n} of {w.streams_per_layer} streams of 1 of {w.n_layers} layers, one layer-step at cell "
                      f"{cur - w.n_text} (cache full, {C} rows), {t_probe:.2f} s each, mean of {reps}, extrapolated to a whole token"}


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


def run_selftest(args, rank, world):
    """--impl selftest: no GPU work.  Every rank reports a made-up time and unit count through the same
    aggregation and printing as the real arms, so that the multi-process plumbing can be checked on CPUs."""
    ms, units = aggregate(10.0 + 5.0 * rank, 16.0 * (rank + 1), world)
    if rank == 0:
        print(json.dumps({"metric": METRIC, "value": units / (ms * 1e-3), "unit": UNIT, "n_gpus": world, "impl": "selftest",
                          "ms": ms, "units": units}), flush=True)


def main(argv=None):
    argv = sys.argv[1:] if argv is None else argv
    args = parse_args(argv)
    if "WORLD_SIZE" not in os.environ and args.gpus > 1 and args.impl != "reference":
        raise SystemExit(spawn_replicas(args.gpus, argv))      # N independent replicas, one process per GPU
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        if rank == 0:
            run_reference(args)
        return
    if args.impl == "selftest":
        if world > 1:
            torch.distributed.init_process_group(args.backend)
        try:
            run_selftest(args, rank, world)
        finally:
            if world > 1:
                torch.distributed.destroy_process_group()
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

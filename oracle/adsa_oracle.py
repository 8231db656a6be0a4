"""ctypes front end of the CPU oracle (test infrastructure only).

Builds `adsa_oracle.c` with gcc on first use and exposes its functions on numpy
arrays.  Nothing here computes anything: every number comes out of the C file,
which states one layer-step of ADSA (Section 4 of the paper) as plain loops.
Only tests, the smoke check and the benchmark's CPU-baseline leg import this
module; the CUDA path never does.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "adsa_oracle.c")
_LIB = os.path.join(_HERE, "libadsa_oracle.so")
_lib = None

REGION_PREFIX, REGION_PREVIOUS, REGION_LOCAL, REGION_INVALID = 0, 1, 2, -1


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP across streams only)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp",
                               "-ffp-contract=off", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


class _Params(C.Structure):
    _fields_ = [("n_text", C.c_int), ("grid_w", C.c_int), ("n_prefix", C.c_int),
                ("rows_back", C.c_int), ("score_variant", C.c_int), ("softmax_scale", C.c_double)]


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.adsa_oracle_region.restype = C.c_int
        _lib.adsa_oracle_layer_step.restype = C.c_int
        _lib.adsa_oracle_layer_step_batch.restype = C.c_int
        _lib.adsa_oracle_layer_step_mass_batch.restype = C.c_int
        _lib.adsa_oracle_layer_step_shared_batch.restype = C.c_int
        _lib.adsa_oracle_max_threads.restype = C.c_int
    return _lib


def _p(a, t):
    return a.ctypes.data_as(C.POINTER(t))


def _f32(a):
    a = np.ascontiguousarray(a, dtype=np.float32)
    return a


def region(pos, cur_pos, n_text, grid_w, n_prefix, rows_back=1) -> int:
    return lib().adsa_oracle_region(int(pos), int(cur_pos), int(n_text), int(grid_w), int(n_prefix), int(rows_back))


def score_definition(v) -> np.ndarray:
    """Eq. 1-2 by the double loop over pairs.  v: [p, d] float32 -> S: [p] float32."""
    v = _f32(v)
    p, d = v.shape
    s = np.zeros(p, dtype=np.float32)
    lib().adsa_oracle_score_definition(_p(v, C.c_float), p, d, _p(s, C.c_float))
    return s


def score_rowsum(v) -> np.ndarray:
    """Eq. 1-2 through the row-sum identity (labelled variant, not the oracle of record)."""
    v = _f32(v)
    p, d = v.shape
    s = np.zeros(p, dtype=np.float32)
    lib().adsa_oracle_score_rowsum(_p(v, C.c_float), p, d, _p(s, C.c_float))
    return s


def select_lowest(score, pos, K) -> np.ndarray:
    """Eq. 3 with the (score, position) order.  Returns a 0/1 keep flag per candidate."""
    score = _f32(score)
    pos = np.ascontiguousarray(pos, dtype=np.int32)
    keep = np.zeros(score.shape[0], dtype=np.int32)
    lib().adsa_oracle_select_lowest(_p(score, C.c_float), _p(pos, C.c_int), score.shape[0], int(K), _p(keep, C.c_int))
    return keep


def select_highest(score, pos, K) -> np.ndarray:
    """The K highest scores, equal scores by lower position first (attention-mass pruning, Section 3.4's foil)."""
    score = _f32(score)
    pos = np.ascontiguousarray(pos, dtype=np.int32)
    keep = np.zeros(score.shape[0], dtype=np.int32)
    lib().adsa_oracle_select_highest(_p(score, C.c_float), _p(pos, C.c_int), score.shape[0], int(K), _p(keep, C.c_int))
    return keep


def attend(q, k, v, scale=None):
    """softmax(q.k^T * scale) . v over the given rows.  Returns (out[d], weights[n]) in float64."""
    q, k, v = _f32(q), _f32(k), _f32(v)
    n, d = k.shape
    out = np.zeros(d, dtype=np.float64)
    w = np.zeros(n, dtype=np.float64)
    sc = float(scale) if scale is not None else 1.0 / np.sqrt(d)
    lib().adsa_oracle_attend(_p(q, C.c_float), _p(k, C.c_float), _p(v, C.c_float), n, d, C.c_double(sc),
                             _p(out, C.c_double), _p(w, C.c_double))
    return out, w


def causal_attend(q, k, v, scale=None) -> np.ndarray:
    """Dense causal attention: row i of q attends rows 0..i of k, v.  [n, d] each -> [n, d] float64."""
    q, k, v = _f32(q), _f32(k), _f32(v)
    n, d = k.shape
    out = np.zeros((n, d), dtype=np.float64)
    sc = float(scale) if scale is not None else 1.0 / np.sqrt(d)
    lib().adsa_oracle_causal_attend(_p(q, C.c_float), _p(k, C.c_float), _p(v, C.c_float), n, d, C.c_double(sc), _p(out, C.c_double))
    return out


def rope_2d(x, pos, n_text, grid_w, base=10000.0) -> np.ndarray:
    """Two-dimensional rotary embedding of rows x [n, d] at context positions pos [n] -> [n, d] float64."""
    x = _f32(x)
    pos = np.ascontiguousarray(pos, dtype=np.int32)
    n, d = x.shape
    assert d % 4 == 0
    out = np.zeros((n, d), dtype=np.float64)
    lib().adsa_oracle_rope_2d(_p(x, C.c_float), _p(pos, C.c_int), n, d, int(n_text), int(grid_w), C.c_double(base), _p(out, C.c_double))
    return out


def rmsnorm(x, w, eps=1e-5) -> np.ndarray:
    """Root-mean-square normalisation of every row of x [rows, dim] with weights w [dim] (float64 out)."""
    x, w = _f32(x), _f32(w)
    rows, dim = x.shape
    out = np.empty((rows, dim), dtype=np.float64)
    lib().adsa_oracle_rmsnorm(_p(x, C.c_float), _p(w, C.c_float), rows, dim, C.c_double(eps), _p(out, C.c_double))
    return out


def swiglu(gate, up) -> np.ndarray:
    """silu(gate) * up, element by element (float64 out)."""
    gate, up = _f32(gate), _f32(up)
    out = np.empty(gate.shape, dtype=np.float64)
    lib().adsa_oracle_swiglu(_p(gate, C.c_float), _p(up, C.c_float), C.c_longlong(gate.size), _p(out, C.c_double))
    return out


def cfg_sample(logits_cond, logits_uncond, scale, top_k, temperature, u):
    """Classifier-free guidance, top-k filter and inverse-CDF sampling for one image.
    Returns (token, mixed logits float64 [vocab], running share of the kept mass by token id float64 [vocab])."""
    lc, lu = _f32(logits_cond), _f32(logits_uncond)
    vocab = lc.shape[0]
    mixed, cdf = np.empty(vocab, dtype=np.float64), np.empty(vocab, dtype=np.float64)
    fn = lib().adsa_oracle_cfg_sample
    fn.restype = C.c_int
    tok = fn(_p(lc, C.c_float), _p(lu, C.c_float), vocab, C.c_double(scale), int(top_k), C.c_double(temperature),
             C.c_double(u), _p(mixed, C.c_double), _p(cdf, C.c_double))
    return int(tok), mixed, cdf


@dataclass
class StepResult:
    out: np.ndarray          # [streams, d] float64
    kept_pos: list           # per stream: positions retained from the cache (cache order)
    evict_pos: list          # per stream: positions evicted
    cand_pos: list           # per stream: candidate ("previous") positions
    cand_score: list         # per stream: their Eq. 2 scores, float32


class OracleStreams:
    """Cache state of `n_streams` independent streams plus the step function over them."""

    def __init__(self, n_streams, head_dim, cap_rows, n_text, grid_w, n_prefix, rows_back=1,
                 softmax_scale=0.0, score_variant=0, score_mode=0, share_heads=0):
        """score_mode 0: the paper's rule (Eq. 1-3 on V); 1: attention-mass pruning (Section 3.4's foil), with
        a per-row mass carried beside the rows (zero for rows loaded from outside).
        share_heads = H > 0: consecutive groups of H streams are the heads of one batch row and are scored as
        one (a token's V over all heads is one vector), so they keep the same tokens."""
        self.share_heads = share_heads
        assert share_heads == 0 or (n_streams % share_heads == 0 and score_mode == 0)
        self.n_streams, self.d, self.cap = n_streams, head_dim, cap_rows
        self.score_mode = score_mode
        self.mass = np.zeros((n_streams, cap_rows), dtype=np.float32)
        self.prm = _Params(n_text, grid_w, n_prefix, rows_back, score_variant, softmax_scale)
        self.n_live = np.zeros(n_streams, dtype=np.int32)
        self.pos = np.zeros((n_streams, cap_rows), dtype=np.int32)
        self.k = np.zeros((n_streams, cap_rows, head_dim), dtype=np.float32)
        self.v = np.zeros((n_streams, cap_rows, head_dim), dtype=np.float32)

    def load(self, stream, pos, k, v):
        """Replace one stream's cache with the given rows."""
        n = len(pos)
        assert n <= self.cap
        self.n_live[stream] = n
        self.pos[stream, :n] = pos
        self.k[stream, :n] = k
        self.v[stream, :n] = v
        self.mass[stream, :n] = 0.0

    def append_rows(self, k, v, first_pos):
        """Append rows [streams, n, d] at consecutive positions to every stream (the text condition)."""
        n = k.shape[1]
        for s in range(self.n_streams):
            a = int(self.n_live[s])
            assert a + n <= self.cap
            self.pos[s, a:a + n] = np.arange(first_pos, first_pos + n)
            self.k[s, a:a + n] = k[s]
            self.v[s, a:a + n] = v[s]
            self.mass[s, a:a + n] = 0.0
            self.n_live[s] = a + n

    def rows(self, stream):
        n = int(self.n_live[stream])
        return self.pos[stream, :n].copy(), self.k[stream, :n].copy(), self.v[stream, :n].copy()

    def step(self, q, k_new, v_new, cur_pos, budget, n_threads=0) -> StepResult:
        """One layer-step for all streams.  q, k_new, v_new: [streams, d] float32 (bf16-exact)."""
        S, d, cap = self.n_streams, self.d, self.cap
        q, k_new, v_new = _f32(q).reshape(S, d), _f32(k_new).reshape(S, d), _f32(v_new).reshape(S, d)
        out = np.zeros((S, d), dtype=np.float64)
        n_kept = np.zeros(S, dtype=np.int32)
        n_evict = np.zeros(S, dtype=np.int32)
        n_cand = np.zeros(S, dtype=np.int32)
        kept_pos = np.zeros((S, cap), dtype=np.int32)
        evict_pos = np.zeros((S, cap), dtype=np.int32)
        cand_pos = np.zeros((S, cap), dtype=np.int32)
        cand_score = np.zeros((S, cap), dtype=np.float32)
        if self.share_heads:
            failed = lib().adsa_oracle_layer_step_shared_batch(
                C.byref(self.prm), S // self.share_heads, self.share_heads, d, cap, _p(self.n_live, C.c_int),
                _p(self.pos, C.c_int), _p(self.k, C.c_float), _p(self.v, C.c_float), _p(q, C.c_float), _p(k_new, C.c_float),
                _p(v_new, C.c_float), int(cur_pos), int(budget), _p(out, C.c_double),
                _p(n_kept, C.c_int), _p(kept_pos, C.c_int), _p(n_evict, C.c_int), _p(evict_pos, C.c_int),
                _p(n_cand, C.c_int), _p(cand_pos, C.c_int), _p(cand_score, C.c_float), int(n_threads))
        elif self.score_mode == 1:
            failed = lib().adsa_oracle_layer_step_mass_batch(
                C.byref(self.prm), S, d, cap, _p(self.n_live, C.c_int), _p(self.pos, C.c_int),
                _p(self.k, C.c_float), _p(self.v, C.c_float), _p(self.mass, C.c_float), _p(q, C.c_float),
                _p(k_new, C.c_float), _p(v_new, C.c_float), int(cur_pos), int(budget), _p(out, C.c_double),
                _p(n_kept, C.c_int), _p(kept_pos, C.c_int), _p(n_evict, C.c_int), _p(evict_pos, C.c_int),
                _p(n_cand, C.c_int), _p(cand_pos, C.c_int), _p(cand_score, C.c_float), int(n_threads))
        else:
            failed = lib().adsa_oracle_layer_step_batch(
                C.byref(self.prm), S, d, cap, _p(self.n_live, C.c_int), _p(self.pos, C.c_int),
                _p(self.k, C.c_float), _p(self.v, C.c_float), _p(q, C.c_float), _p(k_new, C.c_float),
                _p(v_new, C.c_float), int(cur_pos), int(budget), _p(out, C.c_double),
                _p(n_kept, C.c_int), _p(kept_pos, C.c_int), _p(n_evict, C.c_int), _p(evict_pos, C.c_int),
                _p(n_cand, C.c_int), _p(cand_pos, C.c_int), _p(cand_score, C.c_float), int(n_threads))
        if failed:
            raise RuntimeError(f"oracle: {failed} stream(s) rejected the step (bad position or overflow)")
        return StepResult(
            out,
            [kept_pos[s, :n_kept[s]].copy() for s in range(S)],
            [evict_pos[s, :n_evict[s]].copy() for s in range(S)],
            [cand_pos[s, :n_cand[s]].copy() for s in range(S)],
            [cand_score[s, :n_cand[s]].copy() for s in range(S)],
        )


def max_threads() -> int:
    return lib().adsa_oracle_max_threads()

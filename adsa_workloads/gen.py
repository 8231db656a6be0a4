"""Counter-based seeded generators for q/k/v rows, rounded once to bf16.

Every tensor is a pure function of (seed, configuration, layer, step, tensor
kind): numpy's Philox bit generator is keyed with those integers, so any
layer-step can be drawn on its own, in any order, on any machine, and both the
CPU oracle and the CUDA path are handed the very same bf16 values (the oracle
as float32 arrays holding bf16-exact numbers, the CUDA path as the raw 16-bit
patterns).
"""
from __future__ import annotations

import numpy as np

from .configs import Workload

_T_Q, _T_K, _T_V, _T_PREFIX_K, _T_PREFIX_V, _T_GLOBAL, _T_STRUCT = range(7)


def _rng(seed: int, w: Workload, layer: int, step: int, tensor: int) -> np.random.Generator:
    k1 = (w.cfg_id << 56) | (tensor << 48) | (layer << 32) | (step & 0xFFFFFFFF)
    return np.random.Generator(np.random.Philox(key=[seed & 0xFFFFFFFFFFFFFFFF, k1]))


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bf16 (round-to-nearest-even) and return the uint16 patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + bias) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """Widen uint16 bf16 patterns to float32 exactly."""
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def _normal_bf16(rng: np.random.Generator, shape, sigma: float) -> np.ndarray:
    x = rng.standard_normal(shape, dtype=np.float32) * np.float32(sigma)
    return f32_to_bf16_bits(x)


def global_key_positions(w: Workload, seed: int) -> np.ndarray:
    """Config 1: the seeded context positions whose key rows are scaled x4."""
    if w.n_global_keys == 0:
        return np.zeros(0, dtype=np.int64)
    rng = _rng(seed, w, 0, 0, _T_GLOBAL)
    return np.sort(rng.choice(w.l_max, size=w.n_global_keys, replace=False))


def _scale_global(bits: np.ndarray, mask: np.ndarray) -> np.ndarray:
    # x4 is exact in bf16 (exponent shift), so scaling after rounding equals rounding after scaling
    f = bf16_bits_to_f32(bits)
    f[..., mask, :] *= np.float32(4.0)
    return f32_to_bf16_bits(f)


def prefix_kv(w: Workload, seed: int, layer: int):
    """K and V rows of the text condition: two uint16 arrays [batch, heads, n_text, head_dim]."""
    shape = (w.batch, w.n_heads, w.n_text, w.head_dim)
    k = _normal_bf16(_rng(seed, w, layer, 0, _T_PREFIX_K), shape, w.sigma)
    v = _normal_bf16(_rng(seed, w, layer, 0, _T_PREFIX_V), shape, w.sigma)
    gpos = global_key_positions(w, seed)
    gpos = gpos[gpos < w.n_text]
    if gpos.size:
        mask = np.zeros(w.n_text, dtype=bool)
        mask[gpos] = True
        k = _scale_global(k, mask)
    return k, v


def layer_step_qkv(w: Workload, seed: int, layer: int, step: int):
    """q, k, v of decode step `step` (grid cell index) at `layer`: uint16 [batch, heads, head_dim]."""
    shape = (w.batch, w.n_heads, w.head_dim)
    q = _normal_bf16(_rng(seed, w, layer, step, _T_Q), shape, w.sigma)
    k = _normal_bf16(_rng(seed, w, layer, step, _T_K), shape, w.sigma)
    v = _normal_bf16(_rng(seed, w, layer, step, _T_V), shape, w.sigma)
    if w.n_global_keys and (w.n_text + step) in set(global_key_positions(w, seed).tolist()):
        k = f32_to_bf16_bits(bf16_bits_to_f32(k) * np.float32(4.0))
    return q, k, v


def structured_values(kind: str, n_rows: int, head_dim: int, seed: int) -> np.ndarray:
    """V rows with structure, so that selection is not decided by pure noise.

    kinds: "clusters" (8 seeded centres + 0.3*N(0,1)), "duplicates" (every row
    appears twice: exact score ties), "equal" (all rows identical), "zeros"
    (a quarter of the rows are all-zero), "iid".  Returns uint16 [n_rows, head_dim].
    """
    rng = np.random.Generator(np.random.Philox(key=[seed, (_T_STRUCT << 48) | n_rows]))
    if kind == "iid":
        x = rng.standard_normal((n_rows, head_dim), dtype=np.float32)
    elif kind == "clusters":
        centres = rng.standard_normal((8, head_dim), dtype=np.float32)
        which = rng.integers(0, 8, size=n_rows)
        x = centres[which] + np.float32(0.3) * rng.standard_normal((n_rows, head_dim), dtype=np.float32)
    elif kind == "duplicates":
        half = rng.standard_normal(((n_rows + 1) // 2, head_dim), dtype=np.float32)
        x = np.concatenate([half, half], axis=0)[:n_rows]
        x = x[rng.permutation(n_rows)]
    elif kind == "equal":
        x = np.repeat(rng.standard_normal((1, head_dim), dtype=np.float32), n_rows, axis=0)
    elif kind == "zeros":
        x = rng.standard_normal((n_rows, head_dim), dtype=np.float32)
        x[rng.permutation(n_rows)[: max(1, n_rows // 4)]] = 0.0
    else:
        raise ValueError(f"unknown kind {kind!r}")
    return f32_to_bf16_bits(x)


def late_state(w: Workload, seed: int, n_rows: int, cur_pos: int, streams=None):
    """A seeded cache state as it could look late in a generation, for every stream of one layer.

    Each stream holds `n_rows` rows: the whole text condition, the 2*grid_w image cells just
    before `cur_pos`, and a per-stream random subset of the older image cells; the physical row
    order is shuffled (it is not part of the cache's meaning).  `streams` restricts the draw to
    some stream indices (each stream's state depends only on (seed, stream)).
    Returns pos int32 [S, n_rows], k and v uint16 [S, n_rows, head_dim].
    """
    d = w.head_dim
    recent = np.arange(max(w.n_text, cur_pos - 2 * w.grid_w), cur_pos)
    older = np.arange(w.n_text, recent[0]) if recent.size else np.arange(w.n_text, cur_pos)
    n_old = n_rows - w.n_text - recent.size
    if not 0 <= n_old <= older.size:
        raise ValueError("n_rows does not fit between the mandatory rows and the context")
    ids = list(range(w.streams_per_layer)) if streams is None else list(streams)
    pos = np.empty((len(ids), n_rows), dtype=np.int32)
    k = np.empty((len(ids), n_rows, d), dtype=np.uint16)
    v = np.empty((len(ids), n_rows, d), dtype=np.uint16)
    for i, s in enumerate(ids):
        rng = np.random.Generator(np.random.Philox(key=[seed & 0xFFFFFFFFFFFFFFFF,
                                                        (w.cfg_id << 56) | (_T_STRUCT << 48) | (1 << 40) | s]))
        pick = rng.choice(older, size=n_old, replace=False)
        row = np.concatenate([np.arange(w.n_text), pick, recent])
        pos[i] = row[rng.permutation(n_rows)]
        k[i] = _normal_bf16(rng, (n_rows, d), w.sigma)
        v[i] = _normal_bf16(rng, (n_rows, d), w.sigma)
    return pos, k, v

"""Shapes of the five benchmark configurations.

Each configuration is an attention stack with the shape of a LlamaGen decoder
(the model family the paper evaluates on, Section 5): a text condition of 120
tokens followed by an H x W grid of image tokens decoded in raster order, with
classifier-free guidance doubling the batch.  Only shapes live here; trained
weights, datasets and the rest of the transformer block are not part of the
decode-attention path.
"""
from __future__ import annotations

from dataclasses import dataclass, replace


@dataclass(frozen=True)
class Workload:
    name: str
    cfg_id: int          # stable id mixed into the random-number key
    n_layers: int
    batch: int           # batch rows (cond + uncond rows under CFG)
    n_heads: int
    head_dim: int
    n_text: int          # T0: text-condition rows written before decoding starts
    grid_h: int
    grid_w: int
    beta: float          # budget fraction of the full context
    sigma: float         # std of the synthetic q/k/v entries
    n_global_keys: int = 0   # config 1: seeded key positions scaled x4
    betas: tuple = ()        # config 5: budget sweep

    @property
    def streams_per_layer(self) -> int:
        return self.batch * self.n_heads

    @property
    def n_cells(self) -> int:
        return self.grid_h * self.grid_w

    @property
    def l_max(self) -> int:
        return self.n_text + self.n_cells

    @property
    def row_stride(self) -> int:
        """Pool row stride in elements: head_dim padded to a 16-byte multiple."""
        return (self.head_dim + 7) // 8 * 8

    def capacity(self, beta: float | None = None) -> int:
        """Fixed cache capacity in rows: floor(beta * L_max)."""
        b = self.beta if beta is None else beta
        # small epsilon keeps exact products such as 0.75 * 2424 from rounding down
        return int(b * self.l_max + 1e-9)

    def dense_kv_bytes(self) -> int:
        """K+V payload bytes of a dense (never evicting) bf16 cache."""
        return self.n_layers * self.streams_per_layer * self.l_max * 2 * self.head_dim * 2

    def with_beta(self, beta: float) -> "Workload":
        return replace(self, beta=beta)


def _sigma(d_model: int) -> float:
    # what W @ RMSNorm(x) gives per entry for W ~ N(0, 0.02^2): 0.02 * sqrt(d_model)
    return 0.02 * d_model ** 0.5


CONFIGS = {
    1: Workload("cfg1-single-layer-16x16", 1, 1, 1, 12, 64, 120, 16, 16, 0.5, 1.0, n_global_keys=8),
    2: Workload("cfg2-llamagen-B-16x16", 2, 12, 2, 12, 64, 120, 16, 16, 0.5, _sigma(768)),
    3: Workload("cfg3-llamagen-L-24x24", 3, 24, 16, 16, 64, 120, 24, 24, 0.5, _sigma(1024)),
    4: Workload("cfg4-llamagen-XL-32x32", 4, 36, 32, 20, 64, 120, 32, 32, 0.5, _sigma(1280)),
    5: Workload("cfg5-3B-stack-48x48", 5, 24, 64, 32, 100, 120, 48, 48, 0.5, 1.0,
                betas=(0.25, 0.5, 0.75)),
}


def get_workload(cfg: int, beta: float | None = None) -> Workload:
    w = CONFIGS[cfg]
    return w if beta is None else w.with_beta(beta)


def pick_page_rows(capacity: int, lo: int = 16, hi: int = 64, default: int = 32) -> int:
    """Rows per page for a pool serving streams of `capacity` rows.

    Prefers the largest page size in [lo, hi] that divides the capacity, so a
    full stream occupies whole pages and the pool's bytes equal the budget's
    share exactly; falls back to `default` (last page partly used) otherwise.
    """
    for pr in range(hi, lo - 1, -1):
        if capacity % pr == 0:
            return pr
    return default

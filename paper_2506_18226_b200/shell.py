"""A LlamaGen-shaped decoder around the ADSA attention, with random weights (Section 5 integrates the method with
LlamaGen; trained weights are not available, so this shell has the decoder's shapes and data flow and nothing of
its quality).

What runs where: the attention, the KV cache, the rotary embedding, the normalisations, the gated activation and
the sampling are libadsa calls; the projections, the residual additions and the embedding look-up are torch
(cuBLAS GEMMs: plain library contractions); the token ids go to a pinned host buffer as they are drawn, one
asynchronous copy per step (Section 4.2: generated ids are kept on the host until the image is decoded).

One block: x -> RMSNorm -> q, k, v projections -> 2-D RoPE on q and k -> ADSA layer-step -> output projection
(+ residual) -> RMSNorm -> gate/up projection -> silu(gate) * up -> down projection (+ residual).  Classifier-free
guidance doubles the batch: rows [0, n_images) are conditional, rows [n_images, 2 n_images) unconditional; both
halves are fed the same sampled ids.
"""
from __future__ import annotations

from dataclasses import dataclass

import torch

from . import binding as B


@dataclass(frozen=True)
class ShellConfig:
    n_layers: int
    dim: int
    n_heads: int
    ffn_hidden: int
    vocab: int = 16384
    n_text: int = 120
    grid_h: int = 32
    grid_w: int = 32
    n_images: int = 16
    budget_fraction: float = 0.5
    cfg_scale: float = 7.5
    top_k: int = 2000
    temperature: float = 1.0
    norm_eps: float = 1e-5

    @property
    def head_dim(self) -> int:
        return self.dim // self.n_heads

    @property
    def batch(self) -> int:
        return 2 * self.n_images

    @property
    def capacity(self) -> int:
        return int(self.budget_fraction * (self.n_text + self.grid_h * self.grid_w) + 1e-9)


# the three decoder sizes the benchmark configurations are shaped after (hidden sizes: 2/3 * 4 * dim rounded up to 256)
SHAPES = {
    "B": dict(n_layers=12, dim=768, n_heads=12, ffn_hidden=2048),
    "L": dict(n_layers=24, dim=1024, n_heads=16, ffn_hidden=2816),
    "XL": dict(n_layers=36, dim=1280, n_heads=20, ffn_hidden=3584),
}


class LlamaGenShell:
    def __init__(self, cfg: ShellConfig, seed: int = 0, device: str = "cuda:0", use_graphs: bool = True):
        self.cfg, self.dev = cfg, torch.device(device)
        self.use_graphs, self.graphs = use_graphs, None
        g = torch.Generator(device=self.dev).manual_seed(seed)
        bf = dict(dtype=torch.bfloat16, device=self.dev)

        def w(*shape):
            return (0.02 * torch.randn(*shape, generator=g, device=self.dev)).to(torch.bfloat16)

        L, D, Hd, V = cfg.n_layers, cfg.dim, cfg.ffn_hidden, cfg.vocab
        self.tok_emb = w(V, D)
        self.wqkv_t = w(L, 3, D, D)         # q, k, v projections, stored transposed: [layer][which][in][out]
        self.wo = w(L, D, D)
        self.w13 = w(L, 2 * Hd, D)          # gate and up projections side by side
        self.w2 = w(L, D, Hd)
        self.norm1 = torch.ones(L, D, **bf)
        self.norm2 = torch.ones(L, D, **bf)
        self.norm_f = torch.ones(D, **bf)
        self.head = w(V, D)
        C = self.budget = max(cfg.capacity, cfg.n_text + 1)   # rows a stream may hold (a row is evicted before one is inserted)
        # rows per pool page: the largest divisor of the capacity up to 1024 rows, so that a full stream fills whole pages
        page_rows = next((pr for pr in range(min(C, 1024), 15, -1) if C % pr == 0), 32)
        self.eng = B.AdsaEngine(n_layers=L, batch=cfg.batch, n_heads=cfg.n_heads, head_dim=cfg.head_dim, n_text=cfg.n_text,
                                grid_h=cfg.grid_h, grid_w=cfg.grid_w, max_rows_per_stream=C,
                                page_rows=page_rows, device=device)
        Bt, H, d = cfg.batch, cfg.n_heads, cfg.head_dim
        self.qkv = torch.empty(3, Bt, H, d, **bf)    # q, k, v of a decode step, each dense [batch, heads, head_dim]
        self.q, self.k, self.v = self.qkv[0], self.qkv[1], self.qkv[2]
        self.o = torch.empty(Bt, H, d, **bf)
        self.h = torch.empty(Bt, D, **bf)
        self.gu = torch.empty(Bt, 2 * Hd, **bf)
        self.act = torch.empty(Bt, Hd, **bf)
        self.logits = torch.empty(Bt, V, **bf)
        self.pos = torch.zeros(2 * Bt * H, dtype=torch.int32, device=self.dev)   # one per row of q and of k
        self.tokens = torch.zeros(cfg.n_images, dtype=torch.int32, device=self.dev)
        self.ids_host = torch.zeros(cfg.grid_h * cfg.grid_w, cfg.n_images, dtype=torch.int32).pin_memory()
        # the random numbers of the whole generation, drawn once (the sampling call takes them as an input)
        self.uniforms = torch.rand(cfg.grid_h * cfg.grid_w, cfg.n_images, generator=g, device=self.dev, dtype=torch.float32)
        self.kernel_calls = 0               # libadsa calls made (each is at least one kernel of the library)
        self.x = torch.empty(Bt, D, **bf)   # the residual stream of a decode step
        self.u = torch.zeros(cfg.n_images, dtype=torch.float32, device=self.dev)   # this step's uniform numbers

    # the projections in the usual [out][in] orientation (views)
    wq = property(lambda self: self.wqkv_t[:, 0].transpose(1, 2))
    wk = property(lambda self: self.wqkv_t[:, 1].transpose(1, 2))
    wv = property(lambda self: self.wqkv_t[:, 2].transpose(1, 2))

    # -- one block on a [rows, dim] activation; `attend` does the attention for this layer ------------------------
    def _block(self, layer, x, attend):
        c = self.cfg
        step = x.shape[0] == c.batch                                       # a decode step reuses its buffers
        h = B.rmsnorm(x, self.norm1[layer], out=self.h if step else None, eps=c.norm_eps)
        attn = attend(layer, h)                                            # [rows, dim]
        x.addmm_(attn, self.wo[layer].t())
        h = B.rmsnorm(x, self.norm2[layer], out=self.h if step else None, eps=c.norm_eps)
        gu = torch.mm(h, self.w13[layer].t(), out=self.gu) if step else h @ self.w13[layer].t()
        act = B.swiglu(gu[:, :c.ffn_hidden], gu[:, c.ffn_hidden:], out=self.act if step else None)
        x.addmm_(act, self.w2[layer].t())
        self.kernel_calls += 3
        return x

    def prefill(self, text_emb):
        """The condition: text_emb [batch, n_text, dim] bf16 (rows of the unconditional half are the caller's null
        condition).  Fills the caches through dense causal attention and returns the first image tokens."""
        c = self.cfg
        Bt, T, H, d = c.batch, c.n_text, c.n_heads, c.head_dim
        self.eng.reset()
        x = text_emb.reshape(Bt * T, c.dim).clone()
        pos = torch.arange(T, dtype=torch.int32, device=self.dev).repeat(Bt * H)            # condition rows are not rotated
        out = torch.empty(Bt, H, T, d, dtype=torch.bfloat16, device=self.dev)

        def attend(layer, h):
            q, k, v = ((h @ self.wqkv_t[layer, i]).view(Bt, T, H, d).transpose(1, 2).contiguous() for i in range(3))
            self.eng.rope_2d(q, pos)
            self.eng.rope_2d(k, pos)
            self.eng.prefill_attn(layer, q, k, v, 0, out)
            self.kernel_calls += 3
            return out.transpose(1, 2).reshape(Bt * T, c.dim)

        for layer in range(c.n_layers):
            x = self._block(layer, x, attend)
        return self._sample(x.view(Bt, T, c.dim)[:, -1].contiguous(), 0)

    # -- a decode step as CUDA graphs around the attention launches ---------------------------------------------------
    # Everything between two attention launches works on fixed buffers with fixed arguments, so it is captured once:
    # graph 0 = embedding look-up and the first block's part before the attention; graph l + 1 = block l's part after
    # the attention and block l + 1's part before it (the last one ends with the LM head and the sampling).  The
    # attention launches stay outside: their arguments (position, budget, carried state) change every step.
    def _pre(self, layer):
        c = self.cfg
        B.rmsnorm(self.x, self.norm1[layer], out=self.h, eps=c.norm_eps)
        torch.bmm(self.h.unsqueeze(0).expand(3, -1, -1), self.wqkv_t[layer], out=self.qkv.view(3, c.batch, c.dim))
        self.eng.rope_2d(self.qkv[:2], self.pos)

    def _post(self, layer):
        c = self.cfg
        self.x.addmm_(self.o.view(c.batch, c.dim), self.wo[layer].t())
        B.rmsnorm(self.x, self.norm2[layer], out=self.h, eps=c.norm_eps)
        torch.mm(self.h, self.w13[layer].t(), out=self.gu)
        B.swiglu(self.gu[:, :c.ffn_hidden], self.gu[:, c.ffn_hidden:], out=self.act)
        self.x.addmm_(self.act, self.w2[layer].t())

    def _first(self):
        n = self.cfg.n_images
        torch.index_select(self.tok_emb, 0, self.tokens, out=self.x[:n])
        self.x[n:].copy_(self.x[:n])                                       # conditional and unconditional rows
        self._pre(0)

    def _last(self):
        c = self.cfg
        B.rmsnorm(self.x, self.norm_f, out=self.h, eps=c.norm_eps)
        torch.mm(self.h, self.head.t(), out=self.logits)
        B.cfg_sample(self.logits, c.cfg_scale, min(c.top_k, c.vocab), c.temperature, self.u, tokens=self.tokens)

    def _segments(self):
        L = self.cfg.n_layers
        segs = [self._first]
        for layer in range(L):
            nxt = (lambda l=layer: (self._post(l), self._pre(l + 1))) if layer + 1 < L else (lambda l=layer: (self._post(l), self._last()))
            segs.append(nxt)
        return segs

    def _capture(self):
        segs = self._segments()
        side = torch.cuda.Stream(device=self.dev)
        side.wait_stream(torch.cuda.current_stream(self.dev))
        with torch.cuda.stream(side):                                      # once eagerly: libraries make their handles and workspaces
            for seg in segs:
                seg()
        torch.cuda.current_stream(self.dev).wait_stream(side)
        torch.cuda.synchronize(self.dev)
        graphs = []
        for seg in segs:
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                seg()
            graphs.append(g)
        self.graphs = graphs

    def decode_step(self, cell):
        """The image token of grid cell `cell` (>= 1) from the token of cell - 1: one pass through every layer."""
        c = self.cfg
        cur = c.n_text + cell - 1                                          # position of the token that is fed in
        if self.use_graphs:
            if self.graphs is None:
                saved = self.tokens.clone()
                self._capture()                                            # (the capture's trial run overwrote the ids)
                self.tokens.copy_(saved)
            self.pos.fill_(cur)
            self.u.copy_(self.uniforms[cell])
            self.graphs[0].replay()
            for layer in range(c.n_layers):
                self.eng.layer_step(layer, cur, self.budget, self.q, self.k, self.v, self.o)
                self.graphs[layer + 1].replay()
            self.ids_host[cell].copy_(self.tokens, non_blocking=True)
            self.kernel_calls += 5 * c.n_layers + 3
            return self.tokens
        emb = self.tok_emb[self.tokens.long()]
        x = torch.cat([emb, emb], dim=0)                                   # conditional and unconditional rows
        self.pos.fill_(cur)

        def attend(layer, h):
            torch.bmm(h.unsqueeze(0).expand(3, -1, -1), self.wqkv_t[layer], out=self.qkv.view(3, c.batch, c.dim))   # one batched GEMM
            self.eng.rope_2d(self.qkv[:2], self.pos)                       # q and k in one call
            self.eng.layer_step(layer, cur, self.budget, self.q, self.k, self.v, self.o)
            self.kernel_calls += 2
            return self.o.view(c.batch, c.dim)

        for layer in range(c.n_layers):
            x = self._block(layer, x, attend)
        return self._sample(x, cell)

    def _sample(self, x_last, cell):
        c = self.cfg
        h = B.rmsnorm(x_last, self.norm_f, eps=c.norm_eps)
        torch.mm(h, self.head.t(), out=self.logits)
        B.cfg_sample(self.logits, c.cfg_scale, min(c.top_k, c.vocab), c.temperature, self.uniforms[cell], tokens=self.tokens)
        self.ids_host[cell].copy_(self.tokens, non_blocking=True)          # ids leave the GPU as they are drawn
        self.kernel_calls += 2
        return self.tokens

    def generate(self, text_emb, n_cells=None):
        """Prefill and decode `n_cells` grid cells (default: the whole grid); returns the ids on the host, [cells, n_images]."""
        n = self.cfg.grid_h * self.cfg.grid_w if n_cells is None else n_cells
        self.prefill(text_emb)
        for cell in range(1, n):
            self.decode_step(cell)
        torch.cuda.synchronize(self.dev)
        return self.ids_host[:n]

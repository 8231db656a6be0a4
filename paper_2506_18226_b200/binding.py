"""Python binding of libadsa: argument marshalling only.

Every step of the path (scoring, selection, attention, cache update, paging)
runs inside the CUDA kernels of libadsa.so; this module turns torch tensors
into device pointers and calls the C functions of the same names.  torch is
used for device memory and streams, nothing else.  There is no CPU fallback:
if the library cannot be loaded or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes as C

import torch

from .build import build_lib

OK, EINVAL, ESTATE, ENOMEM, ECUDA = 0, -1, -2, -3, -4
DEV_POOL_EXHAUSTED, DEV_BAD_POSITION, DEV_ROW_OVERFLOW, DEV_RING_TIMEOUT, DEV_BAD_EVICT, DEV_COPY_TIMEOUT = \
    1, 2, 4, 8, 16, 32

EXPORTS = [
    "adsa_workspace_bytes", "adsa_create", "adsa_destroy", "adsa_reset", "adsa_prefill_rows",
    "adsa_set_stream_rows", "adsa_prefill_attn", "adsa_rope_2d", "adsa_score", "adsa_select", "adsa_sparse_decode_attn", "adsa_kv_update",
    "adsa_layer_step", "adsa_layer_step_host", "adsa_token_step", "adsa_token_step_gated", "adsa_token_step_host", "adsa_plan_attn", "adsa_set_attn_chunk_rows", "adsa_set_staged", "adsa_set_ring_stages", "adsa_set_l2_lookahead", "adsa_set_next_layer_hint", "adsa_set_token_launch", "adsa_set_host_chunks", "adsa_set_stream_warps", "adsa_set_single_sweep",
    "adsa_layer_rows_bound", "adsa_get_status", "adsa_launch_count", "adsa_strerror", "adsa_decode_attn_static",
    "adsa_rmsnorm", "adsa_swiglu", "adsa_cfg_sample",
]


class AdsaConfig(C.Structure):
    _fields_ = [(n, C.c_int32) for n in (
        "n_layers", "batch", "n_heads", "head_dim", "row_stride", "page_rows", "n_pages",
        "max_rows_per_stream", "n_text", "grid_h", "grid_w", "n_prefix", "local_rows_back", "score_mode", "score_share")] + \
        [("softmax_scale", C.c_float)]


class AdsaBuffers(C.Structure):
    _fields_ = [("k_pool", C.c_void_p), ("v_pool", C.c_void_p), ("page_table", C.c_void_p), ("pos", C.c_void_p),
                ("inv_norm", C.c_void_p), ("n_live", C.c_void_p), ("free_ring", C.c_void_p),
                ("free_state", C.c_void_p), ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t)]


class AdsaError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        super().__init__(f"{what}: {strerror(status)} ({status})")


_lib = None


def load(rebuild: bool = False) -> C.CDLL:
    """Load libadsa.so, building it first if it is missing or older than its sources."""
    global _lib
    if _lib is None or rebuild:
        lib = C.CDLL(build_lib(rebuild))
        vp, i32, sz = C.c_void_p, C.c_int, C.c_size_t
        sig = {
            "adsa_workspace_bytes": [C.POINTER(AdsaConfig), C.POINTER(sz)],
            "adsa_create": [C.POINTER(AdsaConfig), C.POINTER(AdsaBuffers), C.POINTER(vp)],
            "adsa_destroy": [vp],
            "adsa_reset": [vp, vp],
            "adsa_prefill_rows": [vp, i32, vp, vp, vp, i32, i32, vp],
            "adsa_set_stream_rows": [vp, i32, i32, i32, vp, vp, vp, i32, vp],
            "adsa_prefill_attn": [vp, i32, vp, vp, vp, i32, i32, vp, vp, vp],
            "adsa_rope_2d": [vp, vp, vp, C.c_longlong, C.c_float, vp],
            "adsa_score": [vp, i32, i32, vp, vp],
            "adsa_select": [vp, i32, i32, i32, vp, vp, vp, vp, vp],
            "adsa_sparse_decode_attn": [vp, i32, i32, vp, vp, vp, vp, vp, vp],
            "adsa_kv_update": [vp, i32, i32, vp, vp, vp],
            "adsa_layer_step": [vp, i32, i32, i32, vp, vp, vp, vp, vp],
            "adsa_layer_step_host": [vp, i32, i32, i32, vp, vp, vp, vp, vp],
            "adsa_token_step": [vp, i32, i32, vp, vp, vp, vp, vp],
            "adsa_token_step_host": [vp, i32, i32, vp, vp, vp, vp, vp],
            "adsa_token_step_gated": [vp, i32, i32, vp, vp, vp, vp, vp, i32, vp],
            "adsa_plan_attn": [vp, i32, C.POINTER(i32), C.POINTER(i32)],
            "adsa_set_attn_chunk_rows": [vp, i32],
            "adsa_set_staged": [vp, i32],
            "adsa_set_ring_stages": [vp, i32],
            "adsa_set_l2_lookahead": [vp, i32],
            "adsa_set_next_layer_hint": [vp, i32],
            "adsa_set_token_launch": [vp, i32],
            "adsa_set_host_chunks": [vp, i32],
            "adsa_set_stream_warps": [vp, i32],
            "adsa_set_single_sweep": [vp, i32],
            "adsa_layer_rows_bound": [vp, i32, C.POINTER(i32)],
            "adsa_get_status": [vp, C.POINTER(C.c_uint32), C.POINTER(C.c_int32 * 4)],
            "adsa_decode_attn_static": [vp, vp, vp, vp, vp, vp, i32, i32, i32, i32, C.c_float, vp, vp, vp],
            "adsa_rmsnorm": [vp, vp, vp, C.c_longlong, i32, C.c_float, vp],
            "adsa_swiglu": [vp, vp, vp, C.c_longlong, i32, C.c_longlong, vp],
            "adsa_cfg_sample": [vp, i32, i32, C.c_float, i32, C.c_float, vp, vp, vp],
        }
        for name, args in sig.items():
            fn = getattr(lib, name)
            fn.argtypes, fn.restype = args, C.c_int
        lib.adsa_launch_count.argtypes, lib.adsa_launch_count.restype = [vp], C.c_int64
        lib.adsa_strerror.argtypes, lib.adsa_strerror.restype = [C.c_int], C.c_char_p
        _lib = lib
    return _lib


def strerror(status: int) -> str:
    return load().adsa_strerror(int(status)).decode()


def workspace_bytes(cfg: AdsaConfig) -> int:
    out = C.c_size_t(0)
    rc = load().adsa_workspace_bytes(C.byref(cfg), C.byref(out))
    if rc:
        raise AdsaError(rc, "adsa_workspace_bytes")
    return out.value


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def decode_attn_static(q, k, v, n_rows, k_new, v_new, out_bf16=None, out_f32=None, head_dim=None,
                       softmax_scale=0.0):
    """adsa_decode_attn_static: attention over dense rows with the library's built-in scratch.

    For hosts that cannot allocate device memory when they need attention (frozen memory plan,
    allocation calls forbidden, memory wholly owned by a pool): no context, no workspace, nothing
    allocated.  k, v: [n_streams, max_rows, row_stride] bf16; q, k_new, v_new: [n_streams, head_dim];
    n_rows: int32 [n_streams].  Calls must not overlap on the GPU (they share the scratch)."""
    n_streams, max_rows, row_stride = k.shape
    d = q.shape[-1] if head_dim is None else head_dim
    rc = load().adsa_decode_attn_static(_ptr(q), _ptr(k), _ptr(v), _ptr(n_rows), _ptr(k_new), _ptr(v_new),
                                        n_streams, max_rows, d, row_stride, softmax_scale, _ptr(out_bf16),
                                        _ptr(out_f32), _stream())
    if rc:
        raise AdsaError(rc, "adsa_decode_attn_static")


def rmsnorm(x, w, out=None, eps=1e-5):
    """adsa_rmsnorm: out[r] = x[r] / sqrt(mean(x[r]^2) + eps) * w, rows of bf16 [.., dim] (contiguous)."""
    out = torch.empty_like(x) if out is None else out
    rc = load().adsa_rmsnorm(_ptr(x), _ptr(w), _ptr(out), x.numel() // x.shape[-1], x.shape[-1], float(eps), _stream())
    if rc:
        raise AdsaError(rc, "adsa_rmsnorm")
    return out


def swiglu(gate, up, out=None):
    """adsa_swiglu: silu(gate) * up.  gate, up: bf16 [rows, hidden], either two contiguous tensors or the two halves
    of one contiguous [rows, 2 * hidden] tensor (views)."""
    rows, hidden = gate.shape
    ld = gate.stride(0)
    if up.stride(0) != ld or gate.stride(1) != 1 or up.stride(1) != 1:
        raise ValueError("gate and up must share a row pitch and be dense along the row")
    out = torch.empty((rows, hidden), dtype=gate.dtype, device=gate.device) if out is None else out
    rc = load().adsa_swiglu(_ptr(gate), _ptr(up), _ptr(out), rows, hidden, ld, _stream())
    if rc:
        raise AdsaError(rc, "adsa_swiglu")
    return out


def cfg_sample(logits, scale, top_k, temperature, uniforms, tokens=None):
    """adsa_cfg_sample: the next image token of every image.  logits: bf16 [2 * n_images, vocab] (conditional rows,
    then unconditional rows), uniforms: f32 [n_images] in [0, 1); returns int32 [n_images]."""
    n_images, vocab = logits.shape[0] // 2, logits.shape[1]
    tokens = torch.empty(n_images, dtype=torch.int32, device=logits.device) if tokens is None else tokens
    rc = load().adsa_cfg_sample(_ptr(logits), n_images, vocab, float(scale), int(top_k), float(temperature), _ptr(uniforms),
                                _ptr(tokens), _stream())
    if rc:
        raise AdsaError(rc, "adsa_cfg_sample")
    return tokens


class AdsaEngine:
    """Owns the device buffers of one context and forwards to the C-ABI.

    Methods carry the names of the C functions without the `adsa_` prefix and
    take torch tensors (bf16 payloads may be passed as bfloat16 or as their
    int16/uint16 bit patterns).  All calls enqueue on torch's current stream.
    """

    def __init__(self, *, n_layers, batch, n_heads, head_dim, n_text, grid_h, grid_w, max_rows_per_stream,
                 page_rows=32, n_pages=None, n_prefix=None, local_rows_back=1, softmax_scale=0.0, row_stride=None,
                 device="cuda:0", allocate=True, score_mode=0, score_share=0):
        self.lib = load()
        self.device = torch.device(device)
        row_stride = (head_dim + 7) // 8 * 8 if row_stride is None else row_stride
        self.max_pages = (max_rows_per_stream + page_rows - 1) // page_rows
        self.n_streams = n_layers * batch * n_heads
        if n_pages is None:
            n_pages = self.n_streams * self.max_pages
        self.cfg = AdsaConfig(n_layers, batch, n_heads, head_dim, row_stride, page_rows, n_pages,
                              max_rows_per_stream, n_text, grid_h, grid_w,
                              n_text if n_prefix is None else n_prefix, local_rows_back, score_mode, score_share, softmax_scale)
        self.S = batch * n_heads
        self.ctx = C.c_void_p(None)
        self._t = {}
        if allocate:
            self._allocate()

    # -- plumbing ----------------------------------------------------------
    def _allocate(self):
        cfg, dev = self.cfg, self.device
        i32 = dict(dtype=torch.int32, device=dev)
        pool_shape = (cfg.n_pages, cfg.page_rows, cfg.row_stride)
        t = self._t
        t["k_pool"] = torch.zeros(pool_shape, dtype=torch.bfloat16, device=dev)
        t["v_pool"] = torch.zeros(pool_shape, dtype=torch.bfloat16, device=dev)
        t["page_table"] = torch.zeros((self.n_streams, self.max_pages), **i32)
        t["pos"] = torch.zeros((self.n_streams, cfg.max_rows_per_stream), **i32)
        t["inv_norm"] = torch.zeros((self.n_streams, cfg.max_rows_per_stream), dtype=torch.float32, device=dev)
        t["n_live"] = torch.zeros(self.n_streams, **i32)
        t["free_ring"] = torch.zeros(cfg.n_pages, **i32)
        t["free_state"] = torch.zeros(4, **i32)
        wsb = workspace_bytes(cfg)
        t["workspace"] = torch.zeros(wsb + 256, dtype=torch.uint8, device=dev)
        ws_ptr = (t["workspace"].data_ptr() + 255) // 256 * 256
        self.buf = AdsaBuffers(t["k_pool"].data_ptr(), t["v_pool"].data_ptr(), t["page_table"].data_ptr(),
                               t["pos"].data_ptr(), t["inv_norm"].data_ptr(), t["n_live"].data_ptr(),
                               t["free_ring"].data_ptr(), t["free_state"].data_ptr(), ws_ptr, wsb)
        with torch.cuda.device(dev):
            rc = self.lib.adsa_create(C.byref(self.cfg), C.byref(self.buf), C.byref(self.ctx))
        if rc:
            raise AdsaError(rc, "adsa_create")
        self.reset()

    def _call(self, name, *args):
        rc = getattr(self.lib, name)(self.ctx, *args)
        if rc:
            raise AdsaError(rc, name)

    def close(self):
        if self.ctx:
            self.lib.adsa_destroy(self.ctx)
            self.ctx = C.c_void_p(None)

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- the C-ABI, one method per function --------------------------------
    def reset(self):
        self._call("adsa_reset", _stream())

    def prefill_rows(self, layer, k, v, first_pos=0, pos=None):
        """k, v: [batch, heads, n_rows, head_dim] bf16 on the device; pos: optional int32 [batch, heads, n_rows]."""
        n_rows = k.shape[-2]
        self._call("adsa_prefill_rows", layer, _ptr(k), _ptr(v), _ptr(pos), n_rows, first_pos, _stream())

    def prefill_attn(self, layer, q, k, v, first_pos=0, out_bf16=None, out_f32=None):
        """Dense causal attention over the given rows, which also enter the (empty) cache.  [batch, heads, n_rows, head_dim]."""
        self._call("adsa_prefill_attn", layer, _ptr(q), _ptr(k), _ptr(v), k.shape[-2], first_pos, _ptr(out_bf16), _ptr(out_f32),
                   _stream())

    def rope_2d(self, x, pos, base=0.0):
        """2-D rotary embedding in place.  x: [..., head_dim] bf16 (contiguous), pos: int32, one per row of x."""
        self._call("adsa_rope_2d", _ptr(x), _ptr(pos), x.numel() // x.shape[-1], float(base), _stream())

    def set_stream_rows(self, layer, b, h, k, v, pos):
        n = 0 if pos is None else int(pos.shape[0])
        self._call("adsa_set_stream_rows", layer, b, h, _ptr(k), _ptr(v), _ptr(pos), n, _stream())

    def score(self, layer, cur_pos, scores_out=None):
        self._call("adsa_score", layer, cur_pos, _ptr(scores_out), _stream())

    def select(self, layer, cur_pos, budget_rows, sel_slots=None, sel_pos=None, evict_pos=None, counts=None):
        self._call("adsa_select", layer, cur_pos, budget_rows, _ptr(sel_slots), _ptr(sel_pos), _ptr(evict_pos),
                   _ptr(counts), _stream())

    def sparse_decode_attn(self, layer, cur_pos, q, k_new, v_new, out_bf16=None, out_f32=None):
        self._call("adsa_sparse_decode_attn", layer, cur_pos, _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(out_bf16),
                   _ptr(out_f32), _stream())

    def kv_update(self, layer, cur_pos, k_new, v_new):
        self._call("adsa_kv_update", layer, cur_pos, _ptr(k_new), _ptr(v_new), _stream())

    def layer_step(self, layer, cur_pos, budget_rows, q, k_new, v_new, out_bf16):
        self._call("adsa_layer_step", layer, cur_pos, budget_rows, _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(out_bf16),
                   _stream())

    def layer_step_host(self, layer, cur_pos, budget_rows, q, k_new, v_new, out):
        """q, k_new, v_new, out: HOST tensors (pinned for asynchronous copies).  Synchronises the stream."""
        for t in (q, k_new, v_new, out):
            if t.is_cuda:
                raise ValueError("layer_step_host takes host tensors")
        self._call("adsa_layer_step_host", layer, cur_pos, budget_rows, _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(out),
                   _stream())

    def token_step(self, cur_pos, budget_rows, q, k_new, v_new, out_bf16):
        """All layers of one token; tensors are [n_layers, batch, heads, head_dim] bf16 on the device."""
        self._call("adsa_token_step", cur_pos, budget_rows, _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(out_bf16),
                   _stream())

    def token_step_gated(self, cur_pos, budget_rows, q, k_new, v_new, out_bf16, ready, epoch):
        """token_step that reads layer l's inputs only once ready[l] - epoch >= 0 (ready: int32 [n_layers] on the device)."""
        self._call("adsa_token_step_gated", cur_pos, budget_rows, _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(out_bf16),
                   _ptr(ready), int(epoch), _stream())

    def token_step_host(self, cur_pos, budget_rows, q, k_new, v_new, out):
        """token_step with HOST tensors (pinned for asynchronous copies).  Synchronises the stream."""
        for t in (q, k_new, v_new, out):
            if t.is_cuda:
                raise ValueError("token_step_host takes host tensors")
        self._call("adsa_token_step_host", cur_pos, budget_rows, _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(out),
                   _stream())

    def plan_attn(self, n_rows):
        a, b = C.c_int(0), C.c_int(0)
        self._call("adsa_plan_attn", n_rows, C.byref(a), C.byref(b))
        return a.value, b.value

    def set_attn_chunk_rows(self, chunk_rows):
        self._call("adsa_set_attn_chunk_rows", chunk_rows)

    def set_staged(self, mode):
        """0 streaming kernels, 1 automatic, 2 cluster kernel, 3 persistent (CUDA cores), 4 persistent (MMA)."""
        self._call("adsa_set_staged", int(mode))

    def set_stream_warps(self, warps):
        self._call("adsa_set_stream_warps", int(warps))

    def set_single_sweep(self, mode):
        """0 always a second sweep, 1 scores during the attention sweep, 2 (default) also the carried evictee."""
        self._call("adsa_set_single_sweep", int(mode))

    def set_ring_stages(self, max_stages):
        self._call("adsa_set_ring_stages", int(max_stages))

    def set_l2_lookahead(self, tiles):
        self._call("adsa_set_l2_lookahead", int(tiles))

    def set_host_chunks(self, chunks):
        self._call("adsa_set_host_chunks", int(chunks))

    def set_token_launch(self, mode):
        """token_step: 1 one launch for every layer (default), 0 one launch per layer."""
        self._call("adsa_set_token_launch", int(mode))

    def set_next_layer_hint(self, tiles):
        self._call("adsa_set_next_layer_hint", int(tiles))

    def layer_rows_bound(self, layer):
        a = C.c_int(0)
        self._call("adsa_layer_rows_bound", layer, C.byref(a))
        return a.value

    def get_status(self):
        st, fs = C.c_uint32(0), (C.c_int32 * 4)()
        self._call("adsa_get_status", C.byref(st), C.byref(fs))
        return st.value, list(fs)

    def launch_count(self):
        return int(self.lib.adsa_launch_count(self.ctx))

    # -- read-back helpers for tests and reports (plain copies, no arithmetic) --
    def stream_index(self, layer, b, h):
        return (layer * self.cfg.batch + b) * self.cfg.n_heads + h

    def read_stream(self, sid):
        """(pos[n], k_bits[n, d], v_bits[n, d]) of one stream, as CPU tensors (bf16 as int16 bit patterns)."""
        t, cfg = self._t, self.cfg
        n = int(t["n_live"][sid].item())
        if n == 0:
            e = torch.zeros((0, cfg.head_dim), dtype=torch.int16)
            return torch.zeros(0, dtype=torch.int32), e, e.clone()
        slots = torch.arange(n, device=self.device)
        pages = t["page_table"][sid][slots // cfg.page_rows].long()
        rows = slots % cfg.page_rows
        k = t["k_pool"][pages, rows][:, :cfg.head_dim].view(torch.int16).cpu()
        v = t["v_pool"][pages, rows][:, :cfg.head_dim].view(torch.int16).cpu()
        return t["pos"][sid, :n].cpu(), k, v

    def pool_bytes_peak(self):
        """Bytes of K+V pages that were in use at the high-water mark since the last reset."""
        _, fs = self.get_status()
        cfg = self.cfg
        return (cfg.n_pages - fs[3]) * cfg.page_rows * cfg.row_stride * 2 * 2

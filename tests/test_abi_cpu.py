"""Host-side checks of libadsa that need no GPU: the library loads, exports every
function the header declares, validates configurations, sizes its workspace and
plans launches.  No kernel is launched here."""
import ctypes as C
import os
import re

import pytest

import paper_2506_18226_b200 as A
from paper_2506_18226_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "adsa.h")).read()
    return sorted(set(re.findall(r"ADSA_API[^;(]*?\b(adsa_[a-z_0-9]+)\s*\(", text)))


def _cfg(**kw):
    base = dict(n_layers=2, batch=2, n_heads=4, head_dim=64, row_stride=64, page_rows=16, n_pages=400,
                max_rows_per_stream=188, n_text=120, grid_h=16, grid_w=16, n_prefix=120, local_rows_back=1,
                score_mode=0, score_share=0, softmax_scale=0.0)
    base.update(kw)
    return A.AdsaConfig(*[base[n] for n, _ in A.AdsaConfig._fields_])


def test_library_exports_every_declared_symbol():
    lib = A.load()
    names = _declared()
    assert len(names) >= 18
    assert sorted(A.EXPORTS) == names
    for n in names:
        assert hasattr(lib, n), n


def test_strerror_and_workspace_size():
    assert A.strerror(0) == "ok"
    assert "order" in A.strerror(B.ESTATE)
    small, big = A.workspace_bytes(_cfg()), A.workspace_bytes(_cfg(batch=32))
    assert 0 < small < big and small % 256 == 0


@pytest.mark.parametrize("bad", [
    dict(head_dim=4), dict(head_dim=300, row_stride=304), dict(row_stride=60), dict(row_stride=100, head_dim=100),
    dict(page_rows=1), dict(n_pages=0), dict(max_rows_per_stream=0), dict(grid_w=0), dict(n_prefix=-1),
    dict(score_mode=3), dict(score_share=2), dict(score_share=1, score_mode=1), dict(softmax_scale=-1.0), dict(n_layers=0),
])
def test_invalid_configurations_are_rejected(bad):
    out = C.c_size_t(0)
    assert A.load().adsa_workspace_bytes(C.byref(_cfg(**bad)), C.byref(out)) == B.EINVAL


def _fake_ctx(cfg, ws_slack=0):
    """A context over made-up (never dereferenced) device addresses: enough for host logic."""
    ws = A.workspace_bytes(cfg)
    buf = A.AdsaBuffers(*([0x10000000 + 0x1000000 * i for i in range(9)] + [ws + ws_slack]))
    ctx = C.c_void_p(None)
    rc = A.load().adsa_create(C.byref(cfg), C.byref(buf), C.byref(ctx))
    return rc, ctx


def test_create_checks_buffers_and_workspace():
    cfg = _cfg()
    rc, ctx = _fake_ctx(cfg)
    assert rc == 0 and ctx.value
    A.load().adsa_destroy(ctx)
    rc, ctx = _fake_ctx(cfg, ws_slack=-1)
    assert rc == B.ENOMEM and not ctx.value
    buf = A.AdsaBuffers(*([0] * 9 + [1 << 30]))
    assert A.load().adsa_create(C.byref(cfg), C.byref(buf), C.byref(ctx)) == B.EINVAL
    buf = A.AdsaBuffers(*([0x10000008] + [0x20000000] * 8 + [1 << 30]))     # k_pool not 16-byte aligned
    assert A.load().adsa_create(C.byref(cfg), C.byref(buf), C.byref(ctx)) == B.EINVAL


def test_attention_plan_covers_all_rows():
    lib = A.load()
    for batch, heads in [(1, 12), (2, 12), (16, 16), (32, 20), (64, 32)]:
        rc, ctx = _fake_ctx(_cfg(batch=batch, n_heads=heads, max_rows_per_stream=2424, n_pages=1 << 20))
        assert rc == 0
        s, ch = C.c_int(0), C.c_int(0)
        for n in (0, 571, 2423):
            # persistent kernel (the default): one CTA walks the whole stream in tiles of 64 rows (head_dim 64)
            assert lib.adsa_plan_attn(ctx, n, C.byref(s), C.byref(ch)) == 0 and (s.value, ch.value) == (1, 64)
        assert lib.adsa_set_staged(ctx, 2) == 0
        for n in (0, 1, 31, 32, 33, 187, 571, 1211, 2423):
            # cluster kernel: a cluster of 1, 2, 4 or 8 CTAs per stream, each with a chunk of whole 8-row units
            assert lib.adsa_plan_attn(ctx, n, C.byref(s), C.byref(ch)) == 0
            assert s.value in (1, 2, 4, 8) and ch.value % 8 == 0 and s.value * ch.value >= n
            assert ch.value * 64 * 4 <= 200 * 1024               # K and V of a chunk fit in shared memory
        assert lib.adsa_set_attn_chunk_rows(ctx, 300) == 0         # chunk target: 571 rows -> 2 CTAs of 288 rows
        assert lib.adsa_plan_attn(ctx, 571, C.byref(s), C.byref(ch)) == 0 and (s.value, ch.value) == (2, 288)
        assert lib.adsa_set_attn_chunk_rows(ctx, 0) == 0
        assert lib.adsa_set_staged(ctx, 0) == 0                    # streaming kernel: up to 32 chunks of whole mask words
        for n in (0, 1, 33, 571, 2423):
            assert lib.adsa_plan_attn(ctx, n, C.byref(s), C.byref(ch)) == 0
            assert 1 <= s.value <= 32 and ch.value % 32 == 0 and s.value * ch.value >= n
            assert (s.value - 1) * ch.value < max(n, 1)          # no empty chunk
        lib.adsa_destroy(ctx)


def test_call_order_and_capacity_are_checked_before_any_launch():
    lib = A.load()
    rc, ctx = _fake_ctx(_cfg(n_pages=10))
    assert rc == 0
    null = C.c_void_p(None)
    ptr = C.c_void_p(0x30000000)
    # select / attend / update before score
    assert lib.adsa_select(ctx, 0, 130, 100, null, null, null, null, null) == B.ESTATE
    assert lib.adsa_sparse_decode_attn(ctx, 0, 130, ptr, ptr, ptr, ptr, null, null) == B.ESTATE
    assert lib.adsa_kv_update(ctx, 0, 130, ptr, ptr, null) == B.ESTATE
    # bad arguments
    assert lib.adsa_score(ctx, 5, 130, null, null) == B.EINVAL
    assert lib.adsa_score(ctx, 0, -1, null, null) == B.EINVAL
    assert lib.adsa_prefill_rows(ctx, 0, null, ptr, null, 4, 0, null) == B.EINVAL
    assert lib.adsa_set_stream_rows(ctx, 0, 9, 0, ptr, ptr, ptr, 4, null) == B.EINVAL
    # 120 rows x 8 streams need 8 * 8 = 64 pages of 16 rows; the pool has 10
    assert lib.adsa_prefill_rows(ctx, 0, ptr, ptr, null, 120, 0, null) == B.ENOMEM
    assert lib.adsa_prefill_rows(ctx, 0, ptr, ptr, null, 500, 0, null) == B.ENOMEM   # beyond max rows
    n = C.c_int(-1)
    assert lib.adsa_layer_rows_bound(ctx, 0, C.byref(n)) == 0 and n.value == 0
    assert lib.adsa_launch_count(ctx) == 0
    lib.adsa_destroy(ctx)


def test_every_layer_has_its_own_selection_scratch():
    """What one call of a layer-step leaves for the next (scores, keep mask, counts) is stored per layer, so
    the steps of several layers may be interleaved.  Seen from the host: each extra layer adds at least
    its scores, its carried sum, its keep mask and its counts to the workspace."""
    base = dict(batch=3, n_heads=5, max_rows_per_stream=700)
    S, R = 15, 700
    per_layer = S * (R * 4 + 256 * 4 + (R + 31) // 32 * 4 + 16)
    sizes = [A.workspace_bytes(_cfg(n_layers=n, **base)) for n in (1, 2, 5)]
    assert sizes[1] - sizes[0] >= per_layer and sizes[2] - sizes[1] >= 3 * per_layer
    # the step order is kept per layer: another layer being mid-step changes nothing for this one
    lib = A.load()
    rc, ctx = _fake_ctx(_cfg(n_pages=4000))
    assert rc == 0
    null, ptr = C.c_void_p(None), C.c_void_p(0x30000000)
    assert lib.adsa_select(ctx, 1, 130, 100, null, null, null, null, null) == B.ESTATE
    assert lib.adsa_kv_update(ctx, 1, 130, ptr, ptr, null) == B.ESTATE
    lib.adsa_destroy(ctx)


def test_page_division_by_multiplication_is_exact():
    # the kernels compute slot // page_rows as umulhi(slot, floor(2^32 / page_rows) + 1)
    for pr in list(range(2, 130)) + [255, 256, 1000, 4096]:
        magic = (1 << 32) // pr + 1
        for slot in list(range(0, 3000)) + [16383, 16384]:
            assert (slot * magic) >> 32 == slot // pr

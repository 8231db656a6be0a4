// C-ABI of libadsa: argument checking, the host-side state machine of a
// layer-step (score -> select -> attend -> update), launch planning, and the
// host-buffer variant.  Row counts are functions of positions and budgets only,
// never of data, so every launch is sized on the host without reading back.
#include <math.h>
#include <new>
#include <stdio.h>
#include <string.h>
#include <vector>

#include "adsa_dev.cuh"
#include "adsa_launch.h"

using namespace adsa;

namespace {

enum Phase { kIdle = 0, kScored = 1, kSelected = 2, kAttended = 3 };

struct LayerState {
    int phase = kIdle;
    int cur_pos = -1;
    int budget = 0;
    int rows_hi = 0;   // upper bound of n_live over the layer's streams
    int scores_pos = -1;  // the carried scores (DevCtx::scores) are Eq. 2 for a step at this position; -1 = stale
    int svec_pos = -1;    // the carried sum of normalised rows (DevCtx::svec) belongs to that position too; -1 = none
    bool launched = false;            // some kernel of this layer has been launched since the reset
    cudaStream_t last_stream = nullptr;   // ... the latest of them on this stream
};

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

struct WorkspaceLayout {
    size_t scores, keep_mask, counts, partials, tickets, svec, carry, cand_mask, wscratch, logit, ml, status, in_flags, staging, total;
};

int mask_words_of(const adsa_config &cfg) { return (cfg.max_rows_per_stream + 31) / 32; }

WorkspaceLayout layout_of(const adsa_config &cfg)
{
    const size_t S = (size_t)cfg.batch * cfg.n_heads, R = (size_t)cfg.max_rows_per_stream;
    WorkspaceLayout w;
    size_t off = 0;
    w.scores = off;      off = align_up(off + S * (size_t)cfg.n_layers * R * sizeof(float), 256);
    w.keep_mask = off;   off = align_up(off + S * (size_t)cfg.n_layers * mask_words_of(cfg) * sizeof(uint32_t), 256);
    w.counts = off;      off = align_up(off + S * (size_t)cfg.n_layers * 4 * sizeof(int32_t), 256);
    w.partials = off;    off = align_up(off + S * kMaxSplits * (size_t)(cfg.row_stride + 2) * sizeof(float), 256);
    w.tickets = off;     off = align_up(off + S * sizeof(int32_t), 256);
    w.svec = off;        off = align_up(off + S * (size_t)cfg.n_layers * 256 * sizeof(float), 256);
    w.carry = off;       off = align_up(off + S * (size_t)cfg.n_layers * 4 * sizeof(int32_t), 256);
    w.cand_mask = off;   off = align_up(off + S * (size_t)cfg.n_layers * mask_words_of(cfg) * sizeof(uint32_t), 256);
    w.wscratch = off;    off = align_up(off + (size_t)kScratchCtas * kScratchGroups * (2 * R + 4) * sizeof(unsigned long long), 256);
    w.logit = off;       off = align_up(off + (cfg.score_mode == 1 ? S * (size_t)cfg.n_layers * R * sizeof(float) : 0), 256);
    w.ml = off;          off = align_up(off + (cfg.score_mode == 1 ? S * (size_t)cfg.n_layers * 4 * sizeof(float) : 0), 256);
    w.status = off;      off = align_up(off + 4 * sizeof(uint32_t), 256);
    w.in_flags = off;    off = align_up(off + (size_t)cfg.n_layers * sizeof(int32_t), 256);
    w.staging = off;     off = align_up(off + 4 * S * (size_t)cfg.n_layers * cfg.head_dim * sizeof(__nv_bfloat16), 256);
    w.total = off;
    return w;
}

int check_config(const adsa_config *c)
{
    if (!c) return ADSA_EINVAL;
    if (c->n_layers < 1 || c->batch < 1 || c->n_heads < 1) return ADSA_EINVAL;
    if (c->head_dim < 8 || c->head_dim > 256) return ADSA_EINVAL;
    if (c->row_stride < c->head_dim || c->row_stride % 8 != 0 || c->row_stride > 256) return ADSA_EINVAL;
    if (c->page_rows < 2 || c->page_rows > 4096) return ADSA_EINVAL;
    if (c->n_pages < 1) return ADSA_EINVAL;
    if (c->max_rows_per_stream < 1 || c->max_rows_per_stream > 16384) return ADSA_EINVAL;
    if (c->n_text < 0 || c->grid_h < 1 || c->grid_w < 1) return ADSA_EINVAL;
    if (c->n_prefix < 0 || c->local_rows_back < 0) return ADSA_EINVAL;
    if (c->score_mode != 0 && c->score_mode != 1) return ADSA_EINVAL;
    if (c->score_share != 0 && (c->score_share != 1 || c->score_mode != 0 || c->n_heads > 256)) return ADSA_EINVAL;
    if (!(c->softmax_scale >= 0.f) || isinf(c->softmax_scale)) return ADSA_EINVAL;
    if ((long long)c->n_layers * c->batch * c->n_heads > (1ll << 24)) return ADSA_EINVAL;
    if ((long long)c->n_pages * c->page_rows * c->row_stride > (1ll << 40)) return ADSA_EINVAL;
    return ADSA_OK;
}

// slot / page_rows == umulhi(slot, magic) for every slot the pool can hold
bool magic_divides(uint32_t magic, int page_rows, int max_rows)
{
    for (int s = 0; s <= max_rows; ++s)
        if ((uint32_t)(((uint64_t)s * magic) >> 32) != (uint32_t)(s / page_rows)) return false;
    return true;
}

}  // namespace

struct adsa_ctx {
    adsa_config cfg;
    adsa_buffers buf;
    DevCtx dev;
    WorkspaceLayout ws;
    std::vector<LayerState> layers;
    int sm_count = 148;
    int chunk_override = 0;
    int kernel_mode = 1;   // adsa_set_staged: 0 streaming, 1 automatic, 2 cluster, 3 persistent (CUDA cores), 4 warp-per-stream (MMA)
    int mma_ok = 0;        // tensor maps of the pools exist: the MMA kernel may run
    WStepMaps maps;
    int max_stages = 0;    // cap on the persistent kernel's ring (0 = as many as fit)
    int stream_warps = 0;  // warps per stream of the warp-group kernel (0 = automatic)
    int l2_ahead = -1;     // tiles per warp the tensor-core kernel asks into L2 ahead of its ring (-1 = automatic)
    int next_tiles = 0;    // tiles per warp of the stream served next (the next layer's, in one-layer launches) a launch asks
                           // into L2 when its own sweep is over
    int host_chunks = 0;   // adsa_token_step_host: chunks of layers (0 = default)
    int token_launch = 1;  // adsa_token_step: 1 = one launch of the tensor-core kernel serves every layer, 0 = one launch per layer
    int sweep_mode = 2;    // adsa_set_single_sweep: 0 the fused tensor-core kernel always makes its second sweep, 1 it scores
                           // during the attention sweep when it can, 2 it also takes the evicted row from the previous step's note
    // What the kernel launched last through this context may still be writing when the next one starts its
    // set-up (launches overlap by programmatic dependent launch): the layer it served (-1 = several or
    // unknown) and whether it writes the cache proper (rows, pages, positions, norms) / the carried scores.
    int prev_layer = -1, prev_writes_cache = 1, prev_writes_scores = 1;
    cudaStream_t prev_stream = nullptr;   // the stream that launch went to: only a launch on the same stream is its successor
    int cuda_error = 0;  // sticky
    int64_t launches = 0;
    __nv_bfloat16 *stage_q, *stage_k, *stage_v, *stage_o;
    // adsa_token_step_host moves its tensors in chunks of layers on two copy streams of its own, so that the
    // copies of later layers travel while earlier layers compute (created on first use, host-side objects only)
    cudaStream_t copy_in = nullptr, copy_out = nullptr;
    int *in_flags = nullptr;      // [n_layers] device words: adsa_token_step_host's inputs of a layer have landed
    int *epoch_src = nullptr;     // [n_layers] pinned host words holding the current call's number, the source of those words
    int host_epoch = 0;
    cudaEvent_t ev_start = nullptr;
    std::vector<cudaEvent_t> ev_in, ev_done;
};

namespace {

int cuda_fail(adsa_ctx *ctx, cudaError_t e)
{
    if (e == cudaSuccess) return ADSA_OK;
    ctx->cuda_error = (int)e;
    return ADSA_ECUDA;
}

int pages_for(const adsa_ctx *ctx, int rows) { return (rows + ctx->cfg.page_rows - 1) / ctx->cfg.page_rows; }

// pages the whole pool may need if `layer` grows to `rows` rows per stream
bool pool_can_hold(const adsa_ctx *ctx, int layer, int rows)
{
    long long need = 0;
    for (int l = 0; l < ctx->cfg.n_layers; ++l)
        need += (long long)ctx->dev.S * pages_for(ctx, l == layer ? rows : ctx->layers[l].rows_hi);
    return need <= ctx->cfg.n_pages;
}

// largest number of rows the prefix and local regions can hold at cur_pos
int mandatory_rows_bound(const adsa_ctx *ctx, int cur_pos)
{
    const adsa_config &c = ctx->cfg;
    int pre = c.n_prefix < cur_pos ? c.n_prefix : cur_pos;
    int loc = 0;
    if (cur_pos >= c.n_text) {
        int g = cur_pos - c.n_text, r = g / c.grid_w, col = g % c.grid_w;
        int back = r < c.local_rows_back ? r : c.local_rows_back;
        loc = back * c.grid_w + col;
    }
    return pre + loc;
}

AttnPlan plan_attn(const adsa_ctx *ctx, int n_rows)
{
    AttnPlan p;
    int rows = n_rows < 1 ? 1 : n_rows;
    int chunk = ctx->chunk_override;
    if (chunk <= 0) {
        // enough blocks to fill every SM several times over, but no chunk below 64 rows
        long long target_blocks = (long long)ctx->sm_count * 8;
        int splits = (int)((target_blocks + ctx->dev.S - 1) / ctx->dev.S);
        if (splits < 1) splits = 1;
        chunk = (rows + splits - 1) / splits;
        if (chunk < 64) chunk = 64;
    }
    chunk = (chunk + 31) / 32 * 32;
    int splits = (rows + chunk - 1) / chunk;
    if (splits > kMaxSplits) {
        splits = kMaxSplits;
        chunk = ((rows + splits - 1) / splits + 31) / 32 * 32;
        splits = (rows + chunk - 1) / chunk;
    }
    p.n_splits = splits;
    p.chunk_rows = chunk;
    return p;
}

// Which of the staged kernels serves this context, in order of preference: the warp-per-stream MMA
// kernel, the persistent CUDA-core kernel, the cluster kernel; none of them = the streaming kernels.
struct StagedChoice {
    WStepPlan wp;
    PStepPlan pp;
    StepPlan sp;
    bool any() const { return wp.n_groups || pp.n_stages || sp.cluster_size; }
};

StagedChoice choose_staged(const adsa_ctx *ctx, int n_rows, bool fused)
{
    StagedChoice ch = {};
    const int m = ctx->kernel_mode;
    if (m == 0) return ch;
    if (ctx->cfg.score_mode != 0 || ctx->cfg.score_share != 0) return ch;   // the comparison method and the per-layer granularity run on the four stand-alone kernels
    if ((m == 1 || m == 4) && ctx->mma_ok) {
        ch.wp = plan_wstep(ctx->dev, fused, ctx->sm_count, ctx->max_stages, ctx->stream_warps);
        if (ctx->l2_ahead >= 0) ch.wp.l2_ahead = ctx->l2_ahead;
        if (ch.wp.n_groups) return ch;
    }
    if (m == 1 || m == 3) {
        ch.pp = plan_pstep(ctx->dev, fused, ctx->sm_count, ctx->max_stages);
        if (ch.pp.n_stages) return ch;
    }
    if (m == 1 || m == 2) ch.sp = plan_step(ctx->dev, n_rows, fused, ctx->sm_count, ctx->chunk_override);
    return ch;
}

void note_launch(adsa_ctx *ctx, int layer, bool writes_cache, bool writes_scores, adsa_stream_t stream)
{
    ctx->prev_stream = (cudaStream_t)stream;
    if (layer >= 0) { ctx->layers[layer].launched = true; ctx->layers[layer].last_stream = (cudaStream_t)stream; }
    ctx->prev_layer = layer;
    ctx->prev_writes_cache = writes_cache ? 1 : 0;
    ctx->prev_writes_scores = writes_scores ? 1 : 0;
}

// May the kernel about to be launched on `stream` read `layer`'s cache state (and, for the fused step, its
// carried scores) before the kernel ahead of it in that stream has completed?  Only when that kernel is the
// context's previous launch (same stream), so that what it writes is known.
bool state_is_quiet(const adsa_ctx *ctx, int layer, bool needs_scores, cudaStream_t stream)
{
    if (ctx->prev_layer < 0 || ctx->prev_stream != stream) return false;
    // the layer's own earlier kernels are known to be complete only if they went to this stream too: every
    // kernel of the library lets its successor in the stream start only after its own dependency wait
    const LayerState &L = ctx->layers[layer];
    if (L.launched && L.last_stream != stream) return false;
    if (ctx->prev_layer != layer) return true;
    return !ctx->prev_writes_cache && !(needs_scores && ctx->prev_writes_scores);
}

cudaError_t launch_staged(const adsa_ctx *ctx, const StagedChoice &ch, bool fused, int layer, int cur_pos,
                          int budget_rows, const void *q, const void *k_new, const void *v_new, void *out_bf16,
                          float *out_f32, cudaStream_t st, bool have_svec = false)
{
    if (ch.wp.n_groups)
        return launch_wstep(ctx->dev, ch.wp, ctx->maps, fused, layer, cur_pos, budget_rows, q, k_new, v_new, out_bf16, out_f32, st,
                            have_svec && ctx->sweep_mode >= 1, state_is_quiet(ctx, layer, fused, st), ctx->sweep_mode >= 2,
                            ctx->next_tiles > 0 ? (layer + 1) % ctx->cfg.n_layers : -1, ctx->next_tiles);
    if (ch.pp.n_stages)
        return launch_pstep(ctx->dev, ch.pp, fused, layer, cur_pos, budget_rows, q, k_new, v_new, out_bf16, out_f32, st);
    return launch_step(ctx->dev, ch.sp, fused, layer, cur_pos, budget_rows, q, k_new, v_new, out_bf16, out_f32, st);
}

int check_layer(const adsa_ctx *ctx, int layer)
{
    if (!ctx) return ADSA_EINVAL;
    if (ctx->cuda_error) return ADSA_ECUDA;
    if (layer < 0 || layer >= ctx->cfg.n_layers) return ADSA_EINVAL;
    return ADSA_OK;
}

}  // namespace

extern "C" {

int adsa_workspace_bytes(const adsa_config *cfg, size_t *out_bytes)
{
    int rc = check_config(cfg);
    if (rc != ADSA_OK || !out_bytes) return ADSA_EINVAL;
    *out_bytes = layout_of(*cfg).total;
    return ADSA_OK;
}

int adsa_create(const adsa_config *cfg, const adsa_buffers *buf, adsa_ctx **out)
{
    int rc = check_config(cfg);
    if (rc != ADSA_OK || !buf || !out) return ADSA_EINVAL;
    if (!buf->k_pool || !buf->v_pool || !buf->page_table || !buf->pos || !buf->inv_norm || !buf->n_live ||
        !buf->free_ring || !buf->free_state || !buf->workspace)
        return ADSA_EINVAL;
    if (((uintptr_t)buf->k_pool | (uintptr_t)buf->v_pool) & 15u) return ADSA_EINVAL;
    if ((uintptr_t)buf->workspace & 255u) return ADSA_EINVAL;
    WorkspaceLayout ws = layout_of(*cfg);
    if (buf->workspace_bytes < ws.total) return ADSA_ENOMEM;
    if ((size_t)cfg->max_rows_per_stream * 9 + 16 > 200 * 1024) return ADSA_EINVAL;

    uint32_t magic = (uint32_t)((1ull << 32) / (uint32_t)cfg->page_rows) + 1u;
    if (!magic_divides(magic, cfg->page_rows, cfg->max_rows_per_stream)) return ADSA_EINVAL;

    adsa_ctx *ctx = new (std::nothrow) adsa_ctx();
    if (!ctx) return ADSA_ENOMEM;
    ctx->cfg = *cfg;
    ctx->buf = *buf;
    ctx->ws = ws;
    ctx->layers.resize(cfg->n_layers);
    char *w = (char *)buf->workspace;
    DevCtx &d = ctx->dev;
    d.k_pool = (__nv_bfloat16 *)buf->k_pool;
    d.v_pool = (__nv_bfloat16 *)buf->v_pool;
    d.page_table = buf->page_table;
    d.pos = buf->pos;
    d.n_live = buf->n_live;
    d.inv_norm = buf->inv_norm;
    d.free_ring = buf->free_ring;
    d.free_state = buf->free_state;
    d.scores = (float *)(w + ws.scores);
    d.keep_mask = (uint32_t *)(w + ws.keep_mask);
    d.counts = (int32_t *)(w + ws.counts);
    d.partials = (float *)(w + ws.partials);
    d.tickets = (int32_t *)(w + ws.tickets);
    d.svec = (float *)(w + ws.svec);
    d.carry = (int32_t *)(w + ws.carry);
    d.cand_mask = (uint32_t *)(w + ws.cand_mask);
    d.wscratch = (unsigned long long *)(w + ws.wscratch);
    d.logit = (float *)(w + ws.logit);
    d.ml = (float *)(w + ws.ml);
    d.score_mode = cfg->score_mode;
    d.score_share = cfg->score_share;
    d.n_heads = cfg->n_heads;
    d.status = (uint32_t *)(w + ws.status);
    d.d = cfg->head_dim;
    d.row_stride = cfg->row_stride;
    d.page_rows = cfg->page_rows;
    d.n_pages = cfg->n_pages;
    d.max_rows = cfg->max_rows_per_stream;
    d.max_pages = (cfg->max_rows_per_stream + cfg->page_rows - 1) / cfg->page_rows;
    d.mask_words = mask_words_of(*cfg);
    d.S = cfg->batch * cfg->n_heads;
    d.partial_stride = cfg->row_stride + 2;
    d.pr_magic = magic;
    d.n_text = cfg->n_text;
    d.grid_w = cfg->grid_w;
    d.n_prefix = cfg->n_prefix;
    d.rows_back = cfg->local_rows_back;
    float scale = cfg->softmax_scale > 0.f ? cfg->softmax_scale : 1.0f / sqrtf((float)cfg->head_dim);
    d.scale_log2e = scale * 1.4426950408889634f;
    size_t stage = (size_t)d.S * cfg->n_layers * cfg->head_dim;
    ctx->stage_q = (__nv_bfloat16 *)(w + ws.staging);
    ctx->in_flags = (int *)(w + ws.in_flags);
    ctx->stage_k = ctx->stage_q + stage;
    ctx->stage_v = ctx->stage_k + stage;
    ctx->stage_o = ctx->stage_v + stage;

    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) == cudaSuccess &&
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && sms > 0) {
        ctx->sm_count = sms;
        cudaError_t e = configure_kernels(d);
        if (e != cudaSuccess) { delete ctx; return ADSA_ECUDA; }
        if (wstep_supported(d) && build_wstep_maps(d, &ctx->maps) == 0) {
            if (configure_wstep_kernel(d) != cudaSuccess) { delete ctx; return ADSA_ECUDA; }
            ctx->mma_ok = 1;
        }
    } else {
        cudaGetLastError();  // no usable device: host-side planning still works, launches will fail
    }
    *out = ctx;
    return ADSA_OK;
}

int adsa_destroy(adsa_ctx *ctx)
{
    if (ctx) {
        for (cudaEvent_t e : ctx->ev_in) cudaEventDestroy(e);
        for (cudaEvent_t e : ctx->ev_done) cudaEventDestroy(e);
        if (ctx->ev_start) cudaEventDestroy(ctx->ev_start);
        if (ctx->copy_in) cudaStreamDestroy(ctx->copy_in);
        if (ctx->epoch_src) cudaFreeHost(ctx->epoch_src);
        if (ctx->copy_out) cudaStreamDestroy(ctx->copy_out);
    }
    delete ctx;
    return ADSA_OK;
}

int adsa_reset(adsa_ctx *ctx, adsa_stream_t stream)
{
    if (!ctx) return ADSA_EINVAL;
    if (ctx->cuda_error) return ADSA_ECUDA;
    for (auto &l : ctx->layers) {
        l = LayerState();
        l.launched = true;   // the reset kernel writes every layer's state
        l.last_stream = (cudaStream_t)stream;
    }
    note_launch(ctx, -1, true, true, stream);
    ++ctx->launches;
    return cuda_fail(ctx, launch_reset(ctx->dev, ctx->cfg.n_layers * ctx->dev.S, (cudaStream_t)stream));
}

int adsa_prefill_rows(adsa_ctx *ctx, int layer, const void *k, const void *v, const int32_t *pos, int n_rows,
                      int first_pos, adsa_stream_t stream)
{
    int rc = check_layer(ctx, layer);
    if (rc) return rc;
    if (!k || !v || n_rows < 1 || first_pos < 0) return ADSA_EINVAL;
    LayerState &L = ctx->layers[layer];
    if (L.phase != kIdle) return ADSA_ESTATE;
    if (L.rows_hi + n_rows > ctx->cfg.max_rows_per_stream) return ADSA_ENOMEM;
    if (!pool_can_hold(ctx, layer, L.rows_hi + n_rows)) return ADSA_ENOMEM;
    L.rows_hi += n_rows;
    L.scores_pos = -1;
    L.svec_pos = -1;
    note_launch(ctx, layer, true, true, stream);
    ++ctx->launches;
    return cuda_fail(ctx, launch_append_rows(ctx->dev, layer, k, v, pos, n_rows, first_pos, (cudaStream_t)stream));
}

int adsa_prefill_attn(adsa_ctx *ctx, int layer, const void *q, const void *k, const void *v, int n_rows, int first_pos,
                      void *out_bf16, float *out_f32, adsa_stream_t stream)
{
    int rc = check_layer(ctx, layer);
    if (rc) return rc;
    if (!q || !k || !v || (!out_bf16 && !out_f32) || n_rows < 1 || first_pos < 0) return ADSA_EINVAL;
    if (((uintptr_t)q | (uintptr_t)k | (uintptr_t)v) & 3u) return ADSA_EINVAL;
    LayerState &L = ctx->layers[layer];
    if (L.phase != kIdle || L.rows_hi != 0) return ADSA_ESTATE;   // the rows attend each other only: the cache must be empty
    rc = adsa_prefill_rows(ctx, layer, k, v, nullptr, n_rows, first_pos, stream);
    if (rc) return rc;
    ++ctx->launches;
    return cuda_fail(ctx, launch_prefill_attn(ctx->dev, q, k, v, out_bf16, out_f32, n_rows, (cudaStream_t)stream));
}

int adsa_rope_2d(adsa_ctx *ctx, void *x, const int32_t *pos, long long n_rows, float base, adsa_stream_t stream)
{
    if (!ctx || !x || !pos || n_rows < 0 || !(base >= 0.f) || ((uintptr_t)x & 3u)) return ADSA_EINVAL;
    if (ctx->cuda_error) return ADSA_ECUDA;
    if (ctx->cfg.head_dim % 4 != 0) return ADSA_EINVAL;
    if (n_rows == 0) return ADSA_OK;
    ++ctx->launches;
    return cuda_fail(ctx, launch_rope_2d(ctx->dev, x, pos, n_rows, base > 0.f ? base : 10000.f, (cudaStream_t)stream));
}

int adsa_set_stream_rows(adsa_ctx *ctx, int layer, int b, int h, const void *k, const void *v, const int32_t *pos,
                         int n_rows, adsa_stream_t stream)
{
    int rc = check_layer(ctx, layer);
    if (rc) return rc;
    if (b < 0 || b >= ctx->cfg.batch || h < 0 || h >= ctx->cfg.n_heads || n_rows < 0) return ADSA_EINVAL;
    if (n_rows > 0 && (!k || !v || !pos)) return ADSA_EINVAL;
    LayerState &L = ctx->layers[layer];
    if (L.phase != kIdle) return ADSA_ESTATE;
    if (n_rows > ctx->cfg.max_rows_per_stream) return ADSA_ENOMEM;
    int hi = n_rows > L.rows_hi ? n_rows : L.rows_hi;
    if (!pool_can_hold(ctx, layer, hi)) return ADSA_ENOMEM;
    L.rows_hi = hi;
    L.scores_pos = -1;
    L.svec_pos = -1;
    int sid = (layer * ctx->cfg.batch + b) * ctx->cfg.n_heads + h;
    note_launch(ctx, layer, true, true, stream);
    ++ctx->launches;
    return cuda_fail(ctx, launch_set_rows(ctx->dev, sid, k, v, pos, n_rows, (cudaStream_t)stream));
}

int adsa_score(adsa_ctx *ctx, int layer, int cur_pos, float *scores_out, adsa_stream_t stream)
{
    int rc = check_layer(ctx, layer);
    if (rc) return rc;
    if (cur_pos < 0) return ADSA_EINVAL;
    LayerState &L = ctx->layers[layer];
    if (L.phase != kIdle) return ADSA_ESTATE;
    L.phase = kScored;
    L.cur_pos = cur_pos;
    if (ctx->cfg.score_mode == 1) {   // the masses are carried with the rows: nothing to compute
        if (!scores_out) return ADSA_OK;
        note_launch(ctx, layer, false, false, stream);
        ++ctx->launches;
        return cuda_fail(ctx, launch_scores_copy(ctx->dev, layer, cur_pos, scores_out, (cudaStream_t)stream));
    }
    if (L.scores_pos == cur_pos) {   // carried in from the previous fused step: nothing to compute
        if (!scores_out) return ADSA_OK;
        note_launch(ctx, layer, false, false, stream);
        ++ctx->launches;
        return cuda_fail(ctx, launch_scores_copy(ctx->dev, layer, cur_pos, scores_out, (cudaStream_t)stream));
    }
    L.scores_pos = cur_pos;
    L.svec_pos = -1;   // the stand-alone score kernel does not leave the sum behind
    note_launch(ctx, layer, false, true, stream);
    ++ctx->launches;
    return cuda_fail(ctx, launch_score(ctx->dev, layer, cur_pos, scores_out, (cudaStream_t)stream));
}

int adsa_select(adsa_ctx *ctx, int layer, int cur_pos, int budget_rows, int32_t *sel_slots, int32_t *sel_pos,
                int32_t *evict_pos, int32_t *counts, adsa_stream_t stream)
{
    int rc = check_layer(ctx, layer);
    if (rc) return rc;
    if (budget_rows < 1) return ADSA_EINVAL;
    LayerState &L = ctx->layers[layer];
    if (L.phase != kScored || L.cur_pos != cur_pos) return ADSA_ESTATE;
    // rows after the update: min(rows + 1, budget), but never below prefix + local + 1
    int mand = mandatory_rows_bound(ctx, cur_pos) + 1;
    int cap = budget_rows > mand ? budget_rows : mand;
    int after = L.rows_hi + 1 < cap ? L.rows_hi + 1 : cap;
    if (after > ctx->cfg.max_rows_per_stream) return ADSA_ENOMEM;
    if (!pool_can_hold(ctx, layer, after > L.rows_hi ? after : L.rows_hi)) return ADSA_ENOMEM;
    L.phase = kSelected;
    L.budget = budget_rows;
    note_launch(ctx, layer, false, false, stream);
    ++ctx->launches;
    return cuda_fail(ctx, launch_select(ctx->dev, layer, cur_pos, budget_rows, sel_slots, sel_pos, evict_pos, counts,
                                        (cudaStream_t)stream));
}

int adsa_sparse_decode_attn(adsa_ctx *ctx, int layer, int cur_pos, const void *q, const void *k_new,
                            const void *v_new, void *out_bf16, float *out_f32, adsa_stream_t stream)
{
    int rc = check_layer(ctx, layer);
    if (rc) return rc;
    if (!q || !k_new || !v_new || (!out_bf16 && !out_f32)) return ADSA_EINVAL;
    LayerState &L = ctx->layers[layer];
    if ((L.phase != kSelected && L.phase != kAttended) || L.cur_pos != cur_pos) return ADSA_ESTATE;
    L.phase = kAttended;
    ++ctx->launches;
    StagedChoice ch = choose_staged(ctx, L.rows_hi, false);
    cudaError_t e;
    if (ch.any()) {
        e = launch_staged(ctx, ch, false, layer, cur_pos, 0, q, k_new, v_new, out_bf16, out_f32, (cudaStream_t)stream);
    } else {
        AttnPlan plan = plan_attn(ctx, L.rows_hi);
        e = launch_attn(ctx->dev, plan, layer, cur_pos, q, k_new, v_new, out_bf16, out_f32, (cudaStream_t)stream);
    }
    note_launch(ctx, layer, false, false, stream);   // attention reads the cache and writes the output only
    return cuda_fail(ctx, e);
}

int adsa_kv_update(adsa_ctx *ctx, int layer, int cur_pos, const void *k_new, const void *v_new, adsa_stream_t stream)
{
    int rc = check_layer(ctx, layer);
    if (rc) return rc;
    if (!k_new || !v_new) return ADSA_EINVAL;
    LayerState &L = ctx->layers[layer];
    if ((L.phase != kSelected && L.phase != kAttended) || L.cur_pos != cur_pos) return ADSA_ESTATE;
    if (ctx->cfg.score_mode == 1 && L.phase != kAttended) return ADSA_ESTATE;   // the masses grow by this step's attention weights
    int mand = mandatory_rows_bound(ctx, cur_pos) + 1;
    int cap = L.budget > mand ? L.budget : mand;
    L.rows_hi = L.rows_hi + 1 < cap ? L.rows_hi + 1 : cap;
    L.phase = kIdle;
    L.scores_pos = -1;   // rows move and the scores of the next step were not computed
    L.svec_pos = -1;
    note_launch(ctx, layer, true, false, stream);
    ++ctx->launches;
    return cuda_fail(ctx, launch_kv_update(ctx->dev, layer, cur_pos, k_new, v_new, (cudaStream_t)stream));
}

int adsa_layer_step(adsa_ctx *ctx, int layer, int cur_pos, int budget_rows, const void *q, const void *k_new,
                    const void *v_new, void *out_bf16, adsa_stream_t stream)
{
    int rc = check_layer(ctx, layer);
    if (rc) return rc;
    if (!q || !k_new || !v_new || !out_bf16 || cur_pos < 0 || budget_rows < 1) return ADSA_EINVAL;
    LayerState &L = ctx->layers[layer];
    if (L.phase != kIdle && !(L.phase == kScored && L.cur_pos == cur_pos)) return ADSA_ESTATE;
    StagedChoice ch = choose_staged(ctx, L.rows_hi, true);
    if (!ch.any()) {   // no staged kernel fits this configuration: four kernels
        if (L.phase == kIdle) {
            rc = adsa_score(ctx, layer, cur_pos, nullptr, stream);
            if (rc) return rc;
        }
        rc = adsa_select(ctx, layer, cur_pos, budget_rows, nullptr, nullptr, nullptr, nullptr, stream);
        if (rc) return rc;
        rc = adsa_sparse_decode_attn(ctx, layer, cur_pos, q, k_new, v_new, out_bf16, nullptr, stream);
        if (rc) return rc;
        return adsa_kv_update(ctx, layer, cur_pos, k_new, v_new, stream);
    }
    // capacity checks of adsa_select, before anything is launched
    int mand = mandatory_rows_bound(ctx, cur_pos) + 1;
    int cap = budget_rows > mand ? budget_rows : mand;
    int after = L.rows_hi + 1 < cap ? L.rows_hi + 1 : cap;
    if (after > ctx->cfg.max_rows_per_stream) return ADSA_ENOMEM;
    if (!pool_can_hold(ctx, layer, after > L.rows_hi ? after : L.rows_hi)) return ADSA_ENOMEM;
    if (L.phase == kIdle && L.scores_pos != cur_pos) {   // no scores carried in (first step, or the cache was rewritten)
        ++ctx->launches;
        L.svec_pos = -1;
        note_launch(ctx, layer, false, true, stream);
        rc = cuda_fail(ctx, launch_score(ctx->dev, layer, cur_pos, nullptr, (cudaStream_t)stream));
        if (rc) return rc;
    }
    const bool have_svec = L.svec_pos == cur_pos;
    ++ctx->launches;
    rc = cuda_fail(ctx, launch_staged(ctx, ch, true, layer, cur_pos, budget_rows, q, k_new, v_new, out_bf16, nullptr,
                                      (cudaStream_t)stream, have_svec));
    note_launch(ctx, layer, true, true, stream);
    L.rows_hi = after;
    L.phase = kIdle;
    L.cur_pos = cur_pos;
    L.scores_pos = cur_pos + 1;   // the fused kernel left the scores of the next position behind
    L.svec_pos = ch.wp.n_groups ? cur_pos + 1 : -1;   // ... and the tensor-core kernel the sum they were made from
    return rc;
}

int adsa_layer_step_host(adsa_ctx *ctx, int layer, int cur_pos, int budget_rows, const void *q_host,
                         const void *k_new_host, const void *v_new_host, void *out_host, adsa_stream_t stream)
{
    int rc = check_layer(ctx, layer);
    if (rc) return rc;
    if (!q_host || !k_new_host || !v_new_host || !out_host) return ADSA_EINVAL;
    cudaStream_t st = (cudaStream_t)stream;
    size_t bytes = (size_t)ctx->dev.S * ctx->cfg.head_dim * sizeof(__nv_bfloat16);
    cudaError_t e = cudaMemcpyAsync(ctx->stage_q, q_host, bytes, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(ctx->stage_k, k_new_host, bytes, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(ctx->stage_v, v_new_host, bytes, cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    rc = adsa_layer_step(ctx, layer, cur_pos, budget_rows, ctx->stage_q, ctx->stage_k, ctx->stage_v, ctx->stage_o, stream);
    if (rc) return rc;
    e = cudaMemcpyAsync(out_host, ctx->stage_o, bytes, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    return cuda_fail(ctx, e);
}

// One step of layers l0 .. l0 + NL - 1 (q, k_new, v_new, out_bf16 point at layer l0's tensors).
// One launch for layers l0 .. l0 + NL - 1: the tensor-core kernel serves the configuration, every layer is between
// steps and all are in the same carried state.
static bool one_launch_possible(const adsa_ctx *ctx, int l0, int NL, int cur_pos, WStepPlan *plan)
{
    bool ok = ctx->token_launch == 1 && NL > 1 && (ctx->kernel_mode == 1 || ctx->kernel_mode == 4) && ctx->mma_ok &&
              ctx->cfg.score_mode == 0 && ctx->cfg.score_share == 0;
    const LayerState &L0 = ctx->layers[l0];
    for (int l = 0; l < NL && ok; ++l) {
        const LayerState &L = ctx->layers[l0 + l];
        ok = L.phase == kIdle && (L.scores_pos == cur_pos) == (L0.scores_pos == cur_pos) && (L.svec_pos == cur_pos) == (L0.svec_pos == cur_pos);
    }
    if (!ok) return false;
    WStepPlan wp = plan_wstep(ctx->dev, true, ctx->sm_count, ctx->max_stages, ctx->stream_warps, NL);
    if (ctx->l2_ahead >= 0) wp.l2_ahead = ctx->l2_ahead;
    if (plan) *plan = wp;
    return wp.n_groups > 0;
}

// in_ready (optional, one launch only): per-layer words that say when a layer's inputs have landed (WStepArgs::in_ready)
static int step_layers(adsa_ctx *ctx, int l0, int NL, int cur_pos, int budget_rows, const void *q, const void *k_new,
                       const void *v_new, void *out_bf16, adsa_stream_t stream, const int *in_ready = nullptr, int in_epoch = 0)
{
    size_t per_layer = (size_t)ctx->dev.S * ctx->cfg.head_dim;
    const __nv_bfloat16 *qb = (const __nv_bfloat16 *)q, *kb = (const __nv_bfloat16 *)k_new,
                        *vb = (const __nv_bfloat16 *)v_new;
    __nv_bfloat16 *ob = (__nv_bfloat16 *)out_bf16;

    // One launch for the whole stack: the caller hands over every layer's q, k_new and v_new at once, so no
    // layer has to wait for another, and the tensor-core kernel walks the streams of all layers as one list.
    // The warps of a multiprocessor then sit in different phases of different streams (locating rows,
    // sweeping, updating) instead of all starting and all draining together once per layer.  Taken when
    // every layer is between steps and in the same carried state; otherwise layer by layer.
    WStepPlan wp = {};
    const bool one_launch = one_launch_possible(ctx, l0, NL, cur_pos, &wp);
    if (!one_launch) {
        if (in_ready) return ADSA_ESTATE;   // (the caller has checked: not reached)
        for (int l = 0; l < NL; ++l) {
            int rc = adsa_layer_step(ctx, l0 + l, cur_pos, budget_rows, qb + l * per_layer, kb + l * per_layer,
                                     vb + l * per_layer, ob + l * per_layer, stream);
            if (rc) return rc;
        }
        return ADSA_OK;
    }
    // capacity checks of adsa_select for every layer, before anything is launched
    const int mand = mandatory_rows_bound(ctx, cur_pos) + 1;
    const int cap = budget_rows > mand ? budget_rows : mand;
    std::vector<int> after(NL);
    {
        long long need = 0;
        for (int l = 0; l < ctx->cfg.n_layers; ++l) {
            const int hi = ctx->layers[l].rows_hi;
            int rows = hi;
            if (l >= l0 && l < l0 + NL) {
                after[l - l0] = hi + 1 < cap ? hi + 1 : cap;
                if (after[l - l0] > ctx->cfg.max_rows_per_stream) return ADSA_ENOMEM;
                rows = after[l - l0] > hi ? after[l - l0] : hi;
            }
            need += (long long)ctx->dev.S * pages_for(ctx, rows);
        }
        if (need > ctx->cfg.n_pages) return ADSA_ENOMEM;
    }
    cudaStream_t st = (cudaStream_t)stream;
    if (ctx->layers[l0].scores_pos != cur_pos) {   // nothing carried in (first step, or the caches were rewritten)
        for (int l = l0; l < l0 + NL; ++l) {
            ++ctx->launches;
            ctx->layers[l].svec_pos = -1;
            note_launch(ctx, l, false, true, stream);
            int rc = cuda_fail(ctx, launch_score(ctx->dev, l, cur_pos, nullptr, st));
            if (rc) return rc;
        }
    }
    const bool have_svec = ctx->layers[l0].svec_pos == cur_pos;
    ++ctx->launches;
    int rc = cuda_fail(ctx, launch_wstep(ctx->dev, wp, ctx->maps, true, l0, cur_pos, budget_rows, q, k_new, v_new, out_bf16, nullptr,
                                         st, have_svec && ctx->sweep_mode >= 1, false, ctx->sweep_mode >= 2, -1, ctx->next_tiles, NL, in_ready, in_epoch));
    for (int l = 0; l < NL; ++l) {
        LayerState &L = ctx->layers[l0 + l];
        L.rows_hi = after[l];
        L.cur_pos = cur_pos;
        L.scores_pos = cur_pos + 1;
        L.svec_pos = cur_pos + 1;
        L.launched = true;
        L.last_stream = st;
    }
    note_launch(ctx, -1, true, true, stream);
    return rc;
}

int adsa_token_step(adsa_ctx *ctx, int cur_pos, int budget_rows, const void *q, const void *k_new,
                    const void *v_new, void *out_bf16, adsa_stream_t stream)
{
    if (!ctx || !q || !k_new || !v_new || !out_bf16) return ADSA_EINVAL;
    if (ctx->cuda_error) return ADSA_ECUDA;
    if (cur_pos < 0 || budget_rows < 1) return ADSA_EINVAL;
    return step_layers(ctx, 0, ctx->cfg.n_layers, cur_pos, budget_rows, q, k_new, v_new, out_bf16, stream);
}

int adsa_token_step_gated(adsa_ctx *ctx, int cur_pos, int budget_rows, const void *q, const void *k_new, const void *v_new,
                          void *out_bf16, const int32_t *ready, int32_t epoch, adsa_stream_t stream)
{
    if (!ctx || !q || !k_new || !v_new || !out_bf16 || !ready) return ADSA_EINVAL;
    if (ctx->cuda_error) return ADSA_ECUDA;
    if (cur_pos < 0 || budget_rows < 1) return ADSA_EINVAL;
    if (!one_launch_possible(ctx, 0, ctx->cfg.n_layers, cur_pos, nullptr)) return ADSA_ESTATE;
    return step_layers(ctx, 0, ctx->cfg.n_layers, cur_pos, budget_rows, q, k_new, v_new, out_bf16, stream, ready, epoch);
}

int adsa_token_step_host(adsa_ctx *ctx, int cur_pos, int budget_rows, const void *q_host, const void *k_new_host,
                         const void *v_new_host, void *out_host, adsa_stream_t stream)
{
    if (!ctx) return ADSA_EINVAL;
    if (ctx->cuda_error) return ADSA_ECUDA;
    if (!q_host || !k_new_host || !v_new_host || !out_host) return ADSA_EINVAL;
    if (cur_pos < 0 || budget_rows < 1) return ADSA_EINVAL;
    cudaStream_t st = (cudaStream_t)stream;
    const int L = ctx->cfg.n_layers;
    // Chunk boundaries.  Every chunk is one launch, and larger launches run closer to the copy rate, so chunks are few;
    // the first is one layer, so that computing starts after a short copy.  By default each chunk is about three
    // times the one before it: a layer's inputs cross PCIe in about a quarter of the time the layer computes, so a
    // chunk's copy ends while the chunk before it still runs.  adsa_set_host_chunks(n >= 2): one layer, then n - 1
    // equal chunks.
    int bound[7], n_chunks = 0;
    bound[0] = 0;
    if (L <= 6) {
        for (int l = 1; l <= L; ++l) bound[l] = l;
        n_chunks = L;
    } else if (ctx->host_chunks >= 2 && ctx->host_chunks <= 6) {
        bound[1] = 1;
        const int parts = ctx->host_chunks - 1, rest = L - 1, per = (rest + parts - 1) / parts;
        n_chunks = 1;
        for (int l = 1; l < L; l += per) { bound[n_chunks + 1] = l + per < L ? l + per : L; ++n_chunks; }
    } else {
        int size = 1, l = 0;
        while (l < L) {
            const int take = n_chunks == 5 || l + size + size / 2 >= L ? L - l : size;   // no small last chunk, six chunks at most
            l += take;
            bound[++n_chunks] = l;
            size *= 3;
        }
    }
    // An output buffer in pinned, mapped host memory is written by the kernels themselves (posted writes of whole
    // rows); any other host memory gets its chunks by copies from a staging buffer.
    __nv_bfloat16 *out_direct = nullptr;
    {
        cudaPointerAttributes attr = {};
        if (cudaPointerGetAttributes(&attr, out_host) == cudaSuccess && attr.type == cudaMemoryTypeHost && attr.devicePointer)
            out_direct = (__nv_bfloat16 *)attr.devicePointer;
        else
            cudaGetLastError();
    }
    cudaError_t e = cudaSuccess;
    if (!ctx->copy_in) {   // first use on this context
        e = cudaStreamCreateWithFlags(&ctx->copy_in, cudaStreamNonBlocking);
        if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&ctx->copy_out, cudaStreamNonBlocking);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->ev_start, cudaEventDisableTiming);
        for (int c = 0; c < 6 && e == cudaSuccess; ++c) {
            cudaEvent_t a = nullptr, b = nullptr;
            e = cudaEventCreateWithFlags(&a, cudaEventDisableTiming);
            if (e == cudaSuccess) e = cudaEventCreateWithFlags(&b, cudaEventDisableTiming);
            if (a) ctx->ev_in.push_back(a);
            if (b) ctx->ev_done.push_back(b);
        }
        if (e != cudaSuccess) return cuda_fail(ctx, e);
    }
    const size_t per_layer = (size_t)ctx->dev.S * ctx->cfg.head_dim;   // elements
    const char *qh = (const char *)q_host, *kh = (const char *)k_new_host, *vh = (const char *)v_new_host;
    char *oh = (char *)out_host;

    // ---- one launch for the whole stack, started before its inputs are there ---------------------------------
    // When the tensor-core kernel can take every layer in one launch and the inputs sit in pinned host memory, the
    // launch is queued at once and the copies run beside it on the inbound stream, in small chunks of layers, each
    // followed by a copy that writes this call's number into the chunk's per-layer words; the kernel waits for a
    // layer's word (for a bounded time) before it reads that layer's q, k_new and v_new.  The copies are queued on
    // their own stream and wait for nothing the kernel does, so they always proceed.
    auto pinned = [](const void *p) {
        cudaPointerAttributes attr = {};
        if (cudaPointerGetAttributes(&attr, p) == cudaSuccess && attr.type == cudaMemoryTypeHost) return true;
        cudaGetLastError();
        return false;
    };
    if (ctx->host_chunks == 0 && L > 1 && pinned(q_host) && pinned(k_new_host) && pinned(v_new_host) &&
        one_launch_possible(ctx, 0, L, cur_pos, nullptr)) {
        if (!ctx->epoch_src) {
            e = cudaHostAlloc((void **)&ctx->epoch_src, (size_t)L * sizeof(int), cudaHostAllocDefault);
            if (e == cudaSuccess) e = cudaMemsetAsync(ctx->in_flags, 0, (size_t)L * sizeof(int), ctx->copy_in);
            if (e == cudaSuccess) e = cudaStreamSynchronize(ctx->copy_in);
            if (e != cudaSuccess) { ctx->epoch_src = nullptr; return cuda_fail(ctx, e); }
            ctx->host_epoch = 0;
        }
        const int epoch = ++ctx->host_epoch;   // (the previous call has drained its streams: the source words are free)
        for (int l = 0; l < L; ++l) ctx->epoch_src[l] = epoch;
        auto copy_layers = [&](int l0, int l1) -> cudaError_t {
            const size_t off = (size_t)l0 * per_layer, bytes = (size_t)(l1 - l0) * per_layer * sizeof(__nv_bfloat16);
            cudaError_t r = cudaMemcpyAsync(ctx->stage_q + off, qh + off * 2, bytes, cudaMemcpyHostToDevice, ctx->copy_in);
            if (r == cudaSuccess) r = cudaMemcpyAsync(ctx->stage_k + off, kh + off * 2, bytes, cudaMemcpyHostToDevice, ctx->copy_in);
            if (r == cudaSuccess) r = cudaMemcpyAsync(ctx->stage_v + off, vh + off * 2, bytes, cudaMemcpyHostToDevice, ctx->copy_in);
            if (r == cudaSuccess)   // after the data, in stream order: the words that release these layers
                r = cudaMemcpyAsync(ctx->in_flags + l0, ctx->epoch_src + l0, (size_t)(l1 - l0) * sizeof(int), cudaMemcpyHostToDevice, ctx->copy_in);
            return r;
        };
        e = cudaEventRecord(ctx->ev_start, st);   // earlier work on the caller's stream may still read the staging buffers
        if (e == cudaSuccess) e = cudaStreamWaitEvent(ctx->copy_in, ctx->ev_start, 0);
        int done = 0, size = 1;
        if (e == cudaSuccess) { e = copy_layers(0, 1); done = 1; }
        int rc = ADSA_OK;
        if (e == cudaSuccess)
            rc = step_layers(ctx, 0, L, cur_pos, budget_rows, ctx->stage_q, ctx->stage_k, ctx->stage_v,
                             out_direct ? out_direct : ctx->stage_o, stream, ctx->in_flags, epoch);
        // The rest of the inputs, whatever the launch returned: a kernel that did start must find every word.
        while (done < L && e == cudaSuccess) {
            size *= 2;
            const int take = done + size + size / 2 >= L ? L - done : size;
            e = copy_layers(done, done + take);
            done += take;
        }
        if (e == cudaSuccess && rc == ADSA_OK && !out_direct)
            e = cudaMemcpyAsync(oh, ctx->stage_o, (size_t)L * per_layer * sizeof(__nv_bfloat16), cudaMemcpyDeviceToHost, st);
        const cudaError_t s_in = cudaStreamSynchronize(ctx->copy_in), s_st = cudaStreamSynchronize(st);
        if (rc != ADSA_OK) return rc;
        if (e == cudaSuccess) e = s_in != cudaSuccess ? s_in : s_st;
        return cuda_fail(ctx, e);
    }
    auto copy_in_chunk = [&](int c) -> cudaError_t {   // inputs of chunk c, on the inbound copy stream
        const size_t off = (size_t)bound[c] * per_layer, bytes = (size_t)(bound[c + 1] - bound[c]) * per_layer * sizeof(__nv_bfloat16);
        cudaError_t r = cudaMemcpyAsync(ctx->stage_q + off, qh + off * 2, bytes, cudaMemcpyHostToDevice, ctx->copy_in);
        if (r == cudaSuccess) r = cudaMemcpyAsync(ctx->stage_k + off, kh + off * 2, bytes, cudaMemcpyHostToDevice, ctx->copy_in);
        if (r == cudaSuccess) r = cudaMemcpyAsync(ctx->stage_v + off, vh + off * 2, bytes, cudaMemcpyHostToDevice, ctx->copy_in);
        if (r == cudaSuccess) r = cudaEventRecord(ctx->ev_in[c], ctx->copy_in);
        return r;
    };
    // the copies start when the work already queued on the caller's stream is done (it may still read the staging buffers)
    e = cudaEventRecord(ctx->ev_start, st);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(ctx->copy_in, ctx->ev_start, 0);
    // copies are queued two chunks ahead of the launches, so that the first kernel is queued early
    for (int c = 0; c < 2 && c < n_chunks && e == cudaSuccess; ++c) e = copy_in_chunk(c);
    int rc = ADSA_OK;
    for (int c = 0; c < n_chunks && e == cudaSuccess && rc == ADSA_OK; ++c) {
        const int l0 = bound[c], l1 = bound[c + 1];
        const size_t off = (size_t)l0 * per_layer, bytes = (size_t)(l1 - l0) * per_layer * sizeof(__nv_bfloat16);
        e = cudaStreamWaitEvent(st, ctx->ev_in[c], 0);
        if (e == cudaSuccess)   // the chunk's layers: one launch when the tensor-core kernel can take them together
            rc = step_layers(ctx, l0, l1 - l0, cur_pos, budget_rows, ctx->stage_q + l0 * per_layer, ctx->stage_k + l0 * per_layer,
                             ctx->stage_v + l0 * per_layer, (out_direct ? out_direct : ctx->stage_o) + l0 * per_layer, stream);
        if (e != cudaSuccess || rc != ADSA_OK) break;
        if (!out_direct) {
            e = cudaEventRecord(ctx->ev_done[c], st);
            if (e == cudaSuccess) e = cudaStreamWaitEvent(ctx->copy_out, ctx->ev_done[c], 0);
            if (e == cudaSuccess) e = cudaMemcpyAsync(oh + off * 2, ctx->stage_o + off, bytes, cudaMemcpyDeviceToHost, ctx->copy_out);
        }
        if (e == cudaSuccess && c + 2 < n_chunks) e = copy_in_chunk(c + 2);
    }
    // One way out, whatever happened: nothing of this call may still be running on the private streams, or
    // reading and writing the caller's host buffers, when it returns.  On success the last output chunk is
    // then on the host and every layer has run.
    const cudaError_t s_out = cudaStreamSynchronize(ctx->copy_out), s_st = cudaStreamSynchronize(st),
                      s_in = cudaStreamSynchronize(ctx->copy_in);
    if (rc != ADSA_OK) return rc;
    if (e == cudaSuccess) e = s_out != cudaSuccess ? s_out : s_st != cudaSuccess ? s_st : s_in;
    return cuda_fail(ctx, e);
}

int adsa_plan_attn(const adsa_ctx *ctx, int n_rows, int *n_splits, int *chunk_rows)
{
    if (!ctx || n_rows < 0) return ADSA_EINVAL;
    StagedChoice ch = choose_staged(ctx, n_rows, false);
    if (ch.wp.n_groups || ch.pp.n_stages) {   // one warp or one CTA walks the whole stream, tile by tile
        if (n_splits) *n_splits = 1;
        if (chunk_rows) *chunk_rows = ch.wp.n_groups ? 32 : ch.pp.tile_rows;
        return ADSA_OK;
    }
    if (ch.sp.cluster_size) {
        if (n_splits) *n_splits = ch.sp.cluster_size;
        if (chunk_rows) *chunk_rows = ch.sp.chunk_rows;
        return ADSA_OK;
    }
    AttnPlan p = plan_attn(ctx, n_rows);
    if (n_splits) *n_splits = p.n_splits;
    if (chunk_rows) *chunk_rows = p.chunk_rows;
    return ADSA_OK;
}

int adsa_set_attn_chunk_rows(adsa_ctx *ctx, int chunk_rows)
{
    if (!ctx || chunk_rows < 0) return ADSA_EINVAL;
    ctx->chunk_override = chunk_rows;
    return ADSA_OK;
}

int adsa_set_staged(adsa_ctx *ctx, int mode)
{
    if (!ctx || mode < 0 || mode > 4) return ADSA_EINVAL;
    ctx->kernel_mode = mode;
    return ADSA_OK;
}

int adsa_set_stream_warps(adsa_ctx *ctx, int warps)
{
    if (!ctx || warps < 0 || warps > 4) return ADSA_EINVAL;
    ctx->stream_warps = warps;
    return ADSA_OK;
}

int adsa_set_single_sweep(adsa_ctx *ctx, int mode)
{
    if (!ctx || mode < 0 || mode > 2) return ADSA_EINVAL;
    ctx->sweep_mode = mode;
    return ADSA_OK;
}

int adsa_set_ring_stages(adsa_ctx *ctx, int max_stages)
{
    if (!ctx || max_stages < 0) return ADSA_EINVAL;
    ctx->max_stages = max_stages;
    return ADSA_OK;
}

int adsa_set_l2_lookahead(adsa_ctx *ctx, int tiles)
{
    if (!ctx || tiles < -1) return ADSA_EINVAL;
    ctx->l2_ahead = tiles;
    return ADSA_OK;
}

int adsa_set_host_chunks(adsa_ctx *ctx, int chunks)
{
    if (!ctx || chunks < 0 || chunks > 6) return ADSA_EINVAL;
    ctx->host_chunks = chunks;
    return ADSA_OK;
}

int adsa_set_token_launch(adsa_ctx *ctx, int mode)
{
    if (!ctx || mode < 0 || mode > 1) return ADSA_EINVAL;
    ctx->token_launch = mode;
    return ADSA_OK;
}

int adsa_set_next_layer_hint(adsa_ctx *ctx, int tiles)
{
    if (!ctx || tiles < 0 || tiles > 64) return ADSA_EINVAL;
    ctx->next_tiles = tiles;
    return ADSA_OK;
}

int adsa_layer_rows_bound(const adsa_ctx *ctx, int layer, int *n_rows)
{
    if (!ctx || !n_rows || layer < 0 || layer >= ctx->cfg.n_layers) return ADSA_EINVAL;
    *n_rows = ctx->layers[layer].rows_hi;
    return ADSA_OK;
}

int adsa_get_status(adsa_ctx *ctx, uint32_t *dev_status, int32_t free_state[4])
{
    if (!ctx) return ADSA_EINVAL;
    cudaError_t e = cudaDeviceSynchronize();
    if (e == cudaSuccess && dev_status) e = cudaMemcpy(dev_status, ctx->dev.status, sizeof(uint32_t), cudaMemcpyDeviceToHost);
    if (e == cudaSuccess && free_state) e = cudaMemcpy(free_state, ctx->dev.free_state, 4 * sizeof(int32_t), cudaMemcpyDeviceToHost);
    return cuda_fail(ctx, e);
}

int64_t adsa_launch_count(const adsa_ctx *ctx) { return ctx ? ctx->launches : 0; }

const char *adsa_strerror(int status)
{
    switch (status) {
    case ADSA_OK: return "ok";
    case ADSA_EINVAL: return "invalid argument or configuration";
    case ADSA_ESTATE: return "call out of order for this layer-step";
    case ADSA_ENOMEM: return "pool, workspace or row capacity too small";
    case ADSA_ECUDA: return "a CUDA call failed";
    default: return "unknown status";
    }
}

}  // extern "C"

namespace adsa {

// Opt in to large dynamic shared memory where a configuration needs it.
cudaError_t configure_kernels(const DevCtx &c)
{
    cudaError_t e = configure_select_kernel(c);
    if (e == cudaSuccess) e = configure_score_kernel(c);
    if (e == cudaSuccess) e = configure_update_kernel(c);
    if (e == cudaSuccess) e = configure_step_kernel(c);
    return e != cudaSuccess ? e : configure_pstep_kernel(c);
}

}  // namespace adsa

/*
 * libadsa: decode attention with Adaptive Dynamic Sparse Attention (ADSA) on a
 * paged bf16 KV pool, for one NVIDIA B200 (sm_100a).
 *
 * The library implements one layer-step of the method of "Make It Efficient:
 * Dynamic Sparse Attention for Autoregressive Image Generation" (Section 4):
 *
 *   adsa_score               Eq. 1-2   mean pairwise cosine similarity of the cached V rows
 *   adsa_select              Eq. 3     keep prefix + 2D-local window + the K lowest-scoring rows
 *   adsa_sparse_decode_attn  Eq. 4     softmax(q.K^T).V over the retained rows and the new row
 *   adsa_kv_update           Sec. 4.2  evict what was not retained, insert the new row, compact
 *
 * Vocabulary.  A *stream* is one (layer, batch row, head); it owns a private
 * cache of rows (pos, k[d], v[d]).  Stream index = (layer*batch + b)*n_heads + h.
 * Context position `pos` counts the text condition first (0 .. n_text-1) and
 * then the image grid in raster order: cell g = pos - n_text, row g / grid_w,
 * column g % grid_w.  Live rows of a stream occupy slots 0 .. n_live-1; slot s
 * lives in page page_table[stream][s / page_rows] at row s % page_rows.  The
 * order of rows inside a stream is not part of the contract (compaction moves
 * rows); a stream is the *set* of its (pos, k, v) rows.
 *
 * General rules.
 *   - Every function returns 0 (ADSA_OK) or a negative adsa_status.  Nothing
 *     throws or aborts.  A CUDA error is sticky: later calls return ADSA_ECUDA.
 *   - Pointers marked [device] must be device memory of the current device,
 *     owned by the caller and alive for as long as the context uses them;
 *     pointers marked [host] are ordinary host memory.  The library allocates
 *     no device memory; it owns only the host-side adsa_ctx.
 *   - Calls taking a cudaStream_t only enqueue work on that stream; they do not
 *     synchronise (the *_host variants and adsa_get_status say so where they do).
 *   - Inconsistencies that only the device can see (pool exhausted, a cached
 *     position at or after cur_pos) set bits of a status word, skip the
 *     offending access and never trap; read it with adsa_get_status.
 *   - A context is not thread-safe: use it from one host thread at a time.
 *   - Launches overlap.  The attention and layer-step kernels are launched with
 *     programmatic stream serialization: their set-up runs while the kernel
 *     ahead of them in the stream drains, and when that kernel is this context's
 *     previous launch, went to the same stream and served another layer (or does
 *     not write what is about to be read), they also read this layer's cache state
 *     (rows, page table, positions, norms, carried scores) before it has finished.
 *     Three rules follow.  The buffers of adsa_buffers belong to the library between
 *     calls: nothing else may write them while work of this context is in flight.
 *     The calls of one context must reach the device in the order they are made:
 *     use one stream, or order the streams with events (work on a second stream
 *     that is not ordered after the first races on the shared scratch and on the
 *     cache state).  And a kernel of the caller's own that is put between two
 *     calls on the same stream must not itself start early under programmatic
 *     stream serialization, or must wait for its predecessor before it lets its
 *     successor start.  q, k_new, v_new and the keep mask are read only after the
 *     kernel ahead has completed, so producing them in the kernel launched just
 *     before the call is fine.
 *   - bf16 tensors are dense, row-major, innermost dimension head_dim
 *     ([batch][n_heads][head_dim] unless stated); all arithmetic is fp32.
 */
#ifndef ADSA_H_
#define ADSA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define ADSA_API __attribute__((visibility("default")))
#else
#define ADSA_API
#endif

typedef struct CUstream_st *adsa_stream_t; /* a cudaStream_t; 0 = the default stream */
typedef struct adsa_ctx adsa_ctx;          /* opaque, host side only */

typedef enum {
    ADSA_OK = 0,
    ADSA_EINVAL = -1, /* bad argument or configuration */
    ADSA_ESTATE = -2, /* calls out of order, or cur_pos differs between the calls of one layer-step */
    ADSA_ENOMEM = -3, /* pool, workspace or row capacity too small (found on the host, nothing launched) */
    ADSA_ECUDA = -4   /* a CUDA call failed; sticky */
} adsa_status;

/* bits of the device status word (adsa_get_status) */
#define ADSA_DEV_POOL_EXHAUSTED 1u /* a page was needed and the free ring was empty */
#define ADSA_DEV_BAD_POSITION 2u   /* a cached row had pos < 0 or pos >= cur_pos */
#define ADSA_DEV_ROW_OVERFLOW 4u   /* a stream would exceed max_rows_per_stream */
#define ADSA_DEV_RING_TIMEOUT 8u   /* bounded wait on a free-ring entry ran out */
#define ADSA_DEV_BAD_EVICT 16u     /* hole/survivor pairing of the compaction did not balance */
#define ADSA_DEV_COPY_TIMEOUT 32u  /* bounded wait on a bulk copy into shared memory ran out */

typedef struct {
    int32_t n_layers, batch, n_heads; /* multi-head attention: one KV head per query head */
    int32_t head_dim;                 /* d, 8 .. 256 */
    int32_t row_stride;               /* elements per pool row: >= head_dim, a multiple of 8 (16 bytes), <= 256 */
    int32_t page_rows;                /* rows per page, 2 .. 4096 */
    int32_t n_pages;                  /* pages in k_pool (and in v_pool) */
    int32_t max_rows_per_stream;      /* largest n_live any stream may reach */
    int32_t n_text, grid_h, grid_w;   /* position -> grid cell mapping */
    int32_t n_prefix;                 /* rows with pos < n_prefix are always kept (Section 4.1 "prefix") */
    int32_t local_rows_back;          /* R: the local window holds the current grid row and R rows above it */
    int32_t score_mode;               /* 0 = mean V-cosine similarity, keep the lowest (Eq. 1-3): the paper's rule.
                                         1 = attention mass, keep the highest: the attention-score pruning that
                                         Section 3.4 argues against, as a comparison (see below) */
    int32_t score_share;              /* 0 = one score per stream (a head's V row).  1 = one score per batch row and token:
                                         Eq. 1-2 on the token's V rows of all heads of the layer laid end to end, so
                                         every head keeps the same tokens (the paper does not fix the granularity of
                                         the comparison).  Needs score_mode 0; the heads of a batch row must be loaded
                                         and stepped together (same positions slot by slot, ADSA_DEV_BAD_POSITION
                                         otherwise); runs on the four stand-alone kernels */
    float softmax_scale;              /* 0 => 1/sqrt(head_dim) */
} adsa_config;

typedef struct {
    void *k_pool, *v_pool;   /* [device] bf16 [n_pages][page_rows][row_stride], 16-byte aligned */
    int32_t *page_table;     /* [device] [n_streams][ceil(max_rows_per_stream / page_rows)] */
    int32_t *pos;            /* [device] [n_streams][max_rows_per_stream] context position per slot */
    float *inv_norm;         /* [device] [n_streams][max_rows_per_stream] 1 / max(|v|, 1e-8) per slot */
    int32_t *n_live;         /* [device] [n_streams] */
    int32_t *free_ring;      /* [device] [n_pages] ring of free page ids */
    int32_t *free_state;     /* [device] [4]: head, tail, free count, low-water mark of the free count */
    void *workspace;         /* [device] scratch of adsa_workspace_bytes() bytes, 256-byte aligned */
    size_t workspace_bytes;
} adsa_buffers;
/* n_streams = n_layers * batch * n_heads.  All buffers are initialised by adsa_reset. */

/* Scratch size the configuration needs (per layer: scores, carried sums, keep
 * masks, counts, staging for the *_host calls; once: split partials, status
 * word).  No CUDA call is made. */
ADSA_API int adsa_workspace_bytes(const adsa_config *cfg, size_t *out_bytes);

/* Validate cfg and buffers and build the host-side context.  Queries the
 * current device's SM count; launches nothing.  ADSA_EINVAL / ADSA_ENOMEM
 * (workspace too small) on failure, *out untouched. */
ADSA_API int adsa_create(const adsa_config *cfg, const adsa_buffers *buf, adsa_ctx **out);
ADSA_API int adsa_destroy(adsa_ctx *ctx);

/* Empty every stream, put all pages on the free ring, clear the status word. */
ADSA_API int adsa_reset(adsa_ctx *ctx, adsa_stream_t stream);

/* Append n_rows rows to every stream of `layer` (how the text condition, or a
 * saved cache, enters the pool).  k, v: [device] bf16
 * [batch][n_heads][n_rows][head_dim].  Positions are first_pos ..
 * first_pos+n_rows-1 when pos is NULL, else pos: [device] int32
 * [batch][n_heads][n_rows] gives each row's position (distinct per stream, and
 * distinct from the rows already cached).  Pages are taken from the free ring
 * as needed.  ADSA_ENOMEM if rows or pages cannot fit. */
ADSA_API int adsa_prefill_rows(adsa_ctx *ctx, int layer, const void *k, const void *v, const int32_t *pos, int n_rows,
                               int first_pos, adsa_stream_t stream);

/* The condition entering an EMPTY cache with its attention computed on the way (Section 4.2: while the cache
 * has room the method is plain attention): for every stream of `layer`, row i of q attends rows 0 .. i of
 * k, v (dense causal attention, fp32 softmax), and the n_rows rows of k, v are appended to the cache at
 * positions first_pos .. first_pos+n_rows-1 exactly as adsa_prefill_rows does.  q, k, v: [device] bf16
 * [batch][n_heads][n_rows][head_dim], 4-byte aligned (k and q already rotated, see adsa_rope_2d).
 * out_bf16 / out_f32: [device] same shape; either may be NULL, not both.  ADSA_ESTATE if the layer's cache
 * is not empty. */
ADSA_API int adsa_prefill_attn(adsa_ctx *ctx, int layer, const void *q, const void *k, const void *v, int n_rows, int first_pos,
                               void *out_bf16, float *out_f32, adsa_stream_t stream);

/* Two-dimensional rotary position embedding of q or k rows, in place (Section 4.1: the embedding sits on Q and
 * K, which is why the V rows are what Eq. 1-2 compare).  x: [device] bf16 [n_rows][head_dim], pos: [device] int32
 * [n_rows] context positions.  Elements turn in consecutive pairs (2i, 2i+1): the first head_dim/4 pairs by the
 * token's grid row, the next head_dim/4 by its grid column, pair i of either half by the angle
 * index * base^(-i / (head_dim/4)); rows of the text condition (pos < n_text) are left as they are.
 * head_dim must be a multiple of 4; base 0 => 10000.  fp32 arithmetic, bf16 result rounded to nearest even. */
ADSA_API int adsa_rope_2d(adsa_ctx *ctx, void *x, const int32_t *pos, long long n_rows, float base, adsa_stream_t stream);

/* Replace the cache of one stream by the given rows (tests, resynchronisation,
 * restoring a snapshot).  k, v: [device] bf16 [n_rows][head_dim]; pos: [device]
 * int32 [n_rows], distinct.  Pages are freed or taken as needed. */
ADSA_API int adsa_set_stream_rows(adsa_ctx *ctx, int layer, int b, int h, const void *k, const void *v, const int32_t *pos,
                         int n_rows, adsa_stream_t stream);

/* ---- the four calls of one layer-step, in this order, with the same cur_pos ----
 * cur_pos is the context position of the token being decoded (its row is "the
 * new row").  Section 4.1 partitions each stream's live rows by position into
 * prefix (pos < n_prefix), local (image cells before the current one, in the
 * current grid row or the R rows above) and previous (the rest).
 * The order is kept per layer (ADSA_ESTATE otherwise).  What one call leaves for
 * the next (scores, keep mask, counts) is stored per layer, so the steps of
 * different layers may be interleaved in any way: score and select for every
 * layer, then every layer's attention, then every update, is a valid sequence. */

/* score_mode 1 (comparison method, Section 3.4): every cached row carries the attention mass it has received,
 * the sum of its softmax weights over the steps in which it was attended (its insertion step included; rows
 * loaded by adsa_prefill_rows / adsa_set_stream_rows start at 0).  adsa_score then computes nothing and only
 * reports the masses; adsa_select keeps the K previous rows with the HIGHEST mass (equal masses: lower position
 * first); adsa_kv_update adds this step's weights to the retained rows' masses, so it must follow
 * adsa_sparse_decode_attn (ADSA_ESTATE otherwise).  The mode runs on the four stand-alone kernels
 * (adsa_layer_step and adsa_token_step launch them one after the other).
 *
 * Eq. 1-2.  For every row i of the previous region of every stream of `layer`:
 * S_i = (1/(p-1)) sum_{j != i} cos(v_i, v_j), j over the same region (p rows);
 * p <= 1 gives 0.  Computed through the identity sum_j cos = u_i.(sum_j u_j) - u_i.u_i
 * with u = v * inv_norm.  Scores stay in the workspace for adsa_select.
 * scores_out: [device] float [batch*n_heads][max_rows_per_stream] indexed by
 * slot, NaN for rows outside the previous region; may be NULL. */
ADSA_API int adsa_score(adsa_ctx *ctx, int layer, int cur_pos, float *scores_out, adsa_stream_t stream);

/* Eq. 3 plus the always-kept regions.  budget_rows counts the new row:
 * K = min(p, max(0, budget_rows - |prefix| - |local| - 1)) previous rows are
 * kept, the K lowest in the order (score ascending, position ascending).
 * Outputs (each [device], each may be NULL), stream-major with stride
 * max_rows_per_stream, entries in ascending slot order:
 *   sel_slots / sel_pos     retained cached rows (the new row is not listed)
 *   evict_pos               rows that adsa_kv_update will drop
 *   counts                  int32 [batch*n_heads][4]: previous rows p, evicted, retained, K */
ADSA_API int adsa_select(adsa_ctx *ctx, int layer, int cur_pos, int budget_rows, int32_t *sel_slots, int32_t *sel_pos,
                int32_t *evict_pos, int32_t *counts, adsa_stream_t stream);

/* Eq. 4 and the attention of Fig. 3: out = softmax_j(q.k_j * scale) . v_j over
 * the retained rows and the new row (k_new, v_new), maximum subtracted, fp32.
 * q, k_new, v_new: [device] bf16 [batch][n_heads][head_dim].
 * out_bf16: [device] bf16 same shape (round to nearest even); out_f32: [device]
 * float same shape.  Either output may be NULL, not both. */
ADSA_API int adsa_sparse_decode_attn(adsa_ctx *ctx, int layer, int cur_pos, const void *q, const void *k_new,
                            const void *v_new, void *out_bf16, float *out_f32, adsa_stream_t stream);

/* Section 4.2.  Drops the rows adsa_select marked, writes the new row
 * (k_new, v_new, cur_pos, its inverse norm) and compacts so that live rows are
 * slots 0 .. n_live-1: holes are filled by the new row and by survivors from
 * the tail.  Pages that became empty return to the free ring; a page is taken
 * when the stream grows into one.  Evict-before-insert: a stream never holds
 * more than max(budget_rows, |prefix|+|local|+1) rows. */
ADSA_API int adsa_kv_update(adsa_ctx *ctx, int layer, int cur_pos, const void *k_new, const void *v_new,
                   adsa_stream_t stream);

/* The four calls above in one: score, select, attend, update for `layer`. */
ADSA_API int adsa_layer_step(adsa_ctx *ctx, int layer, int cur_pos, int budget_rows, const void *q, const void *k_new,
                    const void *v_new, void *out_bf16, adsa_stream_t stream);

/* adsa_layer_step with HOST tensors: q, k_new, v_new [host] bf16
 * [batch][n_heads][head_dim] are copied to staging space in the workspace,
 * the step runs, out [host] bf16 is copied back, and the call returns after
 * the stream has drained (it synchronises `stream`).  Pinned host memory makes
 * the copies asynchronous up to that point. */
ADSA_API int adsa_layer_step_host(adsa_ctx *ctx, int layer, int cur_pos, int budget_rows, const void *q_host,
                         const void *k_new_host, const void *v_new_host, void *out_host, adsa_stream_t stream);

/* One decoded token through every layer of an attention stack: what adsa_layer_step
 * does, for layer 0 .. n_layers-1 with the same cur_pos and budget.  q, k_new, v_new,
 * out_bf16: [device] bf16 [n_layers][batch][n_heads][head_dim].  Because every layer's
 * inputs are given at once, no layer has to wait for another: when the tensor-core
 * kernel serves the configuration and every layer is between steps, ONE launch walks
 * the streams of all layers (adsa_set_token_launch); otherwise the layers are
 * launched one after the other.  Results are those of adsa_layer_step layer by layer, up to the order in
 * which partial sums are merged (it depends on how many warps share a stream, which the two ways may choose
 * differently). */
ADSA_API int adsa_token_step(adsa_ctx *ctx, int cur_pos, int budget_rows, const void *q, const void *k_new,
                             const void *v_new, void *out_bf16, adsa_stream_t stream);

/* adsa_token_step whose inputs may still be on their way when it is called: layer l's q, k_new and v_new are read
 * only once ready[l] - epoch >= 0 (wrap-around comparison), where ready is an int32 [n_layers] array in device
 * memory that the caller's own copies or kernels write AFTER the layer's tensors, in an order the device sees
 * (the same stream as those copies, or a release at system scope).  Whatever writes the words must not wait for
 * this call's kernel.  A stream waits for its layer's word for about a second; then it sets the device status
 * ADSA_DEV_COPY_TIMEOUT, reads what is there and goes on (later waits of that warp are a millisecond), so the
 * kernel always ends and the context stays usable (adsa_get_status; adsa_reset clears the state).  Needs the one
 * launch for all layers that adsa_token_step describes: ADSA_ESTATE when the tensor-core kernel cannot serve the
 * configuration in one launch or the layers are not all between steps in the same carried state.
 * This is how adsa_token_step_host overlaps its copies with the kernel. */
ADSA_API int adsa_token_step_gated(adsa_ctx *ctx, int cur_pos, int budget_rows, const void *q, const void *k_new,
                                   const void *v_new, void *out_bf16, const int32_t *ready, int32_t epoch,
                                   adsa_stream_t stream);

/* adsa_token_step with HOST tensors of the same shapes.  The inputs cross the bus in chunks of layers on a copy
 * stream that the context creates on its first call here, while earlier layers compute on `stream`:
 *   - inputs in pinned host memory, and one launch of the tensor-core kernel can serve the whole stack (see
 *     adsa_token_step): that launch is queued at once; every chunk of copies is followed by a small copy that marks
 *     its layers as landed, and the kernel waits for a layer's mark (adsa_token_step_gated: bounded, with the
 *     device status ADSA_DEV_COPY_TIMEOUT when a wait runs out) before it reads that layer's q, k_new, v_new;
 *   - otherwise, or after adsa_set_host_chunks(2 .. 6): every chunk of layers is a launch of its own, queued
 *     behind its copies (pageable memory works here, but its copies overlap nothing).
 * An output buffer in pinned, mapped host memory (cudaHostAlloc, cudaHostRegister) is written by the kernels
 * directly; any other host buffer is filled by copies from a staging buffer.  When the call returns every layer
 * has run and the outputs are on the host.  Uses the staging part of the workspace (and, on its first call, creates
 * two streams, a few events and n_layers words of pinned host memory that live as long as the context); results
 * are those of adsa_token_step. */
ADSA_API int adsa_token_step_host(adsa_ctx *ctx, int cur_pos, int budget_rows, const void *q_host,
                                  const void *k_new_host, const void *v_new_host, void *out_host,
                                  adsa_stream_t stream);

/* How adsa_sparse_decode_attn would split a stream of n_rows cached rows:
 * number of chunks per stream and rows per chunk.  Pure host arithmetic. */
ADSA_API int adsa_plan_attn(const adsa_ctx *ctx, int n_rows, int *n_splits, int *chunk_rows);

/* Which kernels adsa_sparse_decode_attn and adsa_layer_step use.  Same results in every mode.
 *   1 (default) automatic: when pool rows are at most 128 elements wide (and head_dim is even), the warp-group
 *               kernel (a few warps own a stream, each with its own TMA tile ring; tensor-core arithmetic); else the
 *               persistent pipelined CUDA-core kernel (one CTA per SM, a producer warp feeding a
 *               ring of K/V tiles); if that does not fit shared memory, the cluster kernel; if a
 *               stream does not fit a cluster either, the streaming kernels
 *   0 streaming kernels only (register-streaming attention; four kernels per layer-step)
 *   2 cluster kernel (one thread-block cluster per stream), else streaming
 *   3 persistent CUDA-core kernel, else streaming
 *   4 warp-group tensor-core kernel, else streaming */
ADSA_API int adsa_set_staged(adsa_ctx *ctx, int mode);

/* Warps that share a stream in the tensor-core kernel: 1 .. 4, or 0 = chosen from the number of
 * streams per SM and the shared memory the configuration needs. */
ADSA_API int adsa_set_stream_warps(adsa_ctx *ctx, int warps);

/* How much the fused tensor-core kernel takes over from the step before (same results up to rounding of
 * the carried sum of normalised rows):
 *   0  nothing but the scores: it always makes a second sweep over V for the next step's scores;
 *   1  it scores the next step's rows during its attention sweep whenever the sum of normalised rows
 *      carried in from the previous step can be updated in closed form (no eviction, or one; no rows
 *      leaving the local window);
 *   2  (default) as 1, and when the cache is exactly full it evicts the row the previous step noted as
 *      the highest-scoring of this step's previous region instead of classifying and comparing the rows
 *      again (the previous step leaves no note when two rows tie for the highest score or rows moved). */
ADSA_API int adsa_set_single_sweep(adsa_ctx *ctx, int mode);

/* Cap the tile ring (per CTA of the persistent kernel, per warp of the tensor-core kernel) at
 * max_stages stages (0 = as many as fit). */
ADSA_API int adsa_set_ring_stages(adsa_ctx *ctx, int max_stages);

/* The tensor-core kernel asks the K/V tiles that come after the ones its ring holds into L2 while it is
 * still selecting rows, so that HBM is busy before the attention sweep starts.  tiles = how many 32-row
 * tiles per warp beyond the ring (0 = none, -1 = choose automatically, the default).  Results do not
 * depend on it. */
ADSA_API int adsa_set_l2_lookahead(adsa_ctx *ctx, int tiles);

/* adsa_token_step_host: 0 (default): one launch that waits for its inputs layer by layer when that is possible,
 * else one launch per chunk with chunks that grow threefold from a single layer.  2 .. 6: always one launch per
 * chunk: one layer, then chunks - 1 equal chunks. */
ADSA_API int adsa_set_host_chunks(adsa_ctx *ctx, int chunks);

/* adsa_token_step: 1 (default) = one launch serves every layer when it can, 0 = one launch per layer
 * (what a decoder whose layers feed each other has to do, through adsa_layer_step). */
ADSA_API int adsa_set_token_launch(adsa_ctx *ctx, int mode);

/* Between the end of a launch's sweep and the moment the next launch has located its first rows HBM is
 * idle.  A decoder runs its layers in order, so when a launch of the tensor-core kernel has fetched its
 * last tile it asks the first `tiles` 32-row tiles per warp of the same streams of layer (layer + 1) mod
 * n_layers into L2 (the 126 MB L2 holds them until that launch reads them).  A hint only: if another layer
 * comes next the prefetch is wasted, nothing else.  In a launch that serves several layers the hint is
 * for the stream the same warps serve next.  0 = off (default: measured, it did not pay). */
ADSA_API int adsa_set_next_layer_hint(adsa_ctx *ctx, int tiles);

/* Override the rows per attention chunk (0 = choose automatically). */
ADSA_API int adsa_set_attn_chunk_rows(adsa_ctx *ctx, int chunk_rows);

/* Upper bound, tracked on the host, of n_live over the streams of `layer`. */
ADSA_API int adsa_layer_rows_bound(const adsa_ctx *ctx, int layer, int *n_rows);

/* Synchronises the device, then copies out the device status word (OR of
 * ADSA_DEV_* bits since the last reset) and the free-ring state
 * {head, tail, free pages, fewest free pages seen}.  Either pointer may be NULL. */
ADSA_API int adsa_get_status(adsa_ctx *ctx, uint32_t *dev_status, int32_t free_state[4]);

/* Number of kernels this context has launched so far (host counter). */
ADSA_API int64_t adsa_launch_count(const adsa_ctx *ctx);

/* Decode attention without a context, a workspace or any allocation (the paper has no counterpart:
 * this exists for the integration, not for the method).  For callers that cannot allocate device
 * memory where they need attention - a serving loop whose memory plan was frozen at start-up, a
 * plugin interface that forbids the allocation calls, a process whose device memory belongs wholly
 * to a framework's pool - and therefore cannot provide the workspace a context needs.
 *
 * out[s] = softmax_j(q[s].k_j * scale) . v_j over rows j = 0 .. n_rows[s]-1 of stream s and the new
 * row (k_new[s], v_new[s]), fp32 arithmetic, the split reduction of adsa_sparse_decode_attn.
 *   q, k_new, v_new   [device] bf16 [n_streams][head_dim]
 *   k, v              [device] bf16 [n_streams][max_rows][row_stride], 16-byte aligned; row_stride >=
 *                     head_dim, a multiple of 8, <= 256; elements past head_dim are ignored
 *   n_rows            [device] int32 [n_streams], each clamped to 0 .. max_rows
 *   out_bf16/out_f32  [device] [n_streams][head_dim]; either may be NULL, not both
 *   softmax_scale     0 => 1/sqrt(head_dim)
 * The scratch of the split reduction is a fixed 4 MiB array inside the library image: every GPU that
 * loads the library holds it until the process exits.  Limits: n_streams <= 4096, max_rows <= 2^20
 * (ADSA_ENOMEM beyond them; fewer chunks per stream are used when the partial states of more would
 * not fit, down to a single chunk, which needs no partial state at all).  No cudaMalloc, cudaFree or allocating routine is called; the call only enqueues a
 * counter clear and one kernel on `stream`.
 * The first call on each device looks up the array's device address (that device must be current);
 * make that first call before any stream capture begins.  All calls share the array and it keeps
 * the previous call's contents, so calls whose kernels may overlap on the GPU (other streams, other
 * host threads) race: serialise them. */
ADSA_API int adsa_decode_attn_static(const void *q, const void *k, const void *v, const int32_t *n_rows,
                                     const void *k_new, const void *v_new, int n_streams, int max_rows, int head_dim,
                                     int row_stride, float softmax_scale, void *out_bf16, float *out_f32,
                                     adsa_stream_t stream);

/* ---- the host model around the attention -------------------------------------------------------------------------
 * Section 5 integrates the method with a LlamaGen decoder.  The paper defines none of that decoder's own operations;
 * these three are its published element-wise and sampling steps, stateless calls on caller-owned buffers (no
 * context, no workspace; the projections between them are plain GEMMs and are left to the caller's BLAS).  All
 * pointers [device], 16-byte aligned where rows are read in 16-byte pieces; fp32 arithmetic; each call enqueues one
 * kernel on `stream` and returns (ADSA_EINVAL for a null pointer, a misaligned buffer or a size outside the stated
 * range, before anything is launched). */

/* Root-mean-square normalisation, row by row: out[r][i] = x[r][i] / sqrt(mean_j x[r][j]^2 + eps) * w[i].
 *   x, out  bf16 [rows][dim] (out may be x);  w  bf16 [dim];  dim a multiple of 8, >= 8;  eps >= 0 */
ADSA_API int adsa_rmsnorm(const void *x, const void *w, void *out, long long rows, int dim, float eps,
                          adsa_stream_t stream);

/* The gated activation of the feed-forward block: out[r][i] = silu(gate[r][i]) * up[r][i], silu(g) = g / (1 + e^-g).
 *   gate, up  bf16, rows of `hidden` elements ld_in elements apart (ld_in = hidden for two separate tensors,
 *             2 * hidden with up = gate + hidden for one tensor that holds both halves side by side)
 *   out       bf16 [rows][hidden];  hidden and ld_in multiples of 8 */
ADSA_API int adsa_swiglu(const void *gate, const void *up, void *out, long long rows, int hidden, long long ld_in,
                         adsa_stream_t stream);

/* The next image token of every image from the logits of its conditional and unconditional rows:
 *   mixed = uncond + scale * (cond - uncond)                       (classifier-free guidance)
 *   keep the top_k largest mixed logits (equal logits at the threshold: the lower token ids)
 *   p_i proportional to exp((mixed_i - max) / temperature) over the kept ids
 *   token = the first kept id, in ascending order of id, at which the running sum of p reaches u * (sum of p)
 * The random numbers are the caller's: uniforms [n_images] f32 in [0, 1).
 *   logits  bf16 [2 * n_images][vocab]: the conditional rows of all images, then their unconditional rows
 *   tokens  int32 [n_images];  1 <= top_k <= vocab <= 32768;  temperature > 0
 * One block per image; sums are taken in fp32 in a fixed order, so a call is reproducible. */
ADSA_API int adsa_cfg_sample(const void *logits, int n_images, int vocab, float scale, int top_k, float temperature,
                             const float *uniforms, int32_t *tokens, adsa_stream_t stream);

ADSA_API const char *adsa_strerror(int status);

#ifdef __cplusplus
}
#endif
#endif /* ADSA_H_ */

// Shared device-side definitions of libadsa: the kernel parameter block, pool
// addressing, bf16 unpacking, the page free ring and small warp/block helpers.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/adsa.h"

namespace adsa {

constexpr int kRegionPrefix = 0;
constexpr int kRegionPrevious = 1;
constexpr int kRegionLocal = 2;
constexpr int kRegionInvalid = 3;

constexpr int kMaxSplits = 32;         // attention chunks per stream
constexpr int kScratchCtas = 160;      // CTAs of the tensor-core kernel that own a slice of rare-step scratch (its grid is capped here)
constexpr int kScratchGroups = 8;      // ... and streams such a CTA serves at a time
constexpr float kNormEps = 1e-8f;      // clamp of |v| (an all-zero row has similarity 0 with everything)
constexpr int kRingSpinLimit = 1 << 16;

// Everything a kernel needs, passed by value.
struct DevCtx {
    __nv_bfloat16 *k_pool, *v_pool;
    int32_t *page_table, *pos, *n_live;
    float *inv_norm;
    int32_t *free_ring, *free_state;
    // workspace; S = streams per layer.  What one layer-step hands from call to call (scores, keep mask,
    // counts) exists per layer, so that the steps of several layers may be in flight between their calls;
    // the split partials are scratch of one attention launch and are shared by all layers
    float *scores;          // [n_layers * S][max_rows]  Eq. 2 scores by slot; carried from one step to the next
    uint32_t *keep_mask;    // [n_layers * S][mask_words]   bit s = slot s is retained
    int32_t *counts;        // [n_layers * S][4]            p, evicted, retained, K
    float *partials;        // [S][kMaxSplits][partial_stride]
    int32_t *tickets;       // [S]
    float *svec;            // [n_layers * S][256]  s = sum of the normalised V rows the next step scores (carried with the scores)
    int32_t *carry;         // [n_layers * S][4]    left by a fused step for the next one: slot of the row it will evict (the
                            //                      highest-scoring row of its previous region; -1 = not known), number of rows
                            //                      in that region, bit 0 = some cached V row has a clamped norm, spare
    uint32_t *cand_mask;    // [n_layers * S][mask_words]  bit s = slot s lies in the previous region of the next step
    float *logit;           // [n_layers * S][max_rows]  score_mode 1: this step's logits (log2 units) by slot, from attention to the update
    float *ml;              // [n_layers * S][4]         score_mode 1: softmax maximum, denominator, the new row's logit
    unsigned long long *wscratch;   // [kScratchCtas][kScratchGroups][2 * max_rows + 4]  rare-step scratch of the tensor-core kernel
    uint32_t *status;       // [1]
    int d, row_stride, page_rows, n_pages, max_rows, max_pages, mask_words, S;
    int partial_stride;     // floats per split partial: row_stride + 2 (m, l)
    uint32_t pr_magic;      // slot / page_rows == __umulhi(slot, pr_magic)
    int n_text, grid_w, n_prefix, rows_back;
    int n_heads;            // heads per batch row (streams b * n_heads .. of a layer belong to batch row b)
    int score_share;        // 1: Eq. 1-2 on a token's V over all heads of the layer (one score per batch row and token)
    int score_mode;         // 0: Eq. 1-3 (mean V-cosine similarity, keep the lowest); 1: attention mass, keep the highest
    float scale_log2e;      // softmax scale * log2(e)
};

__device__ __forceinline__ void set_status(const DevCtx &c, uint32_t bit) { atomicOr(c.status, bit); }

// Section 4.1 partition of a cached position relative to the current one.
__device__ __forceinline__ int region_of(const DevCtx &c, int pos, int cur_pos)
{
    if (pos < 0 || pos >= cur_pos) return kRegionInvalid;
    if (pos < c.n_prefix) return kRegionPrefix;
    if (pos >= c.n_text && cur_pos >= c.n_text) {
        int row = (pos - c.n_text) / c.grid_w, cur_row = (cur_pos - c.n_text) / c.grid_w;
        if (cur_row - row <= c.rows_back) return kRegionLocal;
    }
    return kRegionPrevious;
}

// Element offset of slot `slot` of stream `sid` inside k_pool / v_pool.
__device__ __forceinline__ size_t row_offset(const DevCtx &c, const int32_t *pt, int slot)
{
    uint32_t pg = __umulhi((uint32_t)slot, c.pr_magic);
    uint32_t in = (uint32_t)slot - pg * (uint32_t)c.page_rows;
    return ((size_t)pt[pg] * c.page_rows + in) * (size_t)c.row_stride;
}

// 8 bf16 packed in a uint4 -> 8 floats (a bf16 is the upper half of a float)
__device__ __forceinline__ void unpack8(const uint4 &r, float (&f)[8])
{
    f[0] = __uint_as_float(r.x << 16); f[1] = __uint_as_float(r.x & 0xffff0000u);
    f[2] = __uint_as_float(r.y << 16); f[3] = __uint_as_float(r.y & 0xffff0000u);
    f[4] = __uint_as_float(r.z << 16); f[5] = __uint_as_float(r.z & 0xffff0000u);
    f[6] = __uint_as_float(r.w << 16); f[7] = __uint_as_float(r.w & 0xffff0000u);
}

__device__ __forceinline__ uint4 ldg128(const void *p) { return __ldg(reinterpret_cast<const uint4 *>(p)); }

// streaming 16-byte load: KV rows are read once per step, keep them out of L1
__device__ __forceinline__ uint4 ldg128_stream(const void *p)
{
    uint4 r;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
                 : "l"(p));
    return r;
}

// ---- page free ring -------------------------------------------------------
// free_state = {head, tail, free count, low-water mark}.  Entries are page ids,
// or -1 once taken.  Pops and pushes may run concurrently from many blocks: the
// free count admits a pop only after the matching push has published its entry
// (entry write, fence, count increment); if a neighbouring push with an earlier
// ticket is still in flight the pop waits for its entry, with a bound.
__device__ inline int pool_pop(const DevCtx &c)
{
    int before = atomicSub(&c.free_state[2], 1);
    if (before <= 0) {
        atomicAdd(&c.free_state[2], 1);
        set_status(c, ADSA_DEV_POOL_EXHAUSTED);
        return -1;
    }
    atomicMin(&c.free_state[3], before - 1);
    uint32_t h = atomicInc(reinterpret_cast<unsigned int *>(&c.free_state[0]), (unsigned)c.n_pages - 1u);
    for (int spin = 0; spin < kRingSpinLimit; ++spin) {
        int pg = atomicExch(&c.free_ring[h], -1);
        if (pg >= 0) return pg;
        __nanosleep(64);
    }
    set_status(c, ADSA_DEV_RING_TIMEOUT);
    return -1;
}

__device__ inline void pool_push(const DevCtx &c, int page)
{
    uint32_t t = atomicInc(reinterpret_cast<unsigned int *>(&c.free_state[1]), (unsigned)c.n_pages - 1u);
    atomicExch(&c.free_ring[t], page);
    __threadfence();
    atomicAdd(&c.free_state[2], 1);
}

// ---- reductions -----------------------------------------------------------
__device__ __forceinline__ float warp_sum(float x)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    return x;
}

// ---- rows and pages --------------------------------------------------------
// Bring the number of pages a stream holds from `have` to `need` (one thread).
// Returns false if the pool ran dry.
__device__ inline bool resize_pages(const DevCtx &c, int32_t *pt, int have, int need)
{
    for (int pg = have; pg < need; ++pg) {
        int page = pool_pop(c);
        if (page < 0) {
            for (int q = have; q < pg; ++q) pool_push(c, pt[q]);  // give back what this call took
            return false;
        }
        pt[pg] = page;
    }
    for (int pg = need; pg < have; ++pg) pool_push(c, pt[pg]);
    return true;
}

// Write one cache row: bf16 payload (padding elements zeroed), position and the
// inverse V norm.  One warp per row; src rows hold d elements.
__device__ inline void write_row(const DevCtx &c, const int32_t *pt, int sid, int slot, const __nv_bfloat16 *ksrc,
                          const __nv_bfloat16 *vsrc, int pos)
{
    int lane = threadIdx.x & 31;
    size_t off = row_offset(c, pt, slot);
    float ss = 0.f;
    const __nv_bfloat16 zero = __float2bfloat16(0.f);
    for (int e = lane; e < c.row_stride; e += 32) {
        __nv_bfloat16 kk = e < c.d ? ksrc[e] : zero;
        __nv_bfloat16 vv = e < c.d ? vsrc[e] : zero;
        c.k_pool[off + e] = kk;
        c.v_pool[off + e] = vv;
        float f = __bfloat162float(vv);
        ss = fmaf(f, f, ss);
    }
    ss = warp_sum(ss);
    if (lane == 0) {
        c.pos[(size_t)sid * c.max_rows + slot] = pos;
        c.inv_norm[(size_t)sid * c.max_rows + slot] = 1.0f / fmaxf(sqrtf(ss), kNormEps);
        if (c.score_mode == 1) c.scores[(size_t)sid * c.max_rows + slot] = 0.f;   // a row from outside has received no attention yet
    }
}


}  // namespace adsa
